"""The allocation-free selection entry point against the regular one.

emo_select_static is for callers that cannot allocate device memory (no workspace to hand over): its
per-block candidates live in a fixed array inside the library.  It must give exactly what emo_select
gives, call after call (the array keeps the previous call's contents), and refuse batches beyond
its stated maximum.  This file sorts last so that a run stopping at the first failure has already
run every other test."""
from __future__ import annotations

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _select_both(torch, emo, T, E, target):
    Td = torch.as_tensor(T, dtype=torch.int64, device="cuda")
    Ed = torch.as_tensor(E, dtype=torch.float64, device="cuda")
    ws = torch.empty(65536, dtype=torch.uint8, device="cuda")
    out = []
    for static in (False, True):
        idx = torch.full((2,), -9, dtype=torch.int64, device="cuda")
        oe = torch.full((1,), -9.0, dtype=torch.float64, device="cuda")
        if static:
            emo.emo_select_static(len(T), Td, Ed, target, idx[0:1], idx[1:2], oe)
        else:
            emo.emo_select(len(T), Td, Ed, target, idx[0:1], idx[1:2], oe, ws)
        torch.cuda.synchronize()
        out.append((int(idx[0].item()), int(idx[1].item()), float(oe.item())))
    return out


def test_static_selection_matches_workspace_selection():
    import torch
    import oracle
    from paper_2607_12324_b200 import build, emo
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)
    build.build()
    rs = np.random.RandomState(5)
    # two calls in a row with different sizes: the second must not see the first call's leftovers
    for B in (300_000, 777, 1, 70_001):
        T = rs.randint(50, 150, B).astype(np.int64)
        E = np.round(rs.rand(B) * 40) / 8.0                  # many exact ties
        for target in (49, 75, 149):
            ref, got = _select_both(torch, emo, T, E, target)
            assert got[0] == ref[0] and got[1] == ref[1]
            assert got[2] == ref[2]                          # same reduction, same bits
            want = oracle.select(T, E, target)               # and directly against the CPU oracle
            assert got[0] == want
            if want >= 0:
                assert got[1] == T[want] and got[2] == E[want]
    # target read on the device, as after a baseline evaluation
    T = rs.randint(1000, 2000, 5000).astype(np.int64)
    E = rs.rand(5000)
    Td = torch.as_tensor(T, device="cuda")
    Ed = torch.as_tensor(E, device="cuda")
    T0 = torch.tensor([1500], dtype=torch.int64, device="cuda")
    a = torch.zeros(1, dtype=torch.int64, device="cuda")
    b = torch.zeros(1, dtype=torch.int64, device="cuda")
    ws = torch.empty(65536, dtype=torch.uint8, device="cuda")
    emo.emo_select(5000, Td, Ed, 0, a, None, None, ws, target_dev=T0, delta_ppm=50_000)
    emo.emo_select_static(5000, Td, Ed, 0, b, target_dev=T0, delta_ppm=50_000)
    torch.cuda.synchronize()
    assert int(a.item()) == int(b.item()) == oracle.select(T, E, oracle.target_from_delta(1500, 50_000)) >= 0
    # beyond the stated maximum: refused, nothing launched
    with pytest.raises(emo.EmoError) as ei:
        emo.emo_select_static(emo.EMO_SELECT_STATIC_MAX_B + 1, Td, Ed, 0, b)
    assert ei.value.code == emo.EMO_E_RANGE
