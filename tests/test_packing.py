"""The library's kernel packing (emo_pack_greedy, emo_pack_tables; host code) against the oracle's."""
from __future__ import annotations

import time

import numpy as np
import pytest

from paper_2607_12324_b200 import workloads as W
from tests.test_oracle_packing import stream_ids


@pytest.fixture(scope="module")
def emo():
    from paper_2607_12324_b200 import build, emo as E
    build.build()
    return E


@pytest.mark.parametrize("name,scale", [("cfg0-tiny", 1.0), ("cfg1-train", 1.0), ("cfg3-8dev", 0.1), ("cfg4-llm", 0.1)])
def test_packing_matches_the_oracle(emo, oracle_mod, name, scale):
    g = W.make_graph(name, scale)
    is_kernel = (g.kind == W.KIND_KERNEL).astype(np.uint8)
    stream_of = stream_ids(g)
    t = g.lat[:, g.L - 1].copy()
    C, crit_o = oracle_mod.crit_pred(g, t)
    for delta_max in (1, 50_000, 5_000_000, 10 ** 12):
        po_o, cnt_o = oracle_mod.pack_greedy(g, is_kernel, stream_of, t, crit_o, delta_max)
        crit, po, cnt = emo.emo_pack_greedy(g.n, g.row_ptr, g.col, is_kernel, stream_of, t, delta_max)
        assert np.array_equal(crit, crit_o)
        assert cnt == cnt_o and np.array_equal(po, po_o)
    pl, pe = emo.emo_pack_tables(g.lat, g.energy, po, cnt)
    for p in (0, cnt // 2, cnt - 1):
        mem = np.flatnonzero(po == p)
        assert np.array_equal(pl[p], g.lat[mem].sum(axis=0))
        assert np.allclose(pe[p], g.energy[mem].sum(axis=0), rtol=1e-12)
    assert int(pl.sum()) == int(g.lat[is_kernel == 1].sum())


def test_packing_on_ties_and_random_streams(emo, oracle_mod):
    rs = np.random.RandomState(2)
    for seed in range(8):
        g = W.random_dag(seed, 60, 0.08, L=2, max_dur=4)
        is_kernel = (rs.rand(g.n) < 0.8).astype(np.uint8)
        stream_of = np.where(is_kernel == 1, rs.randint(0, 3, size=g.n), -1).astype(np.int32)
        t = g.lat[:, 1].copy()
        C, crit_o = oracle_mod.crit_pred(g, t)
        for delta_max in (3, 9, 1000):
            po_o, cnt_o = oracle_mod.pack_greedy(g, is_kernel, stream_of, t, crit_o, delta_max)
            crit, po, cnt = emo.emo_pack_greedy(g.n, g.row_ptr, g.col, is_kernel, stream_of, t, delta_max)
            assert np.array_equal(crit, crit_o) and cnt == cnt_o and np.array_equal(po, po_o)


def test_packing_errors_and_speed(emo):
    g = W.make_graph("cfg1-train", 0.1)
    is_kernel = (g.kind == W.KIND_KERNEL).astype(np.uint8)
    stream_of = stream_ids(g)
    t = g.lat[:, g.L - 1].copy()
    bad = g.col.copy()
    bad[0] = g.n - 1
    with pytest.raises(Exception):
        emo.emo_pack_greedy(g.n, g.row_ptr, bad, is_kernel, stream_of, t, 5_000_000)
    with pytest.raises(Exception):
        emo.emo_pack_greedy(g.n, g.row_ptr, g.col, is_kernel, stream_of, -t, 5_000_000)
    crit, po, cnt = emo.emo_pack_greedy(0, np.zeros(1, np.int64), np.zeros(0, np.int32), np.zeros(0, np.uint8), np.zeros(0, np.int32),
                                        np.zeros(0, np.int64), 5)
    assert cnt == 0


@pytest.mark.gpu
def test_per_pack_policies_on_the_gpu(emo, oracle_mod):
    """The packs as policy rows of the kernel-level graph: one level per pack and policy (Alg. 1 'v is a pack')."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("needs a GPU")
    g = W.make_graph("cfg1-train", 0.3)
    is_kernel = (g.kind == W.KIND_KERNEL).astype(np.uint8)
    t = g.lat[:, g.L - 1].copy()
    crit, po, cnt = emo.emo_pack_greedy(g.n, g.row_ptr, g.col, is_kernel, stream_ids(g), t, 5_000_000)
    assert 0 < cnt < int(is_kernel.sum())
    B = 96
    lv = W.policy_levels(77, cnt, g.L, B, "mixed").numpy()
    h = emo.load_workload(g, group_of=po)
    ld = 96
    lvd = torch.from_numpy(lv).cuda().contiguous()
    T = torch.zeros(B, dtype=torch.int64, device="cuda")
    E = torch.zeros(B, dtype=torch.float64, device="cuda")
    ws = torch.empty(emo.emo_workspace_bytes(h, B, 0), dtype=torch.uint8, device="cuda")
    emo.emo_eval_policies(h, B, lvd, ld, T, E, ws)
    torch.cuda.synchronize()
    r = oracle_mod.batch(g, lv, group_of=po)
    assert np.array_equal(T.cpu().numpy(), r["makespan"])
    assert np.allclose(E.cpu().numpy(), r["energy"], rtol=1e-9, atol=0)
    h.free()


def test_pack_classes_group_equal_name_sequences(emo):
    """Sec. 4.4: packs with the same sequence of kernel names are profiled once.  Checked against the definition
    (a dictionary keyed by the tuple of names), on a workload whose streams repeat their kernels layer by layer."""
    g = W.make_graph("cfg1-train", 1.0)
    is_kernel = (g.kind == W.KIND_KERNEL).astype(np.uint8)
    t = g.lat[:, g.L - 1].copy()
    names = W.kernel_names(g, period=12)
    crit, po, cnt = emo.emo_pack_greedy(g.n, g.row_ptr, g.col, is_kernel, stream_ids(g), t, 300_000)
    cls, ncls = emo.emo_pack_classes(po, names, cnt)
    seen, want = {}, []
    for p in range(cnt):
        key = tuple(names[np.flatnonzero(po == p)].tolist())
        want.append(seen.setdefault(key, len(seen)))
    assert cls.tolist() == want and ncls == len(seen)
    assert 0 < ncls <= cnt
    # permuting the names of one pack changes its class
    names2 = names.copy()
    mem = np.flatnonzero(po == cnt // 2)
    names2[mem[0]] = 999_999
    cls2, _ = emo.emo_pack_classes(po, names2, cnt)
    assert cls2[cnt // 2] not in cls2[: cnt // 2].tolist()
