"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded
inputs.  Integer results (ES, LS, slack, makespan, slack sums, critical counts, selected index) must
be bit-exact; energies within 1e-9 relative."""
from __future__ import annotations

import json
import os

import numpy as np
import pytest

from paper_2607_12324_b200 import workloads as W

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))
E_RTOL = 1e-9


@pytest.fixture(scope="module")
def torch_cuda():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    torch.cuda.set_device(0)
    return torch


@pytest.fixture(scope="module")
def emo(torch_cuda):
    from paper_2607_12324_b200 import build, emo as E
    build.build()
    return E


@pytest.fixture(scope="module")
def golden():
    with open(os.path.join(HERE, "golden", "config_golden.json")) as f:
        return json.load(f)


def gpu_slack_batch(torch, emo, h, lv_dev, B, n, want=("ES", "LS", "slack"), flags=0, ldo=None, sums=True,
                    base=False):
    dev = lv_dev.device
    ldo = int(ldo or max(B, 1))
    out = {k: (torch.full((n, ldo), -7, dtype=torch.int64, device=dev) if k in want else None)
           for k in ("ES", "LS", "slack")}
    T = torch.full((max(B, 1),), -1, dtype=torch.int64, device=dev)
    E = torch.full((max(B, 1),), -1.0, dtype=torch.float64, device=dev)
    ss = torch.full((max(B, 1),), -1, dtype=torch.int64, device=dev)
    nc = torch.full((max(B, 1),), -1, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    aligned = lv_dev.stride(0) % 16 == 0 and lv_dev.data_ptr() % 16 == 0
    ws = torch.empty(emo.emo_workspace_bytes(h, B, 1, flags, aligned), dtype=torch.uint8, device=dev)
    T0 = torch.full((1,), -1, dtype=torch.int64, device=dev) if base else None
    E0 = torch.full((1,), -1.0, dtype=torch.float64, device=dev) if base else None
    emo.emo_slack_batch(h, B, lv_dev, lv_dev.stride(0), out["ES"], out["LS"], out["slack"], ldo, T, E,
                        ss if sums else None, nc if sums else None, ws, status, flags, T0=T0, E0=E0)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    res = {k: v.cpu().numpy() for k, v in out.items() if v is not None}
    if base:
        res["T0"], res["E0"] = int(T0.item()), float(E0.item())
    res.update(makespan=T.cpu().numpy()[:B], energy=E.cpu().numpy()[:B], slack_sum=ss.cpu().numpy()[:B],
               n_critical=nc.cpu().numpy()[:B])
    return res


def gpu_eval(torch, emo, h, lv_dev, B, flags=0):
    dev = lv_dev.device
    T = torch.full((max(B, 1),), -1, dtype=torch.int64, device=dev)
    E = torch.full((max(B, 1),), -1.0, dtype=torch.float64, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = torch.empty(emo.emo_workspace_bytes(h, B, 0), dtype=torch.uint8, device=dev)
    emo.emo_eval_policies(h, B, lv_dev, lv_dev.stride(0), T, E, ws, status, flags)
    torch.cuda.synchronize()
    return T.cpu().numpy()[:B], E.cpu().numpy()[:B], int(status.item())


def gpu_select(torch, emo, T, E, target=0, target_dev=None, delta_ppm=0):
    dev = "cuda"
    Td = torch.as_tensor(T, dtype=torch.int64, device=dev)
    Ed = torch.as_tensor(E, dtype=torch.float64, device=dev)
    out = torch.full((3,), -5, dtype=torch.int64, device=dev)
    oe = torch.zeros(1, dtype=torch.float64, device=dev)
    ws = torch.empty(65536, dtype=torch.uint8, device=dev)
    emo.emo_select(len(T), Td, Ed, target, out[0:1], out[1:2], oe, ws, target_dev, delta_ppm)
    torch.cuda.synchronize()
    return int(out[0].item()), int(out[1].item()), float(oe.item())


def assert_matches(r_gpu, r_or, B, arrays=True):
    assert np.array_equal(r_gpu["makespan"], r_or["makespan"])
    np.testing.assert_allclose(r_gpu["energy"], r_or["energy"], rtol=E_RTOL, atol=0)
    assert np.array_equal(r_gpu["slack_sum"], r_or["slack_sum"])
    assert np.array_equal(r_gpu["n_critical"], r_or["n_critical"])
    if arrays:
        for k in ("ES", "LS", "slack"):
            if k in r_gpu:
                assert np.array_equal(r_gpu[k][:, :B], r_or[k]), k


# ------------------------------------------------------------------------------------------------
def test_tiny_graphs_all_outputs(torch_cuda, emo, oracle_mod):
    """Hand-made and random tiny DAGs (ties, zero durations, duplicate edges, isolated nodes,
    non-monotone rows), every policy, all outputs, several lane counts and a ragged ld."""
    from tests.test_oracle_pins import TINY, all_policies
    torch = torch_cuda
    for gi in range(0, len(TINY), 2):
        g = TINY[gi]
        lv = all_policies(g.n, g.L)
        B = lv.shape[1]
        r_or = oracle_mod.batch(g, lv, want_arrays=True)
        ldb = B + 5 if (B + 5) % 16 else B + 6      # a pitch that rules out 16-byte pieces
        lvp = np.full((g.n, ldb), 0xFF, dtype=np.uint8)
        lvp[:, :B] = lv
        lv_dev = torch.as_tensor(lvp, device="cuda")
        # the same levels at a pitch of whole 16-byte pieces: what the staged kernels need
        ldb16 = (B + 15) // 16 * 16 + 16
        lvq = np.full((g.n, ldb16), 0xFF, dtype=np.uint8)
        lvq[:, :B] = lv
        lv16 = torch.as_tensor(lvq, device="cuda")
        for lanes in (0, 1, 2):
            h = emo.load_workload(g, emo.EMO_F_LANES(lanes))
            assert emo.emo_call_path(h, B, lv_dev, ldb, B + 3, True, 0) == 0, "an odd pitch takes the plain-load kernels"
            assert emo.emo_call_path(h, B, lv16, ldb16, B + 3, True, emo.EMO_F_FLOW_KERNEL) == 2
            for lvx, fl in ((lv_dev, 0), (lv16, emo.EMO_F_PAIR_KERNEL), (lv16, emo.EMO_F_LANE_KERNEL), (lv16, emo.EMO_F_FLOW_KERNEL)):
                r = gpu_slack_batch(torch, emo, h, lvx, B, g.n, ldo=B + 3, flags=fl)
                assert_matches(r, r_or, B)
                for k in ("ES", "LS", "slack"):
                    assert (r[k][:, B:] == -7).all(), "padding columns of the outputs were written"
            T, E, st = gpu_eval(torch, emo, h, lv16, B, emo.EMO_F_VALIDATE | emo.EMO_F_FLOW_KERNEL)
            assert st == 0 and np.array_equal(T, r_or["makespan"])
            np.testing.assert_allclose(E, r_or["energy"], rtol=E_RTOL)
            T, E, st = gpu_eval(torch, emo, h, lv_dev, B, emo.EMO_F_VALIDATE)
            assert st == 0 and np.array_equal(T, r_or["makespan"])
            np.testing.assert_allclose(E, r_or["energy"], rtol=E_RTOL)
            h.free()


def test_hand_worked_example_on_gpu(torch_cuda, emo):
    torch = torch_cuda
    with open(os.path.join(HERE, "golden", "hand_worked_dag.json")) as f:
        gold = json.load(f)
    n = len(gold["nodes"])
    g = W.tiny_graph(n, gold["edges_pred_succ"], gold["lat"], gold["energy"])
    lv = np.array([p["levels"] for p in gold["policies"]], dtype=np.uint8).T.copy()
    h = emo.load_workload(g)
    r = gpu_slack_batch(torch, emo, h, torch.as_tensor(lv, device="cuda"), 2, n)
    for b, p in enumerate(gold["policies"]):
        assert r["makespan"][b] == p["T"] and r["energy"][b] == p["E"]
        assert r["ES"][:, b].tolist() == p["ES"] and r["LS"][:, b].tolist() == p["LS"]
        assert r["slack"][:, b].tolist() == p["slack"]
    for s in gold["selection"]:
        assert emo.emo_target_from_delta(gold["policies"][0]["T"], s["delta_ppm"]) == s["target"]
        assert gpu_select(torch, emo, r["makespan"], r["energy"], s["target"])[0] == s["index"]
    h.free()


@pytest.mark.parametrize("name,scale,B", [("cfg0-tiny", 1.0, 64), ("cfg1-train", 0.25, 333), ("cfg2-packed", 0.5, 1000),
                                            ("cfg3-8dev", 0.03, 200), ("cfg4-llm", 0.02, 257)])
def test_config_graphs_all_outputs(torch_cuda, emo, oracle_mod, name, scale, B):
    """Scaled configuration graphs: several policy tiles and a ragged tail, all per-node outputs."""
    torch = torch_cuda
    g = W.make_graph(name, scale)
    lv_dev = W.policies_for(g, B=B, device="cuda")
    lv = lv_dev.cpu().numpy()
    r_or = oracle_mod.batch(g, lv, B=B, want_arrays=True, threads=os.cpu_count() or 1)
    h = emo.load_workload(g)
    r = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n)
    assert_matches(r, r_or, B)
    # slack only (ES kept in the workspace), same result; then the plain-load kernels
    r2 = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n, want=("slack",))
    assert np.array_equal(r2["slack"][:, :B], r_or["slack"])
    base = oracle_mod.batch(g, np.full((g.n, 1), g.L - 1, dtype=np.uint8))
    # every pass kernel: plain loads, two policies per thread, one policy per thread, 32-bit lane streams
    assert emo.emo_call_path(h, B, lv_dev, lv_dev.stride(0), B, True, emo.EMO_F_FLOW_KERNEL) == 2
    for fl in (emo.EMO_F_NO_STAGING, emo.EMO_F_PAIR_KERNEL, emo.EMO_F_LANE_KERNEL, emo.EMO_F_FLOW_KERNEL):
        r3 = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n, flags=fl, base=True)
        assert_matches(r3, r_or, B)
        assert r3["T0"] == base["makespan"][0]
        assert r3["E0"] == pytest.approx(base["energy"][0], rel=E_RTOL)
    # without the per-policy sums (the configuration the bench times)
    for fl in (0, emo.EMO_F_FLOW_KERNEL):
        r5 = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n, want=("slack",), sums=False, base=True, flags=fl)
        assert np.array_equal(r5["slack"][:, :B], r_or["slack"]) and r5["T0"] == base["makespan"][0]
        assert (r5["slack_sum"] == -1).all()
    T, E, st = gpu_eval(torch, emo, h, lv_dev, B, emo.EMO_F_FLOW_KERNEL)
    assert st == 0 and np.array_equal(T, r_or["makespan"])
    np.testing.assert_allclose(E, r_or["energy"], rtol=E_RTOL)
    # an output pitch that is odd (no 16-byte stores of policy pairs possible) and one that is even
    for ldo in (B + 1, B + 2):
        for fl in (emo.EMO_F_PAIR_KERNEL, emo.EMO_F_LANE_KERNEL, emo.EMO_F_FLOW_KERNEL):
            r4 = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n, ldo=ldo, flags=fl)
            assert_matches(r4, r_or, B)
    # single-policy call
    b = B // 2
    one = lv_dev[:, b].contiguous()
    ES, LS, SL = (torch.zeros(g.n, dtype=torch.int64, device="cuda") for _ in range(3))
    T1 = torch.zeros(1, dtype=torch.int64, device="cuda")
    E1 = torch.zeros(1, dtype=torch.float64, device="cuda")
    ws = torch.empty(emo.emo_workspace_bytes(h, 1, 1), dtype=torch.uint8, device="cuda")
    emo.emo_slack(h, one, ES, LS, SL, T1, E1, ws)
    torch.cuda.synchronize()
    assert int(T1.item()) == r_or["makespan"][b]
    assert np.array_equal(ES.cpu().numpy(), r_or["ES"][:, b])
    assert np.array_equal(LS.cpu().numpy(), r_or["LS"][:, b])
    assert np.array_equal(SL.cpu().numpy(), r_or["slack"][:, b])
    h.free()


@pytest.mark.parametrize("name", ["cfg0-tiny", "cfg1-train", "cfg2-packed", "cfg3-8dev"])
def test_full_configs_against_oracle_and_golden(torch_cuda, emo, oracle_mod, golden, name):
    """Full-size configurations 0-3: every policy's makespan, energy, slack sum and critical count
    against the oracle run here, per-node arrays on a sample of policies, baseline and selection
    against the oracle and against the stored oracle results."""
    torch = torch_cuda
    g = W.make_graph(name)
    B = g.meta["B"]
    gold = golden[name]
    assert (g.n, g.m, B) == (gold["n"], gold["m"], gold["B"])
    lv_dev = W.policies_for(g, device="cuda")
    h = emo.load_workload(g)
    want = ("slack",)
    r = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n, want=want)
    lv = lv_dev.cpu().numpy()
    r_or = oracle_mod.batch(g, lv, B=B, want_slack=True, threads=os.cpu_count() or 1)
    assert_matches(r, r_or, B, arrays=False)
    cols = sorted(set(np.linspace(0, B - 1, 12).astype(int).tolist()))
    sub = np.ascontiguousarray(lv[:, cols])
    r_sub = oracle_mod.batch(g, sub, want_arrays=True)
    assert np.array_equal(r["slack"][:, cols], r_sub["slack"])
    # stored oracle values
    assert [int(r["makespan"][i]) for i in gold["sample_idx"]] == gold["sample_makespan"]
    np.testing.assert_allclose([r["energy"][i] for i in gold["sample_idx"]], gold["sample_energy"], rtol=E_RTOL)
    # baseline (all rows at level L-1) and selection
    T0 = torch.zeros(1, dtype=torch.int64, device="cuda")
    E0 = torch.zeros(1, dtype=torch.float64, device="cuda")
    ws = torch.empty(emo.emo_workspace_bytes(h, B, 0), dtype=torch.uint8, device="cuda")
    emo.emo_baseline(h, T0, E0, ws)
    torch.cuda.synchronize()
    assert int(T0.item()) == gold["T0"]
    assert float(E0.item()) == pytest.approx(gold["E0"], rel=E_RTOL)
    for s in gold["select"]:
        tgt = emo.emo_target_from_delta(int(T0.item()), s["delta_ppm"])
        assert tgt == s["target"] == oracle_mod.target_from_delta(gold["T0"], s["delta_ppm"])
        want_idx = oracle_mod.select(r_or["makespan"], r_or["energy"], tgt)
        assert want_idx == s["index"]
        assert s["margin_rel"] is None or s["margin_rel"] > 2e-9, "selection is ambiguous at the energy tolerance"
        idx, Tsel, Esel = gpu_select(torch, emo, r["makespan"], r["energy"], tgt)
        assert idx == want_idx and Tsel == s["T"]
        assert Esel == pytest.approx(s["E"], rel=E_RTOL)
        idx2, _, _ = gpu_select(torch, emo, r["makespan"], r["energy"], 0, target_dev=T0, delta_ppm=s["delta_ppm"])
        assert idx2 == want_idx
    h.free()


def test_cfg4_full_size_sampled(torch_cuda, emo, oracle_mod, golden):
    """The largest configuration at full size, in the launch configuration the bench times: all
    16 384 policies on the GPU with slack materialised; the oracle checks sampled policies node by
    node, and the stored oracle results check every policy's makespan / slack sum / critical
    count (digests) and the selection."""
    torch = torch_cuda
    import hashlib
    name = "cfg4-llm"
    gold = golden.get(name)
    g = W.make_graph(name)
    B = g.meta["B"]
    lv_dev = W.policies_for(g, device="cuda")
    h = emo.load_workload(g)
    r = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n, want=(), base=True)
    cols = sorted(set(np.linspace(0, B - 1, 16).astype(int).tolist() + [1, 2, B // 2 - 1, B // 2]))
    sub = lv_dev[:, cols].contiguous().cpu().numpy()
    r_sub = oracle_mod.batch(g, sub, want_arrays=True, threads=os.cpu_count() or 1)
    assert np.array_equal(r["makespan"][cols], r_sub["makespan"])
    np.testing.assert_allclose(r["energy"][cols], r_sub["energy"], rtol=E_RTOL)
    assert np.array_equal(r["slack_sum"][cols], r_sub["slack_sum"])
    assert np.array_equal(r["n_critical"][cols], r_sub["n_critical"])
    # per-node slack of the sampled policies: run them as their own small batch with arrays
    sub_dev = torch.as_tensor(sub, device="cuda")
    r2 = gpu_slack_batch(torch, emo, h, sub_dev, len(cols), g.n)
    assert_matches(r2, r_sub, len(cols))
    # the bench's configuration: slack materialised, no per-policy sums, baseline in the same launch
    slack = torch.empty((g.n, B), dtype=torch.int64, device="cuda")
    T = torch.zeros(B, dtype=torch.int64, device="cuda")
    E = torch.zeros(B, dtype=torch.float64, device="cuda")
    T0 = torch.zeros(1, dtype=torch.int64, device="cuda")
    E0 = torch.zeros(1, dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(emo.emo_workspace_bytes(h, B, 1), dtype=torch.uint8, device="cuda")
    assert emo.emo_call_path(h, B, lv_dev, lv_dev.stride(0), B, True, 0) in (2, 5), "the largest workload takes the 32-bit kernels"
    emo.emo_slack_batch(h, B, lv_dev, lv_dev.stride(0), None, None, slack, B, T, E, None, None, ws, status, T0=T0, E0=E0)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(T.cpu().numpy(), r["makespan"])
    # a contiguous slab of 256 policies, element by element: the last two policy tiles (the last one shares
    # its launch with the block of the baseline column)
    slab0 = B - 256
    slab = lv_dev[:, slab0:B].contiguous().cpu().numpy()
    r_slab = oracle_mod.batch(g, slab, want_arrays=True, threads=os.cpu_count() or 1)
    assert np.array_equal(slack[:, slab0:B].cpu().numpy(), r_slab["slack"])
    assert np.array_equal(T.cpu().numpy()[slab0:B], r_slab["makespan"])
    del r_slab, slab
    assert np.array_equal(slack[:, torch.as_tensor(cols, device="cuda")].cpu().numpy(), r_sub["slack"])
    assert np.array_equal(slack.sum(dim=0).cpu().numpy(), r["slack_sum"])
    assert np.array_equal((slack == 0).sum(dim=0).cpu().numpy(), r["n_critical"])
    assert int(T0.item()) == r["T0"]
    del slack, ws
    if gold is not None:
        assert r["T0"] == gold["T0"] and r["E0"] == pytest.approx(gold["E0"], rel=E_RTOL)
        assert (g.n, g.m, B) == (gold["n"], gold["m"], gold["B"])
        assert hashlib.sha256(np.ascontiguousarray(r["makespan"]).tobytes()).hexdigest() == gold["makespan_sha256"]
        assert hashlib.sha256(np.ascontiguousarray(r["slack_sum"]).tobytes()).hexdigest() == gold["slack_sum_sha256"]
        assert hashlib.sha256(np.ascontiguousarray(r["n_critical"]).tobytes()).hexdigest() == gold["n_critical_sha256"]
        np.testing.assert_allclose([r["energy"][i] for i in gold["sample_idx"]], gold["sample_energy"], rtol=E_RTOL)
        for s in gold["select"]:
            assert s["margin_rel"] > 2e-9
            idx, Tsel, Esel = gpu_select(torch, emo, r["makespan"], r["energy"], s["target"])
            assert idx == s["index"] and Tsel == s["T"]
            assert Esel == pytest.approx(s["E"], rel=E_RTOL)
    h.free()


def test_selection_cases(torch_cuda, emo, oracle_mod):
    torch = torch_cuda
    T = np.array([100, 105, 103, 103, 99, 110], dtype=np.int64)
    E = np.array([9.0, 5.0, 7.0, 7.0, 9.5, 1.0])
    for tgt in (98, 99, 100, 102, 103, 104, 105, 109, 110, 1000):
        assert gpu_select(torch, emo, T, E, tgt)[0] == oracle_mod.select(T, E, tgt)
    assert gpu_select(torch, emo, T, E, 98)[0] == -1
    assert gpu_select(torch, emo, T[:1], E[:1], 100)[0] == 0
    e2 = np.array([1.0, np.nextafter(1.0, 0.0), 1.0])
    assert gpu_select(torch, emo, np.ones(3, dtype=np.int64), e2, 1)[0] == 1
    rs = np.random.RandomState(0)
    for B in (1, 31, 32, 33, 1000, 4097, 70001):
        T = rs.randint(50, 150, B).astype(np.int64)
        E = np.round(rs.rand(B) * 20) / 4.0          # many exact ties
        for tgt in (49, 60, 100, 149):
            idx, Ts, Es = gpu_select(torch, emo, T, E, tgt)
            want = oracle_mod.select(T, E, tgt)
            assert idx == want
            if want >= 0:
                assert Ts == T[want] and Es == E[want]


def test_batch_edge_cases(torch_cuda, emo, oracle_mod):
    """B = 0, B = 1, a level out of range with validation on, a graph without nodes, transpose."""
    torch = torch_cuda
    g = W.make_graph("cfg0-tiny")
    h = emo.load_workload(g)
    lv_dev = W.policies_for(g, B=40, device="cuda")
    T = torch.full((4,), -1, dtype=torch.int64, device="cuda")
    E = torch.full((4,), -1.0, dtype=torch.float64, device="cuda")
    emo.emo_eval_policies(h, 0, lv_dev, lv_dev.stride(0), T, E, None, None, 0)
    torch.cuda.synchronize()
    assert (T == -1).all()
    Tg, Eg, st = gpu_eval(torch, emo, h, lv_dev, 1)
    r = oracle_mod.batch(g, lv_dev.cpu().numpy(), B=1)
    assert Tg[0] == r["makespan"][0] and st == 0
    # padding columns hold 0xFF: asking for them with validation reports EMO_E_RANGE
    Tg, Eg, st = gpu_eval(torch, emo, h, lv_dev, 44, emo.EMO_F_VALIDATE)
    assert st == emo.EMO_E_RANGE
    Tg, Eg, st = gpu_eval(torch, emo, h, lv_dev, 40, emo.EMO_F_VALIDATE)
    assert st == 0
    with pytest.raises(emo.EmoError):
        emo.emo_eval_policies(h, 50, lv_dev, 40, T, E, None, None, 0)          # ldb < B
    # transpose helper
    src = torch.randint(0, g.L, (37, g.n), dtype=torch.uint8, device="cuda")
    dst = torch.zeros((g.n, 48), dtype=torch.uint8, device="cuda")
    emo.emo_transpose_policies(37, g.n, src, g.n, dst, 48)
    torch.cuda.synchronize()
    assert torch.equal(dst[:, :37], src.t())
    h.free()
    h0 = emo.emo_graph_load(0, np.zeros(1, np.int64), np.zeros(0, np.int32), None, 3, np.zeros((0, 3), np.int64),
                            np.zeros((0, 3)))
    lv0 = torch.zeros((1, 16), dtype=torch.uint8, device="cuda")
    Tg, Eg, st = gpu_eval(torch, emo, h0, lv0, 5)
    assert (Tg == 0).all() and (Eg == 0).all()
    h0.free()


def test_many_levels(torch_cuda, emo, oracle_mod):
    """200 frequency levels (table rows of 256 entries, far wider than the 32 shared-memory banks),
    non-monotone rows, a ragged batch; every pass kernel."""
    torch = torch_cuda
    L, n, B = 200, 60, 77
    rs = np.random.RandomState(11)
    edges = [(i, j) for i in range(n) for j in range(i + 1, min(n, i + 6)) if rs.rand() < 0.4]
    lat = rs.randint(0, 5000, (n, L)).astype(np.int64)
    en = rs.rand(n, L) * 3.0
    g = W.tiny_graph(n, edges, lat, en)
    lv = rs.randint(0, L, (n, B)).astype(np.uint8)
    r_or = oracle_mod.batch(g, lv, want_arrays=True)
    ldb = 96
    lvp = np.full((n, ldb), 0xFF, dtype=np.uint8)
    lvp[:, :B] = lv
    lv_dev = torch.as_tensor(lvp, device="cuda")
    h = emo.load_workload(g)
    for fl in (emo.EMO_F_NO_STAGING, emo.EMO_F_PAIR_KERNEL, emo.EMO_F_LANE_KERNEL, emo.EMO_F_FLOW_KERNEL, 0):
        r = gpu_slack_batch(torch, emo, h, lv_dev, B, n, flags=fl, base=True)
        assert_matches(r, r_or, B)
    h.free()


def test_group_of_on_gpu(torch_cuda, emo, oracle_mod):
    torch = torch_cuda
    g = W.make_graph("cfg1-train", 0.1)
    group = (np.arange(g.n) // 4).astype(np.int32)
    group[g.kind == W.KIND_CPU] = -1
    rows = int(group.max()) + 1
    B = 70
    lv = np.random.RandomState(3).randint(0, g.L, (rows, B)).astype(np.uint8)
    r_or = oracle_mod.batch(g, lv, want_arrays=True, group_of=group)
    h = emo.load_workload(g, group_of=group)
    lvp = np.zeros((rows, 80), dtype=np.uint8)
    lvp[:, :B] = lv
    for fl in (0, emo.EMO_F_FLOW_KERNEL):
        r = gpu_slack_batch(torch, emo, h, torch.as_tensor(lvp, device="cuda"), B, g.n, flags=fl)
        assert_matches(r, r_or, B)
    h.free()


def test_host_buffer_call(torch_cuda, emo, oracle_mod):
    """emo_slack_batch_host: levels from pinned host memory, per-policy results back to the host."""
    torch = torch_cuda
    g = W.make_graph("cfg1-train", 0.2)
    B, ppm = 500, 30_000
    lv = W.policies_for(g, B=B, device="cpu").pin_memory()
    ldb = lv.stride(0)
    h = emo.load_workload(g)
    dev_lvl = torch.empty((g.n, ldb), dtype=torch.uint8, device="cuda")
    slack = torch.zeros((g.n, B), dtype=torch.int64, device="cuda")
    T = torch.zeros(B, dtype=torch.int64).pin_memory()
    E = torch.zeros(B, dtype=torch.float64).pin_memory()
    ss = torch.zeros(B, dtype=torch.int64).pin_memory()
    nc = torch.zeros(B, dtype=torch.int32).pin_memory()
    sel = torch.zeros(4, dtype=torch.int64)
    ws = torch.empty(emo.emo_workspace_bytes(h, B, 2), dtype=torch.uint8, device="cuda")
    for _ in range(2):
        emo.emo_slack_batch_host(h, B, lv, ldb, dev_lvl, slack, B, ppm, T, E, ss, nc, sel, ws)
    r_or = oracle_mod.batch(g, lv.numpy(), B=B, want_arrays=True)
    assert np.array_equal(T.numpy(), r_or["makespan"])
    np.testing.assert_allclose(E.numpy(), r_or["energy"], rtol=E_RTOL)
    assert np.array_equal(ss.numpy(), r_or["slack_sum"]) and np.array_equal(nc.numpy(), r_or["n_critical"])
    assert np.array_equal(slack.cpu().numpy(), r_or["slack"])
    allmax = np.full((g.n, 1), g.L - 1, dtype=np.uint8)
    T0 = int(oracle_mod.batch(g, allmax)["makespan"][0])
    assert int(sel[3]) == T0
    want = oracle_mod.select(r_or["makespan"], r_or["energy"], oracle_mod.target_from_delta(T0, ppm))
    assert int(sel[0]) == want and int(sel[1]) == r_or["makespan"][want]
    assert np.array([int(sel[2])], dtype=np.int64).view(np.float64)[0] == pytest.approx(r_or["energy"][want], rel=E_RTOL)
    # the same call with the levels packed at 4 bits (16 levels): pack on the device, round trip, then the call
    bits = 4
    ldp = ((B + 7) // 8 * bits + 15) // 16 * 16
    lv_dev = lv.cuda()
    packed = torch.zeros((g.n, ldp), dtype=torch.uint8, device="cuda")
    emo.emo_pack_levels(bits, g.n, B, lv_dev, ldb, packed, ldp)
    back = torch.full_like(lv_dev, 0xEE)
    emo.emo_unpack_levels(bits, g.n, B, packed, ldp, back, ldb)
    torch.cuda.synchronize()
    assert torch.equal(back[:, :B], lv_dev[:, :B])
    pk = packed.cpu().numpy()
    lvn = lv.numpy()
    assert pk[3, 0] == (int(lvn[3, 0]) | (int(lvn[3, 1]) << 4)), "two 4-bit levels per byte, the first in the low bits"
    packed_host = packed.cpu().pin_memory()
    slack.zero_()
    T.zero_()
    for fl in (0, emo.EMO_F_FLOW_KERNEL):
        ws2 = torch.empty(emo.emo_workspace_bytes(h, B, 2, fl), dtype=torch.uint8, device="cuda")
        emo.emo_slack_batch_host_packed(h, B, bits, packed_host, ldp, packed, dev_lvl, ldb, slack, B, ppm, T, E, ss, nc, sel, ws2, flags=fl)
        assert np.array_equal(T.numpy(), r_or["makespan"]) and int(sel[0]) == want
        assert np.array_equal(slack.cpu().numpy(), r_or["slack"])
    # the two-buffer form: the copy of the next batch is enqueued on a stream of its own before the current batch
    # is evaluated; three batches (the same levels, then a second set, then the first again) through two buffers
    lv2 = lv.clone()
    lv2[:, :B] = (g.L - 1) - lv[:, :B]          # a second set of policies: every level mirrored
    sets = [(lv, r_or), (lv2, oracle_mod.batch(g, lv2.numpy(), B=B, want_arrays=True))]
    hosts = []
    for lvx, _ in sets:
        pkx = torch.zeros((g.n, ldp), dtype=torch.uint8, device="cuda")
        emo.emo_pack_levels(bits, g.n, B, lvx.cuda(), ldb, pkx, ldp)
        hosts.append(pkx.cpu().pin_memory())
    bufs = (torch.zeros((g.n, ldp), dtype=torch.uint8, device="cuda"), torch.zeros((g.n, ldp), dtype=torch.uint8, device="cuda"))
    copy_stream = torch.cuda.Stream()
    ready = (torch.cuda.Event(), torch.cuda.Event())
    order = [0, len(sets) - 1, 0]
    emo.emo_levels_prefetch(h, hosts[order[0]], ldp, bufs[0], copy_stream, ready[0])
    for s_, which in enumerate(order):
        if s_ + 1 < len(order):
            emo.emo_levels_prefetch(h, hosts[order[s_ + 1]], ldp, bufs[(s_ + 1) & 1], copy_stream, ready[(s_ + 1) & 1])
        T.zero_()
        slack.zero_()
        emo.emo_slack_batch_prefetched(h, B, bits, bufs[s_ & 1], ldp, ready[s_ & 1], dev_lvl, ldb, slack, B, ppm, T, E, ss, nc, sel, ws)
        rx = sets[which][1]
        assert np.array_equal(T.numpy(), rx["makespan"]) and np.array_equal(ss.numpy(), rx["slack_sum"])
        np.testing.assert_allclose(E.numpy(), rx["energy"], rtol=E_RTOL)
        assert np.array_equal(slack.cpu().numpy(), rx["slack"])
    h.free()


def test_many_groups_per_block(torch_cuda, emo, oracle_mod):
    """A batch large enough for several policy groups per block (more than 2 x 32 x the SM count policies)
    with a ragged last tile: ES, LS and slack of every policy, every staged kernel family."""
    torch = torch_cuda
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    g = W.make_graph("cfg1-train", 0.05)
    B = 2 * 32 * sms + 77
    lv_dev = W.policies_for(g, B=B, device="cuda")
    r_or = oracle_mod.batch(g, lv_dev.cpu().numpy(), B=B, want_arrays=True, threads=os.cpu_count() or 1)
    h = emo.load_workload(g)
    for fl in (emo.EMO_F_FLOW_KERNEL, emo.EMO_F_LANE_KERNEL, emo.EMO_F_PAIR_KERNEL):
        r = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n, flags=fl, base=True)
        assert_matches(r, r_or, B)
    h.free()


def _spread_graph(total_spread: int, n: int = 40):
    """A two-stream graph with cross edges whose completion times spread by about total_spread ns over
    the policies (level 0 is fast, level 1 slow), with rows that are not monotone and zero durations."""
    rs = np.random.RandomState(7)
    per = total_spread // n
    edges = [(i, i + 2) for i in range(n - 2)] + [(i, i + 1) for i in range(0, n - 1, 5)] + [(i, i + 3) for i in range(1, n - 3, 7)]
    lat = np.zeros((n, 3), dtype=np.int64)
    lat[:, 0] = rs.randint(0, 1000, n)
    lat[:, 1] = lat[:, 0] + 2 * per + rs.randint(0, 1000, n)
    lat[:, 2] = rs.randint(0, 500, n)          # faster than level 0 for some nodes: rows are not monotone
    lat[::9] = 0
    en = rs.rand(n, 3)
    return W.tiny_graph(n, edges, lat, en, name="spread")


def test_offset_guard_and_fallback(torch_cuda, emo, oracle_mod):
    """The 32-bit kernels carry times as offsets from static bounds.  A graph whose spread of start times
    stays below 2^32 ns runs on them (non-monotone rows and zero durations included); one whose spread is
    larger must fall back to the 64-bit kernels; both give the oracle's results."""
    torch = torch_cuda
    B = 96
    for total, want32 in ((3_000_000_000, True), (9_000_000_000, False)):
        g = _spread_graph(total)
        lv = np.random.RandomState(1).randint(0, 3, (g.n, B)).astype(np.uint8)
        lv[:, 0] = 1                       # the slowest policy: the largest offsets
        lv[:, 1] = 0
        r_or = oracle_mod.batch(g, lv, want_arrays=True)
        assert (int(r_or["makespan"].max()) - int(r_or["makespan"].min()) > (1 << 32)) == (not want32)
        lv_dev = torch.as_tensor(lv, device="cuda")
        h = emo.load_workload(g)
        path = emo.emo_call_path(h, B, lv_dev, B, B, True, emo.EMO_F_FLOW_KERNEL)
        assert (path == 2) == want32, "the guard decides whether the 32-bit kernels run"
        r = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n, flags=emo.EMO_F_FLOW_KERNEL, base=True)
        assert_matches(r, r_or, B)
        h.free()
    # exactly at the guard: a chain whose completion times spread by 2^32 - 1 ns (fits) and by 2^32 (does not)
    for spread, want32 in ((0xFFFFFFFF, True), (0x100000000, False)):
        a = spread // 2
        lat = np.array([[1, 1 + a], [1, 1 + (spread - a)]], dtype=np.int64)
        g = W.tiny_graph(2, [(0, 1)], lat, name="edge")
        lv = np.zeros((2, 16), dtype=np.uint8)
        lv[:, 1] = 1
        lv[0, 2] = 1
        lv[1, 3] = 1
        r_or = oracle_mod.batch(g, lv, want_arrays=True)
        lv_dev = torch.as_tensor(lv, device="cuda")
        h = emo.load_workload(g)
        assert (emo.emo_call_path(h, 16, lv_dev, 16, 16, True, emo.EMO_F_FLOW_KERNEL) == 2) == want32
        r = gpu_slack_batch(torch, emo, h, lv_dev, 16, 2, flags=emo.EMO_F_FLOW_KERNEL)
        assert_matches(r, r_or, 16)
        h.free()


def test_bounded_waits_report_timeout(torch_cuda, emo, oracle_mod):
    """Every device-side wait of the 32-bit kernels is bounded.  With the test hook the producer warps stop
    half way (no copy is issued, nothing is read out of bounds, nothing spins for ever): the consumers' waits
    run out after the (shortened) limit, EMO_E_TIMEOUT goes to the status word, the kernels return, and the
    next ordinary call gives the oracle's results."""
    torch = torch_cuda
    g = W.make_graph("cfg1-train", 0.05)
    B = 200
    lv_dev = W.policies_for(g, B=B, device="cuda")
    r_or = oracle_mod.batch(g, lv_dev.cpu().numpy(), B=B, want_arrays=True)
    h = emo.load_workload(g)
    emo.emo_set_wait_limit(4_000_000)          # about 2 ms
    try:
        slack = torch.zeros((g.n, B), dtype=torch.int64, device="cuda")
        T = torch.zeros(B, dtype=torch.int64, device="cuda")
        E = torch.zeros(B, dtype=torch.float64, device="cuda")
        fl = emo.EMO_F_FLOW_KERNEL | emo.EMO_F_TEST_STALL
        ws = torch.empty(emo.emo_workspace_bytes(h, B, 1, fl), dtype=torch.uint8, device="cuda")
        for call in ("eval", "slack"):
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            if call == "eval":
                emo.emo_eval_policies(h, B, lv_dev, lv_dev.stride(0), T, E, ws, status, fl)
            else:
                emo.emo_slack_batch(h, B, lv_dev, lv_dev.stride(0), None, None, slack, B, T, E, None, None, ws, status, fl)
            torch.cuda.synchronize()
            assert int(status.item()) == emo.EMO_E_TIMEOUT
    finally:
        emo.emo_set_wait_limit(4_000_000_000)
    r = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n, flags=emo.EMO_F_FLOW_KERNEL, base=True)
    assert_matches(r, r_or, B)
    h.free()


@pytest.mark.gpu
def test_measurement_helpers(torch_cuda, emo):
    """The two measurement helpers run and give plausible figures (they feed the bounds bench.py prints)."""
    torch = torch_cuda
    scratch = torch.zeros(32, dtype=torch.int64, device="cuda")
    ipk = emo.emo_measure_int_issue(scratch)
    assert all(1e10 < v < 1e13 for v in ipk.values()), ipk
    c = emo.emo_measure_warp_costs(scratch)
    assert 1.0 <= c["add_dependent"] <= 12.0
    assert c["add_independent"] <= c["add_dependent"]
    assert 10.0 <= c["shared_load_dependent"] <= 80.0
    assert c["body_without_branch"] <= c["body_with_untaken_branch"]
    assert 5.0 <= c["barrier_5_warps"] <= 400.0


def _wide_graph(ns, seed=0):
    """ns sources, each read later by three of ns sinks: every source's value stays live until the sinks run."""
    rs = np.random.RandomState(seed)
    edges = sorted({(int(k), ns + j) for j in range(ns) for k in rs.choice(ns, 3, replace=False)})
    lat = rs.randint(0, 100, size=(2 * ns, 4)).astype(np.int64)
    return W.tiny_graph(2 * ns, edges, lat, name="wide")


def test_generic_path_takes_what_the_schedules_cannot(torch_cuda, emo, oracle_mod):
    """A graph with more simultaneously live values than there are exchange slots loads and evaluates exactly
    (generic kernels); the same kernels, forced on ordinary graphs, agree with the oracle on every output."""
    torch = torch_cuda
    cases = [(_wide_graph(400), 0, None), (W.make_graph("cfg1-train", 0.1), emo.EMO_F_GENERIC, None),
             (W.make_graph("cfg3-8dev", 0.01), emo.EMO_F_GENERIC, None)]
    g3 = W.make_graph("cfg0-tiny", 0.5)
    cases.append((g3, emo.EMO_F_GENERIC, np.random.RandomState(3).randint(-1, 5, size=g3.n).astype(np.int32)))
    for g, flags, group_of in cases:
        B = 77
        rows = g.n if group_of is None else 5
        lv = np.random.RandomState(1).randint(0, g.L, size=(rows, B)).astype(np.uint8)
        h = emo.load_workload(g, flags=flags, group_of=group_of)
        ld = 80
        lvd = torch.full((rows, ld), 0xFF, dtype=torch.uint8, device="cuda")
        lvd[:, :B] = torch.from_numpy(lv).cuda()
        assert emo.emo_call_path(h, B, lvd, ld, ld, True, 0) == 3
        mk = lambda dt: torch.zeros((g.n, ld), dtype=dt, device="cuda")
        ES, LS, SL = mk(torch.int64), mk(torch.int64), mk(torch.int64)
        T = torch.zeros(B, dtype=torch.int64, device="cuda")
        E = torch.zeros(B, dtype=torch.float64, device="cuda")
        ss = torch.zeros(B, dtype=torch.int64, device="cuda")
        nc = torch.zeros(B, dtype=torch.int32, device="cuda")
        T0 = torch.zeros(1, dtype=torch.int64, device="cuda")
        E0 = torch.zeros(1, dtype=torch.float64, device="cuda")
        ws = torch.empty(emo.emo_workspace_bytes(h, B, 1), dtype=torch.uint8, device="cuda")
        emo.emo_slack_batch(h, B, lvd, ld, ES, LS, SL, ld, T, E, ss, nc, ws, None, T0=T0, E0=E0)
        torch.cuda.synchronize()
        r = oracle_mod.batch(g, lv, want_arrays=True, group_of=group_of)
        assert np.array_equal(T.cpu().numpy(), r["makespan"])
        assert np.allclose(E.cpu().numpy(), r["energy"], rtol=1e-9, atol=0)
        assert np.array_equal(ES.cpu().numpy()[:, :B], r["ES"])
        assert np.array_equal(LS.cpu().numpy()[:, :B], r["LS"])
        assert np.array_equal(SL.cpu().numpy()[:, :B], r["slack"])
        assert np.array_equal(ss.cpu().numpy(), r["slack_sum"]) and np.array_equal(nc.cpu().numpy(), r["n_critical"])
        base_lv = np.full((rows, 1), g.L - 1, np.uint8)
        base = oracle_mod.batch(g, base_lv, group_of=group_of)
        assert int(T0.item()) == int(base["makespan"][0]) and np.isclose(float(E0.item()), base["energy"][0], rtol=1e-9)
        # forward only, and the single-policy call
        T.zero_()
        ws2 = torch.empty(emo.emo_workspace_bytes(h, B, 0), dtype=torch.uint8, device="cuda")
        emo.emo_eval_policies(h, B, lvd, ld, T, E, ws2)
        torch.cuda.synchronize()
        assert np.array_equal(T.cpu().numpy(), r["makespan"])
        one = torch.from_numpy(lv[:, 5].copy()).cuda()
        es1 = torch.zeros(g.n, dtype=torch.int64, device="cuda")
        ls1 = torch.zeros(g.n, dtype=torch.int64, device="cuda")
        sl1 = torch.zeros(g.n, dtype=torch.int64, device="cuda")
        t1 = torch.zeros(1, dtype=torch.int64, device="cuda")
        ws3 = torch.empty(emo.emo_workspace_bytes(h, 1, 1), dtype=torch.uint8, device="cuda")
        emo.emo_slack(h, one, es1, ls1, sl1, t1, None, ws3)
        torch.cuda.synchronize()
        assert int(t1.item()) == int(r["makespan"][5])
        assert np.array_equal(es1.cpu().numpy(), r["ES"][:, 5]) and np.array_equal(sl1.cpu().numpy(), r["slack"][:, 5])
        h.free()
