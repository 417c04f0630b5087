"""Time-interval policies on the GPU (emo_eval_intervals) against the oracle's Alg. 1: makespan bit-exact,
active + idle energy within 1e-9 relative."""
from __future__ import annotations

import json
import os

import numpy as np
import pytest

from paper_2607_12324_b200 import workloads as W

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.fixture(scope="module")
def torch_cuda():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("needs a GPU")
    return torch


@pytest.fixture(scope="module")
def emo():
    from paper_2607_12324_b200 import build, emo as E
    build.build()
    return E


def run_gpu(torch, emo, g, dev_of, breaks, F, p_idle, flags=0, ldb=None, call_flags=0):
    """F: numpy uint8 [D][I][B]."""
    D, I, B = F.shape
    ldb = ldb or (B + 15) // 16 * 16
    Fd = torch.full((D, I, ldb), 0xFF, dtype=torch.uint8, device="cuda")
    Fd[:, :, :B] = torch.from_numpy(F).cuda()
    h = emo.load_workload(g, flags=flags, group_of=np.asarray(dev_of, np.int32))
    T = torch.zeros(B, dtype=torch.int64, device="cuda")
    E = torch.zeros(B, dtype=torch.float64, device="cuda")
    Ei = torch.zeros(B, dtype=torch.float64, device="cuda") if p_idle is not None else None
    pi = torch.from_numpy(np.asarray(p_idle, np.float64)).cuda() if p_idle is not None else None
    ws = torch.empty(emo.emo_workspace_bytes_intervals(h, B, I, p_idle is not None), dtype=torch.uint8, device="cuda")
    emo.emo_eval_intervals(h, B, Fd, ldb, I, np.asarray(breaks, np.int64), pi, T, E, Ei, ws, flags=call_flags)
    torch.cuda.synchronize()
    h.free()
    return T.cpu().numpy(), E.cpu().numpy(), None if Ei is None else Ei.cpu().numpy()


def check(torch, emo, oracle_mod, g, dev_of, breaks, F, p_idle, flags=0, **kw):
    """Both forms of the evaluation: the lane-stream kernel (graph loaded with EMO_F_INTERVALS; uniform grids) and
    the step-program kernel (without the flag, and with EMO_F_NO_STAGING on the prepared handle)."""
    r = oracle_mod.intervals(g, dev_of, breaks, F, p_idle)
    for load_flags, call_flags in ((emo.EMO_F_INTERVALS, 0), (0, 0), (emo.EMO_F_INTERVALS, emo.EMO_F_NO_STAGING)):
        T, E, Ei = run_gpu(torch, emo, g, dev_of, breaks, F, p_idle, flags=flags | load_flags, call_flags=call_flags, **kw)
        assert np.array_equal(T, r["makespan"]), (load_flags, call_flags)
        assert np.allclose(E, r["energy"], rtol=1e-9, atol=0), (load_flags, call_flags)
        if p_idle is not None:
            assert np.allclose(Ei, r["e_idle"], rtol=1e-9, atol=1e-30), (load_flags, call_flags)


def test_hand_worked_example_on_gpu(torch_cuda, emo, oracle_mod):
    d = json.load(open(os.path.join(HERE, "golden", "hand_worked_intervals.json")))
    g = W.tiny_graph(d["n"], d["edges"], np.asarray(d["lat"], np.int64), np.asarray(d["energy"], np.float64))
    T, E, Ei = run_gpu(torch_cuda, emo, g, d["dev_of"], d["breaks"], np.array(d["F"], np.uint8), d["p_idle"])
    assert T.tolist() == d["makespan"]
    assert np.allclose(Ei, np.array(d["idle_ns_times_watts"]) * 1e-9, rtol=1e-12, atol=0)
    assert np.allclose(E, np.array(d["e_active"]) + np.array(d["idle_ns_times_watts"]) * 1e-9, rtol=1e-12, atol=0)


@pytest.mark.parametrize("seed", range(4))
def test_random_dags(torch_cuda, emo, oracle_mod, seed):
    from tests.test_oracle_intervals import _random_case
    g, dev_of, breaks, F, p_idle = _random_case(seed, n=60, L=4, D=3, I=7, B=70)
    check(torch_cuda, emo, oracle_mod, g, dev_of, breaks, F, p_idle)
    check(torch_cuda, emo, oracle_mod, g, dev_of, breaks, F, None)
    check(torch_cuda, emo, oracle_mod, g, dev_of, [0], F[:, :1, :].copy(), p_idle)          # one interval
    check(torch_cuda, emo, oracle_mod, g, dev_of, np.arange(7, dtype=np.int64) * 23, F, p_idle)      # uniform grid
    check(torch_cuda, emo, oracle_mod, g, dev_of, np.arange(7, dtype=np.int64) * 5, F, p_idle)       # packs span several intervals
    check(torch_cuda, emo, oracle_mod, g, dev_of, breaks, F, p_idle, flags=emo.EMO_F_LANES(1))
    check(torch_cuda, emo, oracle_mod, g, dev_of, breaks, F, p_idle, flags=emo.EMO_F_LANES(3) | emo.EMO_F_FLOW_SYNC(8))


@pytest.mark.parametrize("name,scale,B,I", [("cfg0-tiny", 1.0, 64, 9), ("cfg1-train", 0.2, 200, 40), ("cfg3-8dev", 0.02, 100, 24),
                                             ("cfg4-llm", 0.01, 96, 33)])
def test_config_graphs(torch_cuda, emo, oracle_mod, name, scale, B, I):
    g = W.make_graph(name, scale)
    dev_of = W.device_of(g)
    D = int(dev_of.max()) + 1
    lv_max = np.full((g.n, 1), g.L - 1, np.uint8)
    T0 = int(oracle_mod.batch(g, lv_max)["makespan"][0])
    breaks = W.interval_breaks(T0, I)
    F = W.interval_policies(g.meta["policy_seed"], D, I, g.L, B).numpy()[:, :, :B].copy()
    check(torch_cuda, emo, oracle_mod, g, dev_of, breaks, F, W.idle_power(g.L))
    # uneven change points as well
    rs = np.random.RandomState(5)
    br2 = np.concatenate([[0], np.sort(rs.choice(np.arange(1, int(T0 * 1.2)), size=I - 1, replace=False))]).astype(np.int64)
    check(torch_cuda, emo, oracle_mod, g, dev_of, br2, F, W.idle_power(g.L))


def test_pack_with_constant_tables_still_counts_as_busy(torch_cuda, emo, oracle_mod):
    """A pack whose duration and energy do not depend on the level reads no level, but it keeps its device busy."""
    lat = [[4, 4], [10, 10], [8, 5], [4, 4], [6, 6]]
    en = [[0.0, 0.0], [5.0, 5.0], [4.0, 6.0], [0.0, 0.0], [3.0, 3.0]]
    g = W.tiny_graph(5, [(0, 1), (1, 2), (0, 3), (3, 4)], np.asarray(lat, np.int64), np.asarray(en, np.float64))
    F = np.array([[[1, 0, 1, 0], [0, 0, 1, 1], [1, 0, 1, 1]]], np.uint8)
    check(torch_cuda, emo, oracle_mod, g, [-1, 0, 0, -1, 0], [0, 10, 16], F, [2.0, 3.0])
    check(torch_cuda, emo, oracle_mod, g, [-1, 0, 0, -1, 0], [0, 50], F[:, :2, :].copy(), [2.0, 3.0])


def test_argument_errors(torch_cuda, emo):
    torch = torch_cuda
    g = W.make_graph("cfg0-tiny", 0.2)
    h = emo.load_workload(g, group_of=W.device_of(g))
    B, I = 8, 3
    F = torch.zeros((1, I, 16), dtype=torch.uint8, device="cuda")
    T = torch.zeros(B, dtype=torch.int64, device="cuda")
    E = torch.zeros(B, dtype=torch.float64, device="cuda")
    ws = torch.empty(emo.emo_workspace_bytes_intervals(h, B, I, True), dtype=torch.uint8, device="cuda")
    for bad in ([1, 2, 3], [0, 5, 5], [0, 7, 3]):
        with pytest.raises(Exception):
            emo.emo_eval_intervals(h, B, F, 16, I, np.array(bad, np.int64), None, T, E, None, ws)
    with pytest.raises(Exception):      # idle output without idle power
        emo.emo_eval_intervals(h, B, F, 16, I, np.array([0, 4, 9], np.int64), None, T, E, E, ws)
    with pytest.raises(Exception):      # workspace too small
        emo.emo_eval_intervals(h, B, F, 16, I, np.array([0, 4, 9], np.int64), None, T, E, None, ws[:8])
    emo.emo_eval_intervals(h, 0, None, 0, I, np.array([0, 4, 9], np.int64), None, None, None, None, ws)      # B = 0: nothing to do
    h.free()


def test_large_batch_sampled(torch_cuda, emo, oracle_mod):
    """A batch that fills every block with four policy groups (the launch shape of the bench), on the lane-stream
    form; a sample of its columns against the oracle."""
    torch = torch_cuda
    g = W.make_graph("cfg4-llm", 0.1)
    dev_of = W.device_of(g)
    B, D = 16384, 1
    T0 = int(oracle_mod.batch(g, np.full((g.n, 1), g.L - 1, np.uint8))["makespan"][0])
    I = int(T0 * 1.05 / 20e6) + 1
    breaks = W.interval_breaks(T0, I)
    F = W.interval_policies(g.meta["policy_seed"], D, I, g.L, B, device="cuda")
    h = emo.load_workload(g, flags=emo.EMO_F_INTERVALS, group_of=dev_of)
    T = torch.zeros(B, dtype=torch.int64, device="cuda")
    E = torch.zeros(B, dtype=torch.float64, device="cuda")
    Ei = torch.zeros(B, dtype=torch.float64, device="cuda")
    pi = torch.from_numpy(W.idle_power(g.L)).cuda()
    ws = torch.empty(emo.emo_workspace_bytes_intervals(h, B, I, True), dtype=torch.uint8, device="cuda")
    emo.emo_eval_intervals(h, B, F, F.shape[2], I, breaks, pi, T, E, Ei, ws)
    torch.cuda.synchronize()
    cols = np.array([0, 1, 31, 32, 4095, 8192, 16383])
    r = oracle_mod.intervals(g, dev_of, breaks, F[:, :, torch.as_tensor(cols, device="cuda")].cpu().numpy(), W.idle_power(g.L))
    assert np.array_equal(T.cpu().numpy()[cols], r["makespan"])
    assert np.allclose(E.cpu().numpy()[cols], r["energy"], rtol=1e-9, atol=0)
    assert np.allclose(Ei.cpu().numpy()[cols], r["e_idle"], rtol=1e-9, atol=1e-30)
    h.free()


def test_cfg4_full_size_sampled(torch_cuda, emo, oracle_mod):
    """The bench's own workload and launch configuration (cfg4-llm at full size, 16 384 policies, 20 ms grid, idle
    energy on): a few policies one by one against the oracle, both kernels against each other on all of them."""
    torch = torch_cuda
    g = W.make_graph("cfg4-llm", 1.0)
    dev_of = W.device_of(g)
    B, D = int(g.meta["B"]), 1
    T0 = int(oracle_mod.batch(g, np.full((g.n, 1), g.L - 1, np.uint8))["makespan"][0])
    I = int(T0 * 1.05 / 20e6) + 1
    breaks = W.interval_breaks(T0, I)
    F = W.interval_policies(g.meta["policy_seed"], D, I, g.L, B, device="cuda")
    pi = torch.from_numpy(W.idle_power(g.L)).cuda()
    h = emo.load_workload(g, flags=emo.EMO_F_INTERVALS, group_of=dev_of)
    ws = torch.empty(emo.emo_workspace_bytes_intervals(h, B, I, True), dtype=torch.uint8, device="cuda")
    out = []
    for call_flags in (0, emo.EMO_F_NO_STAGING):
        T = torch.zeros(B, dtype=torch.int64, device="cuda")
        E = torch.zeros(B, dtype=torch.float64, device="cuda")
        Ei = torch.zeros(B, dtype=torch.float64, device="cuda")
        emo.emo_eval_intervals(h, B, F, F.shape[2], I, breaks, pi, T, E, Ei, ws, flags=call_flags)
        torch.cuda.synchronize()
        out.append((T.cpu().numpy(), E.cpu().numpy(), Ei.cpu().numpy()))
    assert np.array_equal(out[0][0], out[1][0])
    assert np.allclose(out[0][1], out[1][1], rtol=1e-12, atol=0) and np.allclose(out[0][2], out[1][2], rtol=1e-9, atol=1e-30)
    cols = np.array([0, 5, 8191, 8192, 16383])
    r = oracle_mod.intervals(g, dev_of, breaks, F[:, :, torch.as_tensor(cols, device="cuda")].cpu().numpy(), W.idle_power(g.L))
    assert np.array_equal(out[0][0][cols], r["makespan"])
    assert np.allclose(out[0][1][cols], r["energy"], rtol=1e-9, atol=0)
    assert np.allclose(out[0][2][cols], r["e_idle"], rtol=1e-9, atol=1e-30)
    h.free()
