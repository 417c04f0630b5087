"""GPU parity of the spine kernels (one warp per policy group carries the recurrence of Eq. 1, the other
warps do the look-ups, the sums per segment and the stores) against the CPU oracle, through the C ABI:
makespan, ES, LS, slack, slack sums and critical counts bit-exact, energy within 1e-9 relative."""
from __future__ import annotations

import os

import numpy as np
import pytest

from paper_2607_12324_b200 import workloads as W
from tests.test_gpu_parity import E_RTOL, assert_matches, emo, gpu_eval, gpu_slack_batch, torch_cuda  # noqa: F401  (fixtures)

pytestmark = pytest.mark.gpu


def check(torch, emo, oracle_mod, g, h, lv_dev, B, r_or, ldo=None, flags=None):
    fl = emo.EMO_F_SPINE_KERNEL if flags is None else flags
    base = oracle_mod.batch(g, np.full((g.n, 1), g.L - 1, dtype=np.uint8))
    r = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n, want=("slack",), sums=False, base=True, flags=fl, ldo=ldo)
    assert np.array_equal(r["makespan"], r_or["makespan"])
    np.testing.assert_allclose(r["energy"], r_or["energy"], rtol=E_RTOL, atol=0)
    assert np.array_equal(r["slack"][:, :B], r_or["slack"])
    assert (r["slack"][:, B:] == -7).all(), "padding columns of the slack matrix were written"
    assert r["T0"] == base["makespan"][0]
    assert r["E0"] == pytest.approx(base["energy"][0], rel=E_RTOL)
    # every per-node output and the per-policy sums
    r2 = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n, flags=fl, ldo=ldo)
    assert_matches(r2, r_or, B)
    for k in ("ES", "LS", "slack"):
        assert (r2[k][:, B:] == -7).all(), "padding columns of the outputs were written"
    T, E, st = gpu_eval(torch, emo, h, lv_dev, B, fl | emo.EMO_F_VALIDATE)
    assert st == 0 and np.array_equal(T, r_or["makespan"])
    np.testing.assert_allclose(E, r_or["energy"], rtol=E_RTOL)


def test_tiny_graphs_every_policy(torch_cuda, emo, oracle_mod):
    """Hand-made and random tiny DAGs (ties, zero durations, duplicate edges, isolated nodes, non-monotone
    rows), every policy, several lane counts and stage lengths, a ragged output pitch."""
    from tests.test_oracle_pins import TINY, all_policies
    torch = torch_cuda
    for g in TINY:
        lv = all_policies(g.n, g.L)
        B = lv.shape[1]
        r_or = oracle_mod.batch(g, lv, want_arrays=True)
        ldb = (B + 15) // 16 * 16 + 16
        lvq = np.full((g.n, ldb), 0xFF, dtype=np.uint8)
        lvq[:, :B] = lv
        lv16 = torch.as_tensor(lvq, device="cuda")
        for lanes, k in ((0, 16), (1, 8), (2, 32)):
            h = emo.load_workload(g, emo.EMO_F_LANES(lanes) | emo.EMO_F_SPINE_STAGE(k))
            sp = emo.emo_graph_spine(h)
            assert sp["ok"] == 1 and sp["K"] == k and sp["segments"] <= g.n
            assert emo.emo_call_path(h, B, lv16, ldb, B + 3, True, emo.EMO_F_SPINE_KERNEL) == 4
            check(torch, emo, oracle_mod, g, h, lv16, B, r_or, ldo=B + 3)
            h.free()


@pytest.mark.parametrize("name,scale,B,k", [("cfg0-tiny", 1.0, 64, 16), ("cfg1-train", 0.25, 333, 16), ("cfg1-train", 0.25, 333, 32),
                                              ("cfg2-packed", 0.5, 1000, 8), ("cfg3-8dev", 0.03, 200, 16), ("cfg4-llm", 0.02, 257, 16),
                                              ("cfg4-llm", 0.02, 257, 8)])
def test_config_graphs(torch_cuda, emo, oracle_mod, name, scale, B, k):
    """Scaled configuration graphs (several policy tiles, a ragged tail; the 8-timeline graph has nodes with many
    operands, the 250 000-node one launch nodes whose kernels are folded two stages back)."""
    torch = torch_cuda
    g = W.make_graph(name, scale)
    lv_dev = W.policies_for(g, B=B, device="cuda")
    r_or = oracle_mod.batch(g, lv_dev.cpu().numpy(), B=B, want_arrays=True, threads=os.cpu_count() or 1)
    h = emo.load_workload(g, emo.EMO_F_SPINE_STAGE(k))
    sp = emo.emo_graph_spine(h)
    assert sp["ok"] == 1 and sp["ops_bwd"] >= sp["segments"] > 0 and sp["ops_fwd"] > 0
    check(torch, emo, oracle_mod, g, h, lv_dev, B, r_or, ldo=B + 1)
    # the default: narrow graphs below the large-batch rule take the spine kernels for slack-only calls, every other
    # call (per-node ES / LS, sums) the kernels that produce those outputs
    path = emo.emo_call_path(h, B, lv_dev, lv_dev.stride(0), B, 1, 0)
    assert (path == 4) == (sp["lanes"] <= 8)
    if path == 4:
        check(torch, emo, oracle_mod, g, h, lv_dev, B, r_or, flags=0)
    h.free()


def test_many_groups_and_blocks(torch_cuda, emo, oracle_mod):
    """A batch that fills several groups per block and several blocks; the baseline column falls into the last tile."""
    torch = torch_cuda
    g = W.make_graph("cfg1-train", 0.05)
    for B in (4096 + 31, 160 * 32):
        lv_dev = W.policies_for(g, B=B, device="cuda")
        r_or = oracle_mod.batch(g, lv_dev.cpu().numpy(), B=B, want_arrays=True, threads=os.cpu_count() or 1)
        h = emo.load_workload(g)
        check(torch, emo, oracle_mod, g, h, lv_dev, B, r_or)
        h.free()


def test_bounded_waits_report_timeout(torch_cuda, emo, oracle_mod):
    """With the test hook the producer warps stop half way: every wait of the spine and worker warps runs out after
    the (shortened) limit, EMO_E_TIMEOUT goes to the status word, the kernels return and the next call is right."""
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
        fl = emo.EMO_F_SPINE_KERNEL | emo.EMO_F_TEST_STALL
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
    check(torch, emo, oracle_mod, g, h, lv_dev, B, r_or)
    h.free()


def test_random_dags(torch_cuda, emo, oracle_mod):
    """Random DAGs of varying density, size and level count (merge operations, long segments, isolated nodes), every
    output, through the kernels."""
    torch = torch_cuda
    done = 0
    for seed in range(12):
        rs = np.random.RandomState(2000 + seed)
        n = int(rs.randint(30, 400))
        L = int(rs.randint(2, 9))
        g = W.random_dag(700 + seed, n, float(rs.choice([0.01, 0.03, 0.1, 0.3])), L=L, max_dur=int(rs.choice([5, 40, 100000])))
        B = int(rs.choice([33, 96, 200]))
        ldb = (B + 15) // 16 * 16
        lvq = np.full((g.n, ldb), 0xFF, dtype=np.uint8)
        lvq[:, :B] = rs.randint(0, L, size=(g.n, B))
        lv_dev = torch.as_tensor(lvq, device="cuda")
        r_or = oracle_mod.batch(g, lvq[:, :B].copy(), want_arrays=True)
        h = emo.load_workload(g, emo.EMO_F_SPINE_STAGE(int(rs.choice([8, 16, 32]))))
        if emo.emo_graph_spine(h)["ok"] == 1:      # very dense graphs go to the generic kernels: no spine program
            check(torch, emo, oracle_mod, g, h, lv_dev, B, r_or, ldo=B + 2)
            done += 1
        h.free()
    assert done >= 8


def test_forward_spine_feeds_lane_stream_backward(torch_cuda, emo, oracle_mod):
    """Four policy groups per SM on a narrow graph: the forward spine kernel writes the restore list in the lane-stream
    program's numbering and the lane-stream backward kernel reads it.  Same slack matrix as the lane-stream pair alone,
    and the oracle's on sampled policies."""
    torch = torch_cuda
    g = W.make_graph("cfg4-llm", 0.1)
    B = 16384
    lv_dev = W.policies_for(g, B=B, device="cuda")
    h = emo.load_workload(g)
    path = emo.emo_call_path(h, B, lv_dev, lv_dev.stride(0), B, True, 0)
    assert path in (2, 5)
    if path != 5:
        pytest.skip("this graph's lane-stream program does not share the spine program's schedule")
    r_pair = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n, want=("slack",), sums=False, base=True)
    r_flow = gpu_slack_batch(torch, emo, h, lv_dev, B, g.n, want=("slack",), sums=False, base=True, flags=emo.EMO_F_FLOW_KERNEL)
    assert np.array_equal(r_pair["makespan"], r_flow["makespan"]) and r_pair["T0"] == r_flow["T0"]
    np.testing.assert_allclose(r_pair["energy"], r_flow["energy"], rtol=E_RTOL)
    assert np.array_equal(r_pair["slack"], r_flow["slack"])
    cols = np.linspace(0, B - 1, 24).astype(np.int64)
    sub = lv_dev[:, torch.as_tensor(cols, device="cuda")].contiguous().cpu().numpy()
    r_or = oracle_mod.batch(g, sub, want_arrays=True, threads=os.cpu_count() or 1)
    assert np.array_equal(r_pair["makespan"][cols], r_or["makespan"])
    np.testing.assert_allclose(r_pair["energy"][cols], r_or["energy"], rtol=E_RTOL)
    assert np.array_equal(r_pair["slack"][:, cols], r_or["slack"])
    h.free()
