"""The lane-stream program compiler (the program of the 32-bit pass kernels), checked without a GPU:
interpreted on the host under the kernels' rules (tests/flow_emulator.py) it must reproduce the
oracle bit for bit, and it must exist exactly when every spread of start times fits 32 bits."""
from __future__ import annotations

import numpy as np
import pytest

from paper_2607_12324_b200 import workloads as W
from tests import flow_emulator as FE
from tests.test_oracle_pins import TINY, all_policies


@pytest.fixture(scope="session")
def emo():
    from paper_2607_12324_b200 import build, emo as E
    build.build()
    return E


def check_flow(emo, oracle_mod, g, lv, flags=0, group_of=None, expect_ok=True):
    h = emo.load_workload(g, flags | emo.EMO_F_HOST_ONLY, group_of)
    f = emo.emo_graph_flow(h)
    if not expect_ok:
        assert f["ok32"] == 0
        h.free()
        return f
    assert f["ok32"] == 1
    r = oracle_mod.batch(g, lv, want_arrays=True, group_of=group_of)
    n_rows = lv.shape[0]
    assert int(f["rows"][f["rows"] != FE.NONE].max(initial=0)) < max(n_rows, 1)
    nodes = f["node"][f["node"] != FE.NONE]
    assert sorted(nodes.tolist()) == list(range(g.n)), "every node is scheduled exactly once"
    T, E, restore = FE.run_forward(f, lv, g.L)
    assert np.array_equal(T, r["makespan"])
    assert np.allclose(E, r["energy"], rtol=1e-12, atol=0)
    ES, LS, SL = FE.run_backward(f, lv, g.L, T, restore, g.n)
    assert np.array_equal(ES, r["ES"])
    assert np.array_equal(LS, r["LS"])
    assert np.array_equal(SL, r["slack"])
    # structure: the segments of a lane name every entry once, in walking order; an entry comes as a
    # segment's special entry exactly when it is not simple; a period's first segment carries the barrier
    nper = f["K"] // f["sync"]
    for st in range(f["stages"]):
        for ln in range(f["lanes"]):
            total = int((f["node"][st, ln] != FE.NONE).sum())
            for backward in (False, True):
                segs = FE.segments(f, st, ln, backward)
                order, barriers, period_of_seg = [], 0, []
                for bar, special, run, kind in segs:
                    barriers += bar
                    assert len(run) <= 8
                    if special is not None:
                        order.append(special)
                        w = int(f["rec_bwd" if backward else "rec_fwd"][st, ln, special, 0])
                        assert not (w & FE.B_SIMPLE) if backward else w != FE.F_HASREG
                    for pos in run:
                        order.append(pos)
                        w = int(f["rec_bwd" if backward else "rec_fwd"][st, ln, pos, 0])
                        if backward:
                            assert w & FE.B_SIMPLE
                            assert bool(kind & FE.SEG_IN) == bool(w >> 16) and bool(kind & FE.SEG_OUT) == bool(w & FE.B_OUTSET)
                        else:
                            assert w == FE.F_HASREG and kind == 0
                    pers = {(int(f["step"][st, ln, pos]) % f["K"]) // f["sync"] for pos in ([special] if special is not None else []) + run}
                    assert len(pers) <= 1, "a segment stays inside one period"
                    period_of_seg.append((bar, pers))
                assert barriers == nper
                assert order == (list(range(total - 1, -1, -1)) if backward else list(range(total)))
                # the barrier sits on the first segment of each period
                seen = set()
                for bar, pers in period_of_seg:
                    for q in pers:
                        assert bar or q in seen
                        seen.add(q)
    h.free()
    return f


@pytest.mark.parametrize("gi", range(len(TINY)))
def test_flow_on_tiny_graphs(emo, oracle_mod, gi):
    g = TINY[gi]
    lv = all_policies(g.n, g.L)
    lv = lv[:, :: max(1, lv.shape[1] // 300)].copy()
    for lanes, sync, stage in ((0, 8, 32), (1, 8, 8), (3, 16, 16), (2, 8, 32)):
        check_flow(emo, oracle_mod, g, lv, emo.EMO_F_LANES(lanes) | emo.EMO_F_FLOW_SYNC(sync) | emo.EMO_F_FLOW_STAGE(stage))


@pytest.mark.parametrize("name,scale", [("cfg0-tiny", 1.0), ("cfg1-train", 0.1), ("cfg2-packed", 0.2),
                                          ("cfg3-8dev", 0.02), ("cfg4-llm", 0.01)])
def test_flow_on_config_graphs(emo, oracle_mod, name, scale):
    g = W.make_graph(name, scale)
    lv = W.policy_levels(g.meta["policy_seed"], g.n, g.L, 24, "mixed").numpy()
    f = check_flow(emo, oracle_mod, g, lv)
    assert f["steps"] >= 1 and f["pushes"] <= g.n
    for lanes, look, sync in ((1, 0, 8), (4, 2, 16), (7, 30, 32)):
        check_flow(emo, oracle_mod, g, lv, emo.EMO_F_LANES(lanes) | emo.EMO_F_LOOKAHEAD(look) | emo.EMO_F_FLOW_SYNC(sync))


def test_flow_with_fan_in_and_fan_out(emo, oracle_mod):
    """A node with 20 predecessors and a node with 15 successors: long operand lists, shared slots."""
    n = 37
    edges = [(i, 20) for i in range(20)] + [(20, 21)] + [(21, 22 + i) for i in range(15)]
    rs = np.random.RandomState(5)
    lat = rs.randint(0, 30, size=(n, 3)).astype(np.int64)
    g = W.tiny_graph(n, edges, lat, name="fan")
    lv = rs.randint(0, 3, size=(n, 64)).astype(np.uint8)
    for lanes in (0, 1, 4, 9):
        check_flow(emo, oracle_mod, g, lv, emo.EMO_F_LANES(lanes))


def test_flow_group_of_and_ignored_rows(emo, oracle_mod):
    g = W.make_graph("cfg1-train", 0.03)
    rs = np.random.RandomState(11)
    group_of = rs.randint(-1, 7, size=g.n).astype(np.int32)
    lv = rs.randint(0, g.L, size=(7, 40)).astype(np.uint8)
    check_flow(emo, oracle_mod, g, lv, group_of=group_of)


def _chain_with_spread(spread: int):
    """Two nodes in a row whose completion-time spread over all policies is exactly `spread` ns."""
    a = spread // 2
    lat = np.array([[1, 1 + a], [1, 1 + (spread - a)]], dtype=np.int64)
    return W.tiny_graph(2, [(0, 1)], lat, name="spread")


def test_flow_exists_exactly_up_to_32_bits_of_spread(emo, oracle_mod):
    lv = np.array([[0, 1, 0, 1], [0, 0, 1, 1]], dtype=np.uint8)
    check_flow(emo, oracle_mod, _chain_with_spread(0xFFFFFFFF), lv)                 # sits on the guard
    check_flow(emo, oracle_mod, _chain_with_spread(0x100000000), lv, expect_ok=False)   # one past it
    check_flow(emo, oracle_mod, _chain_with_spread(0x180000000), lv, expect_ok=False)


def test_flow_non_monotone_and_zero_rows(emo, oracle_mod):
    """Rows that are not monotone in the level and zero durations: offsets are taken from the row minimum."""
    rs = np.random.RandomState(3)
    g0 = W.make_graph("cfg0-tiny", 0.3)
    lat = g0.lat.copy()
    for v in range(g0.n):
        if v % 3 == 0:
            lat[v] = rs.permutation(lat[v])
        if v % 7 == 0:
            lat[v] = 0
    g = W.Graph(g0.n, g0.row_ptr, g0.col, g0.level_ptr, g0.L, lat, g0.energy, g0.kind, "nonmono")
    lv = rs.randint(0, g.L, size=(g.n, 50)).astype(np.uint8)
    check_flow(emo, oracle_mod, g, lv)
