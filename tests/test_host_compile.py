"""Host logic of the CUDA library, run without a GPU: the shared object loads and exports every
declared symbol, emo_graph_load validates its input, and the compiled step programs (scheduler,
register/slot assignment, helper ops) reproduce the oracle when interpreted on the host."""
from __future__ import annotations

import ctypes
import os
import re

import numpy as np
import pytest

from paper_2607_12324_b200 import workloads as W
from tests import program_emulator as PE
from tests.test_oracle_pins import TINY, all_policies

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="session")
def emo():
    from paper_2607_12324_b200 import build, emo as E
    build.build()
    return E


def test_library_exports_every_declared_symbol(emo):
    hdr = open(os.path.join(ROOT, "include", "emo.h")).read()
    declared = set(re.findall(r"\b(emo_[a-z0-9_]+)\s*\(", hdr))
    declared -= {"emo_graph", "emo_info"}
    assert declared, "no declarations found"
    L = ctypes.CDLL(emo.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(L, name), f"{name} declared in include/emo.h but not exported"
    assert set(emo.EXPORTS) == declared


def test_target_from_delta_matches_integer_formula(emo):
    for T0, ppm in [(1000, 30_000), (1001, 30_000), (33, 30_000), (0, 50_000), ((1 << 61) + 12345, 50_000),
                    (4_912_345_678, 20_000), (230_300_914, 30_000)]:
        assert emo.emo_target_from_delta(T0, ppm) == T0 + (T0 * ppm) // 1_000_000


def _load(emo, g, flags=0, group_of=None):
    return emo.load_workload(g, flags | emo.EMO_F_HOST_ONLY, group_of)


def check_programs(emo, oracle_mod, g, lv, flags=0, group_of=None):
    h = _load(emo, g, flags, group_of)
    info = h.info
    assert info.n == g.n and info.m == g.m and info.L == g.L
    r = oracle_mod.batch(g, lv, want_arrays=True, group_of=group_of)
    lanes, steps, slots, Lp, ent, rows, lat = emo.emo_graph_program(h, 0)
    assert info.sync_fwd in (8, 16, 32) and info.sync_bwd in (8, 16, 32)
    f = PE.run(ent, rows, lat, Lp, g.L, slots, lv, g.n, False, sync=info.sync_fwd)
    assert (f["seen"] == 1).all()
    assert np.array_equal(f["T"], r["makespan"])
    assert np.array_equal(f["ES"], r["ES"])
    lanes_b, steps_b, slots_b, Lp_b, ent_b, rows_b, lat_b = emo.emo_graph_program(h, 1)
    b = PE.run(ent_b, rows_b, lat_b, Lp_b, g.L, slots_b, lv, g.n, True, ES_in=f["ES"], T_in=f["T"], sync=info.sync_bwd)
    assert (b["seen"] == 1).all()
    # forward entries address the row of the backward program that handles the same node
    pos_b = {}
    for t in range(steps_b):
        for w in range(lanes_b):
            if int(ent_b[t, w, 1]) & 1 and int(ent_b[t, w, 4]) != 0xFFFFFFFF:
                pos_b[int(ent_b[t, w, 4])] = t * lanes_b + w
    assert all(pos_b[node] == row for node, row in f["main_rows"])
    assert all(node == row for node, row in b["main_rows"])
    # runs of simple entries: the stored length counts the simple entries that follow in the same
    # column (15 at most), never crosses a block of the program's barrier distance and keeps one level mask
    for ent_x, sync_x in ((ent, info.sync_fwd), (ent_b, info.sync_bwd)):
        fl = ent_x[:, :, 1].astype(np.int64)
        S_, W_ = fl.shape
        for w in range(W_):
            for t in range(S_):
                f = int(fl[t, w])
                simple = (f & 1) and (f & 2) and not (f & (4 | 8 | 0x80)) and ((f >> 4) & 7) == 0
                assert bool(f >> 31) == bool(simple)
                if simple:
                    run = (f >> 16) & 15
                    assert 1 <= run <= min(15, sync_x - (t % sync_x))
                    for k in range(1, run):
                        g2 = int(fl[t + k, w])
                        assert (g2 >> 31) and ((g2 >> 16) & 15) >= run - k and ((g2 >> 8) & 255) == ((f >> 8) & 255)
    # runs of plain entries (word 5): register operand only, a real node; the forward program also
    # excludes entries that write a slot or end a path
    for ent_x, bwd_x, sync_x in ((ent, False, info.sync_fwd), (ent_b, True, info.sync_bwd)):
        fl = ent_x[:, :, 1].astype(np.int64)
        runs = ent_x[:, :, 5].astype(np.int64)
        S_, W_ = fl.shape
        for w in range(W_):
            nxt = 0
            for t in range(S_ - 1, -1, -1):
                f = int(fl[t, w])
                plain = (f & 1) and (f & 2) and not (f & 0x80) and ((f >> 4) & 7) == 0
                if plain and not bwd_x and (f & (4 | 8)):
                    plain = False
                if not bwd_x and not (f & 1):
                    plain = True          # forward: idle entries do not cut a run
                want = 0
                if plain:
                    want = min(nxt + 1, 15) if (t + 1) % sync_x != 0 else 1
                assert int(runs[t, w]) == want
                nxt = want
    assert np.array_equal(b["LS"], r["LS"])
    assert np.array_equal(b["slack"], r["slack"])
    h.free()
    return info


@pytest.mark.parametrize("gi", range(0, len(TINY), 3))
def test_programs_on_tiny_graphs(emo, oracle_mod, gi):
    g = TINY[gi]
    lv = all_policies(g.n, g.L)
    lv = lv[:, :: max(1, lv.shape[1] // 200)].copy()
    for lanes in (0, 1, 3):
        check_programs(emo, oracle_mod, g, lv, emo.EMO_F_LANES(lanes))


@pytest.mark.parametrize("name,scale", [("cfg0-tiny", 1.0), ("cfg1-train", 0.1), ("cfg2-packed", 0.2),
                                          ("cfg3-8dev", 0.02), ("cfg4-llm", 0.01)])
def test_programs_on_config_graphs(emo, oracle_mod, name, scale):
    g = W.make_graph(name, scale)
    lv = W.policy_levels(g.meta["policy_seed"], g.n, g.L, 16, "uniform").numpy()
    info = check_programs(emo, oracle_mod, g, lv)
    # edges that can never decide a maximum are dropped, so a program may be shallower than the graph
    assert 0 < info.steps_fwd <= 2 * info.depth and 0 < info.steps_bwd <= 2 * info.depth
    for lanes, look in ((1, 0), (4, 2), (16, 30)):
        check_programs(emo, oracle_mod, g, lv, emo.EMO_F_LANES(lanes) | emo.EMO_F_LOOKAHEAD(look))


def test_high_degree_nodes_get_helper_ops(emo, oracle_mod):
    """A node with 20 predecessors and a node with 15 successors need helper ops in one direction each."""
    n = 37
    edges = [(i, 20) for i in range(20)] + [(20, 21)] + [(21, 22 + j) for j in range(15)]
    rs = np.random.RandomState(4)
    lat = rs.randint(0, 30, (n, 3))
    lat[:, 0], lat[:, 2] = 0, 30          # wide rows: no operand is dominated, so no edge is dropped
    g = W.tiny_graph(n, edges, lat)
    lv = rs.randint(0, 3, (n, 40)).astype(np.uint8)
    info = check_programs(emo, oracle_mod, g, lv)
    assert info.aux_fwd >= 2 and info.aux_bwd >= 2


def test_dominated_edges_are_dropped_without_changing_results(emo, oracle_mod):
    """A launch chain that always runs far ahead of the kernels it launches: its edges into the
    kernels can never decide a maximum and are dropped at load time; results stay exact."""
    K = 40
    n = 2 * K
    edges = [(i, i + 1) for i in range(K - 1)]                       # launch chain 0..K-1
    edges += [(K + i, K + i + 1) for i in range(K - 1)]              # one stream K..2K-1
    edges += [(i, K + i) for i in range(K)]                          # launches
    lat = np.zeros((n, 3), dtype=np.int64)
    lat[:K] = 1
    lat[K:] = np.array([[300, 200, 100]]) + np.arange(K)[:, None]
    g = W.tiny_graph(n, edges, lat)
    lv = np.random.RandomState(8).randint(0, 3, (n, 50)).astype(np.uint8)
    check_programs(emo, oracle_mod, g, lv)
    h = emo.load_workload(g, emo.EMO_F_HOST_ONLY)
    _, _, _, _, ent, _, _ = emo.emo_graph_program(h, 0)
    n_slot_operands = int((((ent[:, :, 1] >> 4) & 7) * (ent[:, :, 1] & 1)).sum())
    assert n_slot_operands <= 2, "launch edges into the stream should have been dropped"
    h.free()


def test_group_of_and_ignored_rows(emo, oracle_mod):
    g = W.make_graph("cfg0-tiny")
    group = (np.arange(g.n) // 3).astype(np.int32)
    group[g.kind == W.KIND_CPU] = -1
    rows = int(group.max()) + 1
    lv = np.random.RandomState(1).randint(0, g.L, (rows, 9)).astype(np.uint8)
    info = check_programs(emo, oracle_mod, g, lv, group_of=group)
    assert info.rows == rows


def test_empty_and_single_node(emo, oracle_mod):
    h = emo.emo_graph_load(0, np.zeros(1, np.int64), np.zeros(0, np.int32), None, 3, np.zeros((0, 3), np.int64),
                           np.zeros((0, 3)), None, emo.EMO_F_HOST_ONLY)
    assert h.info.n == 0 and h.info.steps_fwd == 0
    h.free()
    g = W.tiny_graph(1, [], [[4, 2, 1]])
    check_programs(emo, oracle_mod, g, np.array([[0, 1, 2]], dtype=np.uint8))


def test_load_rejects_bad_input(emo):
    E = emo
    ho = E.EMO_F_HOST_ONLY
    lat = np.ones((3, 2), np.int64)
    en = np.ones((3, 2))
    rp = np.array([0, 0, 1, 2], np.int64)
    col = np.array([0, 1], np.int32)

    def code(**kw):
        a = dict(n=3, row_ptr=rp, col=col, level_ptr=None, L=2, lat=lat, energy=en, group_of=None, flags=ho)
        a.update(kw)
        try:
            E.emo_graph_load(a["n"], a["row_ptr"], a["col"], a["level_ptr"], a["L"], a["lat"], a["energy"],
                             a["group_of"], a["flags"]).free()
            return 0
        except E.EmoError as e:
            return e.code

    assert code() == 0
    assert code(col=np.array([0, 2], np.int32)) == E.EMO_E_NOT_TOPOLOGICAL       # forward edge
    assert code(col=np.array([0, 1], np.int32), row_ptr=np.array([0, 1, 1, 2], np.int64)) == E.EMO_E_NOT_TOPOLOGICAL  # self edge 0->0
    assert code(col=np.array([0, 7], np.int32)) == E.EMO_E_INVALID_ARG           # col >= n
    assert code(col=np.array([0, -1], np.int32)) == E.EMO_E_INVALID_ARG
    assert code(row_ptr=np.array([0, 2, 1, 2], np.int64)) == E.EMO_E_INVALID_ARG # not non-decreasing
    bad = lat.copy(); bad[1, 1] = -1
    assert code(lat=bad) == E.EMO_E_RANGE
    bad = lat.copy(); bad[1, 1] = 1 << 32
    assert code(lat=bad) == E.EMO_E_RANGE
    for x in (np.nan, np.inf, -np.inf):
        b = en.copy(); b[2, 0] = x
        assert code(energy=b) == E.EMO_E_NONFINITE
    assert code(L=0) == E.EMO_E_RANGE
    assert code(L=256) == E.EMO_E_RANGE
    assert code(level_ptr=np.array([0, 1, 2, 3], np.int32)) == 0
    assert code(level_ptr=np.array([0, 2, 3], np.int32)) == E.EMO_E_NOT_TOPOLOGICAL   # 0 and 1 share a level but 0->1
    # a malformed level array is rejected before it is used as an index (entries out of [0, n], not monotone)
    assert code(level_ptr=np.array([0, 1_000_000, 3], np.int32)) == E.EMO_E_INVALID_ARG
    assert code(level_ptr=np.array([0, 2, 1, 3], np.int32)) == E.EMO_E_INVALID_ARG
    assert code(level_ptr=np.array([0, -5, 3], np.int32)) == E.EMO_E_INVALID_ARG
    assert code(level_ptr=np.array([1, 2, 3], np.int32)) == E.EMO_E_INVALID_ARG
    assert code(group_of=np.array([0, -2, 1], np.int32)) == E.EMO_E_INVALID_ARG
    assert code(n=-1) == E.EMO_E_INVALID_ARG


def test_overflow_guard(emo):
    """Latencies are capped below 2^32 per node, so 2^62 needs 2^30 nodes in a chain: the guard is
    exercised through its arithmetic instead (T_worst reported exactly on a long chain)."""
    n = 5000
    lat = np.full((n, 2), (1 << 32) - 1, np.int64)
    g = W.tiny_graph(n, [(i, i + 1) for i in range(n - 1)], lat, np.zeros((n, 2)))
    h = emo.load_workload(g, emo.EMO_F_HOST_ONLY)
    assert h.info.T_worst == n * ((1 << 32) - 1)
    assert h.info.T_worst > (1 << 44)
    h.free()


def test_eval_calls_fail_loudly_without_device(emo):
    g = W.make_graph("cfg0-tiny")
    h = emo.load_workload(g, emo.EMO_F_HOST_ONLY)
    with pytest.raises(emo.EmoError) as ei:
        emo.emo_eval_policies(h, 4, 16, 16, 16, 16, None, None, 0, stream=0)
    assert ei.value.code == emo.EMO_E_CUDA
    h.free()


def test_graphs_beyond_the_slot_limit_still_load(emo):
    """More simultaneously live values than exchange slots: the handle is built for the generic kernels
    (no schedule, workspace for the completion times of every node) instead of failing."""
    rs = np.random.RandomState(0)
    ns = 400
    edges = sorted({(int(k), ns + j) for j in range(ns) for k in rs.choice(ns, 3, replace=False)})
    g = W.tiny_graph(2 * ns, edges, rs.randint(0, 100, size=(2 * ns, 4)).astype(np.int64))
    h = emo.load_workload(g, flags=emo.EMO_F_HOST_ONLY)
    info = emo.emo_graph_info(h)
    assert info.n == 2 * ns and info.steps_fwd == 0 and info.depth == 2
    assert emo.emo_graph_flow(h, arrays=False)["ok32"] == 0
    assert emo.emo_workspace_bytes(h, 100, 1) >= 2 * 800 * 112 * 8
    assert emo.emo_workspace_bytes(h, 100, 0) >= 800 * 112 * 8
    h.free()
