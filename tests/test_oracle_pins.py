"""Pins for the CPU oracle: it is checked against things other than itself.

Brute-force path enumeration on tiny DAGs over all 3^n policies, closed forms (chain, fork-join,
series composition, uniform-level energy), the reversal duality of the backward pass, invariants
(slack >= 0, zero exactly on longest paths, monotonicity, relabelling, scaling), a library
longest-path routine, an exactly rounded sum, and a hand-worked example.
"""
from __future__ import annotations

import itertools
import json
import math
import os

import numpy as np
import pytest

from paper_2607_12324_b200 import workloads as W
from tests import bruteforce

HERE = os.path.dirname(os.path.abspath(__file__))


def preds_of(g):
    return [g.preds(v).tolist() for v in range(g.n)]


def all_policies(n, L):
    """uint8 [n][L**n]: column b is the b-th assignment of levels to nodes."""
    P = L ** n
    b = np.arange(P, dtype=np.int64)
    out = np.empty((n, P), dtype=np.uint8)
    for v in range(n):
        out[v] = (b // (L ** v)) % L
    return out


def tiny_family():
    gs = []
    sid = 0
    for n in range(1, 9):
        for p in (0.15, 0.3, 0.6):
            for rep in range(2 if n < 8 else 3):
                gs.append(W.random_dag(1000 + sid, n, p, L=3, max_dur=20, monotone=(rep != 1)))
                sid += 1
    one = lambda n, e, lat: W.tiny_graph(n, e, lat)
    r = np.random.RandomState(7)
    gs.append(one(1, [], [[4, 2, 1]]))                                             # single node
    gs.append(one(8, [(i, i + 1) for i in range(7)], r.randint(0, 9, (8, 3))))     # chain
    gs.append(one(8, [(0, 1), (1, 2), (2, 3), (0, 4), (4, 5), (5, 6), (3, 7), (6, 7)],
                  r.randint(0, 9, (8, 3))))                                        # two chains and a join
    gs.append(one(5, [(0, 1), (1, 2), (2, 4), (0, 3), (3, 4)], [[1] * 3, [5] * 3, [5] * 3, [1] * 3, [2] * 3]))
    gs.append(one(6, [(0, 2), (1, 2), (2, 3), (2, 4), (1, 5)], r.randint(0, 5, (6, 3))))   # 2 sources, 3 sinks
    gs.append(one(5, [(0, 1), (1, 2), (2, 3)], r.randint(1, 9, (5, 3))))           # isolated node beside a chain
    gs.append(one(4, [(0, 1), (0, 1), (1, 2), (0, 2), (2, 3)], r.randint(0, 9, (4, 3))))   # duplicated edge
    gs.append(one(6, [(0, 1), (0, 2), (1, 3), (2, 3), (3, 4), (3, 5)], np.zeros((6, 3))))  # all zero durations
    gs.append(one(6, [(0, 1), (0, 2), (1, 3), (2, 3), (3, 4), (3, 5)],
                  [[0, 0, 0], [3, 9, 1], [2, 2, 2], [0, 5, 0], [7, 1, 4], [1, 1, 1]]))     # non-monotone rows
    return gs


TINY = tiny_family()


@pytest.mark.parametrize("gi", range(len(TINY)))
def test_bruteforce_all_policies(oracle_mod, gi):
    """T, ES, slack of the oracle equal path enumeration for every one of the 3^n policies;
    slack >= 0; slack == 0 exactly on the nodes of a longest path; batch == singles."""
    g = TINY[gi]
    lv = all_policies(g.n, g.L)
    P = lv.shape[1]
    r = oracle_mod.batch(g, lv, want_arrays=True)
    dur = np.stack([g.lat[v, lv[v]] for v in range(g.n)], axis=1)          # [P][n]
    T, ES, slack = bruteforce.evaluate(g.n, preds_of(g), dur)
    assert np.array_equal(r["makespan"], T)
    assert np.array_equal(r["ES"].T, ES)
    assert np.array_equal(r["slack"].T, slack)
    assert np.array_equal(r["LS"], r["slack"] + r["ES"])
    assert (r["slack"] >= 0).all()
    assert np.array_equal(r["slack_sum"], slack.sum(axis=1))
    assert np.array_equal(r["n_critical"], (slack == 0).sum(axis=1))
    # energy: plain definition, exactly rounded
    for b in range(0, P, max(1, P // 50)):
        want = math.fsum(g.energy[v, lv[v, b]] for v in range(g.n))
        assert r["energy"][b] == pytest.approx(want, rel=1e-15, abs=1e-300)
    # one policy evaluated alone gives the same as inside the batch
    for b in (0, P // 2, P - 1):
        single = oracle_mod.batch(g, lv[:, b:b + 1].copy(), want_arrays=True)
        assert single["makespan"][0] == r["makespan"][b]
        assert np.array_equal(single["slack"][:, 0], r["slack"][:, b])


def test_hand_worked_example(oracle_mod):
    """Values derived by hand in tests/golden/hand_worked_dag.json (Eq. 1, Eq. 2, backward pass, Eq. 4)."""
    with open(os.path.join(HERE, "golden", "hand_worked_dag.json")) as f:
        gold = json.load(f)
    n = len(gold["nodes"])
    g = W.tiny_graph(n, gold["edges_pred_succ"], gold["lat"], gold["energy"])
    lv = np.array([p["levels"] for p in gold["policies"]], dtype=np.uint8).T.copy()
    r = oracle_mod.batch(g, lv, want_arrays=True)
    for b, p in enumerate(gold["policies"]):
        assert r["makespan"][b] == p["T"]
        assert r["energy"][b] == p["E"]
        assert r["ES"][:, b].tolist() == p["ES"]
        assert r["LS"][:, b].tolist() == p["LS"]
        assert r["slack"][:, b].tolist() == p["slack"]
    for s in gold["selection"]:
        tgt = oracle_mod.target_from_delta(r["makespan"][0], s["delta_ppm"])
        assert tgt == s["target"]
        assert oracle_mod.select(r["makespan"], r["energy"], tgt) == s["index"]


def test_chain_closed_form(oracle_mod):
    """A single-stream chain: T = sum of durations, ES = prefix sums, every slack 0."""
    n, L = 50, 4
    lat = (W.rand_u64(3, 1, np.arange(n * L)) % np.uint64(1000)).astype(np.int64).reshape(n, L)
    g = W.tiny_graph(n, [(i, i + 1) for i in range(n - 1)], lat)
    lv = (W.rand_u64(3, 2, np.arange(n * 16)) % np.uint64(L)).astype(np.uint8).reshape(n, 16)
    r = oracle_mod.batch(g, lv, want_arrays=True)
    dur = np.stack([lat[v, lv[v]] for v in range(n)], axis=0)        # [n][16]
    assert np.array_equal(r["makespan"], dur.sum(axis=0))
    assert np.array_equal(r["ES"], np.cumsum(dur, axis=0) - dur)
    assert (r["slack"] == 0).all()


def test_fork_join_closed_form(oracle_mod):
    """source -> k parallel chains -> sink: T = d_src + max_i sum(chain_i) + d_sink; a chain's
    nodes all have slack (longest chain) - (this chain)."""
    k, ln = 4, 5
    n = 2 + k * ln
    rs = np.random.RandomState(11)
    lat = rs.randint(1, 50, (n, 2)).astype(np.int64)
    edges = []
    for c in range(k):
        first = 1 + c * ln
        edges.append((0, first))
        for j in range(ln - 1):
            edges.append((first + j, first + j + 1))
        edges.append((first + ln - 1, n - 1))
    g = W.tiny_graph(n, edges, lat)
    lv = rs.randint(0, 2, (n, 32)).astype(np.uint8)
    r = oracle_mod.batch(g, lv, want_arrays=True)
    for b in range(32):
        d = lat[np.arange(n), lv[:, b]]
        sums = [d[1 + c * ln:1 + (c + 1) * ln].sum() for c in range(k)]
        assert r["makespan"][b] == d[0] + max(sums) + d[n - 1]
        for c in range(k):
            assert (r["slack"][1 + c * ln:1 + (c + 1) * ln, b] == max(sums) - sums[c]).all()
        assert r["slack"][0, b] == 0 and r["slack"][n - 1, b] == 0


def test_series_composition(oracle_mod):
    """Two DAGs joined through a single cut node: T = T(left incl. cut) + T(right)."""
    a = W.random_dag(77, 7, 0.4, L=2)
    b = W.random_dag(78, 7, 0.4, L=2)
    ea, eb = a.edges(), b.edges()
    na, nb = a.n, b.n
    cut = na
    sinks_a = [v for v in range(na) if all(v != p for p, _ in ea)]
    sources_b = [v for v in range(nb) if len(b.preds(v)) == 0]
    edges = list(ea) + [(s, cut) for s in sinks_a] + [(cut, cut + 1 + s) for s in sources_b] + \
        [(cut + 1 + p, cut + 1 + s) for p, s in eb]
    lat = np.concatenate([a.lat, np.array([[3, 1]]), b.lat])
    g = W.tiny_graph(na + 1 + nb, edges, lat)
    rs = np.random.RandomState(5)
    lv = rs.randint(0, 2, (g.n, 20)).astype(np.uint8)
    r = oracle_mod.batch(g, lv)
    ra = oracle_mod.batch(a, lv[:na].copy())
    rb = oracle_mod.batch(b, lv[na + 1:].copy())
    dcut = lat[cut, lv[cut]]
    assert np.array_equal(r["makespan"], ra["makespan"] + dcut + rb["makespan"])


@pytest.mark.parametrize("name,scale", [("cfg0-tiny", 1.0), ("cfg1-train", 0.1), ("cfg3-8dev", 0.02), ("cfg4-llm", 0.005)])
def test_reversal_duality_and_edge_conditions(oracle_mod, name, scale):
    """LS_v(G) = T - C_v(G reversed): the backward pass re-derived with the forward routine only.
    Also the edge inequalities of ES and LS with equality on at least one edge."""
    g = W.make_graph(name, scale)
    B = 6
    lv = W.policy_levels(g.meta["policy_seed"], g.n, g.L, max(B, 8), "uniform", cols=(0, B)).numpy()
    r = oracle_mod.batch(g, lv, want_arrays=True)
    # reversed graph in pred-CSR: predecessors of v in G^R = successors of v in G
    succs = [[] for _ in range(g.n)]
    for v in range(g.n):
        for k in g.preds(v):
            succs[int(k)].append(v)
    rp = np.zeros(g.n + 1, dtype=np.int64)
    rp[1:] = np.cumsum([len(s) for s in succs])
    col = np.array([u for s in succs for u in s], dtype=np.int32)
    for b in range(B):
        dur = g.lat[np.arange(g.n), lv[:, b]]
        T, ES, C = oracle_mod.forward(g.n, g.row_ptr, g.col, dur)
        Tr, ESr, Cr = oracle_mod.forward(g.n, rp, col, dur)
        assert T == Tr == r["makespan"][b]
        assert np.array_equal(r["LS"][:, b], T - Cr)
        assert np.array_equal(r["ES"][:, b], ES)
        LS = r["LS"][:, b]
        assert (LS - ES >= 0).all()
        v_of_edge = np.repeat(np.arange(g.n), np.diff(g.row_ptr))
        k_of_edge = g.col.astype(np.int64)
        assert (ES[k_of_edge] + dur[k_of_edge] <= ES[v_of_edge]).all()
        assert (LS[k_of_edge] + dur[k_of_edge] <= LS[v_of_edge]).all()
        tight_in = np.zeros(g.n, dtype=bool)
        np.logical_or.at(tight_in, v_of_edge, ES[k_of_edge] + dur[k_of_edge] == ES[v_of_edge])
        has_pred = np.diff(g.row_ptr) > 0
        assert (tight_in[has_pred]).all() and (ES[~has_pred] == 0).all()
        tight_out = np.zeros(g.n, dtype=bool)
        np.logical_or.at(tight_out, k_of_edge, LS[k_of_edge] + dur[k_of_edge] == LS[v_of_edge])
        has_succ = np.zeros(g.n, dtype=bool)
        has_succ[k_of_edge] = True
        assert tight_out[has_succ].all()
        assert (LS[~has_succ] + dur[~has_succ] == T).all()
        assert (r["slack"][:, b] == 0).sum() >= 1


def test_networkx_longest_path(oracle_mod):
    """Makespan against a textbook library routine on the edge-weighted transform
    (w(u->v) = dur_v, super-source edges w = dur_source)."""
    nx = pytest.importorskip("networkx")
    g = W.make_graph("cfg0-tiny")
    lv = W.policies_for(g, B=8).numpy()
    r = oracle_mod.batch(g, lv, B=8)
    for b in range(8):
        dur = g.lat[np.arange(g.n), lv[:, b]]
        G = nx.DiGraph()
        G.add_node("S")
        for v in range(g.n):
            ps = g.preds(v)
            if len(ps) == 0:
                G.add_edge("S", v, weight=int(dur[v]))
            for k in ps:
                G.add_edge(int(k), v, weight=int(dur[v]))
        assert nx.dag_longest_path_length(G, weight="weight") == r["makespan"][b]


def test_monotone_relabel_scale(oracle_mod):
    """Raising one node's level never increases T when its latency row is non-increasing;
    relabelling to another topological order and scaling all latencies by an integer behave
    as they must."""
    g = W.make_graph("cfg1-train", 0.06)
    n, L = g.n, g.L
    assert (np.diff(g.lat, axis=1) <= 0).all()
    rs = np.random.RandomState(3)
    base = rs.randint(0, L, n).astype(np.uint8)
    nodes = rs.choice(n, 48, replace=False)
    lv = np.repeat(base[:, None], 1 + len(nodes), axis=1)
    for j, v in enumerate(nodes):
        lv[v, 1 + j] = min(L - 1, int(base[v]) + 1 + rs.randint(0, 3))
    r = oracle_mod.batch(g, lv, want_arrays=True)
    assert (r["makespan"][1:] <= r["makespan"][0]).all()
    # relabel: random topological order (Kahn with random tie-break)
    order = random_topo(g, rs)
    new_of_old = np.empty(n, dtype=np.int64)
    new_of_old[order] = np.arange(n)
    edges = [(new_of_old[p], new_of_old[s]) for p, s in g.edges()]
    g2 = W.tiny_graph(n, edges, g.lat[order], g.energy[order])
    r2 = oracle_mod.batch(g2, lv[order], want_arrays=True)
    assert np.array_equal(r2["makespan"], r["makespan"])
    assert np.array_equal(r2["slack"], r["slack"][order])
    assert np.array_equal(r2["ES"], r["ES"][order])
    assert r2["energy"] == pytest.approx(r["energy"], rel=1e-13)
    # scaling
    g3 = W.tiny_graph(n, g.edges(), g.lat * 7, g.energy)
    r3 = oracle_mod.batch(g3, lv, want_arrays=True)
    for k in ("makespan", "ES", "LS", "slack"):
        assert np.array_equal(r3[k], 7 * r[k])


def random_topo(g, rs):
    indeg = np.diff(g.row_ptr).astype(np.int64).copy()
    succs = [[] for _ in range(g.n)]
    for v in range(g.n):
        for k in g.preds(v):
            succs[int(k)].append(v)
    ready = [v for v in range(g.n) if indeg[v] == 0]
    out = []
    while ready:
        i = rs.randint(len(ready))
        v = ready.pop(i)
        out.append(v)
        for u in succs[v]:
            indeg[u] -= 1
            if indeg[u] == 0:
                ready.append(u)
    assert len(out) == g.n
    return np.asarray(out)


def test_energy_closed_forms(oracle_mod):
    """Uniform level l: E = sum_v energy[v][l] = P(f_l) * sum_kernels lat * 1e-9 for the generator's
    tables; E does not depend on the edges; permuting policies permutes the outputs."""
    g = W.make_graph("cfg1-train", 0.2)
    n, L = g.n, g.L
    lv = np.repeat(np.arange(L, dtype=np.uint8)[None, :], n, axis=0)
    r = oracle_mod.batch(g, lv)
    f = W.frequencies_mhz(L)
    power = W.P_STATIC_W + W.P_DYN_W_AT_FMAX / W.F_MAX_MHZ ** 3 * f ** 3
    isk = g.kind == W.KIND_KERNEL
    for l in range(L):
        assert r["energy"][l] == pytest.approx(math.fsum(g.energy[:, l]), rel=1e-15)
        assert r["energy"][l] == pytest.approx(power[l] * g.lat[isk, l].sum() * 1e-9, rel=1e-12)
    rs = np.random.RandomState(9)
    lv2 = rs.randint(0, L, (n, 12)).astype(np.uint8)
    r2 = oracle_mod.batch(g, lv2)
    chain = W.tiny_graph(n, [(i, i + 1) for i in range(n - 1)], g.lat, g.energy)
    r3 = oracle_mod.batch(chain, lv2)
    assert np.array_equal(r2["energy"], r3["energy"])
    perm = rs.permutation(12)
    r4 = oracle_mod.batch(g, lv2[:, perm].copy())
    assert np.array_equal(r4["energy"], r2["energy"][perm])
    assert np.array_equal(r4["makespan"], r2["makespan"][perm])


def test_energy_sum_is_compensated(oracle_mod):
    """The fp64 sum is within one rounding of the exactly rounded sum even when naive summation
    is not."""
    x = np.array([1e16, 1.0, -1e16, 1.0] * 1000 + [0.1] * 1000)
    assert oracle_mod.energy_sum(x) == pytest.approx(math.fsum(x), rel=1e-15)
    y = W.rand_uniform(1, 9, np.arange(250_000)) * 1e-3
    assert oracle_mod.energy_sum(y) == pytest.approx(math.fsum(y), rel=2e-16)


def test_padding_and_groups(oracle_mod):
    """Padding columns (ldb > B) are never read; group_of maps nodes to shared policy rows and a
    negative group ignores the policy."""
    g = W.make_graph("cfg0-tiny")
    lv = W.policies_for(g, B=20, ldb=32).numpy()
    assert (lv[:, 20:] == 0xFF).all()
    r = oracle_mod.batch(g, lv, B=20)
    r2 = oracle_mod.batch(g, np.ascontiguousarray(lv[:, :20]), B=20)
    assert np.array_equal(r["makespan"], r2["makespan"])
    with pytest.raises(oracle_mod.OracleError):
        oracle_mod.batch(g, lv, B=21)                      # reads a padding column: level 255 >= L
    group = (np.arange(g.n) // 2).astype(np.int32)
    group[g.kind == W.KIND_CPU] = -1
    rows = int(group.max()) + 1
    lvg = np.random.RandomState(2).randint(0, g.L, (rows, 5)).astype(np.uint8)
    rg = oracle_mod.batch(g, lvg, group_of=group)
    expanded = np.zeros((g.n, 5), dtype=np.uint8)
    for v in range(g.n):
        expanded[v] = lvg[group[v]] if group[v] >= 0 else 0
    re = oracle_mod.batch(g, expanded)
    assert np.array_equal(rg["makespan"], re["makespan"])
    assert np.array_equal(rg["energy"], re["energy"])


def test_target_rounding(oracle_mod):
    assert oracle_mod.target_from_delta(1000, 30_000) == 1030
    assert oracle_mod.target_from_delta(1001, 30_000) == 1001 + 30          # floor(30.03)
    assert oracle_mod.target_from_delta(33, 30_000) == 33                   # floor(0.99)
    assert oracle_mod.target_from_delta(0, 50_000) == 0
    big = (1 << 61) + 12345
    assert oracle_mod.target_from_delta(big, 50_000) == big + (big * 50_000) // 1_000_000
    assert oracle_mod.target_from_delta(777, 0) == 777


def test_selection_cases(oracle_mod):
    T = np.array([100, 105, 103, 103, 99, 110], dtype=np.int64)
    E = np.array([9.0, 5.0, 7.0, 7.0, 9.5, 1.0])
    brute = lambda tgt: min([(E[b], b) for b in range(len(T)) if T[b] <= tgt], default=(None, -1))[1]
    for tgt in (98, 99, 100, 102, 103, 104, 105, 109, 110, 1000):
        assert oracle_mod.select(T, E, tgt) == brute(tgt)
    assert oracle_mod.select(T, E, 98) == -1                                 # none feasible
    assert oracle_mod.select(T, E, 99) == 4                                  # exactly one
    assert oracle_mod.select(T, E, 103) == 2                                 # exact tie -> lowest index
    assert oracle_mod.select(T, E, 105) == 1                                 # T == target is feasible
    assert oracle_mod.select(T[:1], E[:1], 100) == 0                         # B = 1
    assert oracle_mod.select(T[:0], E[:0], 100) == -1                        # B = 0
    e2 = np.array([1.0, np.nextafter(1.0, 0.0), 1.0])
    assert oracle_mod.select(np.array([1, 1, 1], dtype=np.int64), e2, 1) == 1    # one ulp matters
    # delta = 0 selects among T <= T0; the all-max policy (index 0) is always feasible
    assert oracle_mod.select(T, E, oracle_mod.target_from_delta(T[0], 0)) == brute(100)


def test_packed_graph_bounds_unpacked(oracle_mod):
    """Packing only drops edges and contracts chains: T_packed(P) <= T_unpacked(expand(P)); the
    pack table is the per-level sum of the members' tables."""
    scale = 0.1
    base = W.make_graph("cfg1-train", scale)
    pk = W.make_graph("cfg2-packed", scale)
    assert np.array_equal(base.lat, W.make_graph("cfg1-train", scale).lat)
    B = 24
    lvp = W.policy_levels(5, pk.n, pk.L, B, "mixed", 0.3).numpy()
    expanded = np.full((base.n, B), pk.L - 1, dtype=np.uint8)
    for j, members in enumerate(pk.meta["pack_members"]):
        pid = pk.meta["pack_new_id"][j]
        expanded[np.asarray(members)] = lvp[pid]
        assert np.array_equal(pk.lat[pid], base.lat[np.asarray(members)].sum(axis=0))
    rp = oracle_mod.batch(pk, lvp)
    rb = oracle_mod.batch(base, expanded)
    assert (rp["makespan"] <= rb["makespan"]).all()
    assert rp["makespan"][0] >= 0.98 * rb["makespan"][0]
    assert rp["energy"] == pytest.approx(rb["energy"], rel=1e-12)


def test_cycle_and_range_are_reported(oracle_mod):
    rp = np.array([0, 1, 2], dtype=np.int64)
    col = np.array([1, 0], dtype=np.int32)
    with pytest.raises(oracle_mod.OracleError):
        oracle_mod.topo_order(2, rp, col)
    with pytest.raises(oracle_mod.OracleError):
        oracle_mod.topo_order(2, rp, np.array([5, 0], dtype=np.int32))
