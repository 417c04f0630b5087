"""Pins of the oracle's critical-predecessor tracking (Eq. 5) and dependency-aware greedy packing (Sec. 4.4).

Independent checks: the critical predecessor against an arg-max written from Eq. 5 over completion times of
the pinned forward routine; the packs against a checker written from the three rules as the text states them
(not from the listing's loop), against maximality (every pack boundary is forced by a rule), against a case
worked by hand, and against what the rules are for: with only a pack's first incoming and last outgoing
dependencies kept, the makespan at the default frequency is unchanged."""
from __future__ import annotations

import numpy as np
import pytest

from paper_2607_12324_b200 import workloads as W


def stream_ids(g):
    """Global stream id per kernel (device timeline and stream together), -1 for other nodes."""
    st = np.asarray(g.meta["node_stream"], np.int64)
    tl = np.asarray(g.meta.get("node_timeline", np.zeros(g.n, np.int64)), np.int64)
    ns = int(g.meta.get("n_streams", int(st.max()) + 1))
    return np.where(g.kind == W.KIND_KERNEL, tl * ns + st, -1).astype(np.int32)


def succ_lists(g):
    out = [[] for _ in range(g.n)]
    for v in range(g.n):
        for k in g.preds(v):
            out[int(k)].append(v)
    return out


def check_rules(g, is_kernel, stream_of, t, crit, pack_of, delta_max):
    """The three rules as the text states them, and maximality of the greedy choice."""
    succ = succ_lists(g)
    crit_succ = [[u for u in succ[v] if crit[u] == v] for v in range(g.n)]
    packs = {}
    for v in range(g.n):
        if is_kernel[v]:
            assert pack_of[v] >= 0
            packs.setdefault(int(pack_of[v]), []).append(v)
        else:
            assert pack_of[v] == -1
    assert sorted(packs) == list(range(len(packs)))
    firsts = [min(m) for _, m in sorted(packs.items())]
    assert firsts == sorted(firsts), "packs are numbered by their first member"
    by_stream = {}
    for v in range(g.n):
        if is_kernel[v]:
            by_stream.setdefault(int(stream_of[v]), []).append(v)
    pos = {v: (s, i) for s, vs in by_stream.items() for i, v in enumerate(vs)}

    def r1(v):
        return crit[v] >= 0 and is_kernel[crit[v]] and stream_of[crit[v]] == stream_of[v]

    def r2(u):
        return all(is_kernel[w] and stream_of[w] == stream_of[u] for w in crit_succ[u])

    for _, mem in packs.items():
        s, i0 = pos[mem[0]]
        assert [pos[v] for v in mem] == [(s, i0 + j) for j in range(len(mem))], "a pack is a stretch of one stream"
        for v in mem[1:]:
            assert r1(v), "rule 1: a non-initial member and its critical predecessor share a stream"
        for u in mem[:-1]:
            assert r2(u), "rule 2: every critical successor of a non-final member is in its stream"
        if len(mem) > 1:
            assert sum(int(t[v]) for v in mem) < delta_max, "rule 3: the pack stays below delta_max"
        # maximality: the kernel after the pack on the same stream could not have joined
        nxt = by_stream[s][i0 + len(mem)] if i0 + len(mem) < len(by_stream[s]) else None
        if nxt is not None:
            assert not (r1(nxt) and r2(mem[-1]) and sum(int(t[v]) for v in mem) + int(t[nxt]) < delta_max)
    return packs


def collapse_makespan(g, t, pack_of, packs):
    """Makespan at the given durations when every pack is one node that keeps only its first member's incoming
    and its last member's outgoing dependencies."""
    first = {p: m[0] for p, m in packs.items()}
    last = {p: m[-1] for p, m in packs.items()}
    C = {}
    key = lambda v: ("p", int(pack_of[v])) if pack_of[v] >= 0 else ("n", v)
    dur = {("p", p): sum(int(t[v]) for v in m) for p, m in packs.items()}
    preds = {}
    for v in range(g.n):
        kv = key(v)
        preds.setdefault(kv, set())
        if pack_of[v] >= 0 and v != first[int(pack_of[v])]:
            continue
        for k in g.preds(v):
            k = int(k)
            if pack_of[k] >= 0 and (k != last[int(pack_of[k])] or pack_of[k] == pack_of[v]):
                continue
            preds[kv].add(key(k))
    order = sorted(preds, key=lambda kk: first[kk[1]] if kk[0] == "p" else kk[1])
    T = 0
    for kk in order:
        start = max([C[q] for q in preds[kk]], default=0)
        C[kk] = start + (dur[kk] if kk[0] == "p" else int(t[kk[1]]))
        T = max(T, C[kk])
    return T


@pytest.mark.parametrize("seed", range(6))
def test_critical_predecessor_is_the_argmax(oracle_mod, seed):
    g = W.random_dag(seed, 40, 0.15, L=3, max_dur=6)       # small durations: many ties
    dur = g.lat[:, 1].copy()
    C, crit = oracle_mod.crit_pred(g, dur)
    lv = np.ones((g.n, 1), np.uint8)
    ref = oracle_mod.batch(g, lv, want_arrays=True)
    assert np.array_equal(C, ref["ES"][:, 0] + dur)
    for v in range(g.n):
        ps = [int(k) for k in g.preds(v)]
        if not ps:
            assert crit[v] == -1
            continue
        best = max(C[k] for k in ps)
        assert crit[v] == min(k for k in ps if C[k] == best)      # ties: the one processed first


def test_hand_worked_packing(oracle_mod):
    """Worked by hand.  Nodes: 0, 1 CPU launches (0 -> 1); stream 0 holds kernels 2, 3, 6, 7 in that order, stream 1
    kernels 4, 5 (and 8 in the second case).  Edges: 0->2, 2->3, 3->6, 6->7 (stream 0), 1->4, 4->5 (stream 1), and
    5->6 (kernel 6 waits for the other stream).  Durations 1, 1, 3, 4, 9, 8, 6, 5: completions 1, 2, 4, 8, 11, 19, 25, 30;
    critical predecessors -, 0, 0, 2, 1, 4, 5, 6.
    delta_max = 10: 2 opens a pack, 3 joins (3 + 4 < 10); 6's critical predecessor is kernel 5 of the other stream
    (rule 1): new pack; 7 would make 6 + 5 = 11: new pack; on stream 1, 5 would make 9 + 8 = 17: new pack.
    delta_max = 18: {2, 3}, {6, 7}, {4, 5}.
    With kernel 8 after 5 on stream 1 and delta_max = 30: 5 is the critical predecessor of 6, which is in another
    stream, so nothing may follow 5 in its pack (rule 2): {4, 5} and {8}."""
    n = 8
    edges = [(0, 1), (0, 2), (2, 3), (3, 6), (6, 7), (1, 4), (4, 5), (5, 6)]
    t = np.array([1, 1, 3, 4, 9, 8, 6, 5], np.int64)
    g = W.tiny_graph(n, edges, np.stack([t, t], axis=1))
    is_kernel = np.array([0, 0, 1, 1, 1, 1, 1, 1], np.uint8)
    stream_of = np.array([-1, -1, 0, 0, 1, 1, 0, 0], np.int32)
    C, crit = oracle_mod.crit_pred(g, t)
    assert C.tolist() == [1, 2, 4, 8, 11, 19, 25, 30]
    assert crit.tolist() == [-1, 0, 0, 2, 1, 4, 5, 6]
    pack_of, cnt = oracle_mod.pack_greedy(g, is_kernel, stream_of, t, crit, 10)
    assert pack_of.tolist() == [-1, -1, 0, 0, 1, 2, 3, 4] and cnt == 5
    pack_of, cnt = oracle_mod.pack_greedy(g, is_kernel, stream_of, t, crit, 18)
    assert pack_of.tolist() == [-1, -1, 0, 0, 1, 1, 2, 2] and cnt == 3
    check_rules(g, is_kernel, stream_of, t, crit, pack_of, 18)
    t2 = np.append(t, 1)
    g2 = W.tiny_graph(9, edges + [(5, 8)], np.stack([t2, t2], axis=1))
    isk2, so2 = np.append(is_kernel, 1).astype(np.uint8), np.append(stream_of, 1).astype(np.int32)
    C2, crit2 = oracle_mod.crit_pred(g2, t2)
    assert crit2.tolist() == [-1, 0, 0, 2, 1, 4, 5, 6, 5]
    pack_of, cnt = oracle_mod.pack_greedy(g2, isk2, so2, t2, crit2, 30)
    assert pack_of.tolist() == [-1, -1, 0, 0, 1, 1, 2, 2, 3] and cnt == 4


@pytest.mark.parametrize("name,scale", [("cfg0-tiny", 1.0), ("cfg1-train", 0.2), ("cfg3-8dev", 0.02), ("cfg4-llm", 0.01)])
@pytest.mark.parametrize("delta_ms", [0.05, 5.0])
def test_rules_and_purpose_on_config_graphs(oracle_mod, name, scale, delta_ms):
    g = W.make_graph(name, scale)
    is_kernel = (g.kind == W.KIND_KERNEL).astype(np.uint8)
    stream_of = stream_ids(g)
    t = g.lat[:, g.L - 1].copy()
    C, crit = oracle_mod.crit_pred(g, t)
    delta_max = int(delta_ms * 1e6)
    pack_of, cnt = oracle_mod.pack_greedy(g, is_kernel, stream_of, t, crit, delta_max)
    packs = check_rules(g, is_kernel, stream_of, t, crit, pack_of, delta_max)
    assert cnt == len(packs)
    # what the rules are for: the dropped dependencies are never critical at the default frequency
    assert collapse_makespan(g, t, pack_of, packs) == int(C.max())
    if delta_ms == 5.0:
        assert cnt < int(is_kernel.sum()), "with 5 ms some kernels do pack"
