"""Pins of the oracle's time-interval routine (Alg. 1 with a policy of change points, idle energy of Eq. 2).

The routine is checked against things other than itself: a case worked by hand, the per-node-level oracle
(itself pinned by brute force) fed with the levels the policy realised, closed forms on chains, a
nanosecond-by-nanosecond occupancy count, and invariances that a wrong interval search, a wrong boundary or a
dropped term would break."""
from __future__ import annotations

import json
import os

import numpy as np
import pytest

from paper_2607_12324_b200 import workloads as W

HERE = os.path.dirname(os.path.abspath(__file__))


def _graph(n, edges, lat, energy=None):
    return W.tiny_graph(n, edges, np.asarray(lat, np.int64), None if energy is None else np.asarray(energy, np.float64))


def test_hand_worked_example(oracle_mod):
    d = json.load(open(os.path.join(HERE, "golden", "hand_worked_intervals.json")))
    g = _graph(d["n"], d["edges"], d["lat"], d["energy"])
    r = oracle_mod.intervals(g, d["dev_of"], d["breaks"], np.array(d["F"], np.uint8), d["p_idle"], want_levels=True)
    assert r["makespan"].tolist() == d["makespan"]
    assert np.allclose(r["e_active"], d["e_active"], rtol=1e-15, atol=0)
    assert np.allclose(r["e_idle"], np.array(d["idle_ns_times_watts"]) * 1e-9, rtol=1e-14, atol=0)
    assert r["levels"].tolist() == d["levels"]
    assert np.allclose(r["energy"], r["e_active"] + r["e_idle"])


def _random_case(seed, n=40, L=4, D=2, I=6, B=24, p_edge=0.12):
    rs = np.random.RandomState(seed)
    g0 = W.random_dag(seed, n, p_edge, L=L, max_dur=30)
    dev_of = rs.randint(-1, D, size=n).astype(np.int32)
    lat = g0.lat.copy()
    en = g0.energy.copy()
    for v in range(n):
        if dev_of[v] < 0:
            lat[v] = lat[v, 0]
            en[v] = 0.0
    g = W.Graph(g0.n, g0.row_ptr, g0.col, g0.level_ptr, g0.L, lat, en, g0.kind, "rand")
    steps = rs.randint(1, 40, size=I - 1)
    breaks = np.concatenate([[0], np.cumsum(steps)]).astype(np.int64)
    F = rs.randint(0, L, size=(D, I, B)).astype(np.uint8)
    p_idle = rs.uniform(10.0, 90.0, size=L)
    return g, dev_of, breaks, F, p_idle


@pytest.mark.parametrize("seed", range(6))
def test_realised_levels_reduce_to_the_per_node_oracle(oracle_mod, seed):
    """With the levels the policy realised, Eq. 1 / Eq. 2 of the per-node routines give the same makespan and
    active energy, and every pack's level is the one of the interval that holds its earliest start."""
    g, dev_of, breaks, F, p_idle = _random_case(seed)
    r = oracle_mod.intervals(g, dev_of, breaks, F, p_idle, want_levels=True)
    B = F.shape[2]
    ref = oracle_mod.batch(g, r["levels"], want_arrays=True)
    assert np.array_equal(ref["makespan"], r["makespan"])
    assert np.allclose(ref["energy"], r["e_active"], rtol=1e-13, atol=0)
    ES = ref["ES"]
    for v in range(g.n):
        if dev_of[v] < 0:
            assert (r["levels"][v] == 0).all()
            continue
        idx = np.searchsorted(breaks, ES[v], side="right") - 1      # the interval with breaks[i] <= start < breaks[i+1]
        assert np.array_equal(r["levels"][v], F[dev_of[v], idx, np.arange(B)])


def test_constant_policies_equal_per_node_levels(oracle_mod):
    g, dev_of, breaks, F, p_idle = _random_case(11, L=5)
    B = 5
    Fc = np.zeros((F.shape[0], F.shape[1], B), np.uint8)
    for l in range(B):
        Fc[:, :, l] = l
    r = oracle_mod.intervals(g, dev_of, breaks, Fc, None)
    lv = np.where((dev_of >= 0)[:, None], np.arange(B, dtype=np.uint8)[None, :], 0).astype(np.uint8)
    ref = oracle_mod.batch(g, lv)
    assert np.array_equal(ref["makespan"], r["makespan"])
    assert np.allclose(ref["energy"], r["e_active"], rtol=1e-13, atol=0)
    assert (r["e_idle"] == 0).all()


@pytest.mark.parametrize("seed", range(4))
def test_splitting_an_interval_changes_nothing(oracle_mod, seed):
    g, dev_of, breaks, F, p_idle = _random_case(20 + seed)
    r = oracle_mod.intervals(g, dev_of, breaks, F, p_idle)
    # split every interval that is longer than 1 ns in two, both halves with the old level
    nb, cols = [], []
    for i in range(len(breaks)):
        nb.append(int(breaks[i])); cols.append(i)
        hi = int(breaks[i + 1]) if i + 1 < len(breaks) else int(breaks[i]) + 1000
        if hi - breaks[i] > 1:
            nb.append(int(breaks[i]) + (hi - int(breaks[i])) // 2); cols.append(i)
    r2 = oracle_mod.intervals(g, dev_of, np.array(nb, np.int64), F[:, cols, :], p_idle)
    assert np.array_equal(r["makespan"], r2["makespan"])
    assert np.allclose(r["e_active"], r2["e_active"], rtol=1e-13, atol=0)
    # (idle energy is invariant only where a device's packs do not overlap: the count by nanoseconds below
    # covers that case; with overlapping packs the floor at zero applies per interval)
    assert (r2["e_idle"] >= r["e_idle"] * (1 - 1e-12)).all()


def test_boundary_is_half_open_and_last_interval_is_open_ended(oracle_mod):
    # chain of two packs: the first ends exactly at the change point, so the second takes the new level
    g = _graph(2, [(0, 1)], [[10, 7], [10, 7]])
    for first, expect in ((10, 17), (11, 20), (9, 17)):
        r = oracle_mod.intervals(g, [0, 0], [0, first], np.array([[[0], [1]]], np.uint8), None)
        assert int(r["makespan"][0]) == expect
    # starts far beyond the last change point still use the last level
    r = oracle_mod.intervals(g, [0, 0], [0, 1, 2, 3], np.array([[[0], [0], [0], [1]]], np.uint8), None, want_levels=True)
    assert r["levels"][:, 0].tolist() == [0, 1] and int(r["makespan"][0]) == 17


def test_alternating_chain_closed_form(oracle_mod):
    """CPU, pack, CPU, pack ... on one device: the device idles exactly while the CPU nodes run."""
    rs = np.random.RandomState(3)
    n, L = 30, 3
    lat = rs.randint(1, 50, size=(n, L)).astype(np.int64)
    dev_of = np.array([-1 if v % 2 == 0 else 0 for v in range(n)], np.int32)
    lat[dev_of < 0] = lat[dev_of < 0][:, :1]
    en = rs.uniform(0.5, 2.0, size=(n, L))
    en[dev_of < 0] = 0.0
    g = _graph(n, [(v, v + 1) for v in range(n - 1)], lat, en)
    p_idle = np.array([11.0, 23.0, 47.0])
    for l in range(L):
        r = oracle_mod.intervals(g, dev_of, [0], np.full((1, 1, 1), l, np.uint8), p_idle)
        T = int(lat[dev_of < 0, 0].sum() + lat[dev_of >= 0, l].sum())
        assert int(r["makespan"][0]) == T
        assert np.isclose(r["e_idle"][0], float(lat[dev_of < 0, 0].sum()) * 1e-9 * p_idle[l], rtol=1e-13)
        assert np.isclose(r["e_active"][0], en[dev_of >= 0, l].sum(), rtol=1e-13)


@pytest.mark.parametrize("seed", range(4))
def test_idle_time_by_counting_nanoseconds(oracle_mod, seed):
    """One stream per device (packs of a device form a chain, so they never overlap): the idle time of an
    interval is the number of its nanoseconds, below the makespan, at which no pack of the device runs."""
    rs = np.random.RandomState(100 + seed)
    D, per, L, I = 2, 7, 3, 5
    n = D * per * 2
    edges, dev_of = [], np.full(n, -1, np.int32)
    # device d: packs p_0 -> p_1 -> ...; a CPU chain launches them
    cpu = list(range(0, n, 2)); packs = list(range(1, n, 2))
    for i in range(len(cpu) - 1):
        edges.append((cpu[i], cpu[i + 1]))
    last = {}
    for i, pk in enumerate(packs):
        d = i % D
        dev_of[pk] = d
        edges.append((cpu[i], pk))
        if d in last:
            edges.append((last[d], pk))
        last[d] = pk
    lat = rs.randint(1, 12, size=(n, L)).astype(np.int64)
    lat[dev_of < 0] = lat[dev_of < 0][:, :1]
    g = _graph(n, sorted(edges), lat)
    breaks = np.concatenate([[0], np.cumsum(rs.randint(3, 25, size=I - 1))]).astype(np.int64)
    B = 6
    F = rs.randint(0, L, size=(D, I, B)).astype(np.uint8)
    p_idle = np.array([3.0, 5.0, 7.0])
    r = oracle_mod.intervals(g, dev_of, breaks, F, p_idle, want_levels=True)
    ref = oracle_mod.batch(g, r["levels"], want_arrays=True)
    for b in range(B):
        T = int(r["makespan"][b])
        busy = np.zeros((D, T), bool)
        for v in range(n):
            if dev_of[v] >= 0:
                s = int(ref["ES"][v, b]); c = s + int(lat[v, r["levels"][v, b]])
                assert not busy[dev_of[v], s:c].any()
                busy[dev_of[v], s:c] = True
        e = 0.0
        for d in range(D):
            for i in range(I):
                lo = int(breaks[i]); hi = int(breaks[i + 1]) if i + 1 < I else T
                idle = int((~busy[d, lo:min(hi, T)]).sum()) if lo < T else 0
                e += idle * 1e-9 * p_idle[F[d, i, b]]
        assert np.isclose(r["e_idle"][b], e, rtol=1e-12, atol=1e-30)


def test_idle_power_scales_and_uniform_grid(oracle_mod):
    g, dev_of, breaks, F, p_idle = _random_case(31)
    r1 = oracle_mod.intervals(g, dev_of, breaks, F, p_idle)
    r2 = oracle_mod.intervals(g, dev_of, breaks, F, 2.0 * p_idle)
    assert np.allclose(2.0 * r1["e_idle"], r2["e_idle"], rtol=1e-13)
    assert np.array_equal(r1["makespan"], r2["makespan"])
    # raising a level of a later interval never changes what happened before it
    F2 = F.copy()
    F2[:, -1, :] = (F2[:, -1, :] + 1) % g.L
    r3 = oracle_mod.intervals(g, dev_of, breaks, F2, p_idle, want_levels=True)
    r1l = oracle_mod.intervals(g, dev_of, breaks, F, p_idle, want_levels=True)
    ref = oracle_mod.batch(g, r1l["levels"], want_arrays=True)
    early = ref["ES"] < breaks[-1]
    assert np.array_equal(r3["levels"][early & (dev_of >= 0)[:, None]], r1l["levels"][early & (dev_of >= 0)[:, None]])
