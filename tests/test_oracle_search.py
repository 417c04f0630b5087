"""Pins of the oracle's policy search (Alg. 2).  The DP is a heuristic only where two candidates end in one time
bin (one survives), so it is pinned where something independent exists: the exhaustive optimum for one interval
and, for several intervals, whenever no two policies share a time bin; bounds against exhaustive enumeration
otherwise; feasibility, consistency with Alg. 1 on the reported policy, degenerate inputs."""
from __future__ import annotations

import itertools

import numpy as np
import pytest

from tests.test_oracle_intervals import _random_case


def _all_policies(I, L):
    return np.array(list(itertools.product(range(L), repeat=I)), np.uint8).T      # [I][L^I]


def _pred_all(oracle_mod, g, dev_of, breaks, p_idle, pols):
    D = int(dev_of.max()) + 1
    F = np.repeat(pols[None, :, :], D, axis=0).copy()
    return oracle_mod.intervals(g, dev_of, breaks, F, p_idle)


@pytest.mark.parametrize("seed", range(5))
def test_one_interval_is_exhaustive(oracle_mod, seed):
    g, dev_of, _, _, p_idle = _random_case(seed, n=30, L=5, D=2, I=1, B=1)
    dev_of[0] = 0
    breaks = np.array([0], np.int64)
    r = _pred_all(oracle_mod, g, dev_of, breaks, p_idle, _all_policies(1, g.L))
    t0 = int(r["makespan"][g.L - 1])
    for slack in (0.0, 0.1, 0.5, 10.0):
        T_max = int(t0 * (1 + slack))
        s = oracle_mod.search_dp(g, dev_of, breaks, p_idle, T_max)
        feas = r["makespan"] <= T_max
        assert s["found"] and feas.any()
        best = int(np.flatnonzero(feas)[np.argmin(r["energy"][feas])])
        assert np.isclose(s["E"], r["energy"][best], rtol=1e-15)
        assert s["T"] == int(r["makespan"][int(s["F"][0])]) and s["T"] <= T_max
        assert s["n_pred"] == 1 + g.L


@pytest.mark.parametrize("seed", range(5))
def test_bounds_against_enumeration(oracle_mod, seed):
    """Never better than the exhaustive optimum, never worse than the default policy, always feasible, and the
    reported time and energy are those Alg. 1 gives for the reported policy."""
    g, dev_of, breaks, _, p_idle = _random_case(40 + seed, n=30, L=3, D=2, I=4, B=1)
    dev_of[0] = 0
    pols = _all_policies(4, g.L)
    r = _pred_all(oracle_mod, g, dev_of, breaks, p_idle, pols)
    i0 = pols.shape[1] - 1                      # all L-1
    t0, E0 = int(r["makespan"][i0]), float(r["energy"][i0])
    for slack in (0.0, 0.05, 0.3):
        T_max = int(t0 * (1 + slack))
        feas = r["makespan"] <= T_max
        E_opt = float(r["energy"][feas].min())
        for bin_ns in (1, 7):
            s = oracle_mod.search_dp(g, dev_of, breaks, p_idle, T_max, bin_ns)
            assert s["found"] and s["T"] <= T_max
            assert s["E"] <= E0 * (1 + 1e-15) and s["E"] >= E_opt * (1 - 1e-15)
            col = int(np.flatnonzero((pols == s["F"][:, None]).all(axis=0))[0])
            assert s["T"] == int(r["makespan"][col]) and np.isclose(s["E"], r["energy"][col], rtol=1e-15)
            assert s["n_pred"] >= 1 + g.L and (s["n_pred"] - 1) % g.L == 0


def _chain_case(seed, n=12, L=3, I=3):
    """One stream of n kernels in series on one device: every node is on the critical path, so every interval's level
    changes the end-to-end time; durations 1 000 - 2 000 with random increments (sums of different choices differ),
    longer at lower levels; change points 5 000 apart, so every interval holds several starts under every policy."""
    from paper_2607_12324_b200 import workloads as W
    rs = np.random.RandomState(seed)
    row_ptr = np.concatenate([[0], np.arange(0, n)]).astype(np.int64)      # node v > 0 has the one predecessor v - 1
    col = np.arange(0, n - 1, dtype=np.int32)
    level_ptr = np.arange(0, n + 1, dtype=np.int32)
    top = rs.randint(1000, 1400, size=n)
    lat = np.stack([top + np.cumsum(rs.randint(50, 300, size=(L, n)), axis=0)[L - 1 - l] * (l < L - 1) for l in range(L)], axis=1).astype(np.int64)
    energy = rs.uniform(1.0, 9.0, size=(n, L))
    g = W.Graph(n, row_ptr, col, level_ptr, L, lat, energy, np.zeros(n, np.uint8), "chain")
    breaks = (np.arange(I) * 5000).astype(np.int64)
    return g, np.zeros(n, np.int32), breaks, rs.uniform(10.0, 90.0, size=L)


@pytest.mark.parametrize("seed", range(6))
def test_without_collisions_the_search_is_exhaustive(oracle_mod, seed):
    """Several intervals: when no two policies end in the same time bin (exact keys, all L^I end-to-end times distinct)
    and the constraint admits every policy, nothing is ever merged or dropped, so dp[I] holds every policy: the answer
    must be the exhaustive optimum (earliest time among equal energies) and Alg. 1 runs 1 + L + L^2 + ... + L^I times.
    With a constraint that cuts into the set the same holds among the feasible policies, because here a lower level is
    never faster: a prefix that misses the constraint cannot be repaired by the intervals still at the top level."""
    I, L = 3, 3
    g, dev_of, breaks, p_idle = _chain_case(seed, L=L, I=I)
    pols = _all_policies(I, L)
    r = _pred_all(oracle_mod, g, dev_of, breaks, p_idle, pols)
    assert len(np.unique(r["makespan"])) == pols.shape[1], "the construction should give every policy its own time"
    s = oracle_mod.search_dp(g, dev_of, breaks, p_idle, int(r["makespan"].max()), 1)
    E_opt = float(r["energy"].min())
    cands = np.flatnonzero(r["energy"] == E_opt)
    best = int(cands[np.argmin(r["makespan"][cands])])
    assert s["found"] and s["E"] == E_opt and s["T"] == int(r["makespan"][best])
    assert np.array_equal(s["F"], pols[:, best])
    assert s["n_pred"] == sum(L ** i for i in range(I + 1))
    # a constraint at the median time
    T_max = int(np.median(r["makespan"]))
    feas = r["makespan"] <= T_max
    s = oracle_mod.search_dp(g, dev_of, breaks, p_idle, T_max, 1)
    E_f = float(r["energy"][feas].min())
    cands = np.flatnonzero(feas & (r["energy"] == E_f))
    best = int(cands[np.argmin(r["makespan"][cands])])
    assert s["found"] and s["E"] == E_f and s["T"] == int(r["makespan"][best]) and np.array_equal(s["F"], pols[:, best])


def test_degenerate_inputs(oracle_mod):
    g, dev_of, breaks, _, p_idle = _random_case(7, n=25, L=4, D=1, I=3, B=1)
    dev_of[:] = np.where(dev_of < 0, -1, 0)
    dev_of[0] = 0
    pols = _all_policies(3, g.L)
    r = _pred_all(oracle_mod, g, dev_of, breaks, p_idle, pols)
    t0 = int(r["makespan"][-1])
    # a constraint below the default policy's time: nothing survives the first stage unless a level is faster
    s = oracle_mod.search_dp(g, dev_of, breaks, p_idle, int(r["makespan"].min()) - 1)
    assert not s["found"]
    # a constraint met by everything: the answer is a policy that enumeration also finds feasible, and with
    # exact time keys and one interval left the last stage picks the best level for its states
    s = oracle_mod.search_dp(g, dev_of, breaks, p_idle, int(r["makespan"].max()))
    assert s["found"] and s["E"] <= float(r["energy"][-1])
    # one level: only the default policy exists
    import copy
    g1 = copy.copy(g)
    g1.L, g1.lat, g1.energy = 1, g.lat[:, -1:].copy(), g.energy[:, -1:].copy()
    s = oracle_mod.search_dp(g1, dev_of, breaks, p_idle[-1:], t0)
    assert s["found"] and s["T"] == t0 and s["F"].tolist() == [0, 0, 0] and s["n_pred"] == 1 + 3
