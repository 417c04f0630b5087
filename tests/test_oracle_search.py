"""Pins of the oracle's policy search (Alg. 2).  The DP is a heuristic for several intervals, so it is pinned
where something independent exists: the exhaustive optimum for one interval, bounds against exhaustive
enumeration for several, feasibility, consistency with Alg. 1 on the reported policy, degenerate inputs."""
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
