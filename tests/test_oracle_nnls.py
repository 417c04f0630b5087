"""Pins of the oracle's pack modelling (Eq. 6, Eq. 7): the library routine scipy.optimize.nnls, the optimality
conditions of the constrained problem, closed forms, and the weighted sums of Eq. 7."""
from __future__ import annotations

import numpy as np
import pytest
from scipy.optimize import nnls as scipy_nnls

from paper_2607_12324_b200 import workloads as W


@pytest.mark.parametrize("seed", range(4))
def test_nnls_against_scipy_and_optimality(oracle_mod, seed):
    B, Tb, Eb = W.microbench_model(seed, 16, 12, 8)
    feat = W.pack_features(seed + 10, B, 25, noise=0.1)
    active = 0
    for b in feat:
        x, r2 = oracle_mod.nnls(B, b)
        xs, rn = scipy_nnls(B, b)
        assert np.allclose(x, xs, rtol=1e-8, atol=1e-9)
        assert np.isclose(np.sqrt(r2), rn, rtol=1e-7, atol=1e-9)
        # optimality: x >= 0, gradient w = B^T (b - B x) <= 0, and w_i = 0 wherever x_i > 0
        w = B.T @ (b - B @ x)
        scale = np.abs(B.T @ b).max()
        assert (x >= 0).all() and (w <= 1e-9 * scale).all()
        assert np.abs(w[x > 0]).max(initial=0.0) <= 1e-9 * scale
        active += int((x == 0).sum())
    assert active > 0, "the constraint binds somewhere in the sample"


def test_nnls_closed_forms(oracle_mod):
    # orthogonal columns: x_i = max(0, <B_i, b> / <B_i, B_i>)
    B = np.diag([2.0, 3.0, 4.0])
    x, r2 = oracle_mod.nnls(B, np.array([4.0, -3.0, 2.0]))
    assert np.allclose(x, [2.0, 0.0, 0.5]) and np.isclose(r2, 9.0)
    # b in the cone: exact recovery, zero residual
    B, _, _ = W.microbench_model(3, 10, 6, 4)
    xt = np.array([0.0, 2.0, 0.0, 0.5, 0.0, 3.0])
    x, r2 = oracle_mod.nnls(B, B @ xt)
    assert np.allclose(x, xt, atol=1e-9) and r2 < 1e-16
    # b opposite to every column: x = 0
    x, r2 = oracle_mod.nnls(B, -B.sum(axis=1))
    assert (x == 0).all()


def test_pack_tables_are_the_weighted_sums(oracle_mod):
    B, Tb, Eb = W.microbench_model(5, 16, 12, 6)
    feat = W.pack_features(6, B, 9)
    x, T, E = oracle_mod.pack_model(B, feat, Tb, Eb)
    for p in range(9):
        xs, _ = scipy_nnls(B, feat[p])
        assert np.allclose(T[p], xs @ Tb, rtol=1e-8) and np.allclose(E[p], xs @ Eb, rtol=1e-8)
    # scaling the features scales the weights and the tables (the cone is scale-free)
    x2, T2, E2 = oracle_mod.pack_model(B, 3.0 * feat, Tb, Eb)
    assert np.allclose(x2, 3.0 * x, rtol=1e-9, atol=1e-12) and np.allclose(T2, 3.0 * T, rtol=1e-9)
