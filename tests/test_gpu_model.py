"""Pack modelling on the GPU (emo_pack_model: Eq. 6, Eq. 7) against the oracle: weights and tables within 1e-8
relative to the problem's scale (the minimiser is unique: the metric matrix has independent columns)."""
from __future__ import annotations

import numpy as np
import pytest

from paper_2607_12324_b200 import workloads as W

pytestmark = pytest.mark.gpu


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


def run(torch, emo, B, feat, Tb, Eb):
    P, n = feat.shape
    m, L = Tb.shape
    d = lambda a: torch.from_numpy(np.ascontiguousarray(a, np.float64)).cuda()
    x = torch.zeros((P, m), dtype=torch.float64, device="cuda")
    T = torch.zeros((P, L), dtype=torch.float64, device="cuda")
    E = torch.zeros((P, L), dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    emo.emo_pack_model(P, n, m, L, d(B), d(feat), d(Tb), d(Eb), x, T, E, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return x.cpu().numpy(), T.cpu().numpy(), E.cpu().numpy()


@pytest.mark.parametrize("seed,n,m,L,P,noise", [(0, 16, 12, 16, 300, 0.02), (1, 16, 12, 32, 130, 0.3), (2, 12, 12, 8, 64, 0.1),
                                                  (3, 20, 5, 4, 1, 0.1), (4, 9, 16 - 8, 3, 257, 1.0)])
def test_against_the_oracle(torch_cuda, emo, oracle_mod, seed, n, m, L, P, noise):
    B, Tb, Eb = W.microbench_model(seed, n, m, L)
    feat = W.pack_features(seed + 50, B, P, noise=noise)
    xo, To, Eo = oracle_mod.pack_model(B, feat, Tb, Eb)
    x, T, E = run(torch_cuda, emo, B, feat, Tb, Eb)
    scale = np.abs(xo).max(axis=1, keepdims=True) + 1e-300
    assert np.allclose(x / scale, xo / scale, rtol=0, atol=1e-8)
    assert ((x == 0) == (xo == 0)).mean() > 0.99          # the same variables are held at zero (up to rounding ties)
    assert np.allclose(T, To, rtol=1e-8, atol=1e-8 * np.abs(To).max())
    assert np.allclose(E, Eo, rtol=1e-8, atol=1e-8 * np.abs(Eo).max())
    assert (x >= 0).all()


def test_special_cases(torch_cuda, emo, oracle_mod):
    B, Tb, Eb = W.microbench_model(9, 16, 12, 4)
    xt = np.zeros((4, 12))
    xt[0, 3] = 2.0
    xt[1, [0, 11]] = [1.0, 0.25]
    feat = xt @ B.T
    feat[2] = -B.sum(axis=1)            # opposite to every column: all weights zero
    feat[3] = 0.0
    x, T, E = run(torch_cuda, emo, B, feat, Tb, Eb)
    assert np.allclose(x[:2], xt[:2], atol=1e-9) and (x[2:] == 0).all()
    assert np.allclose(T[:2], xt[:2] @ Tb, rtol=1e-9) and (T[2:] == 0).all()
