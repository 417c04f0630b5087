"""Alg. 2 on the GPU evaluator (emo_search_dp) against the oracle's search: the same chosen policy, time and
number of predictions, energy within 1e-9 relative."""
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


def run_search(torch, emo, g, dev_of, breaks, p_idle, T_max, bin_ns, max_batch=0):
    h = emo.load_workload(g, group_of=np.asarray(dev_of, np.int32))
    pi = torch.from_numpy(np.asarray(p_idle, np.float64)).cuda() if p_idle is not None else None
    ws = torch.empty(emo.emo_workspace_bytes_search(h, len(breaks), max_batch, p_idle is not None), dtype=torch.uint8, device="cuda")
    r = emo.emo_search_dp(h, breaks, pi, T_max, bin_ns, ws, max_batch=max_batch)
    h.free()
    return r


def compare(a, b):
    assert a["found"] == b["found"]
    if a["found"]:
        assert a["T"] == b["T"]
        assert np.isclose(a["E"], b["E"], rtol=1e-9, atol=0)
        assert a["F"].tolist() == b["F"].tolist()
    assert a["n_pred"] == b["n_pred"]


@pytest.mark.parametrize("seed", range(4))
def test_random_dags(torch_cuda, emo, oracle_mod, seed):
    from tests.test_oracle_intervals import _random_case
    g, dev_of, breaks, _, p_idle = _random_case(60 + seed, n=50, L=4, D=2, I=5, B=1)
    dev_of[0] = 0
    t0 = int(oracle_mod.intervals(g, dev_of, breaks, np.full((2, 5, 1), g.L - 1, np.uint8), p_idle)["makespan"][0])
    for slack, bin_ns, mb in ((0.0, 1, 0), (0.1, 1, 0), (0.3, 5, 0), (0.3, 1, 7), (-0.5, 1, 0)):
        T_max = int(t0 * (1 + slack))
        compare(run_search(torch_cuda, emo, g, dev_of, breaks, p_idle, T_max, bin_ns, mb),
                oracle_mod.search_dp(g, dev_of, breaks, p_idle, T_max, bin_ns))
    compare(run_search(torch_cuda, emo, g, dev_of, breaks, None, int(t0 * 1.2), 1),
            oracle_mod.search_dp(g, dev_of, breaks, None, int(t0 * 1.2), 1))


def test_config_graph(torch_cuda, emo, oracle_mod):
    g = W.make_graph("cfg0-tiny", 0.5)
    dev_of = W.device_of(g)
    t0 = int(oracle_mod.batch(g, np.full((g.n, 1), g.L - 1, np.uint8))["makespan"][0])
    breaks = W.interval_breaks(t0, 6)
    p_idle = W.idle_power(g.L)
    T_max = t0 + t0 // 20
    a = run_search(torch_cuda, emo, g, dev_of, breaks, p_idle, T_max, 1000)
    b = oracle_mod.search_dp(g, dev_of, breaks, p_idle, T_max, 1000)
    compare(a, b)
    assert a["found"] and a["T"] <= T_max
