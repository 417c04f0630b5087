"""Host-side check of the spine program (no GPU): the compiled segments, operations, value slots, folds and
position words, interpreted in numpy (tests/spine_emulator.py), reproduce the oracle's makespan, energy, slack,
ES and LS - with the stores of a stage done at once and with them delayed as long as the kernels allow."""
from __future__ import annotations

import numpy as np
import pytest

from paper_2607_12324_b200 import workloads as W
from tests import spine_emulator as SE
from tests.test_oracle_pins import TINY, all_policies


@pytest.fixture(scope="module")
def emo():
    from paper_2607_12324_b200 import build, emo as E
    build.build()
    return E


def compare(emo, oracle_mod, g, lv, flags):
    h = emo.load_workload(g, emo.EMO_F_HOST_ONLY | flags)
    sizes = emo.emo_graph_spine(h)
    view = emo.emo_graph_spine_view(h)
    assert sizes["ok"] == 1 and view["ok"] == 1
    assert sizes["segments"] <= g.n and sizes["ops_bwd"] >= sizes["segments"]
    assert int(view["n_ops_fwd"].sum()) == sizes["ops_fwd"] and int(view["n_ops_bwd"].sum()) == sizes["ops_bwd"]
    # every node sits at exactly one position
    nodes = view["mem"][:, :, 0].ravel()
    nodes = nodes[nodes != 0xFFFFFFFF]
    assert len(nodes) == g.n and len(np.unique(nodes)) == g.n
    r_or = oracle_mod.batch(g, lv, want_arrays=True)
    for late in (False, True):
        r = SE.run(view, lv, g.L, late_stores=late)
        assert np.array_equal(r["makespan"], r_or["makespan"]), late
        np.testing.assert_allclose(r["energy"], r_or["energy"], rtol=1e-9)
        for k in ("slack", "ES", "LS"):
            assert np.array_equal(r[k], r_or[k]), (k, late)
    h.free()
    return sizes


@pytest.mark.parametrize("gi", range(len(TINY)))
def test_spine_program_on_tiny_graphs(emo, oracle_mod, gi):
    g = TINY[gi]
    lv = all_policies(g.n, g.L)
    for lanes, k in ((0, 16), (1, 8), (2, 32), (3, 8)):
        compare(emo, oracle_mod, g, lv, emo.EMO_F_LANES(lanes) | emo.EMO_F_SPINE_STAGE(k))


@pytest.mark.parametrize("name,scale,k", [("cfg0-tiny", 1.0, 16), ("cfg1-train", 0.05, 8), ("cfg2-packed", 0.3, 16),
                                            ("cfg3-8dev", 0.01, 16), ("cfg4-llm", 0.01, 8), ("cfg4-llm", 0.01, 16)])
def test_spine_program_on_config_graphs(emo, oracle_mod, name, scale, k):
    g = W.make_graph(name, scale)
    lv = W.policies_for(g, B=24)
    lv = np.asarray(lv)[:, :24]
    sizes = compare(emo, oracle_mod, g, lv, emo.EMO_F_SPINE_STAGE(k))
    assert sizes["K"] == k or sizes["lanes"] * k > 256
    if name == "cfg4-llm" and k == 8:
        # the launch nodes' kernels are folded, not published: chains of kernels stay segments (where the graph is long
        # enough for the schedule to keep launch nodes two stages ahead of their kernels)
        assert sizes["segments"] < 0.85 * g.n


@pytest.mark.parametrize("seed", range(24))
def test_spine_program_on_random_dags(emo, oracle_mod, seed):
    """Random DAGs of varying density (dense ones have nodes with many operands: merge operations; sparse ones long
    chains: segments of several members), random policies, two lane counts and stage lengths."""
    rs = np.random.RandomState(1000 + seed)
    n = int(rs.randint(30, 140))
    L = int(rs.randint(2, 7))
    g = W.random_dag(500 + seed, n, float(rs.choice([0.02, 0.05, 0.12, 0.3])), L=L, max_dur=int(rs.choice([5, 40, 100000])))
    lv = rs.randint(0, L, size=(g.n, 20)).astype(np.uint8)
    lv[:, 0] = L - 1
    lv[:, 1] = 0
    for lanes, k in ((0, 8), (3, 16)):
        compare(emo, oracle_mod, g, lv, emo.EMO_F_LANES(lanes) | emo.EMO_F_SPINE_STAGE(k))
