"""The seeded input generator: sizes, structure and determinism of the five configurations."""
import numpy as np
import pytest

from hx_synth import CONFIG_NAMES, make_workload, sub_forest

SIZES = {"tiny": (3, 2, 2, 64, 8), "medium": (6, 16, 16, 4096, 512), "large": (8, 64, 64, 65536, 8192),
         "cp_stress": (8, 32, 32, 50000, 16384), "sweep": (8, 128, 128, 262144, 32768)}


def _check_forest(wl):
    N = wl.n_nodes
    rp = wl.row_ptr.astype(np.int64)
    assert rp[0] == 0 and rp[-1] == wl.n_edges and np.all(np.diff(rp) >= 0)
    src = np.repeat(np.arange(N), np.diff(rp))
    assert np.all(src < wl.col)                                   # numbering is a topological order
    assert np.array_equal(wl.node_wf[src], wl.node_wf[wl.col])    # edges stay inside one workflow
    assert np.all(np.diff(wl.node_wf.astype(np.int64)) >= 0) and wl.node_wf.max() == wl.n_workflows - 1


@pytest.mark.parametrize("name", CONFIG_NAMES)
def test_config_sizes_and_structure(name):
    scale = 1.0 if name in ("tiny", "medium") else 0.05
    wl = make_workload(name, scale=scale)
    G, P, D, C, W = SIZES[name]
    assert wl.gpu_types.shape == (G, 2) and (wl.P, wl.D) == (P, D)
    assert wl.ready_nodes.shape[0] == max(1, round(C * scale)) and wl.n_workflows == max(1, round(W * scale))
    assert len(np.unique(wl.ready_nodes)) == wl.ready_nodes.shape[0]
    assert wl.link_gbps.shape == (P + D, P + D) and wl.link_gbps.min() >= 25 and wl.link_gbps.max() <= 400
    assert wl.load_s.min() >= 0 and wl.load_s.max() <= 2
    n, o = wl.node_calls["prompt_tokens"], wl.node_calls["output_tokens"]
    assert n.min() >= 1 and n.max() <= (131072 if name == "large" else 32768)
    assert np.all(n == np.round(n)) and np.all(o == np.round(o))   # token counts are integers
    assert set(np.unique(wl.inst_type[:P])) == set(range(G)) if P >= G else True
    _check_forest(wl)


def test_generator_is_deterministic_and_seeded():
    a, b, c = make_workload("medium"), make_workload("medium"), make_workload("medium", seed=7)
    for f in ("link_gbps", "load_s", "col", "ready_nodes", "elapsed"):
        assert np.array_equal(getattr(a, f), getattr(b, f))
    assert np.array_equal(a.node_calls, b.node_calls)
    assert not np.array_equal(a.link_gbps, c.link_gbps)


@pytest.mark.timeout(120)
def test_cp_stress_full_size_shape():
    wl = make_workload("cp_stress")
    assert wl.n_nodes == 1_000_000 and wl.n_workflows == 16384 and wl.ready_nodes.shape[0] == 50000
    assert np.bincount(wl.col, minlength=wl.n_nodes).max() <= 16           # fan-in
    assert wl.depth.max() == 256
    assert wl.node_cost.shape[0] == wl.n_nodes and wl.node_cost.min() > 0
    _check_forest(wl)


def test_sweep_chunks_and_capacity_pressure():
    wl = make_workload("sweep", scale=1 / 16)
    assert wl.chunk == 16384 and wl.topk == 4 and wl.commit
    demand = (wl.calls["prompt_tokens"] + wl.calls["output_tokens"]).sum()
    assert 0.3 < demand / wl.kv_free[wl.P:].sum() < 1.5                    # capacity is contended


def test_sub_forest_keeps_structure():
    wl = make_workload("medium", scale=0.1)
    pick = np.array([3, 0, 17])
    rp, col, lwf, ids = sub_forest(wl, pick)
    assert np.array_equal(wl.node_wf[ids], pick[lwf])
    deg = np.diff(wl.row_ptr.astype(np.int64))[ids]
    assert np.array_equal(np.diff(rp.astype(np.int64)), deg)
    src = np.repeat(np.arange(len(ids)), deg)
    orig = [(int(ids[s]), int(ids[c])) for s, c in zip(src, col)]
    full_src = np.repeat(np.arange(wl.n_nodes), np.diff(wl.row_ptr.astype(np.int64)))
    keep = np.isin(full_src, ids)
    assert sorted(orig) == sorted(zip(full_src[keep].tolist(), wl.col[keep].tolist()))
