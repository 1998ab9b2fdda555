"""Online horizon refinement on the GPU (cost estimates replaced by observed latencies, Section 5.1)
against the definition: a full longest-path pass of the oracle over the updated costs."""
import numpy as np
import pytest

import hx_helpers as hh
from hx_synth import make_workload
from oracle import hx_oracle as ho

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hx():
    import __graft_entry__ as entry
    entry.build()
    import paper_2605_16637_b200 as mod
    return mod


def _costs(wl, oracle, oc, gc):
    if wl.node_cost is not None:
        return np.asarray(wl.node_cost, np.float32).copy()
    cost = hh.gpu_node_costs(gc, wl.node_calls)
    assert np.array_equal(cost, hh.oracle_node_costs(oracle, oc, wl.node_calls))
    return cost


@pytest.mark.parametrize("name, scale, frac", [("tiny", 1.0, 0.3), ("medium", 1.0, 0.02), ("cp_stress", 1 / 20, 0.001),
                                               ("large", 1 / 16, 0.2)])
def test_cost_updates_equal_full_recompute(hx, oracle, name, scale, frac):
    wl = make_workload(name, scale=scale)
    oc, gc = hh.oracle_cluster(wl), hh.gpu_cluster(wl)
    cost = _costs(wl, oracle, oc, gc)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    before = [a.copy() for a in gc.dag_results()]
    rng = np.random.default_rng(7)
    for rnd in range(3):
        k = max(1, int(frac * wl.n_nodes))
        ids = rng.integers(0, wl.n_nodes, k).astype(np.uint32)
        if k > 2:
            ids[1] = ids[0]                                   # a node listed twice: the last value counts
        new = (cost[ids] * rng.uniform(0.5, 2.0, k)).astype(np.float32)
        gc.update_costs(ids, new)
        for i, v in zip(ids, new):
            cost[i] = v
        want = oracle.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
        cp, tail, H = gc.dag_results()
        assert np.array_equal(cp, want.cp) and np.array_equal(tail, want.tail) and np.array_equal(H, want.H)
        touched = np.zeros(wl.n_workflows, bool); touched[wl.node_wf[ids]] = True
        assert np.array_equal(H[~touched], before[2][~touched])      # nothing else moved
        before = [cp.copy(), tail.copy(), H.copy()]
    assert gc.status() == 0
    gc.close()


def test_updates_before_the_first_pass_and_bad_arguments(hx, oracle):
    wl = make_workload("medium", scale=0.25)
    oc, gc = hh.oracle_cluster(wl), hh.gpu_cluster(wl)
    with pytest.raises(hx.HxError) as e:
        gc.update_costs([0], [1.0])
    assert e.value.code == -4
    cost = _costs(wl, oracle, oc, gc)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.update_costs([3, 5], [0.25, 0.5])                      # no horizons yet: costs only
    cost[3], cost[5] = 0.25, 0.5
    gc.critical_path()
    want = oracle.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
    cp, tail, H = gc.dag_results()
    assert np.array_equal(cp, want.cp) and np.array_equal(H, want.H)
    for ids, vals in (([wl.n_nodes], [1.0]), ([0], [-1.0]), ([0], [np.inf]), ([0, 1], [1.0, np.nan])):
        with pytest.raises(hx.HxError) as e:
            gc.update_costs(ids, vals)
        assert e.value.code == -1
    cp2, _, H2 = gc.dag_results()
    assert np.array_equal(cp2, cp) and np.array_equal(H2, H)    # rejected updates change nothing
    gc.update_costs(np.zeros(0, np.uint32), np.zeros(0, np.float32))
    gc.close()


def test_elapsed_refresh_feeds_the_ratio(hx, oracle):
    wl = make_workload("medium", scale=0.5)
    oc, gc = hh.oracle_cluster(wl), hh.gpu_cluster(wl)
    cost = _costs(wl, oracle, oc, gc)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    dag = oracle.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
    later = (wl.elapsed + np.float32(0.75)).astype(np.float32)
    gc.update_elapsed(later)
    gc.set_options(score_mode=hx.HX_MODE_RATIO, alpha=wl.alpha)
    a, r = gc.schedule_batch(wl.calls)
    ea, er, _ = oracle.schedule(oc, wl.calls, mode=ho.MODE_RATIO, dag=dag, node_wf=wl.node_wf, elapsed=later)
    assert np.array_equal(a.cpu().numpy(), ea)
    hh.assert_costs_close(r.cpu().numpy(), er, "ratio after elapsed refresh")
    assert np.array_equal(r.cpu().numpy(), er)
    with pytest.raises(hx.HxError):
        gc.update_elapsed(later[:-1])
    gc.close()


@pytest.mark.parametrize("name, scale, frac", [("tiny", 1.0, 0.3), ("medium", 1.0, 0.02), ("cp_stress", 1 / 20, 0.001),
                                               ("large", 1 / 16, 0.2), ("sweep", 1 / 8, 0.01)])
def test_forward_pass_equals_oracle_and_follows_cost_updates(hx, oracle, name, scale, frac):
    wl = make_workload(name, scale=scale)
    oc, gc = hh.oracle_cluster(wl), hh.gpu_cluster(wl)
    cost = _costs(wl, oracle, oc, gc)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    with pytest.raises(hx.HxError) as e:
        gc.earliest_results()
    assert e.value.code == -4
    gc.critical_path()
    gc.earliest_start()
    est, eft = gc.earliest_results()
    w_est, w_eft = oracle.earliest_start(wl.row_ptr, wl.col, cost)
    assert np.array_equal(est, w_est) and np.array_equal(eft, w_eft)
    cp, tail, H = gc.dag_results()
    want = oracle.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
    assert np.array_equal(cp, want.cp) and np.array_equal(H, want.H)       # the backward results are untouched
    # longest path through a node never exceeds the horizon by more than the rounding of two sums
    assert np.all(est + cp <= H[wl.node_wf] * (1 + 1e-4))
    rng = np.random.default_rng(17)
    for rnd in range(2):
        k = max(1, int(frac * wl.n_nodes))
        ids = rng.integers(0, wl.n_nodes, k).astype(np.uint32)
        new = (cost[ids] * rng.uniform(0.5, 2.0, k)).astype(np.float32)
        gc.update_costs(ids, new)
        for i, v in zip(ids, new):
            cost[i] = v
        est, eft = gc.earliest_results()
        w_est, w_eft = oracle.earliest_start(wl.row_ptr, wl.col, cost)
        assert np.array_equal(est, w_est) and np.array_equal(eft, w_eft)
        cp, tail, H = gc.dag_results()
        want = oracle.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
        assert np.array_equal(cp, want.cp) and np.array_equal(tail, want.tail) and np.array_equal(H, want.H)
    assert gc.status() == 0
    gc.close()


def test_forward_pass_built_after_cost_updates_and_rebuilt_after_upload(hx, oracle):
    wl = make_workload("medium", scale=0.25)
    oc, gc = hh.oracle_cluster(wl), hh.gpu_cluster(wl)
    cost = _costs(wl, oracle, oc, gc)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.update_costs([3, 5, 3], [0.25, 0.5, 0.75])              # before the transposed forest exists
    cost[3], cost[5] = 0.75, 0.5
    gc.earliest_start()                                        # without hx_critical_path: independent of it
    est, eft = gc.earliest_results()
    w_est, w_eft = oracle.earliest_start(wl.row_ptr, wl.col, cost)
    assert np.array_equal(est, w_est) and np.array_equal(eft, w_eft)
    wl2 = make_workload("tiny")
    cost2 = _costs(wl2, oracle, hh.oracle_cluster(wl2), hh.gpu_cluster(wl2))
    gc.dag_upload(wl2.row_ptr, wl2.col, cost2, wl2.node_wf, wl2.elapsed)
    with pytest.raises(hx.HxError):
        gc.earliest_results()                                  # the old forward results went with the old forest
    gc.earliest_start()
    est, eft = gc.earliest_results()
    w_est, w_eft = oracle.earliest_start(wl2.row_ptr, wl2.col, cost2)
    assert np.array_equal(est, w_est) and np.array_equal(eft, w_eft)
    gc.close()
