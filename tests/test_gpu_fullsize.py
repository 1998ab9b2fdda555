"""Parity at the full sizes of the evaluation configurations, in the launch configuration the
benchmark times.  The oracle is too slow to redo everything, so it recomputes sampled outputs
one by one (with the horizons of exactly the workflows those calls belong to) and, for the
capacity pass, the complete first scheduler invocation; the rest is checked through properties
that hold at any size."""
import numpy as np
import pytest

import hx_helpers as hh
from hx_synth import make_workload, sub_forest
from oracle import hx_oracle as ho

pytestmark = [pytest.mark.gpu, pytest.mark.timeout(900)]


@pytest.fixture(scope="module")
def hx():
    import __graft_entry__ as entry
    entry.build()
    import paper_2605_16637_b200 as mod
    return mod


def _oracle_dag_for(oracle, oc, wl, workflows):
    """Oracle horizons of the given workflows only, scattered into full-size arrays."""
    workflows = np.unique(workflows)
    rp, col, lwf, ids = sub_forest(wl, workflows)
    cost = wl.node_cost[ids] if wl.node_cost is not None else hh.oracle_node_costs(oracle, oc, wl.node_calls[ids])
    sub = oracle.longest_path(rp, col, cost, lwf, workflows.shape[0])
    tail = np.zeros(wl.n_nodes, np.float32); tail[ids] = sub.tail
    cp = np.zeros(wl.n_nodes, np.float32); cp[ids] = sub.cp
    H = np.ones(wl.n_workflows, np.float32); H[workflows] = sub.H
    return ho.DagResult(cp, tail, H), ids, workflows, cost


def _gpu_setup(hx, wl):
    gc = hh.gpu_cluster(wl)
    cost = wl.node_cost if wl.node_cost is not None else hh.gpu_node_costs(gc, wl.node_calls)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    return gc, cost


def test_large_full_sampled(hx, oracle):
    wl = make_workload("large")
    gc, gcost = _gpu_setup(hx, wl)
    calls = wl.calls
    gc.set_options(score_mode=hx.HX_MODE_SLACK, alpha=wl.alpha)
    a, c = gc.schedule_batch(calls)
    a, c = a.cpu().numpy(), c.cpu().numpy()
    assert a.min() >= -1 and a.max() < wl.P * wl.D and gc.status() == 0
    pick = np.random.default_rng(0).choice(len(calls), 400, replace=False)
    oc = hh.oracle_cluster(wl)
    dag, ids, wfs, ocost = _oracle_dag_for(oracle, oc, wl, wl.node_wf[calls["node"][pick]])
    assert np.array_equal(gcost[ids], ocost)
    cp, tail, H = gc.dag_results()
    assert np.array_equal(cp[ids], dag.cp[ids]) and np.array_equal(tail[ids], dag.tail[ids])
    assert np.array_equal(H[wfs], dag.H[wfs])
    oa, ocst, _ = oracle.schedule(oc, calls[pick], mode=ho.MODE_SLACK, alpha=wl.alpha, dag=dag,
                                  node_wf=wl.node_wf, elapsed=wl.elapsed)
    hh.assert_costs_close(c[pick], ocst, "large")
    hh.assert_assign_matches(oracle, oc, calls[pick], a[pick], oa, what="large")
    assert np.array_equal(c[pick], ocst) and np.array_equal(a[pick], oa)
    gc.close()


def test_cp_stress_full(hx, oracle):
    wl = make_workload("cp_stress")
    gc, _ = _gpu_setup(hx, wl)
    cp, tail, H = gc.dag_results()
    r = oracle.longest_path(wl.row_ptr, wl.col, wl.node_cost, wl.node_wf, wl.n_workflows)
    assert np.array_equal(cp, r.cp) and np.array_equal(tail, r.tail) and np.array_equal(H, r.H)
    # invariants that hold at any size: a node's cp is at least its cost plus any successor's cp
    src = np.repeat(np.arange(wl.n_nodes), np.diff(wl.row_ptr.astype(np.int64)))
    assert np.all(cp[src] >= cp[wl.col]) and np.all(tail[src] >= cp[wl.col])
    calls = wl.calls
    gc.set_options(score_mode=hx.HX_MODE_RATIO, alpha=wl.alpha)
    a, c = gc.schedule_batch(calls)
    a, c = a.cpu().numpy(), c.cpu().numpy()
    pick = np.random.default_rng(1).choice(len(calls), 2000, replace=False)
    oc = hh.oracle_cluster(wl)
    oa, ocst, _ = oracle.schedule(oc, calls[pick], mode=ho.MODE_RATIO, dag=r, node_wf=wl.node_wf, elapsed=wl.elapsed)
    assert np.array_equal(c[pick], ocst) and np.array_equal(a[pick], oa)
    gc.close()


def test_sweep_full_as_benchmarked(hx, oracle):
    wl = make_workload("sweep")
    P, D, chunk, K = wl.P, wl.D, wl.chunk, wl.topk
    gc, gcost = _gpu_setup(hx, wl)
    calls = wl.calls
    n_chunks = len(calls) // chunk
    free0 = wl.kv_free[P:].copy()
    gc.set_options(score_mode=hx.HX_MODE_RATIO, topk=K, commit=1, alpha=wl.alpha)
    results = []
    for i in range(n_chunks):
        gc.update_loads(kv_free=free0)
        a, c = gc.schedule_batch(calls[i * chunk:(i + 1) * chunk])
        pair, cost, prio = gc.topk_results(chunk)
        qP, _, free = gc.read_loads()
        results.append((a.cpu().numpy(), c.cpu().numpy(), pair, cost, prio, qP, free))
    assert gc.status() == 0
    m = calls["prompt_tokens"] + calls["output_tokens"]
    for i, (a, c, pair, cost, prio, qP, free) in enumerate(results):
        mi = m[i * chunk:(i + 1) * chunk]
        placed = a >= 0
        assert np.all(free >= 0) and np.all(free <= free0)                  # never over-committed
        used = np.zeros(D); np.add.at(used, a[placed] % D, mi[placed])
        assert np.array_equal((free0 - free).astype(np.float64), used)       # tokens are conserved
        assert np.all((pair == a[:, None]).any(axis=1) | ~placed)            # a call only gets one of its candidates
        assert np.all(np.diff(cost, axis=1)[np.isfinite(cost[:, 1:])] >= 0)  # lists ordered by finish time
        if i:
            assert np.all(qP >= results[i - 1][5])                           # prefill queues only grow
    # the first scheduler invocation, completely, against the oracle
    oc = hh.oracle_cluster(wl)
    c0 = calls[:chunk]
    dag, ids, wfs, ocost = _oracle_dag_for(oracle, oc, wl, wl.node_wf[c0["node"]])
    assert np.array_equal(gcost[ids], ocost)
    a, c, pair, cost, prio, qP, free = results[0]
    op, ocs, opr, om, ots = oracle.topk(oc, c0, K, dag=dag, node_wf=wl.node_wf, elapsed=wl.elapsed)
    assert np.array_equal(pair, op) and np.array_equal(cost, ocs) and np.array_equal(prio, opr)
    oa, ofree, oq = oracle.conflict(op, opr, om, ots, free0, wl.load_s[:P], D)
    assert np.array_equal(a, oa) and np.array_equal(free, ofree) and np.array_equal(qP, oq)
    gc.close()
