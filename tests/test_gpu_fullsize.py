"""Parity at the full sizes of the evaluation configurations, in the launch configuration the
benchmark times.  Every output is compared with the oracle: all 65,536 calls of the large
configuration, the 1,000,000-node forest and all 50,000 calls of the critical-path stress, and all
16 scheduler invocations of the sweep, chained through the prefill queues exactly as the benchmark
chains them.  The oracle is single-threaded; the test spreads independent slices of calls over the
host's cores (the oracle's functions are pure, and ctypes releases the interpreter lock), which
changes no result."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest

import hx_helpers as hh
from hx_synth import make_workload
from oracle import hx_oracle as ho

pytestmark = [pytest.mark.gpu, pytest.mark.timeout(1500)]

N_THREADS = max(1, min(16, (os.cpu_count() or 2) - 1))


@pytest.fixture(scope="module")
def hx():
    import __graft_entry__ as entry
    entry.build()
    import paper_2605_16637_b200 as mod
    return mod


def _sliced(fn, calls, n_out):
    """fn(calls[lo:hi]) over slices of the batch on several host threads; fn returns a tuple of arrays
    with one row per call, of which the first n_out are concatenated again."""
    n = len(calls)
    step = max(256, -(-n // (4 * N_THREADS)))
    bounds = [(lo, min(n, lo + step)) for lo in range(0, n, step)]
    with ThreadPoolExecutor(N_THREADS) as ex:
        parts = list(ex.map(lambda b: fn(calls[b[0]:b[1]]), bounds))
    return tuple(np.concatenate([p[k] for p in parts]) for k in range(n_out))


def _oracle_forest(oracle, oc, wl):
    """Stand-alone node costs and horizons of the whole forest from the oracle."""
    if wl.node_cost is not None:
        cost = wl.node_cost
    else:
        cost = _sliced(lambda c: oracle.schedule(oc, c, flags=ho.FLAG_UNLOADED | ho.FLAG_NO_DAG), wl.node_calls, 3)[2]
    return cost, oracle.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)


def _gpu_setup(hx, wl):
    gc = hh.gpu_cluster(wl)
    cost = wl.node_cost if wl.node_cost is not None else hh.gpu_node_costs(gc, wl.node_calls)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    return gc, cost


def _check_forest(gc, gcost, ocost, dag):
    assert np.array_equal(gcost, ocost), "stand-alone node costs differ"
    cp, tail, H = gc.dag_results()
    assert np.array_equal(cp, dag.cp) and np.array_equal(tail, dag.tail) and np.array_equal(H, dag.H), "horizons differ"


def test_large_full(hx, oracle):
    wl = make_workload("large")
    gc, gcost = _gpu_setup(hx, wl)
    oc = hh.oracle_cluster(wl)
    ocost, dag = _oracle_forest(oracle, oc, wl)
    _check_forest(gc, gcost, ocost, dag)
    calls = wl.calls
    kw = dict(dag=dag, node_wf=wl.node_wf, elapsed=wl.elapsed)
    for mode_g, mode_o in ((hx.HX_MODE_SLACK, ho.MODE_SLACK), (hx.HX_MODE_RATIO, ho.MODE_RATIO)):
        gc.set_options(score_mode=mode_g, alpha=wl.alpha)
        a, c = gc.schedule_batch(calls)
        a, c = a.cpu().numpy(), c.cpu().numpy()
        oa, ocst, _ = _sliced(lambda s: oracle.schedule(oc, s, mode=mode_o, alpha=wl.alpha, **kw), calls, 3)
        hh.assert_costs_close(c, ocst, "large")
        hh.assert_assign_matches(oracle, oc, calls, a, oa, what="large")
        assert np.array_equal(c, ocst) and np.array_equal(a, oa)
    assert gc.status() == 0
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
    oc = hh.oracle_cluster(wl)
    oa, ocst, _ = _sliced(lambda s: oracle.schedule(oc, s, mode=ho.MODE_RATIO, dag=r, node_wf=wl.node_wf,
                                                    elapsed=wl.elapsed), calls, 3)
    assert np.array_equal(c, ocst) and np.array_equal(a, oa)
    assert gc.status() == 0
    gc.close()


def test_sweep_full_as_benchmarked(hx, oracle):
    """All 16 scheduler invocations of the sweep, as the benchmark runs them: the free KV tokens are
    restored ahead of every invocation, the prefill queues carry the commits of the one before."""
    import torch
    wl = make_workload("sweep")
    P, D, chunk, K = wl.P, wl.D, wl.chunk, wl.topk
    gc, gcost = _gpu_setup(hx, wl)
    calls = wl.calls
    n_chunks = len(calls) // chunk
    assert n_chunks == 16 and n_chunks * chunk == len(calls)
    free0 = wl.kv_free[P:].copy()
    qP0 = wl.load_s[:P].copy()
    gc.set_options(score_mode=hx.HX_MODE_RATIO, topk=K, commit=1, alpha=wl.alpha)
    results = []
    for i in range(n_chunks):
        gc.update_loads(kv_free=free0)
        a, c = gc.schedule_batch(calls[i * chunk:(i + 1) * chunk])
        pair, cost, prio = gc.topk_results(chunk)
        qP, _, free = gc.read_loads()
        results.append((a.cpu().numpy(), c.cpu().numpy(), pair, cost, prio, qP, free))
    assert gc.status() == 0

    # the same 16 invocations through the host-buffer entry point (what the end-to-end figure times)
    calls_pin = torch.from_numpy(calls.view(np.uint8).reshape(-1, 16).copy()).pin_memory()
    a_pin = torch.full((len(calls),), -7, dtype=torch.int32).pin_memory()
    c_pin = torch.full((len(calls),), -7.0, dtype=torch.float32).pin_memory()
    free_pin = torch.from_numpy(free0.astype(np.float32)).pin_memory()
    gc.update_loads(qP=qP0, kv_free=free0)
    sp = torch.cuda.current_stream().cuda_stream
    hx.hx_schedule_sweep_host(gc.h, calls_pin.numpy().view(hx.CALL_DTYPE).reshape(-1), chunk, free_pin.numpy(),
                              a_pin.numpy(), c_pin.numpy(), sp)
    torch.cuda.current_stream().synchronize()
    assert np.array_equal(a_pin.numpy(), np.concatenate([r[0] for r in results]))
    assert np.array_equal(c_pin.numpy(), np.concatenate([r[1] for r in results]))
    sw_qP, _, sw_free = gc.read_loads()
    assert np.array_equal(sw_qP, results[-1][5]) and np.array_equal(sw_free, results[-1][6])

    # the oracle, invocation by invocation
    oc = hh.oracle_cluster(wl)
    ocost, dag = _oracle_forest(oracle, oc, wl)
    _check_forest(gc, gcost, ocost, dag)
    kw = dict(dag=dag, node_wf=wl.node_wf, elapsed=wl.elapsed)
    qP = qP0.copy()
    m = calls["prompt_tokens"] + calls["output_tokens"]
    placed_total = 0
    for i, (a, c, pair, cost, prio, gq, gfree) in enumerate(results):
        ci = calls[i * chunk:(i + 1) * chunk]
        oc.qP[:] = qP
        op, ocs, opr, om, ots = _sliced(lambda s: oracle.topk(oc, s, K, **kw), ci, 5)
        what = "sweep invocation %d" % i
        assert np.array_equal(pair, op), what
        assert np.array_equal(cost, ocs) and np.array_equal(prio, opr), what
        oa, ofree, oq = oracle.conflict(op, opr, om, ots, free0, qP, D)
        assert np.array_equal(a, oa), what
        assert np.array_equal(gfree, ofree) and np.array_equal(gq, oq), what
        _, ocost_i, _ = _sliced(lambda s: oracle.schedule(oc, s, mode=ho.MODE_RATIO, **kw), ci, 3)
        assert np.array_equal(c, ocost_i), what
        # properties that hold at any size
        placed = a >= 0
        assert np.all(gfree >= 0) and np.all(gfree <= free0)
        used = np.zeros(D); np.add.at(used, a[placed] % D, m[i * chunk:(i + 1) * chunk][placed])
        assert np.array_equal((free0 - gfree).astype(np.float64), used)
        assert np.all(gq >= qP)
        placed_total += int(placed.sum())
        qP = oq
    assert 0 < placed_total < len(calls)
    gc.close()
