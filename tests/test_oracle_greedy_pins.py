"""Pins of the oracle's recomputing greedy planner (Algorithm 1, the while-loop over the
queue snapshot) against things other than itself: a run worked out in exact rational
arithmetic, a plain-Python loop around the already pinned one-shot scorer, and invariants
of the procedure."""
import json
import os

import numpy as np

from oracle import hx_oracle as ho
from hx_synth import CALL_DTYPE

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _cluster(rng, P, D, G=3, M=2):
    types = np.stack([rng.uniform(50, 2000, G), rng.uniform(0.3, 8, G)], 1)
    models = np.stack([rng.uniform(1e9, 2e11, M), rng.uniform(1e9, 2e11, M),
                       rng.choice([65536.0, 131072.0, 327680.0], M)], 1)
    return ho.Cluster(types, rng.integers(0, G, P), rng.integers(0, G, D), rng.uniform(0, 2, P),
                      rng.uniform(0, 2, D), np.full(D, 1e6), rng.uniform(25, 400, (P, D)), models)


def _calls(rng, C, M=2):
    a = np.zeros(C, dtype=CALL_DTYPE)
    a["node"] = np.arange(C)
    a["model"] = rng.integers(0, M, C)
    a["prompt_tokens"] = np.clip(np.round(rng.lognormal(7, 1, C)), 1, 32768)
    a["output_tokens"] = np.clip(np.round(rng.lognormal(5, 1, C)), 1, 32768)
    return a


def _dag(rng, C):
    """every call is its own workflow: elapsed and horizon per call, no tail"""
    H = rng.uniform(0.5, 4.0, C).astype(np.float32)
    el = rng.uniform(0.0, 2.0, C).astype(np.float32)
    return ho.DagResult(cp=None, tail=np.zeros(C, np.float32), H=H), np.arange(C, dtype=np.uint32), el


def _clone(cl, qP=None, capD=None):
    return ho.Cluster(np.stack([cl.tflops, cl.tbps], 1), cl.typeP, cl.typeD,
                      cl.qP if qP is None else qP, cl.qD, cl.capD if capD is None else capD, cl.link,
                      np.stack([cl.phi, cl.omega, cl.kappa], 1))


def test_greedy_worked_run_in_exact_arithmetic(oracle):
    with open(os.path.join(GOLD, "greedy_hand.json")) as f:
        g = json.load(f)
    i, e = g["inputs"], g["expected"]
    cl = ho.Cluster(i["gpu_types"], i["typeP"], i["typeD"], i["qP"], i["qD"], i["capD"], i["link_gbps"],
                    [i["model"]])
    C = len(i["calls"])
    calls = np.zeros(C, dtype=CALL_DTYPE)
    for c, r in enumerate(i["calls"]):
        calls[c] = (c, 0, r["prompt_tokens"], r["output_tokens"])
    dag = ho.DagResult(cp=None, tail=np.zeros(C, np.float32),
                       H=np.array([r["H"] for r in i["calls"]], np.float32))
    el = np.array([r["elapsed"] for r in i["calls"]], np.float32)
    a, ratio, order, placed, qP, free = oracle.greedy(cl, calls, i["freeD"], dag=dag,
                                                      node_wf=np.arange(C, dtype=np.uint32), elapsed=el)
    assert placed == len(e["order"])
    assert list(order[:placed]) == e["order"] and np.all(order[placed:] == -1)
    assert list(a) == e["assign"]
    for c in range(C):
        if e["ratio"][c] is None:
            assert np.isinf(ratio[c]) and a[c] == -1
        else:
            assert abs(ratio[c] - e["ratio"][c]) <= 2e-6 * e["ratio"][c]
    np.testing.assert_allclose(qP, e["qP"], rtol=2e-6)
    assert list(free) == e["freeD"]


def _python_loop(orc, cl, calls, freeD, dag, node_wf, el):
    """The same procedure written around the one-shot scorer: capacities of the simulated state
    are passed as Cap(d) = min(Cap(d), free(d)), which is the same feasibility test."""
    C = calls.shape[0]
    qP = cl.qP.copy(); free = np.asarray(freeD, np.float32).copy()
    tpre, _, _, m = orc.terms(cl, calls)
    waiting = list(range(C))
    assign = np.full(C, -1, np.int32); ratio = np.full(C, np.inf, np.float32); order = []
    delta = np.full(C, np.inf, np.float32)
    while waiting:
        sim = _clone(cl, qP=qP, capD=np.minimum(cl.capD, free))
        idx = np.array(waiting)
        a, r, dl = orc.schedule(sim, calls[idx], mode=ho.MODE_RATIO, flags=ho.FLAG_NO_TAIL, dag=dag,
                                node_wf=node_wf, elapsed=el)
        ok = np.flatnonzero(a >= 0)
        if ok.size == 0:
            break
        k = ok[np.argmax(r[ok])]                     # first maximum = lowest call index among equals
        c, j = int(idx[k]), int(a[k])
        p, d = divmod(j, cl.D)
        qP[p] = np.float32(qP[p] + tpre[c, cl.typeP[p]])
        free[d] = np.float32(free[d] - m[c])
        assign[c], ratio[c], delta[c] = j, r[k], dl[k]
        order.append(c)
        waiting.remove(c)
    return assign, ratio, order, qP, free, delta


def test_greedy_equals_loop_around_the_one_shot_scorer(oracle):
    rng = np.random.default_rng(21)
    for P, D, C, frac in [(1, 1, 12, 0.5), (2, 2, 30, 0.6), (3, 4, 40, 0.4), (4, 4, 48, 2.0)]:
        cl = _cluster(rng, P, D)
        calls = _calls(rng, C)
        dag, nwf, el = _dag(rng, C)
        _, _, _, m = oracle.terms(cl, calls)
        freeD = np.floor(rng.uniform(0.5, 1.5, D) * frac * m.sum() / D).astype(np.float32)
        a, ratio, order, placed, qP, free, delta = oracle.greedy(cl, calls, freeD, dag=dag, node_wf=nwf, elapsed=el,
                                                                 with_delta=True)
        ea, er, eo, eq, ef, ed = _python_loop(oracle, cl, calls, freeD, dag, nwf, el)
        assert placed == len(eo) and list(order[:placed]) == eo
        assert np.array_equal(a, ea) and np.array_equal(ratio, er)
        assert np.array_equal(delta, ed)                      # the Delta inside the ratio, +inf when passed over
        took = a >= 0
        assert np.array_equal(ratio[took], ((el[nwf[calls["node"][took]]] + delta[took]) / dag.H[nwf[calls["node"][took]]]).astype(np.float32))
        assert np.array_equal(qP, eq) and np.array_equal(free, ef)
        if frac < 1:
            assert (a == -1).any() and (a >= 0).any()        # capacity really binds
        else:
            assert np.all(a >= 0)


def test_greedy_invariants(oracle):
    rng = np.random.default_rng(22)
    cl = _cluster(rng, 3, 3)
    C = 36
    calls = _calls(rng, C)
    dag, nwf, el = _dag(rng, C)
    _, _, _, m = oracle.terms(cl, calls)
    freeD = np.floor(0.5 * m.sum() / 3 * np.ones(3)).astype(np.float32)
    a, ratio, order, placed, qP, free = oracle.greedy(cl, calls, freeD, dag=dag, node_wf=nwf, elapsed=el)
    # the first call taken is the most urgent one of the one-shot projection, on its one-shot pair
    a1, r1, _ = oracle.schedule(cl, calls, mode=ho.MODE_RATIO, flags=ho.FLAG_NO_TAIL, dag=dag, node_wf=nwf,
                                elapsed=el)
    first = int(np.argmax(r1))
    assert order[0] == first and a[first] == a1[first] and ratio[first] == r1[first]
    # KV tokens are never over-committed and are conserved
    assert np.all(free >= 0)
    used = np.zeros(3); np.add.at(used, a[a >= 0] % 3, m[a >= 0])
    np.testing.assert_array_equal(freeD - free, used.astype(np.float32))
    # a call left behind does not fit anywhere in the final state
    for c in np.flatnonzero(a < 0):
        assert np.all(m[c] > free)
    # prefill queues only grow; the projected ratio of a call is never below its one-shot ratio
    assert np.all(qP >= cl.qP)
    assert np.all(ratio[a >= 0] >= r1[a >= 0])
    # a queue of one call is the one-shot placement
    b, rb, ob, pb, _, _ = oracle.greedy(cl, calls[5:6], freeD, dag=dag, node_wf=nwf, elapsed=el)
    assert pb == 1 and b[0] == a1[5] and rb[0] == r1[5]
    # relabelling the calls (no equal ratios here) relabels the result
    perm = rng.permutation(C)
    a2, ratio2, order2, placed2, _, _ = oracle.greedy(cl, calls[perm], freeD, dag=dag, node_wf=nwf, elapsed=el)
    assert placed2 == placed and np.array_equal(a2, a[perm]) and np.array_equal(ratio2, ratio[perm])
    assert np.array_equal(perm[order2[:placed]], order[:placed])
