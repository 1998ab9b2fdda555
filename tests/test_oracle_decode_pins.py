"""Pins of the oracle's decode-stage scheduler (Section 5.4: ranking by Eq. 2, capacity by Eq. 3-4 over
token-capacity intervals, locked and free calls) against things other than itself: a run worked out in
exact rational arithmetic, a brute-force search straight from the definition, and invariants."""
import json
import os

import numpy as np

from oracle import hx_oracle as ho
from hx_synth import CALL_DTYPE

GOLD = os.path.join(os.path.dirname(__file__), "golden")
F32 = np.float32


def _cluster(rng, D, G=3, M=2, caps=(3000.0, 6000.0, 20000.0)):
    types = np.stack([rng.uniform(50, 2000, G), rng.uniform(0.3, 8, G)], 1)
    models = np.stack([rng.uniform(1e9, 2e11, M), rng.uniform(1e9, 2e11, M),
                       rng.choice([65536.0, 131072.0, 327680.0], M)], 1)
    return ho.Cluster(types, [0], rng.integers(0, G, D), [0.0], np.zeros(D), rng.choice(caps, D),
                      np.full((1, D), 100.0), models)


def _calls(rng, C, M=2, hi=1500):
    a = np.zeros(C, dtype=CALL_DTYPE)
    a["node"] = np.arange(C)
    a["model"] = rng.integers(0, M, C)
    a["prompt_tokens"] = rng.integers(50, hi, C)
    a["output_tokens"] = rng.integers(5, 400, C)
    return a


def _running(rng, cl, per=3):
    ptr, end, tok = [0], [], []
    for d in range(cl.D):
        k = int(rng.integers(0, per + 1))
        share = rng.dirichlet(np.ones(k + 1))[:k] * 0.9 * cl.capD[d] if k else []
        for s in share:
            end.append(rng.uniform(0.01, 3.0)); tok.append(np.floor(s))
        ptr.append(len(end))
    return np.array(ptr, np.uint32), np.array(end, F32), np.array(tok, F32)


def _usage(iv, t):
    return sum(m for s, e, m in iv if s <= t < e)


def _earliest_by_definition(iv, cap, m, tau, ready):
    """Candidate starts are the ready time and the ends of intervals after it; a start is feasible when the
    usage at the start and at every interval start inside the window leaves m tokens.  binary32 values,
    exact comparisons; the window end is the one binary32 addition start + tau."""
    for c in sorted({float(ready)} | {e for s, e, _ in iv if e > ready}):
        fin = float(F32(c) + F32(tau))
        if all(_usage(iv, t) + m <= cap for t in [c] + [s for s, e, _ in iv if c < s < fin]):
            return c, fin
    raise AssertionError


def _python_greedy(orc, cl, calls, ptr, end, tok, lock, ready, dag, nwf, el):
    C = calls.shape[0]
    _, tdec, _, m = orc.terms(cl, calls)
    iv = [[(0.0, float(end[i]), float(tok[i])) for i in range(ptr[d], ptr[d + 1])] for d in range(cl.D)]
    waiting = list(range(C))
    inst = np.full(C, -1, np.int32); start = np.full(C, np.inf, F32); ratio = np.full(C, np.inf, F32); order = []
    while waiting:
        best = None
        for c in waiting:
            opt = None
            for d in range(cl.D):
                if (lock[c] >= 0 and lock[c] != d) or m[c] > cl.capD[d]:
                    continue
                s, f = _earliest_by_definition(iv[d], float(cl.capD[d]), float(m[c]), tdec[c, cl.typeD[d]], ready[c])
                if opt is None or f < opt[0]:
                    opt = (f, s, d)
            if opt is None:
                continue
            w = nwf[calls["node"][c]]
            R = F32(F32(el[w]) + F32(opt[0])) / F32(dag.H[w])
            if best is None or R > best[0]:
                best = (R, c, opt)
        if best is None:
            break
        R, c, (f, s, d) = best
        iv[d].append((s, f, float(m[c])))
        inst[c], start[c], ratio[c] = d, s, R
        order.append(c); waiting.remove(c)
    return inst, start, ratio, order, iv


def _dag(rng, C):
    H = rng.uniform(0.5, 4.0, C).astype(F32)
    return ho.DagResult(cp=None, tail=np.zeros(C, F32), H=H), np.arange(C, dtype=np.uint32), rng.uniform(0, 2, C).astype(F32)


def test_decode_worked_run_in_exact_arithmetic(oracle):
    with open(os.path.join(GOLD, "decode_hand.json")) as f:
        g = json.load(f)
    i, e = g["inputs"], g["expected"]
    D, C = len(i["capD"]), len(i["calls"])
    cl = ho.Cluster(i["gpu_types"], [0], i["typeD"], [0.0], np.zeros(D), i["capD"], np.full((1, D), 100.0), [i["model"]])
    calls = np.zeros(C, dtype=CALL_DTYPE)
    for c, r in enumerate(i["calls"]):
        calls[c] = (c, 0, r["prompt_tokens"], r["output_tokens"])
    ptr = np.cumsum([0] + [len(r) for r in i["running"]]).astype(np.uint32)
    end = np.array([x["end"] for r in i["running"] for x in r], F32)
    tok = np.array([x["tokens"] for r in i["running"] for x in r], F32)
    dag = ho.DagResult(cp=None, tail=np.zeros(C, F32), H=np.array([r["H"] for r in i["calls"]], F32))
    inst, start, ratio, order, placed = oracle.decode_greedy(
        cl, calls, ptr, end, tok, [r["lock"] for r in i["calls"]], [r["ready"] for r in i["calls"]], dag=dag,
        node_wf=np.arange(C, dtype=np.uint32), elapsed=np.array([r["elapsed"] for r in i["calls"]], F32))
    assert placed == len(e["order"]) and list(order[:placed]) == e["order"] and list(inst) == e["inst"]
    np.testing.assert_allclose(start, e["start"], rtol=2e-6, atol=1e-9)
    np.testing.assert_allclose(ratio, e["ratio"], rtol=2e-6)


def test_decode_greedy_equals_search_from_the_definition(oracle):
    rng = np.random.default_rng(31)
    for D, C in [(1, 8), (2, 12), (3, 16), (4, 20)]:
        for rep in range(3):
            cl = _cluster(rng, D)
            calls = _calls(rng, C)
            ptr, end, tok = _running(rng, cl)
            lock = np.where(rng.random(C) < 0.3, rng.integers(0, D, C), -1).astype(np.int32)
            ready = np.where(rng.random(C) < 0.5, 0.0, rng.uniform(0, 1.0, C)).astype(F32)
            dag, nwf, el = _dag(rng, C)
            inst, start, ratio, order, placed = oracle.decode_greedy(cl, calls, ptr, end, tok, lock, ready, dag=dag,
                                                                    node_wf=nwf, elapsed=el)
            ei, es, er, eo, _ = _python_greedy(oracle, cl, calls, ptr, end, tok, lock, ready, dag, nwf, el)
            assert placed == len(eo) and list(order[:placed]) == eo
            assert np.array_equal(inst, ei) and np.array_equal(start, es) and np.array_equal(ratio, er)


def test_decode_greedy_invariants(oracle):
    rng = np.random.default_rng(32)
    D, C = 3, 30
    cl = _cluster(rng, D, caps=(4000.0,))
    calls = _calls(rng, C)
    ptr, end, tok = _running(rng, cl)
    lock = np.where(rng.random(C) < 0.4, rng.integers(0, D, C), -1).astype(np.int32)
    ready = rng.uniform(0, 0.5, C).astype(F32)
    dag, nwf, el = _dag(rng, C)
    inst, start, ratio, order, placed = oracle.decode_greedy(cl, calls, ptr, end, tok, lock, ready, dag=dag,
                                                            node_wf=nwf, elapsed=el)
    _, tdec, _, m = oracle.terms(cl, calls)
    assert placed == C                                         # every call fits an empty instance
    assert np.all(start >= ready)                              # nobody decodes before its KV cache is there
    assert np.all(inst[lock >= 0] == lock[lock >= 0])          # locked calls do not migrate
    # the capacity is respected at every instant: usage is piecewise constant, check every breakpoint
    for d in range(D):
        iv = [(0.0, float(end[i]), float(tok[i])) for i in range(ptr[d], ptr[d + 1])]
        iv += [(float(start[c]), float(F32(start[c]) + F32(tdec[c, cl.typeD[d]])), float(m[c])) for c in range(C) if inst[c] == d]
        for t in sorted({s for s, _, _ in iv}):
            assert _usage(iv, t) <= cl.capD[d]
    # without contention every call starts when ready, on the instance that finishes it first
    roomy = ho.Cluster(np.stack([cl.tflops, cl.tbps], 1), [0], cl.typeD, [0.0], np.zeros(D), np.full(D, 1e7),
                       np.full((1, D), 100.0), np.stack([cl.phi, cl.omega, cl.kappa], 1))
    free = np.full(C, -1, np.int32)
    i2, s2, r2, o2, p2 = oracle.decode_greedy(roomy, calls, ptr, end, tok, free, ready, dag=dag, node_wf=nwf, elapsed=el)
    assert p2 == C and np.array_equal(s2, ready)
    fin = ready[:, None] + tdec[:, cl.typeD]
    assert np.array_equal(i2, np.argmin(fin, axis=1))
    # ... and they are taken by decreasing ratio, which no commit changes
    assert np.all(np.diff(r2[o2]) <= 0)
    # a call larger than every instance is passed over
    big = calls.copy(); big["prompt_tokens"][4] = 5000
    i3, s3, r3, o3, p3 = oracle.decode_greedy(cl, big, ptr, end, tok, lock, ready, dag=dag, node_wf=nwf, elapsed=el)
    assert p3 == C - 1 and i3[4] == -1 and np.isinf(r3[4]) and 4 not in o3[:p3]


def _hand_case():
    with open(os.path.join(GOLD, "decode_hand.json")) as f:
        g = json.load(f)
    i = g["inputs"]
    D, C = len(i["capD"]), len(i["calls"])
    cl = ho.Cluster(i["gpu_types"], [0], i["typeD"], [0.0], np.zeros(D), i["capD"], np.full((1, D), 100.0), [i["model"]])
    calls = np.zeros(C, dtype=CALL_DTYPE)
    for c, r in enumerate(i["calls"]):
        calls[c] = (c, 0, r["prompt_tokens"], r["output_tokens"])
    ptr = np.cumsum([0] + [len(r) for r in i["running"]]).astype(np.uint32)
    end = np.array([x["end"] for r in i["running"] for x in r], F32)
    tok = np.array([x["tokens"] for r in i["running"] for x in r], F32)
    dag = ho.DagResult(cp=None, tail=np.zeros(C, F32), H=np.array([r["H"] for r in i["calls"]], F32))
    kw = dict(dag=dag, node_wf=np.arange(C, dtype=np.uint32), elapsed=np.array([r["elapsed"] for r in i["calls"]], F32))
    return g, cl, calls, ptr, end, tok, [r["lock"] for r in i["calls"]], [r["ready"] for r in i["calls"]], kw


def test_decode_one_pass_worked_run_in_exact_arithmetic(oracle):
    """The same inputs as the greedy run; the one-pass order (5, 1, 3, 0, 4, 2) and three of the six instances
    differ from the greedy's, so a mix-up of the two forms fails here."""
    g, cl, calls, ptr, end, tok, lock, ready, kw = _hand_case()
    e = g["expected_one_pass"]
    assert e["order"] != g["expected"]["order"] and e["inst"] != g["expected"]["inst"]
    inst, start, ratio, order, placed = oracle.decode_onepass(cl, calls, ptr, end, tok, lock, ready, **kw)
    assert placed == len(e["order"]) and list(order[:placed]) == e["order"] and list(inst) == e["inst"]
    np.testing.assert_allclose(start, e["start"], rtol=2e-6, atol=1e-9)
    np.testing.assert_allclose(ratio, e["ratio"], rtol=2e-6)


def _python_onepass(orc, cl, calls, ptr, end, tok, lock, ready, dag, nwf, el):
    C = calls.shape[0]
    _, tdec, _, m = orc.terms(cl, calls)
    iv = [[(0.0, float(end[i]), float(tok[i])) for i in range(ptr[d], ptr[d + 1])] for d in range(cl.D)]

    def best(c):
        opt = None
        for d in range(cl.D):
            if (lock[c] >= 0 and lock[c] != d) or m[c] > cl.capD[d]:
                continue
            s, f = _earliest_by_definition(iv[d], float(cl.capD[d]), float(m[c]), tdec[c, cl.typeD[d]], ready[c])
            if opt is None or f < opt[0]:
                opt = (f, s, d)
        return opt

    score = {}
    for c in range(C):
        o = best(c)
        if o is not None:
            w = nwf[calls["node"][c]]
            score[c] = F32(F32(el[w]) + F32(o[0])) / F32(dag.H[w])
    visit = sorted(score, key=lambda c: (-score[c], c))
    inst = np.full(C, -1, np.int32); start = np.full(C, np.inf, F32); ratio = np.full(C, np.inf, F32)
    for c in visit:
        f, s, d = best(c)
        iv[d].append((s, f, float(m[c])))
        inst[c], start[c], ratio[c] = d, s, score[c]
    return inst, start, ratio, visit


def test_decode_one_pass_equals_search_from_the_definition(oracle):
    rng = np.random.default_rng(33)
    differs = 0
    for D, C in [(1, 8), (2, 12), (3, 16), (4, 20)]:
        for rep in range(3):
            cl = _cluster(rng, D)
            calls = _calls(rng, C)
            ptr, end, tok = _running(rng, cl)
            lock = np.where(rng.random(C) < 0.3, rng.integers(0, D, C), -1).astype(np.int32)
            ready = np.where(rng.random(C) < 0.5, 0.0, rng.uniform(0, 1.0, C)).astype(F32)
            dag, nwf, el = _dag(rng, C)
            inst, start, ratio, order, placed = oracle.decode_onepass(cl, calls, ptr, end, tok, lock, ready, dag=dag,
                                                                     node_wf=nwf, elapsed=el)
            ei, es, er, eo = _python_onepass(oracle, cl, calls, ptr, end, tok, lock, ready, dag, nwf, el)
            assert placed == len(eo) and list(order[:placed]) == eo and np.all(order[placed:] == -1)
            assert np.array_equal(inst, ei) and np.array_equal(start, es) and np.array_equal(ratio, er)
            gi = oracle.decode_greedy(cl, calls, ptr, end, tok, lock, ready, dag=dag, node_wf=nwf, elapsed=el)
            differs += not np.array_equal(gi[3], order)
    assert differs >= 6                                         # the two forms are not the same thing


def test_decode_one_pass_invariants(oracle):
    rng = np.random.default_rng(34)
    D, C = 3, 30
    cl = _cluster(rng, D, caps=(4000.0,))
    calls = _calls(rng, C)
    ptr, end, tok = _running(rng, cl)
    lock = np.where(rng.random(C) < 0.4, rng.integers(0, D, C), -1).astype(np.int32)
    ready = rng.uniform(0, 0.5, C).astype(F32)
    dag, nwf, el = _dag(rng, C)
    inst, start, ratio, order, placed = oracle.decode_onepass(cl, calls, ptr, end, tok, lock, ready, dag=dag,
                                                             node_wf=nwf, elapsed=el)
    _, tdec, _, m = oracle.terms(cl, calls)
    assert placed == C and np.all(start >= ready) and np.all(inst[lock >= 0] == lock[lock >= 0])
    assert np.all(np.diff(ratio[order]) <= 0)                   # visited by decreasing score
    for d in range(D):
        iv = [(0.0, float(end[i]), float(tok[i])) for i in range(ptr[d], ptr[d + 1])]
        iv += [(float(start[c]), float(F32(start[c]) + F32(tdec[c, cl.typeD[d]])), float(m[c])) for c in range(C) if inst[c] == d]
        for t in sorted({s for s, _, _ in iv}):
            assert _usage(iv, t) <= cl.capD[d]
    # the score is the greedy's first projection: the first call taken, its instance, start and ratio agree
    gi, gs, gr, go, _ = oracle.decode_greedy(cl, calls, ptr, end, tok, lock, ready, dag=dag, node_wf=nwf, elapsed=el)
    f = order[0]
    assert go[0] == f and gi[f] == inst[f] and gs[f] == start[f] and gr[f] == ratio[f]
    # without contention no placement changes another call's projection: both forms give the same plan
    roomy = ho.Cluster(np.stack([cl.tflops, cl.tbps], 1), [0], cl.typeD, [0.0], np.zeros(D), np.full(D, 1e7),
                       np.full((1, D), 100.0), np.stack([cl.phi, cl.omega, cl.kappa], 1))
    free = np.full(C, -1, np.int32)
    a = oracle.decode_onepass(roomy, calls, ptr, end, tok, free, ready, dag=dag, node_wf=nwf, elapsed=el)
    b = oracle.decode_greedy(roomy, calls, ptr, end, tok, free, ready, dag=dag, node_wf=nwf, elapsed=el)
    assert all(np.array_equal(x, y) for x, y in zip(a[:4], b[:4])) and a[4] == b[4] == C
    # a call larger than every instance is never visited
    big = calls.copy(); big["prompt_tokens"][4] = 5000
    i3, s3, r3, o3, p3 = oracle.decode_onepass(cl, big, ptr, end, tok, lock, ready, dag=dag, node_wf=nwf, elapsed=el)
    assert p3 == C - 1 and i3[4] == -1 and np.isinf(r3[4]) and 4 not in o3[:p3]
