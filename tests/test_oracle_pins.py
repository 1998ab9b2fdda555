"""Pins of the CPU oracle against things other than itself.

Closed forms (tests/golden), brute-force enumeration, textbook routines and
invariants; chosen so that a dropped term, a swapped index, a transposed link
matrix or a wrong tie-break in the oracle fails at least one of them.
"""
import itertools
import json
import os

import numpy as np
import pytest

from oracle import hx_oracle as ho
from hx_synth import CALL_DTYPE, make_workload

GOLD = os.path.join(os.path.dirname(__file__), "golden")
REL = 2e-6     # binary32 sequence of a handful of operations vs exact rational value


def _calls(rows):
    a = np.zeros(len(rows), dtype=CALL_DTYPE)
    for i, (node, model, n, o) in enumerate(rows):
        a[i] = (node, model, n, o)
    return a


def _golden_case(c):
    i = c["inputs"]
    cl = ho.Cluster(i["gpu_types"], i["typeP"], i["typeD"], i["qP"], i["qD"], i["capD"],
                    i["link_gbps"], [i["model"]])
    if i.get("attn_flops_per_token2"):
        cl.set_attention([i["attn_flops_per_token2"]])       # prefill variant with a quadratic attention term
    calls = _calls([(0, 0, i["prompt_tokens"], i["output_tokens"])])
    dag = ho.DagResult(cp=None, tail=np.array([i["tail"]], np.float32), H=np.array([i["H"]], np.float32))
    return cl, calls, dag, i


@pytest.fixture(scope="module")
def golden():
    with open(os.path.join(GOLD, "latency_closed_forms.json")) as f:
        return json.load(f)["cases"]


def test_closed_form_terms_and_candidates(oracle, golden):
    for c in golden:
        cl, calls, dag, i = _golden_case(c)
        e = c["expected"]
        tpre, tdec, kvB, m = oracle.terms(cl, calls)
        np.testing.assert_allclose(tpre[0], e["tpre"], rtol=REL, err_msg=c["name"])
        np.testing.assert_allclose(tdec[0], e["tdec"], rtol=REL, err_msg=c["name"])
        assert kvB[0] == np.float32(e["kvB"]) and m[0] == np.float32(e["m"])
        fin = oracle.fin_all(cl, calls)[0].reshape(-1)
        for got, want in zip(fin, e["fin"]):
            if want is None:
                assert np.isinf(got) and got > 0, c["name"]
            else:
                assert abs(got - want) <= REL * abs(want), (c["name"], got, want)


def test_closed_form_scores_and_tie_break(oracle, golden):
    for c in golden:
        cl, calls, dag, i = _golden_case(c)
        e = c["expected"]
        kw = dict(dag=dag, node_wf=np.zeros(1, np.uint32), elapsed=np.array([i["elapsed"]], np.float32),
                  alpha=i["alpha"])
        a, comp, delta = oracle.schedule(cl, calls, mode=ho.MODE_COMPLETION, **kw)
        assert a[0] == e["assign"], c["name"]
        if e["assign"] < 0:
            assert np.isinf(delta[0]) and np.isinf(comp[0])
            continue
        assert abs(delta[0] - e["delta"]) <= REL * e["delta"]
        assert abs(comp[0] - e["completion"]) <= REL * e["completion"]
        _, ratio, _ = oracle.schedule(cl, calls, mode=ho.MODE_RATIO, **kw)
        assert abs(ratio[0] - e["ratio"]) <= REL * e["ratio"]
        _, r2, _ = oracle.schedule(cl, calls, mode=ho.MODE_RATIO, flags=ho.FLAG_NO_TAIL, **kw)
        assert abs(r2[0] - e["ratio_eq2"]) <= REL * e["ratio_eq2"]          # Eq. 2 as printed
        _, slack, _ = oracle.schedule(cl, calls, mode=ho.MODE_SLACK, **kw)
        assert abs(slack[0] - e["slack"]) <= 4e-6 * max(abs(e["slack"]), e["completion"])
        # priority of the capacity pass is Eq. 2 as printed
        pair, cost, prio, m, _ = oracle.topk(cl, calls, 1, dag=dag, node_wf=kw["node_wf"], elapsed=kw["elapsed"])
        assert pair[0, 0] == e["assign"] and abs(prio[0] - e["ratio_eq2"]) <= REL * e["ratio_eq2"]


def _random_cluster(rng, P, D, G=3, M=2, tight=False):
    types = np.stack([rng.uniform(50, 2000, G), rng.uniform(0.3, 8, G)], 1)
    models = np.stack([rng.uniform(1e9, 2e11, M), rng.uniform(1e9, 2e11, M),
                       rng.choice([65536.0, 131072.0, 327680.0], M)], 1)
    cap = rng.choice([600.0, 3000.0, 1e6], D) if tight else np.full(D, 1e6)
    return ho.Cluster(types, rng.integers(0, G, P), rng.integers(0, G, D), rng.uniform(0, 2, P),
                      rng.uniform(0, 2, D), cap, rng.uniform(25, 400, (P, D)), models)


def _random_calls(rng, C, M=2):
    a = np.zeros(C, dtype=CALL_DTYPE)
    a["node"] = np.arange(C)
    a["model"] = rng.integers(0, M, C)
    a["prompt_tokens"] = np.clip(np.round(rng.lognormal(7, 1, C)), 1, 32768)
    a["output_tokens"] = np.clip(np.round(rng.lognormal(5, 1, C)), 1, 32768)
    return a


def test_binary32_sequence_close_to_textbook_double(oracle):
    rng = np.random.default_rng(11)
    for P, D in [(1, 1), (2, 3), (4, 4), (7, 5)]:
        cl = _random_cluster(rng, P, D, tight=True)
        calls = _random_calls(rng, 40)
        f32 = oracle.fin_all(cl, calls).astype(np.float64)
        f64 = oracle.fin_all_f64(cl, calls)
        assert np.array_equal(np.isinf(f32), np.isinf(f64))
        ok = np.isfinite(f64)
        assert np.max(np.abs(f32[ok] - f64[ok]) / f64[ok]) < 1e-6


def test_argmin_is_lowest_index_of_enumerated_minimum(oracle):
    rng = np.random.default_rng(5)
    for P, D in itertools.product([1, 2, 3, 4], [1, 2, 4]):
        cl = _random_cluster(rng, P, D, tight=True)
        cl.qD[:] = np.round(cl.qD * 2) / 2          # equal admission times produce exact ties
        calls = _random_calls(rng, 64)
        fin = oracle.fin_all(cl, calls).reshape(64, -1)
        a, cost, delta = oracle.schedule(cl, calls)
        for c in range(64):
            order = sorted(range(P * D), key=lambda j: (fin[c, j], j))     # explicit sort
            if np.isinf(fin[c, order[0]]):
                assert a[c] == -1 and np.isinf(delta[c])
            else:
                assert a[c] == order[0] and delta[c] == fin[c, order[0]]
                assert cost[c] == delta[c]        # no DAG: elapsed 0, tail 0


def test_exact_ties_resolve_to_lowest_pair_index(oracle):
    # identical instances and a late decode admission: every pair finishes at qD + decode time
    cl = ho.Cluster([[1000, 1]], [0, 0, 0], [0, 0], [0.1, 0.0, 0.2], [9.0, 9.0], [1e6, 1e6],
                    np.full((3, 2), 100.0), [[2e9, 1e9, 1e5]])
    calls = _calls([(0, 0, 1000, 11)])
    fin = oracle.fin_all(cl, calls).reshape(-1)
    assert np.all(fin == fin[0])
    a, _, _ = oracle.schedule(cl, calls)
    assert a[0] == 0
    pair, cost, _, _, _ = oracle.topk(cl, calls, 2)
    assert list(pair[0]) == [0, 1]                # d = 0 then d = 1, each with p = 0


def test_topk_matches_sorted_enumeration(oracle):
    rng = np.random.default_rng(6)
    for P, D, K in [(1, 1, 1), (3, 4, 2), (4, 4, 4), (2, 3, 4), (4, 2, 3)]:
        cl = _random_cluster(rng, P, D, tight=True)
        calls = _random_calls(rng, 50)
        fin = oracle.fin_all(cl, calls)
        pair, cost, prio, m, tsel = oracle.topk(cl, calls, K)
        tpre, _, _, mm = oracle.terms(cl, calls)
        assert np.array_equal(m, mm)
        for c in range(50):
            best = []
            for d in range(D):
                p = min(range(P), key=lambda q: (fin[c, q, d], q))
                if np.isfinite(fin[c, p, d]):
                    best.append((fin[c, p, d], d, p))
            best.sort()
            for k in range(K):
                if k < len(best):
                    f, d, p = best[k]
                    assert pair[c, k] == p * D + d and cost[c, k] == f
                    assert tsel[c, k] == tpre[c, cl.typeP[p]]
                else:
                    assert pair[c, k] == -1 and np.isinf(cost[c, k])
        a, _, delta = oracle.schedule(cl, calls)
        feas = a >= 0
        assert np.array_equal(cost[feas, 0], delta[feas])        # K-list starts at the minimum


def test_monotonicity_invariants(oracle):
    rng = np.random.default_rng(7)
    cl = _random_cluster(rng, 4, 4)
    calls = _random_calls(rng, 30)
    base = oracle.fin_all(cl, calls)
    # a slower link never makes any candidate finish earlier (Section 5.3, joint planning)
    slow = ho.Cluster(np.stack([cl.tflops, cl.tbps], 1), cl.typeP, cl.typeD, cl.qP, cl.qD, cl.capD,
                      cl.link * 0.5, np.stack([cl.phi, cl.omega, cl.kappa], 1))
    assert np.all(oracle.fin_all(slow, calls) >= base)
    # more queued work never makes any candidate finish earlier
    busy = ho.Cluster(np.stack([cl.tflops, cl.tbps], 1), cl.typeP, cl.typeD, cl.qP + 1.0, cl.qD + 0.5,
                      cl.capD, cl.link, np.stack([cl.phi, cl.omega, cl.kappa], 1))
    assert np.all(oracle.fin_all(busy, calls) >= base)
    # only the link entry [p][d] of a pair matters: transposing the matrix changes results
    tr = ho.Cluster(np.stack([cl.tflops, cl.tbps], 1), cl.typeP, cl.typeD, cl.qP, cl.qD, cl.capD,
                    cl.link.T.copy(), np.stack([cl.phi, cl.omega, cl.kappa], 1))
    assert not np.array_equal(oracle.fin_all(tr, calls), base)
    # the unloaded flag is the same as zero queues
    idle = ho.Cluster(np.stack([cl.tflops, cl.tbps], 1), cl.typeP, cl.typeD, cl.qP * 0, cl.qD * 0,
                      cl.capD, cl.link, np.stack([cl.phi, cl.omega, cl.kappa], 1))
    assert np.array_equal(oracle.fin_all(cl, calls, flags=ho.FLAG_UNLOADED), oracle.fin_all(idle, calls))


def test_feasibility_mask_eq4(oracle):
    rng = np.random.default_rng(8)
    cl = _random_cluster(rng, 3, 4, tight=True)
    calls = _random_calls(rng, 200)
    fin = oracle.fin_all(cl, calls)
    m = calls["prompt_tokens"] + calls["output_tokens"]
    infeasible = m[:, None] > cl.capD[None, :]
    assert np.array_equal(np.isinf(fin), np.broadcast_to(infeasible[:, None, :], fin.shape))
    a, _, _ = oracle.schedule(cl, calls)
    placed = a >= 0
    assert np.all(~infeasible[np.flatnonzero(placed), a[placed] % cl.D])
    assert np.array_equal(~placed, infeasible.all(axis=1))


def test_single_pair_decomposition(oracle):
    # P = D = 1: finish = max(qP + prefill + transfer, qD) + decode, term by term
    cl = ho.Cluster([[500, 2]], [0], [0], [0.5], [0.0], [1e6], [[50.0]], [[1e10, 2e10, 131072.0]])
    calls = _calls([(0, 0, 2048, 64)])
    tpre, tdec, kvB, _ = oracle.terms(cl, calls)
    transfer = 2048 * 131072.0 / 50e9
    fin = oracle.fin_all(cl, calls)[0, 0, 0]
    assert abs(fin - (0.5 + float(tpre[0, 0]) + transfer + float(tdec[0, 0]))) < 1e-6 * fin
    cl.qD[0] = 100.0                               # decode admission dominates
    assert oracle.fin_all(cl, calls)[0, 0, 0] == np.float32(100.0) + tdec[0, 0]


# ---------------------------------------------------------------------------
# horizons
# ---------------------------------------------------------------------------

def _csr(n, edges):
    edges = sorted(edges)
    row = np.zeros(n + 1, np.uint32)
    for u, _ in edges:
        row[u + 1] += 1
    row = np.cumsum(row).astype(np.uint32)
    col = np.array([v for _, v in edges], np.uint32)
    return row, col


def test_dag_hand_cases(oracle):
    with open(os.path.join(GOLD, "dag_hand.json")) as f:
        cases = json.load(f)["cases"]
    for c in cases:
        n = len(c["cost"])
        row, col = _csr(n, [tuple(e) for e in c["edges"]])
        r = oracle.longest_path(row, col, c["cost"], c["node_wf"], len(c["H"]))
        assert list(r.cp) == c["cp"] and list(r.tail) == c["tail"] and list(r.H) == c["H"], c["name"]


def _all_path_sums(n, succ, cost, v):
    if not succ[v]:
        return [cost[v]]
    return [cost[v] + s for u in succ[v] for s in _all_path_sums(n, succ, cost, u)]


def test_longest_path_vs_path_enumeration(oracle):
    rng = np.random.default_rng(3)
    for trial in range(30):
        n = int(rng.integers(1, 15))
        edges = [(u, v) for u in range(n) for v in range(u + 1, n) if rng.random() < 0.3]
        perm = rng.permutation(n)                 # node numbers are not a topological order
        edges = [(int(perm[u]), int(perm[v])) for u, v in edges]
        cost = rng.integers(1, 50, n).astype(np.float32)     # integers: every sum is exact
        row, col = _csr(n, edges)
        succ = [[int(x) for x in col[row[v]:row[v + 1]]] for v in range(n)]
        r = oracle.longest_path(row, col, cost, np.zeros(n, np.uint32), 1)
        for v in range(n):
            sums = _all_path_sums(n, succ, cost, v)
            assert r.cp[v] == max(sums)                        # >= every path, attained by one
            assert r.tail[v] == r.cp[v] - cost[v]
        assert r.H[0] == r.cp.max()


def test_chain_is_a_suffix_sum(oracle):
    rng = np.random.default_rng(4)
    n = 300
    cost = rng.lognormal(0, 1, n).astype(np.float32)
    row = np.arange(n + 1, dtype=np.uint32); row[-1] = n - 1
    col = np.arange(1, n, dtype=np.uint32)
    r = oracle.longest_path(row, col, cost, np.zeros(n, np.uint32), 1)
    suffix = np.cumsum(cost[::-1], dtype=np.float32)[::-1]   # sequential binary32 sums from the sink
    assert np.array_equal(r.cp, suffix)
    assert np.array_equal(r.tail[:-1], suffix[1:]) and r.tail[-1] == 0 and r.H[0] == suffix[0]


def test_longest_path_vs_library_shortest_path(oracle):
    sp = pytest.importorskip("scipy.sparse")
    from scipy.sparse.csgraph import bellman_ford
    wl = make_workload("medium", scale=0.1)
    N = wl.n_nodes
    cost = np.random.default_rng(9).lognormal(0, 1, N).astype(np.float32)
    r = oracle.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
    # longest path to a sink = -(shortest path with negated weights) on the reversed graph
    # from a super sink: edge v->u weighs -cost[u]... use edge (u -> v) weight -cost[v], plus cost[u]
    src = np.repeat(np.arange(N), np.diff(wl.row_ptr.astype(np.int64)))
    g = sp.csr_matrix((-cost[wl.col].astype(np.float64), (src, wl.col.astype(np.int64))), shape=(N, N))
    some = np.random.default_rng(1).choice(N, 40, replace=False)
    dist = bellman_ford(g, directed=True, indices=some)
    longest = cost[some].astype(np.float64) - dist.min(axis=1)
    np.testing.assert_allclose(r.cp[some], longest, rtol=1e-5)
    # H is the largest cp of the workflow and is attained at a source
    Hmax = np.zeros(wl.n_workflows); np.maximum.at(Hmax, wl.node_wf, r.cp)
    assert np.array_equal(r.H, Hmax.astype(np.float32))
    indeg = np.bincount(wl.col, minlength=N)
    Hs = np.zeros(wl.n_workflows); np.maximum.at(Hs, wl.node_wf[indeg == 0], r.cp[indeg == 0])
    assert np.array_equal(r.H, Hs.astype(np.float32))


def test_horizon_grows_with_reveal(oracle):
    # appending newly revealed nodes never shrinks H (Section 5.1, "Refine the horizon progressively")
    edges = [(0, 1), (0, 2), (1, 3)]
    cost = np.array([1, 2, 3, 4, 5, 6], np.float32)
    prev = 0.0
    for n, ed in [(3, edges[:2]), (4, edges), (5, edges + [(3, 4)]), (6, edges + [(3, 4), (2, 5)])]:
        row, col = _csr(n, ed)
        H = oracle.longest_path(row, col, cost[:n], np.zeros(n, np.uint32), 1).H[0]
        assert H >= prev
        prev = H
    assert prev == 1 + 2 + 4 + 5


def test_cycle_is_rejected(oracle):
    row, col = _csr(3, [(0, 1), (1, 2), (2, 0)])
    with pytest.raises(ValueError):
        oracle.longest_path(row, col, [1, 1, 1], [0, 0, 0], 1)


# ---------------------------------------------------------------------------
# capacity-conflict pass
# ---------------------------------------------------------------------------

def _conflict_python(pair, prio, m, tsel, freeD, qP, D):
    free = [np.float32(x) for x in freeD]; q = [np.float32(x) for x in qP]
    order = sorted(range(len(prio)), key=lambda c: (-float(prio[c]), c))
    out = [-1] * len(prio)
    for c in order:
        for k in range(pair.shape[1]):
            j = int(pair[c, k])
            if j >= 0 and free[j % D] >= m[c]:
                free[j % D] = np.float32(free[j % D] - m[c]); q[j // D] = np.float32(q[j // D] + tsel[c, k])
                out[c] = j
                break
    return np.array(out, np.int32), np.array(free, np.float32), np.array(q, np.float32)


def test_conflict_pass_vs_plain_python(oracle):
    rng = np.random.default_rng(12)
    for P, D, K, C in [(2, 2, 2, 40), (4, 4, 4, 200), (3, 5, 3, 150), (4, 3, 4, 100)]:
        cl = _random_cluster(rng, P, D)
        calls = _random_calls(rng, C)
        pair, cost, prio, m, tsel = oracle.topk(cl, calls, K)
        prio[rng.integers(0, C, C // 4)] = prio[0]            # equal priorities -> index order
        freeD = np.floor(rng.uniform(0.2, 0.6, D) * m.sum() / D).astype(np.float32)
        a, f2, q2 = oracle.conflict(pair, prio, m, tsel, freeD, cl.qP, D)
        ea, ef, eq = _conflict_python(pair, prio, m, tsel, freeD, cl.qP, D)
        assert np.array_equal(a, ea) and np.array_equal(f2, ef) and np.array_equal(q2, eq)
        assert (a == -1).any() and (a >= 0).any()             # the case really is contended
        assert np.all(f2 >= 0)                                # never over-committed
        used = np.zeros(D); np.add.at(used, a[a >= 0] % D, m[a >= 0])
        np.testing.assert_array_equal(freeD - f2, used.astype(np.float32))
        first = sorted(range(C), key=lambda c: (-float(prio[c]), c))[0]
        if freeD[pair[first, 0] % D] >= m[first]:
            assert a[first] == pair[first, 0]                 # the most urgent call gets its best pair


def test_conflict_pass_hand_worked_case(oracle):
    """Eight calls, K = 3, worked by hand (tests/golden/make_conflict_case.py): an exact priority tie that
    decides who gets the last room, a first candidate that is full, a call that takes its third candidate,
    calls left unplaced, an equality fit, and prefill-queue sums whose binary32 value depends on the
    order of the additions."""
    with open(os.path.join(GOLD, "conflict_hand.json")) as f:
        g = json.load(f)
    prio = np.array([np.inf if x == "inf" else x for x in g["prio"]], np.float32)
    pair = np.array(g["pair"], np.int32)
    tpre = np.array(g["tpre"], np.float32)
    assert np.array_equal(tpre.astype(np.float64), np.array(g["tpre"]))      # inputs are binary32 values
    a, free, qP = oracle.conflict(pair, prio, np.array(g["m"], np.float32), tpre, g["free"], g["qP"], g["D"])
    e = g["expect"]
    assert a.tolist() == e["assign"]
    assert free.tolist() == e["free"]
    assert [float(x).hex() for x in qP] == e["qP_hex"]
    # the hand-derived visiting order really is the one the rule states
    order = sorted(range(len(prio)), key=lambda c: (-float(prio[c]), c))
    assert order == e["order"]


def test_conflict_pass_equal_calls_are_visited_by_index(oracle):
    """300 identical calls of 1,000 tokens, four decode instances with room for 20 + 5 + 7 + 3 of them,
    every call listing all four instances: all priorities are equal, so the calls are visited by index
    and exactly the first 35 obtain a pair."""
    rng = np.random.default_rng(3)
    cl = _random_cluster(rng, 4, 4)
    calls = np.zeros(300, CALL_DTYPE)
    calls["prompt_tokens"] = 900; calls["output_tokens"] = 100
    pair, cost, prio, m, tsel = oracle.topk(cl, calls, 4)
    assert np.all(prio == prio[0]) and np.all(m == 1000) and np.all(pair >= 0)
    free = np.array([20000, 5000, 7000, 3000], np.float32)
    a, f2, _ = oracle.conflict(pair, prio, m, tsel, free, cl.qP, 4)
    assert (a[:35] >= 0).all() and (a[35:] == -1).all()
    assert f2.tolist() == [0, 0, 0, 0]
    assert np.bincount(a[:35] % 4, minlength=4).tolist() == [20, 5, 7, 3]


def test_conflict_pass_without_contention_is_the_argmin(oracle):
    rng = np.random.default_rng(13)
    cl = _random_cluster(rng, 4, 4)
    calls = _random_calls(rng, 100)
    pair, cost, prio, m, tsel = oracle.topk(cl, calls, 1)
    a, f2, q2 = oracle.conflict(pair, prio, m, tsel, np.full(4, 1e7, np.float32), cl.qP, 4)
    b, _, _ = oracle.schedule(cl, calls)
    # K = 1 orders ties over d first, the plain argmin over p first; with random loads there are none
    assert np.array_equal(a, b)
    # queue growth in priority order, accumulated in binary32
    q = cl.qP.copy()
    for c in sorted(range(100), key=lambda c: (-float(prio[c]), c)):
        q[a[c] // 4] = np.float32(q[a[c] // 4] + tsel[c, 0])
    assert np.array_equal(q, q2)


def test_oracle_runs_on_generated_configs(oracle):
    for name in ("tiny", "medium"):
        wl = make_workload(name)
        cl = ho.Cluster.from_workload(wl)
        cost, _, _ = oracle.schedule(cl, wl.node_calls, flags=ho.FLAG_UNLOADED)[1], None, None
        dag = oracle.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
        assert np.all(dag.H > 0) and np.all(np.isfinite(dag.cp))
        a, score, delta = oracle.schedule(cl, wl.calls, mode=ho.MODE_SLACK, alpha=wl.alpha, dag=dag,
                                          node_wf=wl.node_wf, elapsed=wl.elapsed)
        assert np.all(a >= 0) and np.all(a < wl.P * wl.D) and np.all(np.isfinite(score))


def test_cost_change_stays_inside_its_workflow_and_is_monotone(oracle):
    """Workflows are independent components: replacing a node's cost estimate by an observed latency
    (Section 5.1) can only change the nodes of that workflow that reach the node, a larger cost never
    shortens any path, and the node's own tail is untouched."""
    wl = make_workload("medium", scale=0.25)
    rng = np.random.default_rng(3)
    cost = rng.lognormal(0, 1, wl.n_nodes).astype(np.float32)
    base = oracle.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
    v = int(rng.integers(0, wl.n_nodes))
    up = cost.copy(); up[v] = cost[v] * np.float32(3.0)
    new = oracle.longest_path(wl.row_ptr, wl.col, up, wl.node_wf, wl.n_workflows)
    other = wl.node_wf != wl.node_wf[v]
    assert np.array_equal(new.cp[other], base.cp[other]) and np.array_equal(new.tail[other], base.tail[other])
    keep = np.ones(wl.n_workflows, bool); keep[wl.node_wf[v]] = False
    assert np.array_equal(new.H[keep], base.H[keep])
    assert np.all(new.cp >= base.cp) and np.all(new.H >= base.H)
    assert new.tail[v] == base.tail[v] and new.cp[v] == np.float32(up[v] + base.tail[v])


def test_quadratic_prefill_variant(oracle):
    """psi = 0 is the linear model bit for bit; psi > 0 only lengthens the prefill, by n^2 * psi / F on a
    compute-bound class, and leaves decode time, demand and transfer alone."""
    rng = np.random.default_rng(41)
    cl = _random_cluster(rng, 3, 3)
    calls = _random_calls(rng, 50)
    base = oracle.fin_all(cl, calls)
    t0 = oracle.terms(cl, calls)
    cl.set_attention(np.zeros(cl.M, np.float32))
    assert np.array_equal(oracle.fin_all(cl, calls), base)
    psi = np.array([3e5, 7e5], np.float32)
    cl.set_attention(psi)
    t1 = oracle.terms(cl, calls)
    assert np.array_equal(t1[1], t0[1]) and np.array_equal(t1[2], t0[2]) and np.array_equal(t1[3], t0[3])
    assert np.all(t1[0] >= t0[0]) and np.all(oracle.fin_all(cl, calls) >= base)
    n = calls["prompt_tokens"].astype(np.float64)
    F = cl.tflops.astype(np.float64) * 1e12
    B = cl.tbps.astype(np.float64) * 1e12
    phi, om, ka = (x.astype(np.float64)[calls["model"]] for x in (cl.phi, cl.omega, cl.kappa))
    want = np.maximum((n * phi + n * n * psi.astype(np.float64)[calls["model"]])[:, None] / F[None, :],
                      (om + n * ka)[:, None] / B[None, :])
    assert np.max(np.abs(t1[0] - want) / want) < 1e-6
