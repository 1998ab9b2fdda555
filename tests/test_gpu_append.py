"""Appending newly revealed nodes and edges on the GPU (Section 5.1, progressive refinement of the
horizon) against the definition: the oracle's longest-path pass over the grown graph."""
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


def _csr(n, src, dst):
    order = np.argsort(src, kind="stable")
    row = np.zeros(n + 1, np.uint32)
    np.add.at(row, np.asarray(src, np.int64) + 1, 1)
    return np.cumsum(row, dtype=np.uint32), np.asarray(dst, np.uint32)[order]


def _reveal_plan(wl, cost, rounds, hidden_frac, late_edge_frac, seed):
    """Renumbers a generated forest so that it can be revealed step by step: a random subset of the nodes
    is hidden and handed out over `rounds` appends (new numbers follow the old count), and a few edges
    between nodes of the first upload are held back for a later round as well."""
    rng = np.random.default_rng(seed)
    N = wl.n_nodes
    src = np.repeat(np.arange(N, dtype=np.int64), np.diff(wl.row_ptr.astype(np.int64)))
    dst = wl.col.astype(np.int64)
    stage = np.where(rng.random(N) < hidden_frac, rng.integers(1, rounds + 1, N), 0)
    order = np.argsort(stage, kind="stable")                      # new number -> old number
    new_of = np.empty(N, np.int64); new_of[order] = np.arange(N)
    n_at = [int(np.count_nonzero(stage <= r)) for r in range(rounds + 1)]
    s, d = new_of[src], new_of[dst]
    e_stage = np.maximum(stage[src], stage[dst])
    late = (e_stage == 0) & (rng.random(src.shape[0]) < late_edge_frac)
    e_stage = np.where(late, rng.integers(1, rounds + 1, src.shape[0]), e_stage)
    return dict(cost=np.asarray(cost, np.float32)[order], wf=wl.node_wf[order].astype(np.uint32),
                n_at=n_at, src=s, dst=d, e_stage=e_stage)


def _check(gc, oracle, plan, r, n_workflows):
    n = plan["n_at"][r]
    m = plan["e_stage"] <= r
    row, col = _csr(n, plan["src"][m], plan["dst"][m])
    want = oracle.longest_path(row, col, plan["cost"][:n], plan["wf"][:n], n_workflows)
    cp, tail, H = gc.dag_results()
    assert cp.shape[0] == n
    assert np.array_equal(cp, want.cp) and np.array_equal(tail, want.tail) and np.array_equal(H, want.H), "round %d" % r
    return want, row, col


@pytest.mark.parametrize("name, scale, rounds", [("tiny", 1.0, 3), ("medium", 1.0, 4), ("cp_stress", 1 / 20, 3),
                                                 ("large", 1 / 16, 3)])
def test_appends_equal_a_fresh_pass_over_the_grown_graph(hx, oracle, name, scale, rounds):
    wl = make_workload(name, scale=scale)
    cost = np.random.default_rng(21).lognormal(0, 1, wl.n_nodes).astype(np.float32)
    plan = _reveal_plan(wl, cost, rounds, 0.3, 0.05, seed=22)
    gc = hh.gpu_cluster(wl)
    n0 = plan["n_at"][0]
    m0 = plan["e_stage"] == 0
    row, col = _csr(n0, plan["src"][m0], plan["dst"][m0])
    gc.dag_upload(row, col, plan["cost"][:n0], plan["wf"][:n0], wl.elapsed)
    gc.critical_path()
    prev, _, _ = _check(gc, oracle, plan, 0, wl.n_workflows)
    for r in range(1, rounds + 1):
        a, b = plan["n_at"][r - 1], plan["n_at"][r]
        m = plan["e_stage"] == r
        gc.dag_append(plan["cost"][a:b], plan["wf"][a:b], plan["src"][m], plan["dst"][m])
        want, row, col = _check(gc, oracle, plan, r, wl.n_workflows)
        touched = np.zeros(wl.n_workflows, bool)
        touched[plan["wf"][a:b]] = True; touched[plan["wf"][plan["src"][m]]] = True
        assert np.array_equal(want.H[~touched], prev.H[~touched])
        assert np.all(want.H >= prev.H)                      # revealing more never shrinks a horizon
        prev = want
    # the grown forest behaves like an uploaded one: cost updates, forward pass, a full pass
    n = plan["n_at"][rounds]
    cost_now = plan["cost"][:n].copy()
    ids = np.random.default_rng(23).integers(0, n, max(1, n // 50)).astype(np.uint32)
    new = (cost_now[ids] * 1.5).astype(np.float32)
    gc.update_costs(ids, new)
    for i, v in zip(ids, new):
        cost_now[i] = v
    want = oracle.longest_path(row, col, cost_now, plan["wf"][:n], wl.n_workflows)
    cp, tail, H = gc.dag_results()
    assert np.array_equal(cp, want.cp) and np.array_equal(tail, want.tail) and np.array_equal(H, want.H)
    gc.earliest_start()
    est, eft = gc.earliest_results()
    w_est, w_eft = oracle.earliest_start(row, col, cost_now)
    assert np.array_equal(est, w_est) and np.array_equal(eft, w_eft)
    gc.critical_path()
    cp, tail, H = gc.dag_results()
    assert np.array_equal(cp, want.cp) and np.array_equal(H, want.H)
    assert gc.status() == 0
    gc.close()


def test_scheduling_reads_appended_nodes(hx, oracle):
    wl = make_workload("medium", scale=0.25)
    oc, gc = hh.oracle_cluster(wl), hh.gpu_cluster(wl)
    cost = np.random.default_rng(31).lognormal(0, 1, wl.n_nodes).astype(np.float32)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    # every workflow of the first 40 gets a two-node tail behind its last node
    N = wl.n_nodes
    wfs = np.arange(40, dtype=np.uint32)
    last = np.array([np.flatnonzero(wl.node_wf == w)[-1] for w in wfs], np.uint32)
    new_cost = np.random.default_rng(32).lognormal(0, 1, 80).astype(np.float32)
    new_wf = np.repeat(wfs, 2)
    a = N + 2 * np.arange(40, dtype=np.uint32)
    src = np.concatenate([last, a]); dst = np.concatenate([a, a + 1])
    gc.dag_append(new_cost, new_wf, src, dst)
    all_cost = np.concatenate([cost, new_cost]); all_wf = np.concatenate([wl.node_wf, new_wf]).astype(np.uint32)
    s0 = np.repeat(np.arange(N, dtype=np.int64), np.diff(wl.row_ptr.astype(np.int64)))
    row, col = _csr(N + 80, np.concatenate([s0, src]), np.concatenate([wl.col, dst]))
    dag = oracle.longest_path(row, col, all_cost, all_wf, wl.n_workflows)
    # ready calls on the appended nodes (first of each tail) and on old nodes
    calls = wl.calls[:256].copy()
    calls["node"][:40] = a
    oa, ocost, _ = oracle.schedule(oc, calls, mode=ho.MODE_RATIO, dag=dag, node_wf=all_wf, elapsed=wl.elapsed)
    gc.set_options(score_mode=hx.HX_MODE_RATIO)
    assign, got_cost = gc.schedule_batch(calls)
    hh.assert_assign_matches(oracle, oc, calls, assign.cpu().numpy(), oa, what="after append")
    hh.assert_costs_close(got_cost.cpu().numpy(), ocost, "after append")
    gc.close()


def test_growth_beyond_the_reserve_and_many_small_appends(hx, oracle):
    wl = make_workload("medium", scale=0.25)                 # 128 workflows
    gc = hh.gpu_cluster(wl)
    N, W = wl.n_nodes, wl.n_workflows
    cost = np.random.default_rng(41).integers(1, 100, N).astype(np.float32)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    src = list(np.repeat(np.arange(N, dtype=np.int64), np.diff(wl.row_ptr.astype(np.int64))))
    dst = list(wl.col.astype(np.int64))
    costs = list(cost); wfs = list(wl.node_wf)
    rng = np.random.default_rng(42)
    assert W > 100 and N // 4 < 6000
    # 1. one append of 6,000 chain nodes, more than the reserve of this upload: the arrays move
    w = 0
    first = len(costs)
    k = 6000
    nc = rng.integers(1, 100, k).astype(np.float32)
    es = [int(np.flatnonzero(wl.node_wf == w)[0])] + list(range(first, first + k - 1))
    ed = list(range(first, first + k))
    gc.dag_append(nc, np.full(k, w, np.uint32), es, ed)
    costs += list(nc); wfs += [w] * k; src += es; dst += ed
    # 2. a hundred appends of one node each, round-robin over the workflows: more parts than are kept,
    #    so the forest is regrouped as one on the way
    for i in range(100):
        w = i % W
        v = len(costs)
        parent = int(rng.choice(np.flatnonzero(np.asarray(wfs) == w)))
        c = float(rng.integers(1, 100))
        gc.dag_append([c], [w], [parent], [v])
        costs.append(c); wfs.append(w); src.append(parent); dst.append(v)
    n = len(costs)
    row, col = _csr(n, src, dst)
    want = oracle.longest_path(row, col, np.asarray(costs, np.float32), np.asarray(wfs, np.uint32), W)
    cp, tail, H = gc.dag_results()
    assert cp.shape[0] == n
    assert np.array_equal(cp, want.cp) and np.array_equal(tail, want.tail) and np.array_equal(H, want.H)
    assert gc.status() == 0
    gc.close()


def test_rejected_appends_change_nothing(hx, oracle):
    wl = make_workload("tiny")
    gc = hh.gpu_cluster(wl)
    N = wl.n_nodes
    cost = np.random.default_rng(51).integers(1, 100, N).astype(np.float32)
    with pytest.raises(hx.HxError) as e:
        gc.dag_append([1.0], [0], [], [])
    assert e.value.code == -4
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    before = [a.copy() for a in gc.dag_results()]
    u = int(np.flatnonzero(np.diff(wl.row_ptr.astype(np.int64)) > 0)[0]); v = int(wl.col[wl.row_ptr[u]])
    other = int(np.flatnonzero(wl.node_wf != wl.node_wf[u])[0])
    bad = [
        (([1.0], [wl.n_workflows], [], []), -1),             # workflow out of range
        (([-1.0], [0], [], []), -1),                         # negative cost
        (([np.nan], [0], [], []), -1),
        (([], [], [u], [N]), -1),                            # endpoint out of range
        (([], [], [u], [other]), -1),                        # edge across workflows
        (([1.0], [int(wl.node_wf[other])], [u], [N]), -1),   # new node in another workflow than its parent
        (([], [], [v], [u]), -3),                            # closes a cycle with an uploaded edge
        (([1.0, 1.0], [0, 0], [N, N + 1], [N + 1, N]), -3),  # a cycle among the new nodes
    ]
    for args, code in bad:
        with pytest.raises(hx.HxError) as e:
            gc.dag_append(*args)
        assert e.value.code == code, args
        gc.n_nodes = N                                       # the binding counts only successful appends
        after = gc.dag_results()
        assert all(np.array_equal(x, y) for x, y in zip(before, after))
    gc.dag_append([], [], [], [])                            # nothing to do
    gc.critical_path()
    after = gc.dag_results()
    assert all(np.array_equal(x, y) for x, y in zip(before, after))
    gc.close()


@pytest.mark.parametrize("name, scale, base_frac, rounds", [("tiny", 1.0, 0.5, 3), ("medium", 1.0, 0.4, 5),
                                                            ("large", 1 / 16, 0.7, 4)])
def test_arriving_workflows_equal_a_fresh_upload(hx, oracle, name, scale, base_frac, rounds):
    """Workflows that arrive after the upload (Section 5.2, first trigger of the scheduling loop): only a share
    of the generated workflows is uploaded; the others arrive in rounds, each round registering its workflows,
    handing in their source calls and, interleaved, later calls of workflows that arrived earlier plus a few
    cost updates.  After every round cp, tail and H equal the oracle's pass over the forest as it stands."""
    wl = make_workload(name, scale=scale)
    rng = np.random.default_rng(41)
    N, W = wl.n_nodes, wl.n_workflows
    cost = rng.lognormal(0, 1, N).astype(np.float32)
    src = np.repeat(np.arange(N, dtype=np.int64), np.diff(wl.row_ptr.astype(np.int64)))
    dst = wl.col.astype(np.int64)
    # arrival round of every workflow (0 = uploaded); workflows are renumbered in arrival order
    w_round = np.where(rng.random(W) < base_frac, 0, rng.integers(1, rounds + 1, W))
    w_round[0] = 0
    w_order = np.argsort(w_round, kind="stable"); w_new = np.empty(W, np.int64); w_new[w_order] = np.arange(W)
    indeg = np.bincount(dst, minlength=N)
    # a node is revealed with its workflow if it is a source, else one or two rounds later
    n_round = w_round[wl.node_wf] + np.where(indeg == 0, 0, rng.integers(0, 3, N))
    n_round = np.minimum(n_round, rounds)
    n_round[(w_round[wl.node_wf] == 0) & (rng.random(N) < 0.5)] = 0
    n_order = np.argsort(n_round, kind="stable"); n_new = np.empty(N, np.int64); n_new[n_order] = np.arange(N)
    cost_r, wf_r = cost[n_order], w_new[wl.node_wf[n_order]].astype(np.uint32)
    s, d = n_new[src], n_new[dst]
    e_round = np.maximum(n_round[src], n_round[dst])
    n_at = [int(np.count_nonzero(n_round <= r)) for r in range(rounds + 1)]
    w_at = [int(np.count_nonzero(w_round <= r)) for r in range(rounds + 1)]
    elapsed = rng.uniform(0, 2, W).astype(np.float32)

    def want(r, c):
        m = e_round <= r
        row, col = _csr(n_at[r], s[m], d[m])
        return oracle.longest_path(row, col, c[:n_at[r]], wf_r[:n_at[r]], w_at[r]), row, col

    gc = hh.gpu_cluster(wl)
    m0 = e_round == 0
    row, col = _csr(n_at[0], s[m0], d[m0])
    gc.dag_upload(row, col, cost_r[:n_at[0]], wf_r[:n_at[0]], elapsed[:w_at[0]])
    gc.critical_path()
    cost_now = cost_r.copy()
    for r in range(1, rounds + 1):
        gc.dag_append_workflows(elapsed[w_at[r - 1]:w_at[r]])
        cp, tail, H = gc.dag_results()
        assert H.shape[0] == w_at[r] and np.all(H[w_at[r - 1]:] == 0)         # arrived, nothing revealed yet
        m = e_round == r
        gc.dag_append(cost_now[n_at[r - 1]:n_at[r]], wf_r[n_at[r - 1]:n_at[r]], s[m], d[m])
        ids = rng.integers(0, n_at[r], max(1, n_at[r] // 100)).astype(np.uint32)
        new = (cost_now[ids] * 1.25).astype(np.float32)
        gc.update_costs(ids, new)
        for i, v in zip(ids, new):
            cost_now[i] = v
        w, row, col = want(r, cost_now)
        cp, tail, H = gc.dag_results()
        assert np.array_equal(cp, w.cp) and np.array_equal(tail, w.tail) and np.array_equal(H, w.H), "round %d" % r
    # the grown forest behaves like an uploaded one: elapsed times of the grown count, forward pass, full pass, scoring
    gc.update_elapsed(elapsed[:w_at[rounds]])
    gc.earliest_start()
    est, eft = gc.earliest_results()
    w_est, w_eft = oracle.earliest_start(row, col, cost_now)
    assert np.array_equal(est, w_est) and np.array_equal(eft, w_eft)
    gc.critical_path()
    cp, tail, H = gc.dag_results()
    assert np.array_equal(cp, w.cp) and np.array_equal(H, w.H)
    oc = hh.oracle_cluster(wl)
    calls = wl.node_calls[n_order][-min(N, 300):].copy()
    calls["node"] = np.arange(N - len(calls), N)
    gc.set_options(score_mode=hx.HX_MODE_RATIO)
    a, c = gc.schedule_batch(calls)
    oa, ocst, _ = oracle.schedule(oc, calls, mode=ho.MODE_RATIO, dag=w, node_wf=wf_r, elapsed=elapsed[:w_at[rounds]])
    assert np.array_equal(a.cpu().numpy(), oa) and np.array_equal(c.cpu().numpy(), ocst)
    assert gc.status() == 0
    gc.close()


def test_arriving_workflows_beyond_the_reserve_and_bad_arguments(hx, oracle):
    wl = make_workload("tiny")
    gc = hh.gpu_cluster(wl)
    with pytest.raises(hx.HxError) as e:
        gc.dag_append_workflows([0.0])
    assert e.value.code == -4                                 # nothing uploaded yet
    cost = np.ones(wl.n_nodes, np.float32)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    with pytest.raises(hx.HxError):
        gc.dag_append_workflows([-1.0])
    with pytest.raises(hx.HxError):                           # a node of a workflow that has not arrived
        gc.dag_append([1.0], [wl.n_workflows], [], [])
    W0, N0 = wl.n_workflows, wl.n_nodes
    k = 6000                                                  # more than the reserve of 4,096: the arrays move
    gc.dag_append_workflows(np.zeros(k, np.float32))
    new_cost = np.arange(1, k + 1, dtype=np.float32)
    gc.dag_append(new_cost, np.arange(W0, W0 + k, dtype=np.uint32), [], [])
    cp, tail, H = gc.dag_results()
    base = oracle.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, W0)
    assert np.array_equal(H[:W0], base.H) and np.array_equal(H[W0:], new_cost) and np.array_equal(cp[N0:], new_cost)
    assert gc.status() == 0
    gc.close()
