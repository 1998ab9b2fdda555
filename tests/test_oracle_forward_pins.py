"""Pins of the oracle's forward pass (earliest start / finish of every node).

None of these re-types the recurrence: they enumerate paths, use closed forms of
special graphs, a library shortest-path routine, and the identity that ties the
forward pass to the horizon."""
import numpy as np
import pytest

from oracle import hx_oracle as ho
from hx_synth import make_workload


@pytest.fixture(scope="module")
def oracle():
    return ho.Oracle()


def _csr(n, edges):
    row = np.zeros(n + 1, np.uint32)
    for u, _ in edges:
        row[u + 1] += 1
    row = np.cumsum(row, dtype=np.uint32)
    col = np.zeros(len(edges), np.uint32)
    cur = row[:-1].copy()
    for u, v in sorted(edges):
        col[cur[u]] = v
        cur[u] += 1
    return row, col


def _sums_of_paths_into(pred, cost, v):
    """Cost of every path that ends just before v (v's own cost excluded), summed from the source on."""
    if not pred[v]:
        return [0.0]
    return [s + cost[u] for u in pred[v] for s in _sums_of_paths_into(pred, cost, u)]


def test_earliest_start_vs_path_enumeration(oracle):
    rng = np.random.default_rng(13)
    for trial in range(30):
        n = int(rng.integers(1, 15))
        edges = [(u, v) for u in range(n) for v in range(u + 1, n) if rng.random() < 0.3]
        perm = rng.permutation(n)                 # node numbers are not a topological order
        edges = [(int(perm[u]), int(perm[v])) for u, v in edges]
        cost = rng.integers(1, 50, n).astype(np.float32)     # integers: every sum is exact
        row, col = _csr(n, edges)
        pred = [[] for _ in range(n)]
        for u, v in edges:
            pred[v].append(u)
        est, eft = oracle.earliest_start(row, col, cost)
        for v in range(n):
            assert est[v] == max(_sums_of_paths_into(pred, cost, v))
            assert eft[v] == est[v] + cost[v]


def test_chain_is_a_prefix_sum(oracle):
    rng = np.random.default_rng(14)
    n = 300
    cost = rng.lognormal(0, 1, n).astype(np.float32)
    row = np.arange(n + 1, dtype=np.uint32); row[-1] = n - 1
    col = np.arange(1, n, dtype=np.uint32)
    est, eft = oracle.earliest_start(row, col, cost)
    prefix = np.cumsum(cost, dtype=np.float32)               # sequential binary32 sums from the source
    assert np.array_equal(eft, prefix)
    assert est[0] == 0 and np.array_equal(est[1:], prefix[:-1])


def test_fan_out_and_join(oracle):
    # source 0 -> branches 1..4 -> join 5: the join waits for the slowest branch
    cost = np.array([2, 7, 3, 11, 5, 1], np.float32)
    row, col = _csr(6, [(0, b) for b in range(1, 5)] + [(b, 5) for b in range(1, 5)])
    est, eft = oracle.earliest_start(row, col, cost)
    assert list(est) == [0, 2, 2, 2, 2, 13] and list(eft) == [2, 9, 5, 13, 7, 14]


def test_forward_and_backward_passes_meet_at_the_horizon(oracle):
    # est[v] + cp[v] is the longest path through v: never above H, equal to H on a critical path,
    # and the largest eft of a workflow is H itself.  Integer costs keep every sum exact.
    wl = make_workload("medium", scale=0.1)
    N = wl.n_nodes
    cost = np.random.default_rng(15).integers(1, 1000, N).astype(np.float32)
    r = oracle.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
    est, eft = oracle.earliest_start(wl.row_ptr, wl.col, cost)
    through = est + r.cp
    assert np.all(through <= r.H[wl.node_wf])
    best = np.zeros(wl.n_workflows, np.float32); np.maximum.at(best, wl.node_wf, through)
    assert np.array_equal(best, r.H)
    last = np.zeros(wl.n_workflows, np.float32); np.maximum.at(last, wl.node_wf, eft)
    assert np.array_equal(last, r.H)
    # a source starts at 0, everything else after its predecessors
    indeg = np.bincount(wl.col, minlength=N)
    assert np.all(est[indeg == 0] == 0) and np.all(est[indeg > 0] > 0)


def test_earliest_start_vs_library_shortest_path(oracle):
    sp = pytest.importorskip("scipy.sparse")
    from scipy.sparse.csgraph import bellman_ford
    wl = make_workload("medium", scale=0.1)
    N = wl.n_nodes
    cost = np.random.default_rng(16).lognormal(0, 1, N).astype(np.float32)
    est, eft = oracle.earliest_start(wl.row_ptr, wl.col, cost)
    # earliest start of v = -(shortest distance to v from any node) when edge u -> v weighs -cost[u]
    src = np.repeat(np.arange(N), np.diff(wl.row_ptr.astype(np.int64)))
    g = sp.csr_matrix((-cost[src].astype(np.float64), (src, wl.col.astype(np.int64))), shape=(N, N))
    some = np.random.default_rng(2).choice(N, 40, replace=False)
    dist = bellman_ford(g.T.tocsr(), directed=True, indices=some)    # reversed graph: distances INTO `some`
    np.testing.assert_allclose(est[some], -dist.min(axis=1), rtol=1e-5, atol=1e-6)


def test_cycle_is_rejected(oracle):
    row, col = _csr(3, [(0, 1), (1, 2), (2, 0)])
    with pytest.raises(ValueError):
        oracle.earliest_start(row, col, np.ones(3, np.float32))
