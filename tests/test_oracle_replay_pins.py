"""Pins of the oracle's event-driven replay (oracle/hx_replay.py).  The paper gives no worked example of its
simulator; these pin the replay to what its definition and the paper's metric fix: a workflow alone on the
cluster reproduces its stand-alone horizon (that is how Section 7.3 defines H_w), a two-call hand case with a
closed form built from the pinned service times, causality and capacity invariants, and Req95 / Req99 on a
known list."""
import numpy as np
import pytest

from oracle import hx_oracle as ho
from oracle import hx_replay as hr
from hx_synth import CALL_DTYPE


@pytest.fixture(scope="module")
def oracle():
    return ho.Oracle()


def _cluster(rng, P, D, G=3, M=2, cap=1e6):
    types = np.stack([rng.uniform(50, 2000, G), rng.uniform(0.3, 8, G)], 1)
    models = np.stack([rng.uniform(1e9, 2e11, M), rng.uniform(1e9, 2e11, M),
                       rng.choice([65536.0, 131072.0, 327680.0], M)], 1)
    return ho.Cluster(types, rng.integers(0, G, P), rng.integers(0, G, D), np.zeros(P), np.zeros(D),
                      np.full(D, cap), rng.uniform(25, 400, (P, D)), models)


def _calls(rng, C, M=2):
    a = np.zeros(C, dtype=CALL_DTYPE)
    a["node"] = np.arange(C)
    a["model"] = rng.integers(0, M, C)
    a["prompt_tokens"] = np.clip(np.round(rng.lognormal(7, 1, C)), 1, 32768)
    a["output_tokens"] = np.clip(np.round(rng.lognormal(5, 1, C)), 1, 32768)
    return a


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


def _standalone(oracle, cl, calls, row, col, node_wf, W):
    cost = oracle.schedule(cl, calls, flags=ho.FLAG_UNLOADED | ho.FLAG_NO_DAG)[2]
    return cost, oracle.longest_path(row, col, cost, node_wf, W)


def test_req_is_the_order_statistic_of_the_definition():
    r = np.arange(1, 101, dtype=np.float64)[::-1].copy()
    assert hr.req(r, 0.95) == 95 and hr.req(r, 0.99) == 99 and hr.req(r, 1.0) == 100
    r20 = np.arange(1, 21, dtype=np.float64)
    assert hr.req(r20, 0.95) == 19 and hr.req(r20, 0.99) == 20      # 19 of 20 = 95 %; 99 % needs all 20
    for q in (0.5, 0.9, 0.95, 0.99):
        a = hr.req(r20, q)
        assert np.mean(r20 <= a) >= q and np.mean(r20 <= np.nextafter(a, 0)) < q


def test_a_chain_alone_reproduces_its_horizon(oracle):
    rng = np.random.default_rng(61)
    for trial in range(5):
        cl = _cluster(rng, 3, 4)
        n = int(rng.integers(1, 12))
        calls = _calls(rng, n)
        row, col = _csr(n, [(i, i + 1) for i in range(n - 1)])
        nwf = np.zeros(n, np.uint32)
        cost, dag = _standalone(oracle, cl, calls, row, col, nwf, 1)
        out = hr.replay(oracle, cl, row, col, nwf, 1, calls, [3.25], dag)
        assert out["stuck"] == 0 and out["runs"] == n
        # every call starts when its predecessor completes and runs at its stand-alone best
        want = 3.25 + np.cumsum(cost.astype(np.float64))
        np.testing.assert_allclose(out["fin"], want, rtol=1e-12)
        np.testing.assert_allclose(out["ratio"], [1.0], rtol=1e-5)
        assert out["req95"] == out["req99"] == out["ratio"][0]


def test_any_workflow_alone_is_never_faster_than_its_horizon(oracle):
    rng = np.random.default_rng(62)
    for trial in range(10):
        cl = _cluster(rng, 2, 2)
        n = int(rng.integers(2, 14))
        edges = [(u, v) for u in range(n) for v in range(u + 1, n) if rng.random() < 0.3]
        calls = _calls(rng, n)
        row, col = _csr(n, edges)
        nwf = np.zeros(n, np.uint32)
        cost, dag = _standalone(oracle, cl, calls, row, col, nwf, 1)
        out = hr.replay(oracle, cl, row, col, nwf, 1, calls, [0.0], dag)
        assert out["stuck"] == 0 and out["ratio"][0] >= 1 - 1e-6
        # a call is planned when its last predecessor completes, and completes no sooner than its best case allows
        for v in range(n):
            pred = [u for u, x in edges if x == v]
            assert out["planned"][v] == (max(out["fin"][u] for u in pred) if pred else 0.0)
            assert out["fin"][v] >= out["planned"][v] + cost[v] * (1 - 1e-6)


def test_two_calls_on_one_pair_closed_form(oracle):
    # one prefill and one decode instance, two single-call workflows arriving together: the more urgent call
    # (larger stand-alone ratio = both 1, so the lower index) goes first, the other queues behind its prefill
    rng = np.random.default_rng(63)
    cl = _cluster(rng, 1, 1, G=1, M=1)
    calls = _calls(rng, 2, M=1)
    row, col = _csr(2, [])
    nwf = np.array([0, 1], np.uint32)
    cost, dag = _standalone(oracle, cl, calls, row, col, nwf, 2)
    out = hr.replay(oracle, cl, row, col, nwf, 2, calls, [1.0, 1.0], dag)
    tpre, tdec, kvB, m = oracle.terms(cl, calls)
    xfer = kvB.astype(np.float64) / (float(cl.link[0, 0]) * 1e9)
    first, second = (0, 1) if out["fin"][0] - cost[0] <= 1.0 + 1e-9 else (1, 0)
    assert first == 0                                            # equal ratios: lower index first
    np.testing.assert_allclose(out["fin"][0], 1.0 + tpre[0, 0] + xfer[0] + tdec[0, 0], rtol=1e-6)
    np.testing.assert_allclose(out["fin"][1], 1.0 + tpre[0, 0] + tpre[1, 0] + xfer[1] + tdec[1, 0], rtol=1e-6)
    np.testing.assert_allclose(out["ratio"][1], (out["fin"][1] - 1.0) / cost[1], rtol=1e-6)
    # far apart they do not meet: both run at their horizon
    far = hr.replay(oracle, cl, row, col, nwf, 2, calls, [1.0, 1000.0], dag)
    np.testing.assert_allclose(far["ratio"], [1.0, 1.0], rtol=1e-5)


def test_invariants_on_a_loaded_trace(oracle):
    rng = np.random.default_rng(64)
    cl = _cluster(rng, 2, 3, cap=40000.0)                        # tight KV room: calls get passed over and wait
    W, per = 30, 5
    N = W * per
    calls = _calls(rng, N)
    calls["prompt_tokens"] = np.minimum(calls["prompt_tokens"], 8000)
    calls["output_tokens"] = np.minimum(calls["output_tokens"], 2000)
    edges = []
    for w in range(W):
        b = w * per
        edges += [(b, b + 1), (b, b + 2), (b + 1, b + 3), (b + 2, b + 3), (b + 3, b + 4)]
    row, col = _csr(N, edges)
    nwf = np.repeat(np.arange(W), per).astype(np.uint32)
    cost, dag = _standalone(oracle, cl, calls, row, col, nwf, W)
    arrival = np.sort(rng.uniform(0, 0.5 * float(dag.H.sum()) / 4, W))
    out = hr.replay(oracle, cl, row, col, nwf, W, calls, arrival, dag, qmax=16)
    assert out["stuck"] == 0 and np.all(np.isfinite(out["fin"]))
    fin, planned, pair = out["fin"], out["planned"], out["pair"]
    for u, v in edges:
        assert planned[v] >= fin[u]                              # precedence
    assert np.all(planned >= arrival[nwf])
    assert np.all(fin >= planned + cost.astype(np.float64) * (1 - 1e-6))
    assert np.all(out["ratio"] >= 1 - 1e-6) and out["ratio"].max() > 1.05      # the load is felt
    assert out["req99"] >= out["req95"] >= out["ratio"].min()
    # KV tokens held on a decode instance never exceed its capacity (Eq. 4 over time)
    m = calls["prompt_tokens"].astype(np.float64) + calls["output_tokens"]
    d = pair % cl.D
    for t in np.unique(planned):
        live = (planned <= t) & (fin > t)
        used = np.bincount(d[live], weights=m[live], minlength=cl.D)
        assert np.all(used <= cl.capD + 0.5)
    # the chunk size of the planner runs changes who is planned with whom, not the validity of the outcome
    again = hr.replay(oracle, cl, row, col, nwf, W, calls, arrival, dag, qmax=4096)
    assert again["stuck"] == 0 and again["runs"] <= out["runs"]


# ---------------------------------------------------------------------------
# replay with separate stages, a scheduled decode stage and estimation error
# ---------------------------------------------------------------------------

def _service(oracle, cl, calls):
    tpre, tdec, kvB, m = oracle.terms(cl, calls)
    inv = np.float32(1.0) / (cl.link.astype(np.float32) * np.float32(1e9))
    return tpre.astype(np.float64), tdec.astype(np.float64), kvB, inv, m.astype(np.float64)


def test_lifecycle_chain_alone_reproduces_its_horizon_whatever_the_error(oracle):
    """One prefill and one decode instance leave the schedulers nothing to decide, so a chain alone completes at
    arrival + the sum of (prefill + transfer + decode) of its calls, i.e. at its stand-alone horizon, for every
    error level: the error changes what the scheduler sees, never the service a call gets (Section 7.6)."""
    rng = np.random.default_rng(71)
    for trial in range(4):
        cl = _cluster(rng, 1, 1, G=2, M=2)
        n = int(rng.integers(1, 9))
        calls = _calls(rng, n)
        row, col = _csr(n, [(i, i + 1) for i in range(n - 1)])
        nwf = np.zeros(n, np.uint32)
        cost, dag = _standalone(oracle, cl, calls, row, col, nwf, 1)
        tpre, tdec, kvB, inv, m = _service(oracle, cl, calls)
        g_p, g_d = cl.typeP[0], cl.typeD[0]
        step = tpre[:, g_p] + (kvB * inv[0, 0]).astype(np.float64) + tdec[:, g_d]
        for eps in (0.0, 0.1, 0.3):
            out = hr.replay_lifecycle(oracle, cl, row, col, nwf, 1, calls, [2.5], dag, est_error=eps)
            assert out["stuck"] == 0 and out["runs"] == n and out["decode_runs"] == n
            np.testing.assert_allclose(out["fin"], 2.5 + np.cumsum(step), rtol=1e-12)
            np.testing.assert_allclose(out["ratio"], [1.0], rtol=2e-6)     # binary32 horizon vs binary64 clock


def test_lifecycle_without_error_an_idle_cluster_gives_ratio_one(oracle):
    """With exact estimates the planner sends a call that finds the cluster idle to its stand-alone best pair."""
    rng = np.random.default_rng(72)
    cl = _cluster(rng, 3, 4)
    calls = _calls(rng, 6)
    row, col = _csr(6, [(i, i + 1) for i in range(5)])
    nwf = np.zeros(6, np.uint32)
    cost, dag = _standalone(oracle, cl, calls, row, col, nwf, 1)
    out = hr.replay_lifecycle(oracle, cl, row, col, nwf, 1, calls, [0.0], dag)
    np.testing.assert_allclose(out["fin"], np.cumsum(cost.astype(np.float64)), rtol=2e-6)
    np.testing.assert_allclose(out["ratio"], [1.0], rtol=2e-6)
    wrong = hr.replay_lifecycle(oracle, cl, row, col, nwf, 1, calls, [0.0], dag, est_error=0.3)
    assert wrong["ratio"][0] >= 1 - 2e-6                       # a misled choice can only be slower


def test_lifecycle_two_calls_the_error_flips_the_order(oracle):
    """Two single-call workflows arrive together on one prefill and one decode instance.  Their horizons are
    chosen so that call 0 is slightly more urgent when the estimates are exact (ratio 1.000 against 0.999)
    and call 1 is when they are off by 20 % in opposite directions; whoever goes first keeps the prefill
    instance busy for its prefill time, the decode instance holds both."""
    assert hr.error_sign(0) != hr.error_sign(1)
    rng = np.random.default_rng(73)
    cl = _cluster(rng, 1, 1, G=1, M=1)
    calls = _calls(rng, 2, M=1)
    row, col = _csr(2, [])
    nwf = np.array([0, 1], np.uint32)
    cost, dag = _standalone(oracle, cl, calls, row, col, nwf, 2)
    dag.H[:] = cost * np.array([1.0, 1.001], np.float32)
    tpre, tdec, kvB, inv, m = _service(oracle, cl, calls)
    serve = tpre[:, 0] + (kvB * inv[0, 0]).astype(np.float64) + tdec[:, 0]
    exact = hr.replay_lifecycle(oracle, cl, row, col, nwf, 2, calls, [1.0, 1.0], dag)
    np.testing.assert_allclose(exact["fin"], [1.0 + serve[0], 1.0 + tpre[0, 0] + serve[1]], rtol=1e-12)
    assert exact["prefill_start"][0] == 1.0 and exact["prefill_start"][1] == 1.0 + tpre[0, 0]
    eps = 0.2
    up = 0 if hr.error_sign(0) > 0 else 1                      # the call whose estimates are too long looks more urgent
    off = hr.replay_lifecycle(oracle, cl, row, col, nwf, 2, calls, [1.0, 1.0], dag, est_error=eps)
    first, second = up, 1 - up
    np.testing.assert_allclose(off["fin"][first], 1.0 + serve[first], rtol=1e-12)
    np.testing.assert_allclose(off["fin"][second], 1.0 + tpre[first, 0] + serve[second], rtol=1e-12)
    if up == 1:
        assert off["prefill_start"][1] < off["prefill_start"][0]      # the order really flipped


def test_lifecycle_decode_stage_admits_in_the_order_of_the_decode_plan(oracle):
    """A decode instance with room for one call at a time and three single-call workflows whose KV caches arrive
    while it is busy: when it frees up, the waiting call with the larger projected ratio (Eq. 2; the horizons are
    set so that this is the call with the higher number) is admitted first."""
    rng = np.random.default_rng(74)
    cl = _cluster(rng, 3, 1, G=1, M=1, cap=3000.0)
    calls = _calls(rng, 3, M=1)
    calls["prompt_tokens"] = [1500, 1400, 1300]; calls["output_tokens"] = [300, 300, 300]
    row, col = _csr(3, [])
    nwf = np.arange(3, dtype=np.uint32)
    cost, dag = _standalone(oracle, cl, calls, row, col, nwf, 3)
    dag.H[:] = cost * np.array([1.0, 4.0, 1.0], np.float32)    # workflow 1 has the most slack
    out = hr.replay_lifecycle(oracle, cl, row, col, nwf, 3, calls, [0.0, 0.0, 0.0], dag)
    assert out["stuck"] == 0 and np.all(np.isfinite(out["fin"]))
    ds = out["decode_start"]
    order = np.argsort(ds)
    assert order[0] == 0 or ds[order[0]] < ds[order[1]]
    # the planner reserves the tokens at planning time, so the three prefills are planned one after the other as
    # room is released; decodes never overlap on this instance
    for a in range(3):
        for b in range(3):
            if a != b:
                assert ds[a] >= out["fin"][b] or ds[b] >= out["fin"][a]


def test_lifecycle_invariants_on_a_loaded_trace(oracle):
    rng = np.random.default_rng(75)
    cl = _cluster(rng, 2, 3, cap=40000.0)
    W, per = 30, 5
    N = W * per
    calls = _calls(rng, N)
    calls["prompt_tokens"] = np.minimum(calls["prompt_tokens"], 8000)
    calls["output_tokens"] = np.minimum(calls["output_tokens"], 2000)
    edges = []
    for w in range(W):
        b = w * per
        edges += [(b, b + 1), (b, b + 2), (b + 1, b + 3), (b + 2, b + 3), (b + 3, b + 4)]
    row, col = _csr(N, edges)
    nwf = np.repeat(np.arange(W), per).astype(np.uint32)
    cost, dag = _standalone(oracle, cl, calls, row, col, nwf, W)
    arrival = np.sort(rng.uniform(0, 0.5 * float(dag.H.sum()) / 4, W))
    tpre, tdec, kvB, inv, m = _service(oracle, cl, calls)
    for eps in (0.0, 0.3):
        out = hr.replay_lifecycle(oracle, cl, row, col, nwf, W, calls, arrival, dag, est_error=eps, qmax=16)
        assert out["stuck"] == 0 and np.all(np.isfinite(out["fin"]))
        fin, pair, ps, ds, planned = out["fin"], out["pair"], out["prefill_start"], out["decode_start"], out["planned"]
        p, d = pair // cl.D, pair % cl.D
        for u, v in edges:
            assert planned[v] >= fin[u]                          # precedence
        assert np.all(planned >= arrival[nwf]) and np.all(ps >= planned)
        # the stages follow one another with the real service times
        pend = ps + tpre[np.arange(N), cl.typeP[p]]
        tend = pend + (kvB * inv[p, d]).astype(np.float64)
        assert np.all(ds >= tend - 1e-12)
        np.testing.assert_allclose(fin, ds + tdec[np.arange(N), cl.typeD[d]], rtol=1e-12)
        for q in range(cl.P):                                   # a prefill instance serves one call at a time
            mine = np.flatnonzero(p == q)
            o = mine[np.argsort(ps[mine])]
            assert np.all(ps[o[1:]] >= pend[o[:-1]] - 1e-12)
        for t in np.unique(ds):                                 # Eq. 4 over time, on the tokens really held
            live = (ds <= t) & (fin > t)
            assert np.all(np.bincount(d[live], weights=m[live], minlength=cl.D) <= cl.capD + 0.5)
        assert np.all(out["ratio"] >= 1 - 2e-6) and out["req99"] >= out["req95"]
    assert out["ratio"].max() > 1.05
