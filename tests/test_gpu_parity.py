"""GPU-vs-oracle parity through the C ABI binding.

Bars (stated once in hx_helpers): binary32 costs within 1e-5 relative of the oracle,
placements identical unless the oracle's own cost gap is below that tolerance,
horizons bit-exact, integer outputs of the capacity pass bit-exact.  The kernels
are designed to reproduce the oracle's binary32 sequence exactly, so most checks
also demand identical bits; where they do it is an additional, stricter assertion.
"""
import numpy as np
import pytest

import hx_helpers as hh
from hx_synth import CALL_DTYPE, make_workload, sub_forest
from oracle import hx_oracle as ho

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hx():
    import __graft_entry__ as entry
    entry.build()
    import paper_2605_16637_b200 as mod
    return mod


def _cluster_pair(hx, P, D, G=4, M=2, seed=0, tight=False, qd_round=False):
    rng = np.random.default_rng(seed)
    types = np.stack([rng.uniform(50, 2000, G), rng.uniform(0.3, 8, G)], 1).astype(np.float32)
    models = np.stack([rng.uniform(1e9, 2e11, M), rng.uniform(1e9, 2e11, M),
                       rng.choice([65536.0, 131072.0, 327680.0], M)], 1).astype(np.float32)
    inst = np.zeros(P + D, hx.INSTANCE_DTYPE)
    inst["type"] = rng.integers(0, G, P + D)
    inst["role"][P:] = 1
    inst["load_s"] = rng.uniform(0, 2, P + D)
    if qd_round:
        inst["load_s"] = np.round(inst["load_s"] * 2) / 2
    cap = rng.choice([600.0, 3000.0, 1e6], P + D) if tight else np.full(P + D, 1e6)
    inst["kv_cap_tokens"] = cap
    inst["kv_free_tokens"] = cap
    link = rng.uniform(25, 400, (P + D, P + D)).astype(np.float32)
    gc = hx.Cluster(types, inst, link, models)
    oc = ho.Cluster(types, inst["type"][:P], inst["type"][P:], inst["load_s"][:P], inst["load_s"][P:],
                    inst["kv_cap_tokens"][P:], link[:P, P:], models)
    return gc, oc


def _calls(n, M=2, seed=1, lo_mu=7.0):
    rng = np.random.default_rng(seed)
    a = np.zeros(n, CALL_DTYPE)
    a["node"] = np.arange(n)
    a["model"] = rng.integers(0, M, n)
    a["prompt_tokens"] = np.clip(np.round(rng.lognormal(lo_mu, 1, n)), 1, 32768)
    a["output_tokens"] = np.clip(np.round(rng.lognormal(5, 1, n)), 1, 32768)
    return a


def _prepare(hx, oracle, wl):
    """Cluster on both sides, stand-alone node costs, horizons; returns everything needed to score."""
    oc, gc = hh.oracle_cluster(wl), hh.gpu_cluster(wl)
    if wl.node_cost is not None:
        cost_o = cost_g = wl.node_cost
    else:
        cost_o = hh.oracle_node_costs(oracle, oc, wl.node_calls)
        cost_g = hh.gpu_node_costs(gc, wl.node_calls)
        hh.assert_costs_close(cost_g, cost_o, "stand-alone node costs")
        assert np.array_equal(cost_g, cost_o)
    dag = oracle.longest_path(wl.row_ptr, wl.col, cost_o, wl.node_wf, wl.n_workflows)
    gc.dag_upload(wl.row_ptr, wl.col, cost_g, wl.node_wf, wl.elapsed)
    gc.critical_path()
    return oc, gc, dag


CONFIGS = [("tiny", 1.0), ("medium", 1.0), ("large", 1 / 16), ("cp_stress", 1 / 20), ("sweep", 1 / 64)]


@pytest.mark.parametrize("name, scale", CONFIGS)
def test_horizons_bit_exact(hx, oracle, name, scale):
    wl = make_workload(name, scale=scale)
    oc, gc, dag = _prepare(hx, oracle, wl)
    cp, tail, H = gc.dag_results()
    assert np.array_equal(cp, dag.cp) and np.array_equal(tail, dag.tail) and np.array_equal(H, dag.H)
    gc.close()


@pytest.mark.parametrize("name, scale", CONFIGS)
def test_scoring_all_modes(hx, oracle, name, scale):
    wl = make_workload(name, scale=scale)
    oc, gc, dag = _prepare(hx, oracle, wl)
    calls = wl.calls
    kw = dict(dag=dag, node_wf=wl.node_wf, elapsed=wl.elapsed, alpha=wl.alpha)
    for mode, flags in [(0, 0), (1, 0), (2, 0), (2, hx.HX_FLAG_NO_TAIL), (0, hx.HX_FLAG_UNLOADED)]:
        gc.set_options(score_mode=mode, flags=flags, alpha=wl.alpha)
        a, c = gc.schedule_batch(calls)
        a, c = a.cpu().numpy(), c.cpu().numpy()
        oa, ocost, _ = oracle.schedule(oc, calls, mode=mode, flags=flags, **kw)
        hh.assert_costs_close(c, ocost, "%s mode %d flags %d" % (name, mode, flags))
        hh.assert_assign_matches(oracle, oc, calls, a, oa, flags=flags & hx.HX_FLAG_UNLOADED, what=name)
        assert np.array_equal(c, ocost) and np.array_equal(a, oa)       # identical bits by construction
    assert gc.status() == 0
    gc.close()


SHAPES = [(1, 1, 5), (2, 3, 17), (5, 3, 64), (4, 9, 100), (17, 16, 333), (33, 70, 500), (130, 129, 300),
          (128, 200, 257), (40, 512, 130), (600, 64, 200), (1024, 128, 150)]


@pytest.mark.parametrize("P, D, n", SHAPES)
def test_scoring_ragged_shapes(hx, oracle, P, D, n):
    """Pool sizes that are not multiples of the tiles, several warps along d, chunked prefill dimension."""
    gc, oc = _cluster_pair(hx, P, D, seed=P * 1000 + D, tight=True)
    calls = _calls(n, seed=n)
    gc.set_options(flags=hx.HX_FLAG_NO_DAG)
    a, c = gc.schedule_batch(calls)
    oa, ocost, _ = oracle.schedule(oc, calls)
    assert np.array_equal(a.cpu().numpy(), oa) and np.array_equal(c.cpu().numpy(), ocost)
    K = min(4, D)
    gc.set_options(topk=K, flags=hx.HX_FLAG_NO_DAG)
    gc.schedule_batch(calls)
    pair, cost, prio = gc.topk_results(n)
    op, ocs, opr, _, _ = oracle.topk(oc, calls, K)
    assert np.array_equal(pair, op) and np.array_equal(cost, ocs) and np.array_equal(prio, opr)
    gc.close()


@pytest.mark.parametrize("D, LD", [(5, 1), (12, 2), (24, 4)])
@pytest.mark.parametrize("TC", [1, 2, 4, 8])
def test_scoring_thread_tile_heights_of_narrow_pools(hx, oracle, D, LD, TC):
    """For decode pools of at most 32 instances the kernel keeps eight warps per block and picks the thread
    tile height (1, 2, 4 or 8 calls) from the batch size: a batch of 148 tiles of that height selects it on
    a 148-SM device.  Every height of every lane layout is compared with the oracle, plain argmin and top-2."""
    import torch
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    rows = 8 * (32 // LD)                        # calls per block and unit of tile height
    n = n_sm * rows * TC - 3                     # ragged last tile
    P = 3
    gc, oc = _cluster_pair(hx, P, D, seed=D * 10 + TC, tight=True)
    calls = _calls(n, seed=n % 1000)
    gc.set_options(flags=hx.HX_FLAG_NO_DAG)
    a, c = gc.schedule_batch(calls)
    oa, ocost, _ = oracle.schedule(oc, calls)
    assert np.array_equal(a.cpu().numpy(), oa) and np.array_equal(c.cpu().numpy(), ocost)
    m = min(n, 16000)                            # the capacity pass takes at most 65,536 calls
    gc.set_options(topk=2, flags=hx.HX_FLAG_NO_DAG)
    gc.schedule_batch(calls[:m])
    pair, cost, prio = gc.topk_results(m)
    op, ocs, opr, _, _ = oracle.topk(oc, calls[:m], 2)
    assert np.array_equal(pair, op) and np.array_equal(cost, ocs) and np.array_equal(prio, opr)
    gc.close()


def test_exact_ties_and_infeasible_calls(hx, oracle):
    # identical instances, late decode admission: every pair of a decode type ties exactly
    P, D = 6, 5
    inst = np.zeros(P + D, hx.INSTANCE_DTYPE)
    inst["role"][P:] = 1
    inst["load_s"][:P] = [0.1, 0.0, 0.2, 0.0, 0.3, 0.05]
    inst["load_s"][P:] = 9.0
    inst["kv_cap_tokens"] = [0] * P + [1e6, 1e6, 500, 1e6, 1e6]
    inst["kv_free_tokens"] = inst["kv_cap_tokens"]
    types = np.array([[1000.0, 1.0]], np.float32)
    models = np.array([[2e9, 1e9, 1e5]], np.float32)
    link = np.full((P + D, P + D), 100.0, np.float32)
    gc = hx.Cluster(types, inst, link, models)
    oc = ho.Cluster(types, inst["type"][:P], inst["type"][P:], inst["load_s"][:P], inst["load_s"][P:],
                    inst["kv_cap_tokens"][P:], link[:P, P:], models)
    calls = np.zeros(4, CALL_DTYPE)
    calls["prompt_tokens"] = [1000, 200, 3e6, 100]       # the third call fits nowhere
    calls["output_tokens"] = [11, 50, 10, 100]
    gc.set_options(flags=hx.HX_FLAG_NO_DAG)
    a, c = gc.schedule_batch(calls)
    a, c = a.cpu().numpy(), c.cpu().numpy()
    oa, ocost, _ = oracle.schedule(oc, calls)
    assert list(a) == list(oa) == [0, 0, -1, 0]
    assert np.array_equal(c, ocost) and np.isinf(c[2])
    gc.set_options(topk=4, flags=hx.HX_FLAG_NO_DAG)
    a2, _ = gc.schedule_batch(calls)
    pair, cost, prio = gc.topk_results(4)
    op, ocs, opr, om, ots = oracle.topk(oc, calls, 4)
    assert np.array_equal(pair, op) and np.array_equal(cost, ocs) and np.array_equal(prio, opr)
    assert list(pair[0]) == [0, 1, 3, 4]                 # d = 2 is too small for call 0; ties ordered by d
    assert list(pair[2]) == [-1] * 4
    gc.close()


def test_single_call_single_pair_closed_form(hx):
    """P = D = 1, one call: the hand-computed finish of the golden 'hand' case (0.2651055 s)."""
    inst = np.zeros(2, hx.INSTANCE_DTYPE)
    inst["role"][1] = 1
    inst["load_s"] = [0.25, 0.1]
    inst["kv_cap_tokens"] = inst["kv_free_tokens"] = 1e6
    gc = hx.Cluster(np.array([[1000.0, 1.0]]), inst, np.full((2, 2), 100.0), np.array([[2e9, 1e9, 1e5]]))
    calls = np.zeros(1, CALL_DTYPE)
    calls["prompt_tokens"] = 1000; calls["output_tokens"] = 11
    gc.set_options(flags=hx.HX_FLAG_NO_DAG)
    a, c = gc.schedule_batch(calls)
    assert int(a[0]) == 0 and abs(float(c[0]) - 0.2651055) < 2e-6 * 0.2651055
    gc.close()


def test_empty_batch_not_ready_and_bad_ids(hx, oracle):
    import torch
    wl = make_workload("tiny")
    gc = hh.gpu_cluster(wl)
    assert hx.hx_schedule_batch(gc.h, None, 0, None, None, 0) is None        # n_calls = 0 is a no-op
    with pytest.raises(hx.HxError) as e:                                      # horizons not computed yet
        gc.schedule_batch(wl.calls)
    assert e.value.code == -4
    with pytest.raises(hx.HxError):
        gc.set_options(topk=9)
    with pytest.raises(hx.HxError) as e:                                      # cycle
        gc.dag_upload([0, 1, 2], [1, 0], [1.0, 1.0], [0, 0], [0.0])
    assert e.value.code == -3
    with pytest.raises(hx.HxError):                                           # edge across workflows
        gc.dag_upload([0, 1, 1], [1], [1.0, 1.0], [0, 1], [0.0, 0.0])
    # a record with an unknown model or node is flagged, gets no pair, and does not disturb the others
    gc.set_options(flags=hx.HX_FLAG_NO_DAG)
    calls = wl.calls.copy()
    calls["model"][3] = 77
    a, c = gc.schedule_batch(calls)
    a, c = a.cpu().numpy(), c.cpu().numpy()
    assert a[3] == -1 and np.isinf(c[3]) and gc.status() == -1
    good = np.arange(len(calls)) != 3
    oa, ocost, _ = oracle.schedule(hh.oracle_cluster(wl), wl.calls)
    assert np.array_equal(a[good], oa[good]) and np.array_equal(c[good], ocost[good])
    assert gc.status() == 0                               # reading the status word clears it
    a, _ = gc.schedule_batch(wl.calls)
    assert gc.status() == 0                               # a clean batch after a bad one reports clean
    gc.close()


def test_fractional_token_counts_are_refused_by_the_capacity_pass(hx, oracle):
    """The capacity pass takes its decisions on whole token counts.  A record with a fractional prompt or
    output length is flagged (status word, no pair) when the pass is on, while the plain argmin, which
    compares in binary32 like the oracle, scores it; free KV tokens that are not whole numbers are
    refused by the host."""
    gc, oc = _cluster_pair(hx, 5, 6, seed=11)
    calls = _calls(200, seed=12)
    calls["prompt_tokens"][17] += 0.5
    calls["output_tokens"][90] += 0.25
    gc.set_options(flags=hx.HX_FLAG_NO_DAG)
    a, c = gc.schedule_batch(calls)
    oa, ocost, _ = oracle.schedule(oc, calls)
    assert np.array_equal(a.cpu().numpy(), oa) and np.array_equal(c.cpu().numpy(), ocost) and gc.status() == 0
    gc.set_options(topk=3, commit=1, flags=hx.HX_FLAG_NO_DAG)
    a, c = gc.schedule_batch(calls)
    a, c = a.cpu().numpy(), c.cpu().numpy()
    assert gc.status() == -1
    assert a[17] == -1 and a[90] == -1 and np.isinf(c[17]) and np.isinf(c[90])
    good = np.ones(200, bool); good[[17, 90]] = False
    op, ocs, opr, om, ots = oracle.topk(oc, calls[good], 3)
    oa, ofree, oq = oracle.conflict(op, opr, om, ots, np.full(6, 1e6, np.float32), oc.qP, 6)
    assert np.array_equal(a[good], oa)
    gq, _, gfree = gc.read_loads()
    assert np.array_equal(gfree, ofree) and np.array_equal(gq, oq)
    with pytest.raises(hx.HxError) as e:
        gc.update_loads(kv_free=np.full(6, 1000.5, np.float32))
    assert e.value.code == -1
    with pytest.raises(hx.HxError):
        gc.update_loads(kv_free=np.full(6, 2.0 ** 24, np.float32))
    gc.close()


@pytest.mark.parametrize("kind", ["single", "chain_staged", "chain_block", "chain_global", "mixed"])
def test_horizon_workflow_classes(hx, oracle, kind):
    """Workflows small enough for a warp's staging area, for a block's, and too large for either."""
    rng = np.random.default_rng(5)
    if kind == "single":
        n_w = [1]
    elif kind == "chain_staged":
        n_w = [900]
    elif kind == "chain_block":
        n_w = [6000]
    elif kind == "chain_global":
        n_w = [30000]
    else:
        n_w = [1, 40, 1500, 3, 9000, 200, 25000, 7]
    rows, cols, wf = [0], [], []
    base = 0
    for w, n in enumerate(n_w):
        for i in range(n):
            succ = []
            if i + 1 < n:
                succ.append(base + i + 1)
                if i + 5 < n and rng.random() < 0.3:
                    succ.append(base + i + 5)
            cols += succ
            rows.append(len(cols))
            wf.append(w)
        base += n
    N = base
    cost = rng.lognormal(0, 1, N).astype(np.float32)
    wl = make_workload("tiny")
    gc = hh.gpu_cluster(wl)
    gc.dag_upload(rows, cols, cost, wf, np.zeros(len(n_w)))
    gc.critical_path()
    cp, tail, H = gc.dag_results()
    r = oracle.longest_path(rows, cols, cost, wf, len(n_w))
    assert np.array_equal(cp, r.cp) and np.array_equal(tail, r.tail) and np.array_equal(H, r.H)
    gc.close()


def test_horizons_of_a_forest_whose_workflows_are_interleaved(hx, oracle):
    """Node numbers in random order (no workflow is a contiguous range): the upload regroups such a forest along
    another path than one listed workflow by workflow; both must give the oracle's horizons, and the same values
    node for node as the ordered listing."""
    wl = make_workload("medium", scale=0.25)
    rng = np.random.default_rng(12)
    N = wl.n_nodes
    cost = rng.lognormal(0, 1, N).astype(np.float32)
    new_id = rng.permutation(N).astype(np.uint32)                 # old node v becomes new_id[v]
    old_of = np.argsort(new_id)
    rows, cols = [0], []
    for v_new in range(N):
        v = old_of[v_new]
        cols += [int(new_id[u]) for u in wl.col[wl.row_ptr[v]:wl.row_ptr[v + 1]]]
        rows.append(len(cols))
    wf_new, cost_new = wl.node_wf[old_of], cost[old_of]
    assert (np.diff(wf_new.astype(np.int64)) < 0).any()           # really interleaved
    gc = hh.gpu_cluster(wl)
    gc.dag_upload(rows, cols, cost_new, wf_new, wl.elapsed)
    gc.critical_path()
    cp, tail, H = gc.dag_results()
    r = oracle.longest_path(rows, cols, cost_new, wf_new, wl.n_workflows)
    assert np.array_equal(cp, r.cp) and np.array_equal(tail, r.tail) and np.array_equal(H, r.H)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    cp0, tail0, H0 = gc.dag_results()
    assert np.array_equal(cp0, cp[new_id]) and np.array_equal(tail0, tail[new_id]) and np.array_equal(H0, H)
    assert gc.status() == 0
    gc.close()


@pytest.mark.parametrize("name, scale, K", [("tiny", 1.0, 2), ("medium", 1.0, 4), ("large", 1 / 32, 4),
                                            ("cp_stress", 1 / 50, 1), ("sweep", 1 / 64, 4), ("sweep", 1 / 64, 8)])
def test_topk_and_capacity_pass(hx, oracle, name, scale, K):
    wl = make_workload(name, scale=scale)
    oc, gc, dag = _prepare(hx, oracle, wl)
    calls = wl.calls
    P, D = wl.P, wl.D
    free0 = wl.kv_free[P:].copy()
    if name != "sweep":                                   # make capacity scarce so that the pass matters
        m = calls["prompt_tokens"] + calls["output_tokens"]
        free0 = np.floor(np.minimum(free0, 0.7 * m.sum() / D)).astype(np.float32)
    kw = dict(dag=dag, node_wf=wl.node_wf, elapsed=wl.elapsed)
    n_chunks = 3
    step = max(1, len(calls) // n_chunks)
    qP = wl.load_s[:P].copy()
    gc.set_options(score_mode=hx.HX_MODE_RATIO, topk=K, commit=1, alpha=wl.alpha)
    for i in range(n_chunks):
        chunk = calls[i * step:(i + 1) * step]
        gc.update_loads(kv_free=free0)                    # decode capacity is refreshed between invocations
        a, c = gc.schedule_batch(chunk)
        a, c = a.cpu().numpy(), c.cpu().numpy()
        pair, cost, prio = gc.topk_results(len(chunk))
        oc.qP[:] = qP
        op, ocs, opr, om, ots = oracle.topk(oc, chunk, K, **kw)
        assert np.array_equal(pair, op) and np.array_equal(cost, ocs) and np.array_equal(prio, opr)
        oa, ofree, oq = oracle.conflict(op, opr, om, ots, free0, qP, D)
        gq, _, gfree = gc.read_loads()
        assert np.array_equal(a, oa), "%s chunk %d" % (name, i)
        assert np.array_equal(gfree, ofree) and np.array_equal(gq, oq)
        _, ocost, _ = oracle.schedule(oc, chunk, mode=ho.MODE_RATIO, **kw)
        assert np.array_equal(c, ocost)
        assert np.all(gfree >= 0)
        qP = oq
    assert gc.status() == 0
    gc.close()


def test_capacity_pass_without_commit_leaves_loads(hx, oracle):
    wl = make_workload("sweep", scale=1 / 64)
    oc, gc, dag = _prepare(hx, oracle, wl)
    before = gc.read_loads()
    gc.set_options(score_mode=hx.HX_MODE_RATIO, topk=4, commit=0)
    a, _ = gc.schedule_batch(wl.calls)
    after = gc.read_loads()
    assert all(np.array_equal(x, y) for x, y in zip(before, after))
    op, ocs, opr, om, ots = oracle.topk(oc, wl.calls, 4, dag=dag, node_wf=wl.node_wf, elapsed=wl.elapsed)
    oa, _, _ = oracle.conflict(op, opr, om, ots, wl.kv_free[wl.P:], wl.load_s[:wl.P], wl.D)
    assert np.array_equal(a.cpu().numpy(), oa)
    gc.close()


def test_equal_priorities_visit_lower_call_first(hx, oracle):
    """All calls identical: the order of the pass is the call index, capacity runs out part way."""
    gc, oc = _cluster_pair(hx, 4, 4, seed=3)
    calls = np.zeros(300, CALL_DTYPE)
    calls["prompt_tokens"] = 900; calls["output_tokens"] = 100
    free = np.array([20000, 5000, 7000, 3000], np.float32)
    gc.update_loads(kv_free=free)
    gc.set_options(topk=4, commit=1, flags=hx.HX_FLAG_NO_DAG)
    a, _ = gc.schedule_batch(calls)
    a = a.cpu().numpy()
    op, ocs, opr, om, ots = oracle.topk(oc, calls, 4)
    oa, ofree, oq = oracle.conflict(op, opr, om, ots, free, oc.qP, 4)
    assert np.array_equal(a, oa) and (a >= 0).sum() == 35 and np.all(a[35:] == -1)
    gq, _, gfree = gc.read_loads()
    assert np.array_equal(gfree, ofree) and np.array_equal(gq, oq)
    gc.close()


@pytest.mark.parametrize("n, K, P, D", [(20000, 4, 8, 12), (16384, 4, 8, 12), (16385, 2, 5, 40), (5000, 8, 300, 9),
                                       (33, 3, 2, 5), (1, 1, 1, 1)])
def test_capacity_pass_batch_sizes_and_pool_shapes(hx, oracle, n, K, P, D):
    """Batches on both sides of the size up to which the pass runs as one block-resident kernel, a prefill
    pool too wide for the fused queue sums, and the smallest shapes; a tenth of the calls fits no decode
    instance at all (priority +inf: visited first, placed nowhere) and a fifth are exact duplicates of one
    another (equal priorities: visited by call number)."""
    gc, oc = _cluster_pair(hx, P, D, seed=n + K, tight=True)
    calls = _calls(n, seed=n)
    rng = np.random.default_rng(n)
    dup = rng.random(n) < 0.2
    calls["model"][dup] = 0; calls["prompt_tokens"][dup] = 777; calls["output_tokens"][dup] = 33
    calls["prompt_tokens"][rng.random(n) < 0.1] = 2.0e6
    m = calls["prompt_tokens"] + calls["output_tokens"]
    free = np.floor(rng.uniform(0.05, 0.6, D) * np.minimum(m, 40000).sum() / D).astype(np.float32)
    free = np.minimum(free, 2.0 ** 24 - 1).astype(np.float32)
    qP = oc.qP.copy()
    gc.set_options(score_mode=hx.HX_MODE_RATIO, topk=K, commit=1, flags=hx.HX_FLAG_NO_DAG)
    for rep in range(2):                                  # the second batch sees the committed queues
        gc.update_loads(kv_free=free)
        a, _ = gc.schedule_batch(calls)
        oc.qP[:] = qP
        op, ocs, opr, om, ots = oracle.topk(oc, calls, K)
        pair, cost, prio = gc.topk_results(n)
        assert np.array_equal(pair, op) and np.array_equal(cost, ocs) and np.array_equal(prio, opr)
        oa, ofree, oq = oracle.conflict(op, opr, om, ots, free, qP, D)
        gq, _, gfree = gc.read_loads()
        assert np.array_equal(a.cpu().numpy(), oa), "placements differ"
        assert np.array_equal(gfree, ofree) and np.array_equal(gq, oq), "committed loads differ"
        qP = oq
    if n > 100:
        assert np.isinf(opr).any() and (oa >= 0).any() and (oa < 0).any()
    assert gc.status() == 0
    gc.close()


def test_host_buffer_entry_point_matches_device_path(hx, oracle):
    wl = make_workload("medium")
    oc, gc, dag = _prepare(hx, oracle, wl)
    gc.set_options(score_mode=hx.HX_MODE_SLACK, alpha=wl.alpha)
    a, c = gc.schedule_batch(wl.calls)
    ha, hc = gc.schedule_batch_host(wl.calls)
    assert np.array_equal(a.cpu().numpy(), ha) and np.array_equal(c.cpu().numpy(), hc)
    gc.close()


def test_async_host_entry_point_chains_dependent_batches(hx, oracle):
    """Four ready batches whose commits feed the next one, enqueued from page-locked memory without a
    synchronisation in between, equal the same batches run one by one through the device entry point."""
    import torch
    wl = make_workload("sweep", scale=1 / 32)
    oc, gc, dag = _prepare(hx, oracle, wl)
    gc.set_options(score_mode=hx.HX_MODE_RATIO, topk=4, commit=1, alpha=wl.alpha)
    n = len(wl.calls) // 4
    qP0, free0 = wl.load_s[:wl.P].copy(), wl.kv_free[wl.P:].copy()
    want = []
    for i in range(4):
        a, c = gc.schedule_batch(wl.calls[i * n:(i + 1) * n])
        want.append((a.cpu().numpy(), c.cpu().numpy()))
    loads_want = gc.read_loads()
    gc.update_loads(qP=qP0, kv_free=free0)
    calls_pin = torch.from_numpy(wl.calls[:4 * n].view(np.uint8).reshape(-1, 16).copy()).pin_memory()
    a_pin = torch.empty(4 * n, dtype=torch.int32).pin_memory()
    c_pin = torch.empty(4 * n, dtype=torch.float32).pin_memory()
    cn = calls_pin.numpy().view(hx.CALL_DTYPE).reshape(-1)
    sp = torch.cuda.current_stream().cuda_stream
    for i in range(4):
        hx.hx_schedule_batch_host_async(gc.h, cn[i * n:(i + 1) * n], a_pin.numpy()[i * n:(i + 1) * n],
                                        c_pin.numpy()[i * n:(i + 1) * n], sp)
    torch.cuda.current_stream().synchronize()
    for i in range(4):
        assert np.array_equal(a_pin.numpy()[i * n:(i + 1) * n], want[i][0])
        assert np.array_equal(c_pin.numpy()[i * n:(i + 1) * n], want[i][1])
    for x, y in zip(gc.read_loads(), loads_want):
        assert np.array_equal(x, y)
    gc.close()


@pytest.mark.parametrize("reset", [False, True])
def test_sweep_entry_point_equals_the_batches_one_by_one(hx, oracle, reset):
    """hx_schedule_sweep_host (copies on their own streams, overlapped with the kernels) against the same chunks
    run one by one through the device entry point, with and without the reset of the free KV tokens ahead of
    every chunk; a ragged last chunk; twice in a row on the same handle."""
    import torch
    wl = make_workload("sweep", scale=1 / 32)
    oc, gc, dag = _prepare(hx, oracle, wl)
    gc.set_options(score_mode=hx.HX_MODE_RATIO, topk=4, commit=1, alpha=wl.alpha)
    total = len(wl.calls) - 37
    n = 1500                                               # 6 chunks, the last one shorter
    qP0, free0 = wl.load_s[:wl.P].copy(), wl.kv_free[wl.P:].copy()
    want_a, want_c = [], []
    for lo in range(0, total, n):
        if reset:
            gc.update_loads(kv_free=free0)
        a, c = gc.schedule_batch(wl.calls[lo:min(total, lo + n)])
        want_a.append(a.cpu().numpy()); want_c.append(c.cpu().numpy())
    want_a, want_c = np.concatenate(want_a), np.concatenate(want_c)
    loads_want = gc.read_loads()
    calls_pin = torch.from_numpy(wl.calls[:total].view(np.uint8).reshape(-1, 16).copy()).pin_memory()
    a_pin = torch.empty(total, dtype=torch.int32).pin_memory()
    c_pin = torch.empty(total, dtype=torch.float32).pin_memory()
    free_pin = torch.from_numpy(free0.astype(np.float32)).pin_memory()
    cn = calls_pin.numpy().view(hx.CALL_DTYPE).reshape(-1)
    sp = torch.cuda.current_stream().cuda_stream
    for rep in range(2):
        a_pin.fill_(-7); c_pin.fill_(-7.0)
        gc.update_loads(qP=qP0, kv_free=free0)
        hx.hx_schedule_sweep_host(gc.h, cn, n, free_pin.numpy() if reset else None, a_pin.numpy(), c_pin.numpy(), sp)
        torch.cuda.current_stream().synchronize()
        assert np.array_equal(a_pin.numpy(), want_a) and np.array_equal(c_pin.numpy(), want_c)
        for x, y in zip(gc.read_loads(), loads_want):
            assert np.array_equal(x, y)
    with pytest.raises(hx.HxError):
        hx.hx_schedule_sweep_host(gc.h, cn, 0, None, a_pin.numpy(), c_pin.numpy(), sp)
    assert gc.status() == 0
    gc.close()


@pytest.mark.parametrize("commit", [1, 0])
def test_restored_capacity_equals_a_load_refresh_ahead_of_every_batch(hx, oracle, commit):
    """hx_set_kv_free_restore once against hx_cluster_update_loads(kv_free) ahead of every batch: same pairs, costs
    and loads after every batch; switched off, the committed capacities carry over again; a bad value changes nothing."""
    wl = make_workload("sweep", scale=1 / 32)
    oc, gc, dag = _prepare(hx, oracle, wl)
    gc.set_options(score_mode=hx.HX_MODE_RATIO, topk=4, commit=commit, alpha=wl.alpha)
    qP0, free0 = wl.load_s[:wl.P].copy(), wl.kv_free[wl.P:].copy()
    n, chunks = 2000, 4
    want = []
    gc.update_loads(qP=qP0, kv_free=free0)
    for i in range(chunks):
        gc.update_loads(kv_free=free0)
        a, c = gc.schedule_batch(wl.calls[i * n:(i + 1) * n])
        want.append((a.cpu().numpy(), c.cpu().numpy(), gc.read_loads()))
    gc.update_loads(qP=qP0, kv_free=np.zeros_like(free0))    # the table itself says "nothing free": the restore must win
    gc.set_kv_free_restore(free0)
    for i in range(chunks):
        a, c = gc.schedule_batch(wl.calls[i * n:(i + 1) * n])
        assert np.array_equal(a.cpu().numpy(), want[i][0]) and np.array_equal(c.cpu().numpy(), want[i][1])
        for x, y in zip(gc.read_loads(), want[i][2]):
            assert np.array_equal(x, y)
    assert (want[0][0] >= 0).any() and gc.status() == 0
    bad = free0.copy(); bad[0] = 10.5
    with pytest.raises(hx.HxError):
        gc.set_kv_free_restore(bad)
    a, c = gc.schedule_batch(wl.calls[:n])                    # still restored to free0
    if commit == 0:
        assert np.array_equal(a.cpu().numpy(), want[0][0])
    gc.set_kv_free_restore(None)                              # off: the table's values count again
    gc.update_loads(qP=qP0, kv_free=np.zeros_like(free0))
    a, c = gc.schedule_batch(wl.calls[:n])
    assert (a.cpu().numpy() == -1).all()
    gc.close()


@pytest.mark.parametrize("P, D, n", [(4, 9, 300), (70, 130, 700)])
def test_quadratic_prefill_variant(hx, oracle, P, D, n):
    """Attention FLOPs per token pair set on both sides: scoring, top-K lists and the greedy planner agree
    bit for bit; with zeros the results are those of the linear model."""
    gc, oc = _cluster_pair(hx, P, D, seed=P + D)
    calls = _calls(n, seed=P)
    gc.set_options(flags=hx.HX_FLAG_NO_DAG)
    base_a, base_c = (x.cpu().numpy() for x in gc.schedule_batch(calls))
    gc.set_attention_flops([0.0, 0.0])
    a, c = (x.cpu().numpy() for x in gc.schedule_batch(calls))
    assert np.array_equal(a, base_a) and np.array_equal(c, base_c)
    psi = np.array([2.5e5, 9e5], np.float32)
    gc.set_attention_flops(psi)
    oc.set_attention(psi)
    a, c = (x.cpu().numpy() for x in gc.schedule_batch(calls))
    oa, ocost, _ = oracle.schedule(oc, calls)
    assert np.array_equal(a, oa) and np.array_equal(c, ocost) and np.all(c >= base_c) and (c > base_c).any()
    gc.set_options(topk=3, flags=hx.HX_FLAG_NO_DAG)
    gc.schedule_batch(calls)
    pair, cost, prio = gc.topk_results(n)
    op, ocs, opr, _, _ = oracle.topk(oc, calls, 3)
    assert np.array_equal(pair, op) and np.array_equal(cost, ocs) and np.array_equal(prio, opr)
    gc.set_options(score_mode=hx.HX_MODE_RATIO, flags=hx.HX_FLAG_NO_DAG, commit=0)
    m = min(n, 200)
    ga, gr, go = (x.cpu().numpy() for x in gc.schedule_greedy(calls[:m]))
    ea, er, eo, _, _, _ = oracle.greedy(oc, calls[:m], np.full(D, 1e6, np.float32))
    assert np.array_equal(ga, ea) and np.array_equal(gr, er) and np.array_equal(go, eo)
    with pytest.raises(hx.HxError):
        gc.set_attention_flops([-1.0, 0.0])
    gc.close()


def test_runs_are_deterministic(hx, oracle):
    wl = make_workload("sweep", scale=1 / 32)
    outs = []
    for _ in range(2):
        oc, gc, dag = _prepare(hx, oracle, wl)
        gc.set_options(score_mode=hx.HX_MODE_RATIO, topk=4, commit=1)
        a, c = gc.schedule_batch(wl.calls)
        outs.append((a.cpu().numpy().tobytes(), c.cpu().numpy().tobytes(),
                     b"".join(x.tobytes() for x in gc.read_loads())))
        gc.close()
    assert outs[0] == outs[1]
