"""GPU-vs-oracle parity of the recomputing greedy planner (Algorithm 1, the while-loop over the
queue snapshot) through the C ABI binding: taken order, pairs, ratios and the committed state
must be identical; ratios are additionally checked against the 1e-5 relative bar."""
import json
import os

import numpy as np
import pytest

import hx_helpers as hh
from hx_synth import CALL_DTYPE, make_workload
from oracle import hx_oracle as ho

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def hx():
    import __graft_entry__ as entry
    entry.build()
    import paper_2605_16637_b200 as mod
    return mod


def _compare(hx, gc, oc, oracle, calls, free0, P, D, dag=None, node_wf=None, elapsed=None, flags=0):
    gc.set_options(score_mode=hx.HX_MODE_RATIO, commit=1, flags=flags)
    a, r, o, dl = (t.cpu().numpy() for t in gc.schedule_greedy(calls, with_delta=True))
    ea, er, eo, placed, eq, ef, ed = oracle.greedy(oc, calls, free0, dag=dag, node_wf=node_wf, elapsed=elapsed,
                                                   with_delta=True)
    assert np.array_equal(o, eo), "order differs"
    assert np.array_equal(dl, ed), "projected completions differ"
    assert np.array_equal(a, ea), "pairs differ"
    hh.assert_costs_close(r, er, "ratios")
    assert np.array_equal(r, er)
    qP, _, free = gc.read_loads()
    assert np.array_equal(qP, eq) and np.array_equal(free, ef)
    assert gc.status() == 0
    return placed, a


# the last case is the whole medium configuration: 4,096 calls (the largest queue the planner takes) x 16 x 16 pairs
@pytest.mark.parametrize("name, scale", [("tiny", 1.0), ("medium", 1 / 8), ("medium", 1 / 2), ("medium", 1.0)])
def test_greedy_on_generated_queues(hx, oracle, name, scale):
    wl = make_workload(name, scale=scale)
    oc, gc = hh.oracle_cluster(wl), hh.gpu_cluster(wl)
    cost = hh.gpu_node_costs(gc, wl.node_calls)
    assert np.array_equal(cost, hh.oracle_node_costs(oracle, oc, wl.node_calls))
    dag = oracle.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    placed, a = _compare(hx, gc, oc, oracle, wl.calls, wl.kv_free[wl.P:], wl.P, wl.D, dag=dag,
                         node_wf=wl.node_wf, elapsed=wl.elapsed)
    assert placed == len(wl.calls)               # capacities of these configurations do not bind
    gc.close()


@pytest.mark.parametrize("P, D, n, frac", [(1, 1, 9, 0.5), (2, 2, 64, 0.5), (3, 5, 200, 0.3), (16, 16, 700, 0.6),
                                           (33, 7, 333, 0.4), (64, 64, 256, 0.5),
                                           (128, 64, 300, 0.5),     # per-class times cached, no room for the row minima
                                           (200, 200, 500, 0.4)])   # the last: no room for the cached per-class times
def test_greedy_with_binding_capacity(hx, oracle, P, D, n, frac):
    rng = np.random.default_rng(100 + P + D)
    G, M = 4, 2
    types = np.stack([rng.uniform(50, 2000, G), rng.uniform(0.3, 8, G)], 1).astype(np.float32)
    models = np.stack([rng.uniform(1e9, 2e11, M), rng.uniform(1e9, 2e11, M),
                       rng.choice([65536.0, 131072.0, 327680.0], M)], 1).astype(np.float32)
    calls = np.zeros(n, CALL_DTYPE)
    calls["model"] = rng.integers(0, M, n)
    calls["prompt_tokens"] = np.clip(np.round(rng.lognormal(7, 1, n)), 1, 32768)
    calls["output_tokens"] = np.clip(np.round(rng.lognormal(5, 1, n)), 1, 32768)
    m = calls["prompt_tokens"] + calls["output_tokens"]
    inst = np.zeros(P + D, hx.INSTANCE_DTYPE)
    inst["type"] = rng.integers(0, G, P + D)
    inst["role"][P:] = 1
    inst["load_s"] = np.round(rng.uniform(0, 2, P + D) * 4) / 4      # equal admission times: exact ties
    inst["kv_cap_tokens"] = rng.choice([3000.0, 1e6], P + D)
    inst["kv_free_tokens"] = np.floor(rng.uniform(0.5, 1.5, P + D) * frac * m.sum() / D)
    link = rng.uniform(25, 400, (P + D, P + D)).astype(np.float32)
    gc = hx.Cluster(types, inst, link, models)
    oc = ho.Cluster(types, inst["type"][:P], inst["type"][P:], inst["load_s"][:P], inst["load_s"][P:],
                    inst["kv_cap_tokens"][P:], link[:P, P:], models)
    placed, a = _compare(hx, gc, oc, oracle, calls, inst["kv_free_tokens"][P:], P, D, flags=hx.HX_FLAG_NO_DAG)
    assert 0 < placed < n                        # some calls are left behind
    gc.close()


def test_greedy_worked_run(hx):
    with open(os.path.join(GOLD, "greedy_hand.json")) as f:
        g = json.load(f)
    i, e = g["inputs"], g["expected"]
    C = len(i["calls"])
    inst = np.zeros(4, hx.INSTANCE_DTYPE)
    inst["type"] = i["typeP"] + i["typeD"]
    inst["role"][2:] = 1
    inst["load_s"] = i["qP"] + i["qD"]
    inst["kv_cap_tokens"][2:] = i["capD"]
    inst["kv_free_tokens"][2:] = i["freeD"]
    link = np.ones((4, 4), np.float32)
    link[:2, 2:] = i["link_gbps"]
    gc = hx.Cluster(i["gpu_types"], inst, link, [i["model"]])
    calls = np.zeros(C, CALL_DTYPE)
    for c, r in enumerate(i["calls"]):
        calls[c] = (c, 0, r["prompt_tokens"], r["output_tokens"])
    # every call is its own one-node workflow: cost = H, so the horizon kernel reproduces H
    H = np.array([r["H"] for r in i["calls"]], np.float32)
    gc.dag_upload(np.zeros(C + 1, np.uint32), np.zeros(0, np.uint32), H, np.arange(C, dtype=np.uint32),
                  np.array([r["elapsed"] for r in i["calls"]], np.float32))
    gc.critical_path()
    gc.set_options(score_mode=hx.HX_MODE_RATIO, commit=1)
    a, r, o = (t.cpu().numpy() for t in gc.schedule_greedy(calls))
    n = len(e["order"])
    assert list(o[:n]) == e["order"] and np.all(o[n:] == -1) and list(a) == e["assign"]
    for c in range(C):
        if e["ratio"][c] is None:
            assert np.isinf(r[c])
        else:
            assert abs(r[c] - e["ratio"][c]) <= 2e-6 * e["ratio"][c]
    qP, _, free = gc.read_loads()
    np.testing.assert_allclose(qP, e["qP"], rtol=2e-6)
    assert list(free) == e["freeD"]
    gc.close()


def test_greedy_argument_checks(hx):
    wl = make_workload("tiny")
    gc = hh.gpu_cluster(wl)
    gc.set_options(flags=0)
    with pytest.raises(hx.HxError) as e:
        gc.schedule_greedy(wl.calls)             # horizons missing
    assert e.value.code == -4
    gc.set_options(flags=hx.HX_FLAG_NO_DAG | hx.HX_FLAG_UNLOADED)
    with pytest.raises(hx.HxError):
        gc.schedule_greedy(wl.calls)
    gc.set_options(flags=hx.HX_FLAG_NO_DAG)
    big = np.zeros(5000, CALL_DTYPE)
    big["prompt_tokens"] = 10; big["output_tokens"] = 10
    with pytest.raises(hx.HxError) as e:
        gc.schedule_greedy(big)
    assert "4096" in str(e.value)
    bad = wl.calls.copy()
    bad["model"][3] = 77
    a, r, o = (t.cpu().numpy() for t in gc.schedule_greedy(bad))
    assert a[3] == -1 and np.isinf(r[3]) and 3 not in o and gc.status() == -1
    gc.close()
