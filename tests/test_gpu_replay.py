"""Event-driven replay of the library (hx_replay, planner runs on the GPU) against the oracle's replay
(oracle/hx_replay.py, planner runs on the CPU): identical completion times, ratios and Req95 / Req99."""
import numpy as np
import pytest

import hx_helpers as hh
from hx_synth import make_workload
from oracle import hx_oracle as ho
from oracle import hx_replay as hr

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hx():
    import __graft_entry__ as entry
    entry.build()
    import paper_2605_16637_b200 as mod
    return mod


def _trace(wl, load, seed):
    """Stand-alone costs, horizons and Poisson-like arrivals scaled so that the offered work is `load` times
    what the prefill pool can serve."""
    orc = ho.Oracle()
    oc = hh.oracle_cluster(wl)
    cost = orc.schedule(oc, wl.node_calls, flags=ho.FLAG_UNLOADED | ho.FLAG_NO_DAG)[2]
    dag = orc.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
    rng = np.random.default_rng(seed)
    span = float(cost.sum()) / (wl.P * load)
    arrival = np.sort(rng.uniform(0, span, wl.n_workflows))
    return orc, oc, cost, dag, arrival


@pytest.mark.parametrize("name, scale, load, qmax", [("tiny", 1.0, 2.0, 4096), ("medium", 0.25, 1.5, 4096),
                                                     ("medium", 0.25, 4.0, 64), ("large", 1 / 64, 2.0, 512)])
def test_replay_equals_oracle_replay(hx, name, scale, load, qmax):
    wl = make_workload(name, scale=scale)
    orc, oc, cost, dag, arrival = _trace(wl, load, seed=71)
    gc = hh.gpu_cluster(wl)
    gcost = hh.gpu_node_costs(gc, wl.node_calls)
    assert np.array_equal(gcost, cost)
    gc.dag_upload(wl.row_ptr, wl.col, gcost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    gc.set_options(score_mode=hx.HX_MODE_SLACK, topk=2, commit=0, alpha=2.0)
    got = gc.replay(wl.row_ptr, wl.col, wl.node_wf, wl.node_calls, arrival, qmax=qmax)
    want = hr.replay(orc, oc, wl.row_ptr, wl.col, wl.node_wf, wl.n_workflows, wl.node_calls, arrival, dag, qmax=qmax)
    assert got["stuck"] == want["stuck"] == 0 and got["runs"] == want["runs"]
    assert np.array_equal(got["fin"], want["fin"])
    assert np.array_equal(got["ratio"], want["ratio"])
    assert got["req95"] == want["req95"] and got["req99"] == want["req99"]
    assert want["ratio"].min() >= 1 - 1e-6 and want["req99"] > 1.0
    assert gc.status() == 0
    # the options of the handle are back as they were
    a, c = gc.schedule_batch(wl.calls[:64])
    assert gc.topk == 2
    gc.close()


def test_replay_with_tight_kv_room_and_bad_arguments(hx):
    wl = make_workload("medium", scale=0.25)
    m = (wl.node_calls["prompt_tokens"] + wl.node_calls["output_tokens"]).max()
    wl.kv_cap[wl.P:] = float(2 * m)                           # two of the largest calls fill an instance
    wl.kv_free[wl.P:] = 0                                     # the replay starts idle whatever the loads say
    orc, oc, cost, dag, arrival = _trace(wl, 6.0, seed=72)
    gc = hh.gpu_cluster(wl)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    with pytest.raises(hx.HxError) as e:
        gc.replay(wl.row_ptr, wl.col, wl.node_wf, wl.node_calls, arrival)
    assert e.value.code == -4                                 # no horizons yet
    gc.critical_path()
    got = gc.replay(wl.row_ptr, wl.col, wl.node_wf, wl.node_calls, arrival)
    want = hr.replay(orc, oc, wl.row_ptr, wl.col, wl.node_wf, wl.n_workflows, wl.node_calls, arrival, dag)
    assert got["stuck"] == want["stuck"] == 0
    assert np.array_equal(got["fin"], want["fin"]) and got["req95"] == want["req95"] and got["req99"] == want["req99"]
    assert want["runs"] > wl.n_nodes // 8                     # calls were passed over and planned at later events
    for kw in (dict(qmax=0), dict(qmax=5000)):
        with pytest.raises(hx.HxError) as e:
            gc.replay(wl.row_ptr, wl.col, wl.node_wf, wl.node_calls, arrival, **kw)
        assert e.value.code == -1
    bad = arrival.copy(); bad[3] = -1.0
    with pytest.raises(hx.HxError):
        gc.replay(wl.row_ptr, wl.col, wl.node_wf, wl.node_calls, bad)
    shuffled = wl.node_calls.copy(); shuffled["node"][5] = 6
    with pytest.raises(hx.HxError):
        gc.replay(wl.row_ptr, wl.col, wl.node_wf, shuffled, arrival)
    gc.close()


def test_estimator_equals_oracle_terms(hx):
    """hx_estimate_calls (the Estimator of Section 4.2) against the oracle's per-class service times, bit for bit,
    with and without the quadratic attention term; a record with an unknown model is flagged."""
    wl = make_workload("large", scale=1 / 64)
    orc, oc = ho.Oracle(), hh.oracle_cluster(wl)
    gc = hh.gpu_cluster(wl)
    for psi in (None, np.array([3.0e5, 1.0e6], np.float32)[:gc.M]):
        if psi is not None:
            gc.set_attention_flops(psi); oc.set_attention(psi)
        tp, td, kv, tok = (x.cpu().numpy() for x in gc.estimate_calls(wl.node_calls))
        wtp, wtd, wkv, wm = orc.terms(oc, wl.node_calls)
        assert np.array_equal(tp, wtp) and np.array_equal(td, wtd) and np.array_equal(kv, wkv) and np.array_equal(tok, wm)
    assert gc.status() == 0
    bad = wl.node_calls[:8].copy(); bad["model"][2] = 31
    tp, td, kv, tok = (x.cpu().numpy() for x in gc.estimate_calls(bad))
    assert np.all(np.isinf(tp[2])) and np.all(np.isfinite(tp[[0, 1, 3]])) and gc.status() == -1
    gc.close()


@pytest.mark.parametrize("name, scale, load, qmax, eps", [("tiny", 1.0, 2.0, 4096, 0.0), ("tiny", 1.0, 2.0, 4096, 0.2),
                                                          ("medium", 0.25, 8.0, 4096, 0.0), ("medium", 0.25, 8.0, 4096, 0.2),
                                                          ("medium", 0.25, 32.0, 64, 0.3), ("large", 1 / 64, 8.0, 512, 0.1)])
def test_lifecycle_replay_equals_oracle_replay(hx, name, scale, load, qmax, eps):
    """The stages of a call kept apart, decode-stage events planned with locks, estimation error on what the
    schedulers see: completion times, ratios, Req95 / Req99 and the number of planner runs identical to the
    oracle's replay."""
    wl = make_workload(name, scale=scale)
    orc, oc, cost, dag, arrival = _trace(wl, load, seed=73)
    gc = hh.gpu_cluster(wl)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    gc.set_options(score_mode=hx.HX_MODE_SLACK, topk=2, commit=1, alpha=2.0)
    got = gc.replay_lifecycle(wl.node_calls, arrival, est_error=eps, qmax=qmax)
    want = hr.replay_lifecycle(orc, oc, wl.row_ptr, wl.col, wl.node_wf, wl.n_workflows, wl.node_calls, arrival, dag,
                               est_error=eps, qmax=qmax)
    assert got["stuck"] == want["stuck"] == 0
    assert got["runs"] == want["runs"] and got["decode_runs"] == want["decode_runs"] > 0
    assert np.array_equal(got["fin"], want["fin"])
    assert np.array_equal(got["ratio"], want["ratio"])
    assert got["req95"] == want["req95"] and got["req99"] == want["req99"]
    assert gc.status() == 0
    a, c = gc.schedule_batch(wl.calls[:64])                  # options and model table are back as they were
    assert gc.topk == 2
    gc.close()


def test_lifecycle_replay_with_tight_kv_room_and_bad_arguments(hx):
    wl = make_workload("medium", scale=0.25)
    m = (wl.node_calls["prompt_tokens"] + wl.node_calls["output_tokens"]).max()
    wl.kv_cap[wl.P:] = float(2 * m)                           # two of the largest calls fill an instance
    wl.kv_free[wl.P:] = 0
    orc, oc, cost, dag, arrival = _trace(wl, 16.0, seed=74)
    gc = hh.gpu_cluster(wl)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    with pytest.raises(hx.HxError) as e:
        gc.replay_lifecycle(wl.node_calls, arrival)
    assert e.value.code == -4                                 # no horizons yet
    gc.critical_path()
    for eps in (0.0, 0.3):
        got = gc.replay_lifecycle(wl.node_calls, arrival, est_error=eps)
        want = hr.replay_lifecycle(orc, oc, wl.row_ptr, wl.col, wl.node_wf, wl.n_workflows, wl.node_calls, arrival, dag,
                                   est_error=eps)
        assert got["stuck"] == want["stuck"] == 0
        assert np.array_equal(got["fin"], want["fin"]) and got["req95"] == want["req95"] and got["req99"] == want["req99"]
        assert want["req99"] > 1.2                            # calls wait for KV room
    for kw in (dict(qmax=0), dict(qmax=5000), dict(est_error=1.0), dict(est_error=-0.1)):
        with pytest.raises(hx.HxError) as e:
            gc.replay_lifecycle(wl.node_calls, arrival, **kw)
        assert e.value.code == -1
    shuffled = wl.node_calls.copy(); shuffled["node"][5] = 6
    with pytest.raises(hx.HxError):
        gc.replay_lifecycle(shuffled, arrival)
    # the older replay checks the graph it is given against the uploaded one
    col = wl.col.copy(); col[3] = wl.n_nodes + 7
    with pytest.raises(hx.HxError) as e:
        gc.replay(wl.row_ptr, col, wl.node_wf, wl.node_calls, arrival)
    assert e.value.code == -1
    row = wl.row_ptr.copy(); row[-1] += 5
    with pytest.raises(hx.HxError):
        gc.replay(row, wl.col, wl.node_wf, wl.node_calls, arrival)
    gc.close()
