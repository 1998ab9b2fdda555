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
