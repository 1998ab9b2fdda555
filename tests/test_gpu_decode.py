"""GPU-vs-oracle parity of the decode-stage scheduler (Section 5.4) through the C ABI binding: chosen
instances, planned starts, ratios and the order must be identical."""
import json
import os

import numpy as np
import pytest

import hx_helpers as hh
from hx_synth import CALL_DTYPE
from oracle import hx_oracle as ho

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(__file__), "golden")
F32 = np.float32


@pytest.fixture(scope="module")
def hx():
    import __graft_entry__ as entry
    entry.build()
    import paper_2605_16637_b200 as mod
    return mod


def _pair(hx, rng, D, caps, G=4, M=2):
    types = np.stack([rng.uniform(50, 2000, G), rng.uniform(0.3, 8, G)], 1).astype(F32)
    models = np.stack([rng.uniform(1e9, 2e11, M), rng.uniform(1e9, 2e11, M),
                       rng.choice([65536.0, 131072.0, 327680.0], M)], 1).astype(F32)
    inst = np.zeros(1 + D, hx.INSTANCE_DTYPE)
    inst["type"] = rng.integers(0, G, 1 + D)
    inst["role"][1:] = 1
    inst["kv_cap_tokens"][1:] = rng.choice(caps, D)
    inst["kv_free_tokens"] = inst["kv_cap_tokens"]
    link = np.full((1 + D, 1 + D), 100.0, F32)
    gc = hx.Cluster(types, inst, link, models)
    oc = ho.Cluster(types, inst["type"][:1], inst["type"][1:], [0.0], np.zeros(D), inst["kv_cap_tokens"][1:],
                    link[:1, 1:], models)
    return gc, oc


def _queue(rng, C, D, M=2, hi=1500):
    calls = np.zeros(C, CALL_DTYPE)
    calls["node"] = np.arange(C)
    calls["model"] = rng.integers(0, M, C)
    calls["prompt_tokens"] = rng.integers(50, hi, C)
    calls["output_tokens"] = rng.integers(5, 400, C)
    lock = np.where(rng.random(C) < 0.3, rng.integers(0, D, C), -1).astype(np.int32)
    ready = np.where(rng.random(C) < 0.5, 0.0, rng.uniform(0, 1.0, C)).astype(F32)
    return calls, lock, ready


def _running(rng, oc, per):
    ptr, end, tok = [0], [], []
    for d in range(oc.D):
        k = int(rng.integers(0, per + 1))
        share = rng.dirichlet(np.ones(k + 1))[:k] * 0.9 * oc.capD[d] if k else []
        for s in share:
            end.append(np.round(rng.uniform(0.01, 3.0), 2)); tok.append(np.floor(s))     # rounded: equal ends occur
        ptr.append(len(end))
    return np.array(ptr, np.uint32), np.array(end, F32), np.array(tok, F32)


def _check(hx, gc, oc, oracle, calls, lock, ready, ptr, end, tok, commit=0, run_start=None, one_pass=False):
    gc.set_options(score_mode=hx.HX_MODE_RATIO, commit=commit,
                   flags=hx.HX_FLAG_NO_DAG | (hx.HX_FLAG_ONE_PASS if one_pass else 0))
    got = [t.cpu().numpy() for t in gc.schedule_decode(calls, lock, ready)]
    plan = oracle.decode_onepass if one_pass else oracle.decode_greedy
    want = plan(oc, calls, ptr, end, tok, lock, ready, run_start=run_start)
    for g, w, name in zip(got, want[:4], ("instance", "start", "ratio", "order")):
        assert np.array_equal(g, w), name
    hh.assert_costs_close(got[2], want[2], "ratio")
    assert gc.status() == 0
    return want


@pytest.mark.parametrize("D, C, per, caps", [(1, 10, 2, (4000.0,)), (2, 40, 3, (3000.0, 6000.0)),
                                             (5, 150, 4, (3000.0, 6000.0, 20000.0)), (16, 400, 6, (4000.0, 8000.0)),
                                             (40, 700, 3, (6000.0,)), (64, 1024, 2, (5000.0, 9000.0)),
                                             (16, 2048, 4, (4000.0, 8000.0))])     # the longest queue accepted
def test_decode_scheduler_matches_oracle(hx, oracle, D, C, per, caps):
    rng = np.random.default_rng(200 + D)
    gc, oc = _pair(hx, rng, D, caps)
    calls, lock, ready = _queue(rng, C, D)
    ptr, end, tok = _running(rng, oc, per)
    gc.decode_set_running(ptr, end, tok)
    inst, start, ratio, order, placed = _check(hx, gc, oc, oracle, calls, lock, ready, ptr, end, tok)
    assert placed == C and (start > ready).any()         # some calls wait for capacity
    # without commit the snapshot is untouched: the same queue gives the same plan again
    _check(hx, gc, oc, oracle, calls, lock, ready, ptr, end, tok)
    # the one-pass ordering on the same queue: another plan (the order changes once calls wait for capacity)
    o_inst, o_start, o_ratio, o_order, o_placed = _check(hx, gc, oc, oracle, calls, lock, ready, ptr, end, tok,
                                                         one_pass=True)
    assert o_placed == C and (C < 40 or not np.array_equal(o_order, order))
    gc.close()


@pytest.mark.parametrize("C", [100, 300])
def test_decode_scheduler_with_a_snapshot_too_long_for_shared_memory(hx, oracle, C):
    # 40 instances x 700 running calls: the step functions do not fit the shared-memory pool, so every block works
    # on its copy in global memory (one block for 100 calls, the cluster for 300)
    rng = np.random.default_rng(300 + C)
    D = 40
    gc, oc = _pair(hx, rng, D, (1.0e6,))
    calls, lock, ready = _queue(rng, C, D, hi=20000)
    ptr, end, tok = [0], [], []
    for d in range(D):
        share = rng.dirichlet(np.ones(701))[:700] * 0.995 * oc.capD[d]
        end += list(rng.uniform(0.01, 3.0, 700).astype(F32)); tok += list(np.floor(share))
        ptr.append(len(end))
    ptr, end, tok = np.array(ptr, np.uint32), np.array(end, F32), np.array(tok, F32)
    gc.decode_set_running(ptr, end, tok)
    inst, start, ratio, order, placed = _check(hx, gc, oc, oracle, calls, lock, ready, ptr, end, tok)
    assert placed == C and (start > ready).any()
    _check(hx, gc, oc, oracle, calls, lock, ready, ptr, end, tok, one_pass=True)
    gc.close()


def test_decode_commit_carries_the_plan_into_the_next_invocation(hx, oracle):
    rng = np.random.default_rng(77)
    D = 6
    gc, oc = _pair(hx, rng, D, (5000.0, 8000.0))
    ptr, end, tok = _running(rng, oc, 3)
    gc.decode_set_running(ptr, end, tok)
    q1 = _queue(rng, 60, D)
    inst, start, ratio, order, placed = _check(hx, gc, oc, oracle, *q1, ptr, end, tok, commit=1)
    # the oracle's second run sees the planned intervals of the first as part of the state
    _, tdec, _, m = oracle.terms(oc, q1[0])
    iv = [[(0.0, float(end[i]), float(tok[i])) for i in range(ptr[d], ptr[d + 1])] for d in range(D)]
    for c in order[:placed]:
        d = inst[c]
        iv[d].append((float(start[c]), float(F32(start[c]) + F32(tdec[c, oc.typeD[d]])), float(m[c])))
    ptr2 = np.cumsum([0] + [len(v) for v in iv]).astype(np.uint32)
    flat = [x for v in iv for x in v]
    q2 = _queue(rng, 80, D)
    _check(hx, gc, oc, oracle, *q2, ptr2, [x[1] for x in flat], [x[2] for x in flat], commit=1,
           run_start=[x[0] for x in flat])
    gc.close()


def test_decode_worked_run(hx):
    with open(os.path.join(GOLD, "decode_hand.json")) as f:
        g = json.load(f)
    i, e = g["inputs"], g["expected"]
    D, C = len(i["capD"]), len(i["calls"])
    inst = np.zeros(1 + D, hx.INSTANCE_DTYPE)
    inst["type"][1:] = i["typeD"]
    inst["role"][1:] = 1
    inst["kv_cap_tokens"][1:] = i["capD"]
    inst["kv_free_tokens"][1:] = i["capD"]
    gc = hx.Cluster(i["gpu_types"], inst, np.full((1 + D, 1 + D), 100.0, F32), [i["model"]])
    calls = np.zeros(C, CALL_DTYPE)
    for c, r in enumerate(i["calls"]):
        calls[c] = (c, 0, r["prompt_tokens"], r["output_tokens"])
    H = np.array([r["H"] for r in i["calls"]], F32)
    gc.dag_upload(np.zeros(C + 1, np.uint32), np.zeros(0, np.uint32), H, np.arange(C, dtype=np.uint32),
                  np.array([r["elapsed"] for r in i["calls"]], F32))
    gc.critical_path()
    ptr = np.cumsum([0] + [len(r) for r in i["running"]]).astype(np.uint32)
    gc.decode_set_running(ptr, [x["end"] for r in i["running"] for x in r], [x["tokens"] for r in i["running"] for x in r])
    gc.set_options(score_mode=hx.HX_MODE_RATIO)
    got = [t.cpu().numpy() for t in gc.schedule_decode(calls, [r["lock"] for r in i["calls"]],
                                                       [r["ready"] for r in i["calls"]])]
    assert list(got[3]) == e["order"] and list(got[0]) == e["inst"]
    np.testing.assert_allclose(got[1], e["start"], rtol=2e-6, atol=1e-9)
    np.testing.assert_allclose(got[2], e["ratio"], rtol=2e-6)
    # the one-pass ordering of the same queue, also worked out in exact arithmetic
    e = g["expected_one_pass"]
    gc.set_options(score_mode=hx.HX_MODE_RATIO, flags=hx.HX_FLAG_ONE_PASS)
    got = [t.cpu().numpy() for t in gc.schedule_decode(calls, [r["lock"] for r in i["calls"]],
                                                       [r["ready"] for r in i["calls"]])]
    assert list(got[3]) == e["order"] and list(got[0]) == e["inst"]
    np.testing.assert_allclose(got[1], e["start"], rtol=2e-6, atol=1e-9)
    np.testing.assert_allclose(got[2], e["ratio"], rtol=2e-6)
    gc.close()


def test_decode_argument_checks_and_oversized_calls(hx, oracle):
    rng = np.random.default_rng(5)
    gc, oc = _pair(hx, rng, 3, (3000.0,))
    calls, lock, ready = _queue(rng, 20, 3)
    gc.set_options(flags=hx.HX_FLAG_NO_DAG)
    with pytest.raises(hx.HxError) as e:
        gc.schedule_decode(calls, lock, ready)
    assert e.value.code == -4                                   # no snapshot yet
    for ends, toks in (([0.0], [10.0]), ([np.inf], [10.0]), ([1.0], [10.5]), ([1.0], [-1.0])):
        with pytest.raises(hx.HxError):
            gc.decode_set_running([0, 1, 1, 1], ends, toks)
    gc.decode_set_running([0, 0, 0, 0], [], [])                 # idle instances
    calls["prompt_tokens"][7] = 5000                            # fits nowhere
    lock[:] = -1
    got = [t.cpu().numpy() for t in gc.schedule_decode(calls, lock, ready)]
    want = oracle.decode_greedy(oc, calls, [0, 0, 0, 0], [], [], lock, ready)
    assert got[0][7] == -1 and np.isinf(got[2][7]) and want[4] == 19
    for g, w in zip(got, want[:4]):
        assert np.array_equal(g, w)
    assert gc.status() == 0
    gc.set_options(flags=hx.HX_FLAG_NO_DAG | hx.HX_FLAG_ONE_PASS)   # the oversized call is never visited
    got = [t.cpu().numpy() for t in gc.schedule_decode(calls, lock, ready)]
    want = oracle.decode_onepass(oc, calls, [0, 0, 0, 0], [], [], lock, ready)
    assert got[0][7] == -1 and np.isinf(got[2][7]) and want[4] == 19 and got[3][19] == -1
    for g, w in zip(got, want[:4]):
        assert np.array_equal(g, w)
    with pytest.raises(hx.HxError):
        gc.set_options(flags=16)                                # not a flag
    gc.set_options(flags=hx.HX_FLAG_NO_DAG)
    bad = lock.copy(); bad[2] = 9                               # lock beyond the pool
    got = [t.cpu().numpy() for t in gc.schedule_decode(calls, bad, ready)]
    assert got[0][2] == -1 and gc.status() == -1
    gc.close()
