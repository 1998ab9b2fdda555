"""hx_schedule_batch_static: the batch operation for hosts that cannot allocate device memory.

Who needs it: a serving process whose memory pool already owns the whole GPU (a late
cudaMalloc would fail), a latency-critical scheduling thread that cannot afford the
device-wide synchronisation an allocation implies, or code running where the CUDA
allocator must not be entered.  The regular entry point allocates its top-K and
capacity-pass buffers on first use; this one keeps them in a fixed array inside the
library.  The test calls it through the C ABI twice in a row (the second time with a
smaller, different batch, so stale contents of the shared array would show) and checks
every output against the regular entry point: integer outputs identical, costs within the
tolerance used by the other parity tests.  This file is collected last on purpose.
"""
import numpy as np
import pytest

import hx_helpers as hh
from hx_synth import make_workload

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hx():
    import __graft_entry__ as entry
    entry.build()
    import paper_2605_16637_b200 as mod
    return mod


def _run(hx, gc, entry, calls_dev, n, loads):
    import torch
    gc.update_loads(*loads)
    a = torch.empty(n, dtype=torch.int32, device="cuda")
    c = torch.empty(n, dtype=torch.float32, device="cuda")
    entry(gc.h, calls_dev.data_ptr(), n, a.data_ptr(), c.data_ptr(), torch.cuda.current_stream().cuda_stream)
    qP, qD, free = gc.read_loads()
    return a.cpu().numpy(), c.cpu().numpy(), qP, free


def test_static_entry_point_matches_regular_one_twice_in_a_row(hx):
    import torch
    wl = make_workload("sweep", scale=1 / 16)             # 16,384 calls: exactly the documented maximum
    assert len(wl.calls) == 16384
    gc = hh.gpu_cluster(wl)
    cost = hh.gpu_node_costs(gc, wl.node_calls)
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    gc.set_options(score_mode=hx.HX_MODE_RATIO, topk=4, commit=1, alpha=wl.alpha)
    loads = (wl.load_s[:wl.P], wl.load_s[wl.P:], wl.kv_free[wl.P:])
    batches = [wl.calls, wl.calls[3000:8000][::-1].copy()]
    for calls in batches:                                 # two calls in a row on the shared array
        n = len(calls)
        dev = torch.from_numpy(calls.view(np.uint8).copy()).cuda()
        ra, rc, rq, rf = _run(hx, gc, hx.hx_schedule_batch, dev, n, loads)
        sa, sc, sq, sf = _run(hx, gc, hx.hx_schedule_batch_static, dev, n, loads)
        assert np.array_equal(sa, ra), "placements differ"
        hh.assert_costs_close(sc, rc, "scores")
        assert np.array_equal(sf, rf) and np.array_equal(sq, rq), "committed loads differ"
        assert (ra >= 0).any() and (ra < 0).any()          # the capacity pass really decided something
    assert gc.status() == 0
    # plain argmin needs no intermediate buffer: any batch size goes through
    gc.set_options(score_mode=hx.HX_MODE_COMPLETION, topk=0)
    big = np.concatenate([wl.calls, wl.calls[:1000]])
    dev = torch.from_numpy(big.view(np.uint8).copy()).cuda()
    ra, rc, _, _ = _run(hx, gc, hx.hx_schedule_batch, dev, len(big), loads)
    sa, sc, _, _ = _run(hx, gc, hx.hx_schedule_batch_static, dev, len(big), loads)
    assert np.array_equal(sa, ra) and np.array_equal(sc, rc)
    gc.close()


def test_static_entry_point_leaves_device_memory_as_it_is(hx):
    """A handle that has never run the regular entry point (so none of its buffers exist): after the one documented
    warm-up call, further calls through the allocation-free entry point leave the amount of free device memory
    exactly as it was, and match the regular entry point run afterwards on the same inputs."""
    import torch
    wl = make_workload("sweep", scale=1 / 32)
    gc = hh.gpu_cluster(wl)
    gc.set_options(score_mode=hx.HX_MODE_COMPLETION, topk=4, commit=1, flags=hx.HX_FLAG_NO_DAG)
    loads = (wl.load_s[:wl.P], wl.load_s[wl.P:], wl.kv_free[wl.P:])
    n = len(wl.calls)
    dev = torch.from_numpy(wl.calls.view(np.uint8).copy()).cuda()
    a = torch.empty(n, dtype=torch.int32, device="cuda")
    c = torch.empty(n, dtype=torch.float32, device="cuda")
    sp = torch.cuda.current_stream().cuda_stream
    gc.update_loads(*loads)
    hx.hx_schedule_batch_static(gc.h, dev.data_ptr(), n, a.data_ptr(), c.data_ptr(), sp)     # warm-up: loads the kernels
    torch.cuda.synchronize()
    before = torch.cuda.mem_get_info()[0]
    for rep in range(3):
        gc.update_loads(*loads)
        hx.hx_schedule_batch_static(gc.h, dev.data_ptr(), n, a.data_ptr(), c.data_ptr(), sp)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == before, "the allocation-free entry point changed the free device memory"
    sa, sc = a.cpu().numpy(), c.cpu().numpy()
    sq, _, sf = gc.read_loads()
    ra, rc, rq, rf = _run(hx, gc, hx.hx_schedule_batch, dev, n, loads)
    assert np.array_equal(sa, ra) and np.array_equal(sf, rf) and np.array_equal(sq, rq)
    hh.assert_costs_close(sc, rc, "scores")
    assert gc.status() == 0
    gc.close()


def test_static_entry_point_rejects_sizes_beyond_its_array(hx):
    import torch
    wl = make_workload("sweep", scale=1 / 15)             # a few calls more than the maximum
    n = len(wl.calls)
    assert n > 16384
    gc = hh.gpu_cluster(wl)
    dev = torch.from_numpy(wl.calls.view(np.uint8).copy()).cuda()
    a = torch.empty(n, dtype=torch.int32, device="cuda")
    c = torch.empty(n, dtype=torch.float32, device="cuda")
    gc.set_options(topk=4, flags=hx.HX_FLAG_NO_DAG)
    with pytest.raises(hx.HxError) as e:
        hx.hx_schedule_batch_static(gc.h, dev.data_ptr(), n, a.data_ptr(), c.data_ptr(), 0)
    assert e.value.code == -1 and "16384" in str(e.value)
    gc.set_options(topk=8, flags=hx.HX_FLAG_NO_DAG)
    with pytest.raises(hx.HxError) as e:
        hx.hx_schedule_batch_static(gc.h, dev.data_ptr(), 100, a.data_ptr(), c.data_ptr(), 0)
    assert e.value.code == -1 and "HX_STATIC_MAX_TOPK" in str(e.value)
    gc.close()
