"""ctypes binding of the C ABI declared in include/hx.h.

Module-level functions carry the names of the C entry points and take plain
pointers / numpy arrays; `Cluster` is a small convenience wrapper that keeps the
handle and passes torch tensors' data pointers and the current CUDA stream.
PyTorch is used for device memory and streams only.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from .build import LIB_PATH

HX_OK = 0
HX_MODE_COMPLETION, HX_MODE_SLACK, HX_MODE_RATIO = 0, 1, 2
HX_FLAG_NO_DAG, HX_FLAG_NO_TAIL, HX_FLAG_UNLOADED, HX_FLAG_ONE_PASS = 1, 2, 4, 8

CALL_DTYPE = np.dtype([("node", "<u4"), ("model", "<u4"),
                       ("prompt_tokens", "<f4"), ("output_tokens", "<f4")])
INSTANCE_DTYPE = np.dtype([("type", "<u4"), ("role", "<u4"), ("load_s", "<f4"),
                           ("kv_cap_tokens", "<f4"), ("kv_free_tokens", "<f4")])


class HxError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("hx error %d: %s" % (code, msg))
        self.code = code


class _Options(C.Structure):
    _fields_ = [("score_mode", C.c_int), ("topk", C.c_int), ("commit", C.c_int),
                ("flags", C.c_int), ("alpha", C.c_float)]


def lib_path() -> str:
    return LIB_PATH


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError("libhx.so is not built (run: python paper_2605_16637_b200/build.py); "
                          "this package has no fallback path")
    lib = C.CDLL(LIB_PATH)
    vp, ci, u32 = C.c_void_p, C.c_int, C.c_uint32
    sig = {
        "hx_cluster_create": [vp, ci, vp, ci, vp, vp, ci, C.POINTER(vp)],
        "hx_cluster_update_loads": [vp, vp, vp, vp, vp],
        "hx_cluster_read_loads": [vp, vp, vp, vp, vp],
        "hx_set_kv_free_restore": [vp, vp, vp],
        "hx_cluster_destroy": [vp],
        "hx_dag_upload": [vp, vp, vp, vp, vp, vp, u32, u32, u32],
        "hx_critical_path": [vp, vp],
        "hx_dag_update_costs": [vp, vp, vp, u32, vp],
        "hx_dag_update_elapsed": [vp, vp, vp],
        "hx_get_dag_results": [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp)],
        "hx_dag_append": [vp, C.c_uint32, vp, vp, C.c_uint32, vp, vp, vp],
        "hx_dag_append_workflows": [vp, C.c_uint32, vp, vp],
        "hx_earliest_start": [vp, vp],
        "hx_get_earliest_results": [vp, C.POINTER(vp), C.POINTER(vp)],
        "hx_set_options": [vp, C.POINTER(_Options)],
        "hx_set_attention_flops": [vp, vp],
        "hx_schedule_batch": [vp, vp, ci, vp, vp, vp],
        "hx_schedule_batch_host": [vp, vp, ci, vp, vp, vp],
        "hx_schedule_batch_host_async": [vp, vp, ci, vp, vp, vp],
        "hx_schedule_sweep_host": [vp, vp, ci, ci, vp, vp, vp, vp],
        "hx_schedule_batch_static": [vp, vp, ci, vp, vp, vp],
        "hx_schedule_greedy": [vp, vp, ci, vp, vp, vp, vp],
        "hx_schedule_greedy_plan": [vp, vp, ci, vp, vp, vp, vp, vp],
        "hx_replay": [vp, vp, vp, vp, C.c_uint32, C.c_uint32, vp, vp, ci, vp, vp, vp, vp, vp],
        "hx_replay_lifecycle": [vp, vp, vp, C.c_double, ci, vp, vp, vp, vp, vp],
        "hx_estimate_calls": [vp, vp, ci, vp, vp, vp, vp, vp],
        "hx_decode_set_running": [vp, vp, vp, vp],
        "hx_schedule_decode": [vp, vp, vp, vp, ci, vp, vp, vp, vp, vp],
        "hx_get_topk": [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp)],
        "hx_get_status": [vp, C.POINTER(ci), vp],
        "hx_measure_fp32_rates": [vp, vp, vp, vp],
        "hx_enable_kernel_timing": [vp, ci],
        "hx_read_kernel_timing": [vp, C.POINTER(C.c_float), C.POINTER(ci)],
    }
    for name, args in sig.items():
        f = getattr(lib, name)
        f.argtypes = args
        f.restype = ci
    lib.hx_last_error.argtypes = [vp]
    lib.hx_last_error.restype = C.c_char_p
    lib.hx_launch_count.argtypes = [vp]
    lib.hx_launch_count.restype = C.c_longlong
    return lib


_lib = _load()


def _check(rc, h=None):
    if rc != HX_OK:
        raise HxError(rc, _lib.hx_last_error(h).decode())


def _np(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


# --- functions named after the C entry points ----------------------------------------------

def hx_cluster_create(gpu_types, instances, link_bw_gbps, models):
    gpu_types = _np(gpu_types, np.float32).reshape(-1, 2)
    instances = _np(instances, INSTANCE_DTYPE)
    n = instances.shape[0]
    link = _np(link_bw_gbps, np.float32).reshape(n, n)
    models = _np(models, np.float32).reshape(-1, 3)
    h = C.c_void_p()
    _check(_lib.hx_cluster_create(_p(gpu_types), gpu_types.shape[0], _p(instances), n, _p(link),
                                  _p(models), models.shape[0], C.byref(h)))
    return h


def hx_cluster_update_loads(h, qP=None, qD=None, kv_free=None, stream=0):
    arrs = [None if a is None else _np(a, np.float32) for a in (qP, qD, kv_free)]
    _check(_lib.hx_cluster_update_loads(h, _p(arrs[0]), _p(arrs[1]), _p(arrs[2]), stream), h)


def hx_set_kv_free_restore(h, kv_free=None, stream=0):
    a = None if kv_free is None else _np(kv_free, np.float32)
    _check(_lib.hx_set_kv_free_restore(h, _p(a), stream), h)


def hx_cluster_read_loads(h, n_prefill, n_decode, stream=0):
    qP = np.zeros(n_prefill, np.float32); qD = np.zeros(n_decode, np.float32)
    free = np.zeros(n_decode, np.float32)
    _check(_lib.hx_cluster_read_loads(h, _p(qP), _p(qD), _p(free), stream), h)
    return qP, qD, free


def hx_cluster_destroy(h):
    _check(_lib.hx_cluster_destroy(h))


def hx_dag_upload(h, row_ptr, col_idx, node_costs, node_workflow, workflow_elapsed_s):
    row_ptr = _np(row_ptr, np.uint32); col_idx = _np(col_idx, np.uint32)
    node_costs = _np(node_costs, np.float32); node_workflow = _np(node_workflow, np.uint32)
    el = _np(workflow_elapsed_s, np.float32)
    if row_ptr.shape[0] != node_workflow.shape[0] + 1 or node_costs.shape[0] != node_workflow.shape[0]:
        raise HxError(-1, "row_ptr, node_costs and node_workflow disagree on the node count")
    _check(_lib.hx_dag_upload(h, _p(row_ptr), _p(col_idx), _p(node_costs), _p(node_workflow), _p(el),
                              node_workflow.shape[0], col_idx.shape[0], el.shape[0]), h)


def hx_critical_path(h, stream=0):
    _check(_lib.hx_critical_path(h, stream), h)


def hx_dag_update_costs(h, node_ids, new_costs, stream=0):
    """Replace node cost estimates (e.g. by observed latencies) and refresh the horizons of the
    workflows they belong to."""
    node_ids = _np(node_ids, np.uint32); new_costs = _np(new_costs, np.float32)
    if node_ids.shape[0] != new_costs.shape[0]:
        raise HxError(-1, "node_ids and new_costs differ in length")
    _check(_lib.hx_dag_update_costs(h, _p(node_ids), _p(new_costs), node_ids.shape[0], stream), h)


def hx_dag_update_elapsed(h, workflow_elapsed_s, stream=0):
    el = _np(workflow_elapsed_s, np.float32)
    _check(_lib.hx_dag_update_elapsed(h, _p(el), stream), h)


def hx_get_dag_results(h):
    """Device addresses (int) of cp, tail, H."""
    cp, tail, H = C.c_void_p(), C.c_void_p(), C.c_void_p()
    _check(_lib.hx_get_dag_results(h, C.byref(cp), C.byref(tail), C.byref(H)), h)
    return cp.value, tail.value, H.value


def hx_dag_append(h, new_costs, new_node_workflow, edge_src, edge_dst, stream=0):
    """Appends nodes (costs, workflows) and edges (src, dst); the new nodes are numbered on from the old count."""
    c, w = _np(new_costs, np.float32), _np(new_node_workflow, np.uint32)
    es, ed = _np(edge_src, np.uint32), _np(edge_dst, np.uint32)
    if c.shape[0] != w.shape[0] or es.shape[0] != ed.shape[0]:
        raise HxError(-1, "array lengths differ")
    _check(_lib.hx_dag_append(h, c.shape[0], _p(c), _p(w), es.shape[0], _p(es), _p(ed), stream), h)


def hx_dag_append_workflows(h, new_elapsed_s, stream=0):
    """Registers len(new_elapsed_s) arriving workflows (numbered on from the old count, no nodes yet)."""
    el = _np(new_elapsed_s, np.float32)
    _check(_lib.hx_dag_append_workflows(h, el.shape[0], _p(el), stream), h)


def hx_earliest_start(h, stream=0):
    _check(_lib.hx_earliest_start(h, stream), h)


def hx_get_earliest_results(h):
    """Device addresses (int) of est, eft."""
    est, eft = C.c_void_p(), C.c_void_p()
    _check(_lib.hx_get_earliest_results(h, C.byref(est), C.byref(eft)), h)
    return est.value, eft.value


def hx_set_options(h, score_mode=HX_MODE_COMPLETION, topk=0, commit=0, flags=0, alpha=1.5):
    o = _Options(int(score_mode), int(topk), int(commit), int(flags), float(alpha))
    _check(_lib.hx_set_options(h, C.byref(o)), h)


def hx_set_attention_flops(h, per_model):
    """Attention FLOPs per pair of prompt tokens, one value per model (quadratic prefill variant)."""
    a = _np(per_model, np.float32)
    _check(_lib.hx_set_attention_flops(h, _p(a)), h)


def hx_schedule_batch(h, calls_ptr, n_calls, out_assign_ptr, out_cost_ptr, stream=0):
    _check(_lib.hx_schedule_batch(h, calls_ptr, int(n_calls), out_assign_ptr, out_cost_ptr, stream), h)


def hx_schedule_batch_static(h, calls_ptr, n_calls, out_assign_ptr, out_cost_ptr, stream=0):
    """hx_schedule_batch without any allocation: intermediates live in a fixed device array
    (at most 16384 calls with topk <= 4); see include/hx.h for who needs this and the rules."""
    _check(_lib.hx_schedule_batch_static(h, calls_ptr, int(n_calls), out_assign_ptr, out_cost_ptr, stream), h)


def hx_schedule_greedy(h, calls_ptr, n_calls, out_assign_ptr, out_ratio_ptr, out_order_ptr, stream=0):
    """Recomputing greedy planner for small queues (Algorithm 1); device pointers."""
    _check(_lib.hx_schedule_greedy(h, calls_ptr, int(n_calls), out_assign_ptr, out_ratio_ptr, out_order_ptr,
                                   stream), h)


def hx_schedule_greedy_plan(h, calls_ptr, n_calls, out_assign_ptr, out_ratio_ptr, out_order_ptr, out_delta_ptr,
                            stream=0):
    """hx_schedule_greedy plus the projected completion Delta of every call; device pointers."""
    _check(_lib.hx_schedule_greedy_plan(h, calls_ptr, int(n_calls), out_assign_ptr, out_ratio_ptr, out_order_ptr,
                                        out_delta_ptr, stream), h)


def hx_replay(h, row_ptr, col_idx, node_workflow, n_workflows, node_calls, arrival_s, qmax=4096, stream=0):
    """Event-driven replay; host arrays in, dict(fin, ratio, req95, req99, runs, stuck) out."""
    row, col, nwf = _np(row_ptr, np.uint32), _np(col_idx, np.uint32), _np(node_workflow, np.uint32)
    calls, arr = _np(node_calls, CALL_DTYPE), _np(arrival_s, np.float64)
    n, w = nwf.shape[0], int(n_workflows)
    if row.shape[0] != n + 1 or calls.shape[0] != n or arr.shape[0] != w:
        raise HxError(-1, "array lengths differ")
    fin, ratio = np.zeros(n, np.float64), np.zeros(w, np.float64)
    req, stats = np.zeros(2, np.float64), np.zeros(2, np.int32)
    _check(_lib.hx_replay(h, _p(row), _p(col), _p(nwf), n, w, _p(calls), _p(arr), int(qmax), _p(fin), _p(ratio),
                          _p(req), _p(stats), stream), h)
    return dict(fin=fin, ratio=ratio, req95=float(req[0]), req99=float(req[1]), runs=int(stats[0]),
                stuck=int(stats[1]))


def hx_replay_lifecycle(h, n_workflows, node_calls, arrival_s, est_error=0.0, qmax=4096, stream=0):
    """Replay with separate stages, a scheduled decode stage and estimation error; host arrays in,
    dict(fin, ratio, req95, req99, runs, decode_runs, stuck) out."""
    calls, arr = _np(node_calls, CALL_DTYPE), _np(arrival_s, np.float64)
    n, w = calls.shape[0], int(n_workflows)
    if arr.shape[0] != w:
        raise HxError(-1, "array lengths differ")
    fin, ratio = np.zeros(n, np.float64), np.zeros(w, np.float64)
    req, stats = np.zeros(2, np.float64), np.zeros(3, np.int32)
    _check(_lib.hx_replay_lifecycle(h, _p(calls), _p(arr), float(est_error), int(qmax), _p(fin), _p(ratio), _p(req),
                                    _p(stats), stream), h)
    return dict(fin=fin, ratio=ratio, req95=float(req[0]), req99=float(req[1]), runs=int(stats[0]),
                decode_runs=int(stats[1]), stuck=int(stats[2]))


def hx_estimate_calls(h, calls_ptr, n_calls, out_tpre_ptr, out_tdec_ptr, out_kv_ptr, out_tokens_ptr, stream=0):
    _check(_lib.hx_estimate_calls(h, calls_ptr, int(n_calls), out_tpre_ptr, out_tdec_ptr, out_kv_ptr, out_tokens_ptr,
                                  stream), h)


KV_INTERVAL_DTYPE = np.dtype([("end_s", "<f4"), ("tokens", "<f4")])


def hx_decode_set_running(h, inst_ptr, running, stream=0):
    """inst_ptr: CSR offsets per decode instance; running: KV_INTERVAL_DTYPE records (host)."""
    inst_ptr = _np(inst_ptr, np.uint32); running = _np(running, KV_INTERVAL_DTYPE)
    if inst_ptr.shape[0] < 1 or inst_ptr[-1] != running.shape[0]:
        raise HxError(-1, "inst_ptr does not span the running calls")
    _check(_lib.hx_decode_set_running(h, _p(inst_ptr), _p(running), stream), h)


def hx_schedule_decode(h, calls_ptr, lock_ptr, ready_ptr, n_calls, out_inst_ptr, out_start_ptr, out_ratio_ptr,
                       out_order_ptr, stream=0):
    """Decode-stage scheduler over token-capacity intervals (Section 5.4); device pointers."""
    _check(_lib.hx_schedule_decode(h, calls_ptr, lock_ptr, ready_ptr, int(n_calls), out_inst_ptr, out_start_ptr,
                                   out_ratio_ptr, out_order_ptr, stream), h)


def hx_schedule_batch_host(h, calls, out_assign=None, out_cost=None, stream=0):
    """calls: host array of CALL_DTYPE (numpy; may be a view of pinned memory)."""
    calls = _np(calls, CALL_DTYPE)
    n = calls.shape[0]
    if out_assign is None:
        out_assign = np.empty(n, np.int32)
    if out_cost is None:
        out_cost = np.empty(n, np.float32)
    _check(_lib.hx_schedule_batch_host(h, _p(calls), n, _p(out_assign), _p(out_cost), stream), h)
    return out_assign, out_cost


def hx_schedule_batch_host_async(h, calls, out_assign, out_cost, stream=0):
    """Enqueue only: calls / out_assign / out_cost are numpy views of page-locked memory that the
    caller keeps alive until the stream has been synchronised."""
    if calls.dtype != CALL_DTYPE or out_assign.dtype != np.int32 or out_cost.dtype != np.float32:
        raise HxError(-1, "hx_schedule_batch_host_async takes CALL_DTYPE, int32 and float32 arrays as they are")
    if not (calls.flags.c_contiguous and out_assign.flags.c_contiguous and out_cost.flags.c_contiguous):
        raise HxError(-1, "hx_schedule_batch_host_async needs contiguous arrays")
    _check(_lib.hx_schedule_batch_host_async(h, _p(calls), calls.shape[0], _p(out_assign), _p(out_cost), stream), h)


def hx_schedule_sweep_host(h, calls, chunk_calls, kv_free_reset, out_assign, out_cost, stream=0):
    """Enqueue a whole sweep (chunks of chunk_calls, copies overlapped with the kernels); arrays as for
    hx_schedule_batch_host_async, kv_free_reset a float32 array (page-locked for overlap) or None."""
    if calls.dtype != CALL_DTYPE or out_assign.dtype != np.int32 or out_cost.dtype != np.float32:
        raise HxError(-1, "hx_schedule_sweep_host takes CALL_DTYPE, int32 and float32 arrays as they are")
    if not (calls.flags.c_contiguous and out_assign.flags.c_contiguous and out_cost.flags.c_contiguous):
        raise HxError(-1, "hx_schedule_sweep_host needs contiguous arrays")
    if kv_free_reset is not None and (kv_free_reset.dtype != np.float32 or not kv_free_reset.flags.c_contiguous):
        raise HxError(-1, "kv_free_reset must be a contiguous float32 array")
    _check(_lib.hx_schedule_sweep_host(h, _p(calls), calls.shape[0], int(chunk_calls), _p(kv_free_reset),
                                       _p(out_assign), _p(out_cost), stream), h)


def hx_get_topk(h):
    """Device addresses (int) of pairs, costs, prio."""
    a, b, c = C.c_void_p(), C.c_void_p(), C.c_void_p()
    _check(_lib.hx_get_topk(h, C.byref(a), C.byref(b), C.byref(c)), h)
    return a.value, b.value, c.value


def hx_get_status(h, stream=0):
    s = C.c_int(0)
    _check(_lib.hx_get_status(h, C.byref(s), stream), h)
    return s.value


def hx_measure_fp32_rates(h, stream=0):
    """Lane-instructions per second of fma.f32, fma.f32x2, three-input min and their mix; ms of each launch."""
    rates, ms = np.zeros(4, np.float64), np.zeros(4, np.float32)
    _check(_lib.hx_measure_fp32_rates(h, _p(rates), _p(ms), stream), h)
    return dict(zip(("fma", "fma2", "min3", "mix"), (float(x) for x in rates))), ms.tolist()


def hx_enable_kernel_timing(h, enable=True):
    _check(_lib.hx_enable_kernel_timing(h, int(bool(enable))), h)


def hx_read_kernel_timing(h):
    """Returns {family: (milliseconds, enqueues)} for scoring, conflict, horizon."""
    ms = (C.c_float * 3)(); n = (C.c_int * 3)()
    _check(_lib.hx_read_kernel_timing(h, ms, n), h)
    return {name: (float(ms[i]), int(n[i])) for i, name in enumerate(("scoring", "conflict", "horizon"))}


def hx_last_error(h=None):
    return _lib.hx_last_error(h).decode()


def hx_launch_count(h):
    return int(_lib.hx_launch_count(h))


# --- convenience wrapper ----------------------------------------------------------------------

class _Borrowed:
    """A borrowed device buffer exposed through the CUDA array interface."""

    def __init__(self, ptr, count, typestr):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": typestr, "data": (int(ptr), False),
                                         "version": 2}


def _dev_to_numpy(ptr, count, typestr):
    """Copy `count` items from a borrowed device address into a new numpy array."""
    import torch
    if count == 0:
        return np.zeros(0, dtype=typestr)
    torch.cuda.current_stream().synchronize()
    return torch.as_tensor(_Borrowed(ptr, count, typestr), device="cuda").cpu().numpy()


class Cluster:
    """Owns one hx_cluster handle; methods mirror the C entry points."""

    def __init__(self, gpu_types, instances, link_bw_gbps, models):
        self.h = None
        self.h = hx_cluster_create(gpu_types, instances, link_bw_gbps, models)
        inst = _np(instances, INSTANCE_DTYPE)
        self.P = int((inst["role"] == 0).sum())
        self.D = int(inst.shape[0] - self.P)
        self.M = int(_np(models, np.float32).reshape(-1, 3).shape[0])
        self.G = int(_np(gpu_types, np.float32).reshape(-1, 2).shape[0])
        self.n_nodes = 0
        self.n_workflows = 0
        self.topk = 0

    @classmethod
    def from_workload(cls, wl):
        """Build from an object with the attributes of hx_synth.Workload."""
        I = wl.P + wl.D
        inst = np.zeros(I, INSTANCE_DTYPE)
        inst["type"] = wl.inst_type
        inst["role"][wl.P:] = 1
        inst["load_s"] = wl.load_s
        inst["kv_cap_tokens"] = wl.kv_cap
        inst["kv_free_tokens"] = wl.kv_free
        return cls(wl.gpu_types, inst, wl.link_gbps, wl.models)

    @staticmethod
    def _stream():
        import torch
        return torch.cuda.current_stream().cuda_stream

    def update_loads(self, qP=None, qD=None, kv_free=None):
        hx_cluster_update_loads(self.h, qP, qD, kv_free, self._stream())

    def set_kv_free_restore(self, kv_free=None):
        if kv_free is not None and np.asarray(kv_free).shape[0] != self.D:
            raise HxError(-1, "one value per decode instance is needed")
        hx_set_kv_free_restore(self.h, kv_free, self._stream())

    def read_loads(self):
        return hx_cluster_read_loads(self.h, self.P, self.D, self._stream())

    def dag_upload(self, row_ptr, col_idx, node_costs, node_workflow, workflow_elapsed_s):
        hx_dag_upload(self.h, row_ptr, col_idx, node_costs, node_workflow, workflow_elapsed_s)
        self.n_nodes = int(np.asarray(node_workflow).shape[0])
        self.n_workflows = int(np.asarray(workflow_elapsed_s).shape[0])

    def critical_path(self):
        hx_critical_path(self.h, self._stream())

    def update_costs(self, node_ids, new_costs):
        hx_dag_update_costs(self.h, node_ids, new_costs, self._stream())

    def update_elapsed(self, workflow_elapsed_s):
        el = _np(workflow_elapsed_s, np.float32)
        if el.shape[0] != self.n_workflows:
            raise HxError(-1, "one elapsed time per workflow is needed")
        hx_dag_update_elapsed(self.h, el, self._stream())

    def dag_results(self):
        """cp, tail, H as numpy arrays (synchronises)."""
        cp, tail, H = hx_get_dag_results(self.h)
        return (_dev_to_numpy(cp, self.n_nodes, "<f4"), _dev_to_numpy(tail, self.n_nodes, "<f4"),
                _dev_to_numpy(H, self.n_workflows, "<f4"))

    def dag_append(self, new_costs, new_node_workflow, edge_src, edge_dst):
        hx_dag_append(self.h, new_costs, new_node_workflow, edge_src, edge_dst, self._stream())
        self.n_nodes += int(np.asarray(new_costs).shape[0])

    def dag_append_workflows(self, new_elapsed_s):
        hx_dag_append_workflows(self.h, new_elapsed_s, self._stream())
        self.n_workflows += int(np.asarray(new_elapsed_s).shape[0])

    def earliest_start(self):
        hx_earliest_start(self.h, self._stream())

    def earliest_results(self):
        """est, eft as numpy arrays (synchronises)."""
        est, eft = hx_get_earliest_results(self.h)
        return _dev_to_numpy(est, self.n_nodes, "<f4"), _dev_to_numpy(eft, self.n_nodes, "<f4")

    def set_options(self, score_mode=HX_MODE_COMPLETION, topk=0, commit=0, flags=0, alpha=1.5):
        hx_set_options(self.h, score_mode, topk, commit, flags, alpha)
        self.topk = int(topk)

    def set_attention_flops(self, per_model):
        a = _np(per_model, np.float32)
        if a.shape[0] != self.M:
            raise HxError(-1, "one value per model is needed")
        hx_set_attention_flops(self.h, a)

    def schedule_batch(self, calls, out_assign=None, out_cost=None):
        """calls: CUDA tensor holding n records of 16 bytes, or a numpy CALL_DTYPE array
        (copied to the device first).  Returns (assign, cost) CUDA tensors."""
        import torch
        if isinstance(calls, np.ndarray):
            calls = torch.from_numpy(_np(calls, CALL_DTYPE).view(np.uint8).copy()).cuda()
        n = calls.numel() * calls.element_size() // 16
        if out_assign is None:
            out_assign = torch.empty(n, dtype=torch.int32, device="cuda")
        if out_cost is None:
            out_cost = torch.empty(n, dtype=torch.float32, device="cuda")
        hx_schedule_batch(self.h, calls.data_ptr(), n, out_assign.data_ptr(), out_cost.data_ptr(), self._stream())
        return out_assign, out_cost

    def schedule_greedy(self, calls, with_delta=False):
        """calls as for schedule_batch.  Returns (assign, ratio, order) CUDA tensors, plus delta on request."""
        import torch
        if isinstance(calls, np.ndarray):
            calls = torch.from_numpy(_np(calls, CALL_DTYPE).view(np.uint8).copy()).cuda()
        n = calls.numel() * calls.element_size() // 16
        assign = torch.empty(n, dtype=torch.int32, device="cuda")
        ratio = torch.empty(n, dtype=torch.float32, device="cuda")
        order = torch.empty(n, dtype=torch.int32, device="cuda")
        if not with_delta:
            hx_schedule_greedy(self.h, calls.data_ptr(), n, assign.data_ptr(), ratio.data_ptr(), order.data_ptr(),
                               self._stream())
            return assign, ratio, order
        delta = torch.empty(n, dtype=torch.float32, device="cuda")
        hx_schedule_greedy_plan(self.h, calls.data_ptr(), n, assign.data_ptr(), ratio.data_ptr(), order.data_ptr(),
                                delta.data_ptr(), self._stream())
        return assign, ratio, order, delta

    def replay(self, row_ptr, col_idx, node_workflow, node_calls, arrival_s, qmax=4096):
        return hx_replay(self.h, row_ptr, col_idx, node_workflow, self.n_workflows, node_calls, arrival_s, qmax,
                         self._stream())

    def replay_lifecycle(self, node_calls, arrival_s, est_error=0.0, qmax=4096):
        return hx_replay_lifecycle(self.h, len(arrival_s), node_calls, arrival_s, est_error, qmax, self._stream())

    def estimate_calls(self, calls):
        """Service-time terms of the given calls: (tpre[n, G], tdec[n, G], kv_bytes[n], tokens[n]) device tensors."""
        import torch
        calls = _np(calls, CALL_DTYPE)
        n = calls.shape[0]
        dev = torch.from_numpy(calls.view(np.uint8).reshape(-1, 16).copy()).cuda()
        tp = torch.empty((n, self.G), dtype=torch.float32, device="cuda"); td = torch.empty_like(tp)
        kv = torch.empty(n, dtype=torch.float32, device="cuda"); tok = torch.empty_like(kv)
        hx_estimate_calls(self.h, dev.data_ptr(), n, tp.data_ptr(), td.data_ptr(), kv.data_ptr(), tok.data_ptr(),
                          self._stream())
        torch.cuda.current_stream().synchronize()
        return tp, td, kv, tok

    def decode_set_running(self, inst_ptr, end_s, tokens):
        run = np.zeros(len(end_s), KV_INTERVAL_DTYPE)
        run["end_s"] = end_s; run["tokens"] = tokens
        hx_decode_set_running(self.h, inst_ptr, run, self._stream())

    def schedule_decode(self, calls, lock=None, ready_s=None):
        """Returns (inst, start, ratio, order) CUDA tensors."""
        import torch
        if isinstance(calls, np.ndarray):
            calls = torch.from_numpy(_np(calls, CALL_DTYPE).view(np.uint8).copy()).cuda()
        n = calls.numel() * calls.element_size() // 16
        lk = None if lock is None else torch.as_tensor(np.ascontiguousarray(lock, np.int32)).cuda()
        rd = None if ready_s is None else torch.as_tensor(np.ascontiguousarray(ready_s, np.float32)).cuda()
        inst = torch.empty(n, dtype=torch.int32, device="cuda")
        start = torch.empty(n, dtype=torch.float32, device="cuda")
        ratio = torch.empty(n, dtype=torch.float32, device="cuda")
        order = torch.empty(n, dtype=torch.int32, device="cuda")
        hx_schedule_decode(self.h, calls.data_ptr(), None if lk is None else lk.data_ptr(),
                           None if rd is None else rd.data_ptr(), n, inst.data_ptr(), start.data_ptr(),
                           ratio.data_ptr(), order.data_ptr(), self._stream())
        torch.cuda.current_stream().synchronize()      # lk / rd are temporaries of this call
        return inst, start, ratio, order

    def schedule_batch_host(self, calls, out_assign=None, out_cost=None):
        return hx_schedule_batch_host(self.h, calls, out_assign, out_cost, self._stream())

    def topk_results(self, n_calls):
        a, b, c = hx_get_topk(self.h)
        K = self.topk
        return (_dev_to_numpy(a, n_calls * K, "<i4").reshape(n_calls, K),
                _dev_to_numpy(b, n_calls * K, "<f4").reshape(n_calls, K),
                _dev_to_numpy(c, n_calls, "<f4"))

    def status(self):
        return hx_get_status(self.h, self._stream())

    def enable_kernel_timing(self, enable=True):
        hx_enable_kernel_timing(self.h, enable)

    def read_kernel_timing(self):
        return hx_read_kernel_timing(self.h)

    def launch_count(self):
        return hx_launch_count(self.h)

    def close(self):
        if self.h is not None:
            hx_cluster_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
