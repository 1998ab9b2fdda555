"""ctypes front-end of the CPU oracle (oracle/hx_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
CPU-baseline leg of the benchmark.  Nothing in the CUDA library or its Python
binding imports this module, and this module imports nothing from them.
It only marshals numpy arrays into the C entry points; all arithmetic is in
the C++ file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hx_oracle.cpp")
_LIB = os.path.join(_HERE, "libhx_oracle.so")

MODE_COMPLETION, MODE_SLACK, MODE_RATIO = 0, 1, 2
FLAG_NO_DAG, FLAG_NO_TAIL, FLAG_UNLOADED = 1, 2, 4

CALL_DTYPE = np.dtype([("node", "<u4"), ("model", "<u4"),
                       ("prompt_tokens", "<f4"), ("output_tokens", "<f4")])


def build(force: bool = False) -> str:
    """Compile the oracle with the host compiler; returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-ffp-contract=off", "-std=c++17", "-shared", "-fPIC",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class _Cluster(C.Structure):
    _fields_ = [("G", C.c_int32), ("P", C.c_int32), ("D", C.c_int32), ("M", C.c_int32),
                ("peak_tflops", C.c_void_p), ("hbm_tbps", C.c_void_p),
                ("typeP", C.c_void_p), ("typeD", C.c_void_p),
                ("qP", C.c_void_p), ("qD", C.c_void_p), ("capD", C.c_void_p),
                ("link_gbps", C.c_void_p),
                ("flops_per_token", C.c_void_p), ("weight_bytes", C.c_void_p),
                ("kv_bytes_per_token", C.c_void_p), ("attn_flops_per_token2", C.c_void_p)]


class _Dag(C.Structure):
    _fields_ = [("node_wf", C.c_void_p), ("tail", C.c_void_p), ("H", C.c_void_p),
                ("elapsed", C.c_void_p)]


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _u32(a):
    return np.ascontiguousarray(a, dtype=np.uint32)


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p)


@dataclass
class DagResult:
    cp: np.ndarray
    tail: np.ndarray
    H: np.ndarray


class Cluster:
    """Cluster snapshot in the oracle's own layout (plain arrays)."""

    def __init__(self, gpu_types, typeP, typeD, qP, qD, capD, link_pd_gbps, models):
        gpu_types = _f32(gpu_types).reshape(-1, 2)
        models = _f32(models).reshape(-1, 3)
        self.tflops = _f32(gpu_types[:, 0]); self.tbps = _f32(gpu_types[:, 1])
        self.typeP = _u32(typeP); self.typeD = _u32(typeD)
        self.qP = _f32(qP).copy(); self.qD = _f32(qD).copy(); self.capD = _f32(capD)
        self.P, self.D = self.typeP.shape[0], self.typeD.shape[0]
        self.link = _f32(link_pd_gbps).reshape(self.P, self.D)
        self.phi = _f32(models[:, 0]); self.omega = _f32(models[:, 1]); self.kappa = _f32(models[:, 2])
        self.G, self.M = self.tflops.shape[0], self.phi.shape[0]
        self.psi = None                 # optional attention FLOPs per token pair, one per model (set_attention)

    def set_attention(self, psi):
        self.psi = _f32(psi)
        assert self.psi.shape[0] == self.M

    @classmethod
    def from_workload(cls, wl):
        P, D = wl.P, wl.D
        return cls(wl.gpu_types, wl.inst_type[:P], wl.inst_type[P:], wl.load_s[:P], wl.load_s[P:],
                   wl.kv_cap[P:], wl.link_gbps[:P, P:], wl.models)

    def _c(self):
        return _Cluster(self.G, self.P, self.D, self.M, _ptr(self.tflops), _ptr(self.tbps),
                        _ptr(self.typeP), _ptr(self.typeD), _ptr(self.qP), _ptr(self.qD),
                        _ptr(self.capD), _ptr(self.link), _ptr(self.phi), _ptr(self.omega),
                        _ptr(self.kappa), None if self.psi is None else _ptr(self.psi))


class Oracle:
    def __init__(self):
        self.lib = C.CDLL(build())

    # -- horizons ---------------------------------------------------------
    def longest_path(self, row_ptr, col, cost, node_wf, n_workflows) -> DagResult:
        row_ptr, col, node_wf, cost = _u32(row_ptr), _u32(col), _u32(node_wf), _f32(cost)
        N = node_wf.shape[0]
        cp = np.zeros(N, np.float32); tail = np.zeros(N, np.float32)
        H = np.zeros(n_workflows, np.float32)
        rc = self.lib.orc_longest_path(_ptr(row_ptr), _ptr(col), _ptr(cost), _ptr(node_wf),
                                       C.c_uint32(N), C.c_uint32(n_workflows),
                                       _ptr(cp), _ptr(tail), _ptr(H))
        if rc != 0:
            raise ValueError("graph has a cycle")
        return DagResult(cp, tail, H)

    def earliest_start(self, row_ptr, col, cost):
        """est, eft of every node (forward pass over the same DAG)."""
        row_ptr, col, cost = _u32(row_ptr), _u32(col), _f32(cost)
        N = cost.shape[0]
        est = np.zeros(N, np.float32); eft = np.zeros(N, np.float32)
        rc = self.lib.orc_earliest_start(_ptr(row_ptr), _ptr(col), _ptr(cost), C.c_uint32(N), _ptr(est), _ptr(eft))
        if rc != 0:
            raise ValueError("graph has a cycle")
        return est, eft

    # -- scoring ----------------------------------------------------------
    @staticmethod
    def _calls(calls):
        calls = np.ascontiguousarray(calls, dtype=CALL_DTYPE)
        return calls, calls.shape[0]

    @staticmethod
    def _dag(dag, node_wf, elapsed):
        if dag is None:
            return None, ()
        keep = (_u32(node_wf), _f32(dag.tail), _f32(dag.H), _f32(elapsed))
        return _Dag(*[_ptr(a) for a in keep]), keep

    def fin_all(self, cl: Cluster, calls, flags=0) -> np.ndarray:
        calls, n = self._calls(calls)
        out = np.zeros((n, cl.P, cl.D), np.float32)
        c = cl._c()
        self.lib.orc_fin_all(C.byref(c), _ptr(calls), n, flags, _ptr(out))
        return out

    def fin_all_f64(self, cl: Cluster, calls, flags=0) -> np.ndarray:
        calls, n = self._calls(calls)
        out = np.zeros((n, cl.P, cl.D), np.float64)
        c = cl._c()
        self.lib.orc_fin_all_f64(C.byref(c), _ptr(calls), n, flags, _ptr(out))
        return out

    def terms(self, cl: Cluster, calls):
        calls, n = self._calls(calls)
        tpre = np.zeros((n, cl.G), np.float32); tdec = np.zeros((n, cl.G), np.float32)
        kvB = np.zeros(n, np.float32); m = np.zeros(n, np.float32)
        c = cl._c()
        self.lib.orc_terms(C.byref(c), _ptr(calls), n, _ptr(tpre), _ptr(tdec), _ptr(kvB), _ptr(m))
        return tpre, tdec, kvB, m

    def schedule(self, cl: Cluster, calls, mode=MODE_COMPLETION, alpha=1.5, flags=0,
                 dag: DagResult | None = None, node_wf=None, elapsed=None):
        """Returns (assign i32[C], cost f32[C], delta f32[C])."""
        calls, n = self._calls(calls)
        assign = np.zeros(n, np.int32); cost = np.zeros(n, np.float32); delta = np.zeros(n, np.float32)
        c = cl._c()
        d, keep = self._dag(dag, node_wf, elapsed)
        if d is None:
            flags |= FLAG_NO_DAG
        self.lib.orc_schedule(C.byref(c), C.byref(d) if d is not None else None, _ptr(calls), n,
                              int(mode), C.c_float(alpha), int(flags),
                              _ptr(assign), _ptr(cost), _ptr(delta))
        return assign, cost, delta

    def topk(self, cl: Cluster, calls, K, flags=0, dag: DagResult | None = None, node_wf=None,
             elapsed=None):
        """Returns (pair i32[C,K], cost f32[C,K], prio f32[C], m f32[C], tpre_sel f32[C,K])."""
        calls, n = self._calls(calls)
        pair = np.zeros((n, K), np.int32); cost = np.zeros((n, K), np.float32)
        prio = np.zeros(n, np.float32); m = np.zeros(n, np.float32)
        tsel = np.zeros((n, K), np.float32)
        c = cl._c()
        d, keep = self._dag(dag, node_wf, elapsed)
        if d is None:
            flags |= FLAG_NO_DAG
        self.lib.orc_topk(C.byref(c), C.byref(d) if d is not None else None, _ptr(calls), n, int(K),
                          int(flags), _ptr(pair), _ptr(cost), _ptr(prio), _ptr(m), _ptr(tsel))
        return pair, cost, prio, m, tsel

    def conflict(self, pair, prio, m, tpre_sel, freeD, qP, D):
        """Sequential capacity pass; returns (assign i32[C], freeD', qP')."""
        pair = np.ascontiguousarray(pair, np.int32)
        n, K = pair.shape
        prio, m, tpre_sel = _f32(prio), _f32(m), _f32(tpre_sel)
        freeD = _f32(freeD).copy(); qP = _f32(qP).copy()
        assign = np.zeros(n, np.int32)
        self.lib.orc_conflict(n, K, int(D), _ptr(pair), _ptr(prio), _ptr(m), _ptr(tpre_sel),
                              _ptr(freeD), _ptr(qP), _ptr(assign))
        return assign, freeD, qP

    def greedy(self, cl: Cluster, calls, freeD, flags=0, dag: DagResult | None = None, node_wf=None,
               elapsed=None, with_delta=False):
        """Recomputing greedy of Algorithm 1 over one queue snapshot.
        Returns (assign i32[C], ratio f32[C], order i32[C], n_placed, qP', freeD'), plus delta f32[C] with
        with_delta."""
        calls, n = self._calls(calls)
        assign = np.zeros(n, np.int32); ratio = np.zeros(n, np.float32); order = np.zeros(n, np.int32)
        delta = np.zeros(n, np.float32)
        qP = _f32(cl.qP).copy(); free = _f32(freeD).copy()
        c = cl._c()
        d, keep = self._dag(dag, node_wf, elapsed)
        if d is None:
            flags |= FLAG_NO_DAG
        self.lib.orc_greedy.restype = C.c_int
        placed = self.lib.orc_greedy(C.byref(c), C.byref(d) if d is not None else None, _ptr(calls), n,
                                     int(flags), _ptr(qP), _ptr(free), _ptr(assign), _ptr(ratio), _ptr(order),
                                     _ptr(delta) if with_delta else None)
        if with_delta:
            return assign, ratio, order, int(placed), qP, free, delta
        return assign, ratio, order, int(placed), qP, free

    def decode_greedy(self, cl: Cluster, calls, run_ptr, run_end, run_tok, lock, ready, flags=0,
                      dag: DagResult | None = None, node_wf=None, elapsed=None, run_start=None):
        """Decode-stage greedy over capacity intervals (Section 5.4).
        Returns (inst i32[C], start f32[C], ratio f32[C], order i32[C], n_placed)."""
        calls, n = self._calls(calls)
        run_ptr = _u32(run_ptr); run_end = _f32(run_end); run_tok = _f32(run_tok)
        run_start = None if run_start is None else _f32(run_start)
        lock = np.ascontiguousarray(lock, np.int32); ready = _f32(ready)
        inst = np.zeros(n, np.int32); start = np.zeros(n, np.float32); ratio = np.zeros(n, np.float32)
        order = np.zeros(n, np.int32)
        c = cl._c()
        d, keep = self._dag(dag, node_wf, elapsed)
        if d is None:
            flags |= FLAG_NO_DAG
        self.lib.orc_decode_greedy.restype = C.c_int
        placed = self.lib.orc_decode_greedy(C.byref(c), C.byref(d) if d is not None else None, _ptr(calls), n,
                                            int(flags), _ptr(run_ptr), None if run_start is None else _ptr(run_start),
                                            _ptr(run_end), _ptr(run_tok), _ptr(lock),
                                            _ptr(ready), _ptr(inst), _ptr(start), _ptr(ratio), _ptr(order))
        return inst, start, ratio, order, int(placed)

    def decode_onepass(self, cl: Cluster, calls, run_ptr, run_end, run_tok, lock, ready, flags=0,
                       dag: DagResult | None = None, node_wf=None, elapsed=None, run_start=None):
        """Decode stage with the one-pass ordering (Section 5.4 fallback, Section 5.3 last sentence):
        ranked once against the snapshot, then placed in that order.  Returns as decode_greedy."""
        calls, n = self._calls(calls)
        run_ptr = _u32(run_ptr); run_end = _f32(run_end); run_tok = _f32(run_tok)
        run_start = None if run_start is None else _f32(run_start)
        lock = np.ascontiguousarray(lock, np.int32); ready = _f32(ready)
        inst = np.zeros(n, np.int32); start = np.zeros(n, np.float32); ratio = np.zeros(n, np.float32)
        order = np.zeros(n, np.int32)
        c = cl._c()
        d, keep = self._dag(dag, node_wf, elapsed)
        if d is None:
            flags |= FLAG_NO_DAG
        self.lib.orc_decode_onepass.restype = C.c_int
        placed = self.lib.orc_decode_onepass(C.byref(c), C.byref(d) if d is not None else None, _ptr(calls), n,
                                             int(flags), _ptr(run_ptr), None if run_start is None else _ptr(run_start),
                                             _ptr(run_end), _ptr(run_tok), _ptr(lock),
                                             _ptr(ready), _ptr(inst), _ptr(start), _ptr(ratio), _ptr(order))
        return inst, start, ratio, order, int(placed)
