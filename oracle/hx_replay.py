"""Minimal event-driven replay around the oracle's greedy planner.

TEST INFRASTRUCTURE ONLY: the plain definition that the library's replay is checked
against.  It shares no code with the CUDA path and is never called from it.

What it models (Section 6, the stand-alone simulator; Section 7.3, Req95 / Req99):
workflows arrive over time, a call becomes ready when all its predecessors have
completed (Section 4.1), and at every event time the scheduler plans all ready
calls with the recomputing greedy of Algorithm 1 (projected ratio of Eq. 2) against
the state of the cluster at that time.  The life of a call -- waiting for prefill,
prefill, KV transfer, waiting for decode, decode, completion -- is the sequence of
terms inside its projected completion Delta, and the replay takes the planner's
projection as what happens: the call completes Delta after it was planned.  A
workflow completes with its last call; its ratio is completion time over stand-alone
horizon H_w, and Req95 / Req99 are the smallest SLO scales that 95 % / 99 % of the
workflows meet.

The paper prints no pseudo-code of its simulator, so the rules below are this
project's reading (PARITY UNPINNED against the paper; pinned as defined by
tests/test_oracle_replay_pins.py):
  * time is binary64 on the host; whatever the planner sees is rounded to binary32;
  * events: arrival of a workflow (its source calls become ready) and completion of a
    call (successors whose predecessors are all complete become ready); all events with
    the same time stamp are taken together, then the scheduler runs once;
  * state shown to the planner at time t: prefill queue qP[p] = max(0, busy_p - t);
    free KV tokens of decode instance d = Cap(d) - tokens of the calls planned onto d
    that have not completed by t (a call holds m = L_in + L_out tokens, Eq. 3, from the
    moment it is planned until it completes); decode availability hint qD = 0; elapsed
    time of workflow w = t - a_w;
  * ready calls are offered in increasing node number, at most `qmax` per planner run,
    run after run until every ready call has been offered once; a call the planner
    passes over (no KV room anywhere) stays ready for the next event;
  * a planned call completes at t + Delta; the prefill instance it was given is busy
    until t + (its simulated queue after the run).
"""
import heapq
import math

import numpy as np

from . import hx_oracle as ho


def replay(orc, cl, row_ptr, col, node_wf, n_workflows, node_calls, arrival, dag, qmax=4096):
    """cl: ho.Cluster (its qP/qD are ignored: the replay starts idle).  node_calls: one CALL_DTYPE
    record per node (record v describes node v).  arrival: seconds, one per workflow.  dag: the
    stand-alone horizons (ho.DagResult).  Returns dict(fin f64[N], planned f64[N] (when the call was
    planned), pair i64[N], ratio f64[W], req95, req99, runs, stuck)."""
    row_ptr = np.asarray(row_ptr, np.int64); col = np.asarray(col, np.int64)
    node_wf = np.asarray(node_wf, np.uint32)
    N, W, P, D = node_wf.shape[0], int(n_workflows), cl.P, cl.D
    arrival = np.asarray(arrival, np.float64)
    left = np.bincount(col, minlength=N).astype(np.int64)          # predecessors not complete yet
    is_source = left == 0
    fin = np.full(N, np.inf)
    planned = np.full(N, np.inf); pair = np.full(N, -1, np.int64)
    busy = np.zeros(P)                                               # prefill instance p is busy until busy[p]
    holds = []                                                       # (completion time, decode instance, tokens)
    events = [(float(arrival[w]), 0, w) for w in range(W)]
    heapq.heapify(events)
    ready = set()
    m_tok = (node_calls["prompt_tokens"].astype(np.float32) + node_calls["output_tokens"].astype(np.float32))
    runs = 0
    while events:
        t = events[0][0]
        while events and events[0][0] == t:
            _, kind, x = heapq.heappop(events)
            if kind == 0:
                ready.update(int(v) for v in np.flatnonzero((node_wf == x) & is_source))
            else:
                for u in col[row_ptr[x]:row_ptr[x + 1]]:
                    left[u] -= 1
                    if left[u] == 0:
                        ready.add(int(u))
        offered = sorted(ready)
        for s in range(0, len(offered), qmax):
            chunk = np.array(offered[s:s + qmax], np.int64)
            qP = np.maximum(0.0, busy - t).astype(np.float32)
            used = np.zeros(D)
            for end, d, tok in holds:
                if end > t:
                    used[d] += tok
            free = (cl.capD.astype(np.float64) - used).astype(np.float32)
            elapsed = np.maximum(0.0, t - arrival).astype(np.float32)
            now = ho.Cluster(np.stack([cl.tflops, cl.tbps], 1), cl.typeP, cl.typeD, qP, np.zeros(D, np.float32),
                             cl.capD, cl.link, np.stack([cl.phi, cl.omega, cl.kappa], 1))
            if cl.psi is not None:
                now.set_attention(cl.psi)
            a, _, _, placed, qP2, _, delta = orc.greedy(now, node_calls[chunk], free, dag=dag, node_wf=node_wf,
                                                         elapsed=elapsed, with_delta=True)
            runs += 1
            touched = set()
            for i in np.flatnonzero(a >= 0):
                v = int(chunk[i]); p, d = divmod(int(a[i]), D)
                fin[v] = t + float(delta[i])
                planned[v] = t; pair[v] = int(a[i])
                heapq.heappush(events, (fin[v], 1, v))
                holds.append((fin[v], d, float(m_tok[v])))
                ready.discard(v)
                touched.add(p)
            for p in touched:
                busy[p] = t + float(qP2[p])
        holds = [h for h in holds if h[0] > t]
    C = np.full(W, -np.inf)
    np.maximum.at(C, node_wf, fin)
    ratio = (C - arrival) / dag.H.astype(np.float64)
    return dict(fin=fin, planned=planned, pair=pair, ratio=ratio, req95=req(ratio, 0.95), req99=req(ratio, 0.99), runs=runs, stuck=len(ready))


def req(ratio, q):
    """Smallest SLO scale alpha such that at least a fraction q of the workflows has ratio <= alpha."""
    r = np.sort(np.asarray(ratio, np.float64))
    return float(r[max(0, math.ceil(q * r.shape[0]) - 1)])
