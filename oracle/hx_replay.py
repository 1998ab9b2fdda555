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


# ----------------------------------------------------------------------------------------------
# Replay with the stages of a call's life kept apart, the decode stage scheduled, and
# scheduler-visible estimates that may differ from the service a call really gets.
# ----------------------------------------------------------------------------------------------

TINY_S = 1e-6          # estimated time left of a call that runs longer than its estimate


def error_sign(v):
    """Deterministic sign of the estimation error of call v: +1 or -1 from a multiplicative hash of the
    node number (the robustness study injects a deterministic multiplicative error, Section 7.6)."""
    return 1 if ((int(v) * 2654435761) >> 31) & 1 else -1


def error_factors(eps):
    """binary32 factors (1 + eps), (1 - eps) applied to the model constants the scheduler sees."""
    return np.float32(1.0 + eps), np.float32(1.0 - eps)


def replay_lifecycle(orc, cl, row_ptr, col, node_wf, n_workflows, node_calls, arrival, dag, est_error=0.0,
                     qmax=4096, dmax=2048):
    """Event-driven replay in which every call goes through waiting for prefill, prefill, KV transfer,
    waiting for decode, decode and completion (Section 6), the prefill stage is planned by the recomputing
    greedy of Algorithm 1 and the decode stage by the decode-stage greedy of Section 5.4 with the planned
    decode instance as the lock, and the durations the schedulers see are the real ones times (1 + eps s_c),
    s_c = +-1 per call (Section 7.6: the error is injected into the scheduler-visible estimates, the service
    durations are unchanged).  The paper prints no pseudo-code of its simulator: the rules are this
    project's reading (PARITY UNPINNED against the paper; pinned as defined by
    tests/test_oracle_replay_pins.py).

    What really happens
      * prefill instance p serves the calls planned onto it one at a time, in the order they were planned;
        call c takes tpre(c, class of p);
      * the KV cache then travels for kvB(c) / link(p, d) and the call waits at its decode instance d;
      * d admits waiting calls whenever a plan, an arrival or a completion changed its state: in the order of the
        latest decode plan (calls of equal rank by node number), every waiting call whose m = L_in + L_out
        tokens (Eq. 3) fit the tokens really free is started; it holds them for tdec(c, class of d);
      * a call completes with its decode; successors whose predecessors are all complete become ready.
    What the schedulers see (all service times from the same latency model with the model constants of the
    call scaled by the binary32 factor 1 + eps s_c)
      * prefill queue of p: estimated time left of the call in service (at least 0) plus the estimated prefill
        times of the calls queued behind it; free KV tokens of d: Cap(d) minus the tokens of every call
        planned onto d and not complete; decode hint 0; elapsed time t - a_w;
      * decode snapshot of d: every call decoding there, until its estimated end (at least TINY_S from now).
    Scheduler invocations: the prefill planner at every event time at which calls are ready (increasing node
    number, at most qmax per run, run after run); the decode planner at every event time at which a KV
    transfer completed, over all calls waiting for decode (increasing node number, the first dmax of them),
    without commit.  Events with equal time stamps are taken together, in the order (kind, number).
    Time is binary64; service times are the binary32 values of the latency model.

    Returns dict(fin, ratio, req95, req99, runs, decode_runs, stuck, pair, planned, prefill_start, decode_start)."""
    row_ptr = np.asarray(row_ptr, np.int64); col = np.asarray(col, np.int64)
    node_wf = np.asarray(node_wf, np.uint32)
    N, W, P, D, M = node_wf.shape[0], int(n_workflows), cl.P, cl.D, cl.M
    arrival = np.asarray(arrival, np.float64)
    # the cluster as the schedulers see it: every model once more with its constants scaled up and scaled down
    fp, fm = error_factors(est_error)
    base = np.stack([cl.phi, cl.omega, cl.kappa], 1).astype(np.float32)
    ext = np.concatenate([base, base * fp, base * fm]).astype(np.float32)
    seen_calls = np.array(node_calls, copy=True)
    sign = np.array([error_sign(v) for v in range(N)])
    seen_calls["model"] = node_calls["model"] + np.where(sign > 0, M, 2 * M).astype(np.uint32)

    def cluster(qP):
        c = ho.Cluster(np.stack([cl.tflops, cl.tbps], 1), cl.typeP, cl.typeD, qP, np.zeros(D, np.float32), cl.capD,
                       cl.link, ext)
        if cl.psi is not None:
            c.set_attention(np.concatenate([cl.psi, cl.psi * fp, cl.psi * fm]).astype(np.float32))
        return c

    idle = cluster(np.zeros(P, np.float32))
    tpre, tdec, kvB, m_tok = orc.terms(idle, node_calls)            # what really happens
    tpre_s, tdec_s, _, _ = orc.terms(idle, seen_calls)              # what the schedulers believe
    inv_link = (np.float32(1.0) / (cl.link.astype(np.float32) * np.float32(1e9))).astype(np.float32)

    left = np.bincount(col, minlength=N).astype(np.int64)
    is_source = left == 0
    fin = np.full(N, np.inf); pair = np.full(N, -1, np.int64); dstart = np.full(N, np.inf)
    pstart = np.full(N, np.inf); planned = np.full(N, np.inf)
    queue = [[] for _ in range(P)]                                   # planned, prefill not started
    serving = [None] * P                                             # (call, start) in prefill service
    waiting = [[] for _ in range(D)]                                 # KV arrived, decode not started
    running = [dict() for _ in range(D)]                             # call -> decode start
    free_act = cl.capD.astype(np.float64).copy()                     # tokens really free
    reserved = np.zeros(D)                                           # tokens of calls planned and not complete
    dprio = np.full(N, np.inf)                                       # rank in the latest decode plan
    events = [(float(arrival[w]), 0, w) for w in range(W)]           # kinds: 0 arrival, 1 prefill done, 2 transfer done, 3 decode done
    heapq.heapify(events)
    ready = set()
    runs = decode_runs = 0
    while events:
        t = events[0][0]
        arrived = False
        while events and events[0][0] == t:
            _, kind, x = heapq.heappop(events)
            if kind == 0:
                ready.update(int(v) for v in np.flatnonzero((node_wf == x) & is_source))
            elif kind == 1:
                p, d = divmod(int(pair[x]), D)
                serving[p] = None
                heapq.heappush(events, (t + float(np.float32(kvB[x] * inv_link[p, d])), 2, x))
            elif kind == 2:
                waiting[int(pair[x]) % D].append(x)
                arrived = True
            else:
                d = int(pair[x]) % D
                del running[d][x]
                free_act[d] += float(m_tok[x]); reserved[d] -= float(m_tok[x])
                fin[x] = t
                for u in col[row_ptr[x]:row_ptr[x + 1]]:
                    left[u] -= 1
                    if left[u] == 0:
                        ready.add(int(u))
        elapsed = np.maximum(0.0, t - arrival).astype(np.float32)
        # prefill stage
        offered = sorted(ready)
        for s in range(0, len(offered), qmax):
            chunk = np.array(offered[s:s + qmax], np.int64)
            qP = np.zeros(P)
            for p in range(P):
                if serving[p] is not None:
                    c, st = serving[p]
                    qP[p] = max(0.0, st + float(tpre_s[c, cl.typeP[p]]) - t)
                for c in queue[p]:
                    qP[p] += float(tpre_s[c, cl.typeP[p]])
            free = (cl.capD.astype(np.float64) - reserved).astype(np.float32)
            a, _, order, placed, _, _ = orc.greedy(cluster(qP.astype(np.float32)), seen_calls[chunk], free, dag=dag,
                                                   node_wf=node_wf, elapsed=elapsed)
            runs += 1
            for i in order[:placed]:
                v = int(chunk[i]); p, d = divmod(int(a[i]), D)
                pair[v] = int(a[i]); queue[p].append(v); reserved[d] += float(m_tok[v]); ready.discard(v)
                planned[v] = t
        # decode stage
        if arrived:
            wait_all = sorted(v for d in range(D) for v in waiting[d])[:dmax]
            ptr, end, tok = [0], [], []
            for d in range(D):
                for c, st in sorted(running[d].items()):
                    end.append(max(st + float(tdec_s[c, cl.typeD[d]]) - t, TINY_S)); tok.append(float(m_tok[c]))
                ptr.append(len(end))
            idx = np.array(wait_all, np.int64)
            lock = (pair[idx] % D).astype(np.int32)
            _, _, _, dorder, dplaced = orc.decode_greedy(cluster(np.zeros(P, np.float32)), seen_calls[idx],
                                                         np.array(ptr, np.uint32), np.array(end, np.float32),
                                                         np.array(tok, np.float32), lock, np.zeros(len(idx), np.float32),
                                                         dag=dag, node_wf=node_wf, elapsed=elapsed)
            decode_runs += 1
            for v in wait_all:
                dprio[v] = np.inf
            for r, i in enumerate(dorder[:dplaced]):
                dprio[wait_all[i]] = r
        for d in range(D):
            waiting[d].sort(key=lambda v: (dprio[v], v))
            still = []
            for v in waiting[d]:
                if float(m_tok[v]) <= free_act[d]:
                    free_act[d] -= float(m_tok[v]); running[d][v] = t; dstart[v] = t
                    heapq.heappush(events, (t + float(tdec[v, cl.typeD[d]]), 3, v))
                else:
                    still.append(v)
            waiting[d] = still
        for p in range(P):
            if serving[p] is None and queue[p]:
                c = queue[p].pop(0)
                serving[p] = (c, t); pstart[c] = t
                heapq.heappush(events, (t + float(tpre[c, cl.typeP[p]]), 1, c))
    C = np.full(W, -np.inf)
    np.maximum.at(C, node_wf, fin)
    ratio = (C - arrival) / dag.H.astype(np.float64)
    return dict(fin=fin, ratio=ratio, req95=req(ratio, 0.95), req99=req(ratio, 0.99), runs=runs,
                decode_runs=decode_runs, stuck=len(ready), pair=pair, decode_start=dstart,
                prefill_start=pstart, planned=planned)
