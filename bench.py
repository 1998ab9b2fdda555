#!/usr/bin/env python
"""Benchmark of the placement-scoring hot path on the throughput-sweep workload.

One step = one pass of the whole path over the sweep configuration: horizon
kernels over the workflow forest, then 16 scheduler invocations of 16,384 ready
calls each against 128 x 128 instance pairs (scoring with top-4 lists,
capacity-conflict pass that starts from the restored free KV tokens, commit).  Prints one JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "placement candidates scored/sec"
UNIT = "candidates/s"
FP32_LANES_PER_SM = 128
ALGO_LANE_OPS_PER_CANDIDATE = 4      # fma, max, add, min of the per-candidate cost definition
EXEC_LANE_OPS_PER_CANDIDATE = 2      # what the candidate loop executes: fma and min
SCORE_DRAM_BYTES_PER_LAUNCH = 3262208   # ncu, one launch of 16,384 calls x 128 x 128 pairs with top-4 lists


def _peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f), "measured"
    except Exception:
        return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------
# CPU oracle legs (reference arm and cpu_baseline)
# ----------------------------------------------------------------------------------------------

def pin_to_one_core():
    """The oracle is single-threaded: keep it on one core of the host for the whole measurement.  Returns the
    core, or None where the platform has no affinity call."""
    try:
        core = sorted(os.sched_getaffinity(0))[0]
        os.sched_setaffinity(0, {core})
        return core
    except (AttributeError, OSError):
        return None


def unpin(cores):
    try:
        os.sched_setaffinity(0, cores)
    except (AttributeError, OSError):
        pass


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count()


def oracle_chunks(wl, n_chunks, with_dag):
    """Runs the oracle, as it stands, on the first n_chunks scheduler invocations of the
    workload; returns (candidates, seconds)."""
    from oracle import hx_oracle as ho
    orc = ho.Oracle()
    oc = ho.Cluster.from_workload(wl)
    calls = wl.calls
    dag = None
    t0 = time.perf_counter()
    if with_dag:
        # horizons from the stand-alone node costs of the workflows touched by these chunks
        from hx_synth import sub_forest
        touched = np.unique(wl.node_wf[wl.ready_nodes[: n_chunks * wl.chunk]])
        rp, col, lwf, ids = sub_forest(wl, touched)
        cost = orc.schedule(oc, wl.node_calls[ids], flags=ho.FLAG_UNLOADED | ho.FLAG_NO_DAG)[2]
        sub = orc.longest_path(rp, col, cost, lwf, touched.shape[0])
        tail = np.zeros(wl.n_nodes, np.float32); tail[ids] = sub.tail
        H = np.ones(wl.n_workflows, np.float32); H[touched] = sub.H
        dag = ho.DagResult(None, tail, H)
    free0 = wl.kv_free[wl.P:].copy()
    cand = 0
    for i in range(n_chunks):
        c = calls[i * wl.chunk:(i + 1) * wl.chunk]
        pair, cost, prio, m, tsel = orc.topk(oc, c, wl.topk, dag=dag, node_wf=wl.node_wf, elapsed=wl.elapsed)
        _, _, qP = orc.conflict(pair, prio, m, tsel, free0, oc.qP, wl.D)
        oc.qP[:] = qP
        cand += c.shape[0] * wl.P * wl.D
    return cand, time.perf_counter() - t0


def run_reference(args):
    from hx_synth import make_workload
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = make_workload("sweep")
    n_chunks = 1                      # bounded sample per step: 1 of the 16 invocations
    n_host = host_cores()
    core = pin_to_one_core()
    times = []
    for i in range(args.warmup + args.steps):
        cand, dt = oracle_chunks(wl, n_chunks, with_dag=False)
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * float(np.mean(times))
    value = cand / (ms * 1e-3)
    sample = "%d of 16 invocations (%d calls x 16384 pairs, top-4 + conflict pass) per step" % (
        n_chunks, n_chunks * wl.chunk)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "sweep: 128x128 instances, 262,144 ready calls in chunks of 16,384, top-4 + commit",
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "host_cores": n_host, "pinned_to_core": core,
                         "kind": "oracle", "sample": sample, "omits": "horizons (the scores use elapsed = 0, tail = 0, H = 1)"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ----------------------------------------------------------------------------------------------
# CUDA arm
# ----------------------------------------------------------------------------------------------

def rank_seed(rank):
    """Every rank schedules its own, differently seeded, sweep: the path has no exchange step."""
    return 4 + rank


def reduce_times(dist, total_ms, e2e_s, device="cuda"):
    """Device time and end-to-end time of the job = MAX over ranks."""
    import torch
    tot = torch.tensor([total_ms, e2e_s], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(tot, op=dist.ReduceOp.MAX)
    return float(tot[0]), float(tot[1])


def job_value(world, cand_per_step, ms_per_step):
    """Whole-job candidates per second: every rank processes cand_per_step per step."""
    return world * cand_per_step / (ms_per_step * 1e-3)


def run_cuda(args):
    import torch
    import paper_2605_16637_b200 as hx
    from hx_synth import make_workload

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    wl = make_workload("sweep", seed=rank_seed(rank))
    gc = hx.Cluster.from_workload(wl)
    P, D, chunk = wl.P, wl.D, wl.chunk
    n_calls = wl.ready_nodes.shape[0]
    n_chunks = n_calls // chunk
    cand_per_step = n_calls * P * D

    # stand-alone node costs come from the library itself (unloaded scoring of every node)
    gc.set_options(score_mode=hx.HX_MODE_COMPLETION, flags=hx.HX_FLAG_UNLOADED | hx.HX_FLAG_NO_DAG)
    node_cost = gc.schedule_batch(wl.node_calls)[1].cpu().numpy()
    gc.dag_upload(wl.row_ptr, wl.col, node_cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    gc.set_options(score_mode=hx.HX_MODE_RATIO, topk=wl.topk, commit=1, alpha=wl.alpha)

    calls_host = torch.from_numpy(wl.calls.view(np.uint8).reshape(-1, 16).copy()).pin_memory()
    calls_dev = calls_host.cuda()
    out_assign = torch.empty(n_calls, dtype=torch.int32, device="cuda")
    out_cost = torch.empty(n_calls, dtype=torch.float32, device="cuda")
    host_assign = torch.empty(n_calls, dtype=torch.int32).pin_memory()
    host_cost = torch.empty(n_calls, dtype=torch.float32).pin_memory()
    # refreshed loads come from pinned host memory (also what a captured copy needs)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a, np.float32).copy()).pin_memory().numpy()
    qP0, qD0, free0 = pin(wl.load_s[:P]), pin(wl.load_s[P:]), pin(wl.kv_free[P:])
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")      # larger than the 126 MB L2
    stream = torch.cuda.current_stream()
    sptr = stream.cuda_stream
    h = gc.h

    ptrs = [(calls_dev[i * chunk:(i + 1) * chunk].data_ptr(), out_assign[i * chunk:(i + 1) * chunk].data_ptr(),
             out_cost[i * chunk:(i + 1) * chunk].data_ptr()) for i in range(n_chunks)]

    def step_device(sp, strm=None, chunk_events=None):
        hx.hx_critical_path(h, sp)
        hx.hx_cluster_update_loads(h, qP0, qD0, free0, sp)
        # decode completions between two scheduler invocations: every capacity pass starts from free0 again
        hx.hx_set_kv_free_restore(h, free0, sp)
        for i in range(n_chunks):
            if chunk_events is not None:
                chunk_events[i][0].record(strm)
            hx.hx_schedule_batch(h, ptrs[i][0], chunk, ptrs[i][1], ptrs[i][2], sp)
            if chunk_events is not None:
                chunk_events[i][1].record(strm)

    ch_np = calls_host.numpy().view(hx.CALL_DTYPE).reshape(-1)
    ha_np, hc_np = host_assign.numpy(), host_cost.numpy()

    def step_host():
        hx.hx_critical_path(h, sptr)
        hx.hx_cluster_update_loads(h, qP0, qD0, free0, sptr)
        hx.hx_schedule_sweep_host(h, ch_np, chunk, free0, ha_np, hc_np, sptr)
        torch.cuda.current_stream().synchronize()        # results of all 16 batches are in host memory

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    launches0 = gc.launch_count()
    step_device(sptr)
    launches_per_step = gc.launch_count() - launches0
    for _ in range(max(args.warmup, 3) - 1):
        step_device(sptr)
    barrier()

    # One step = 16 scheduler invocations of three short kernels each: launch-bound.  The whole step is
    # captured once into a CUDA graph through the same C entry points and replayed (every pointer and
    # size is the same in every step); if the capture is refused the step is enqueued call by call.
    graph, mode = None, "eager"
    if not args.no_graph:
        try:
            cap = torch.cuda.Stream()
            cap.wait_stream(stream)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=cap):
                step_device(torch.cuda.current_stream().cuda_stream)
            stream.wait_stream(cap)
            g.replay(); g.replay()
            torch.cuda.synchronize()
            graph, mode = g, "cuda graph replay"
        except Exception as exc:                          # keep measuring, say why
            mode = "eager (capture refused: %s)" % str(exc).splitlines()[0][:80]
            torch.cuda.synchronize()
    barrier()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    for k in range(args.steps):
        flush.zero_()                                   # L2 flush between timed iterations (not timed)
        ev[k][0].record(stream)
        if graph is not None:
            graph.replay()
        else:
            step_device(sptr)
        ev[k][1].record(stream)
    barrier()
    launches = launches_per_step * args.steps
    step_ms = np.array([a.elapsed_time(b) for a, b in ev])
    status = gc.status()
    placed = (out_assign >= 0).view(n_chunks, chunk).sum(dim=1).cpu().numpy() / float(chunk)
    replay_ok = None
    if graph is not None:                               # a replayed step leaves the same placements as one enqueued call by call
        got_a, got_c = out_assign.clone(), out_cost.clone()
        step_device(sptr)
        torch.cuda.synchronize()
        replay_ok = bool(torch.equal(got_a, out_assign) and torch.equal(got_c, out_cost))

    # second timed region, call by call with event pairs around every kernel family and every ready
    # batch: per-kernel times (roofline of the scoring kernel, shares) and the ready-batch latency
    n_inst = min(args.steps, 10)
    gc.enable_kernel_timing(True)
    gc.read_kernel_timing()
    ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_inst)]
    cev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_chunks)]
           for _ in range(n_inst)]
    for k in range(n_inst):
        flush.zero_()
        ev2[k][0].record(stream)
        step_device(sptr, stream, cev[k])
        ev2[k][1].record(stream)
    barrier()
    kt = gc.read_kernel_timing()
    gc.enable_kernel_timing(False)
    inst_ms = float(np.sum([a.elapsed_time(b) for a, b in ev2]))
    chunk_us = np.array([[a.elapsed_time(b) * 1e3 for a, b in row] for row in cev]).reshape(-1)

    # end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    for _ in range(2):
        step_host()
    barrier()
    t0 = time.perf_counter()
    for k in range(args.steps):
        step_host()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    barrier()
    clocks = sampler.stop() if rank == 0 else None

    total_ms, e2e_s = reduce_times(dist, float(step_ms.sum()), e2e_s)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ms_per_step = total_ms / args.steps
    value = job_value(world, cand_per_step, ms_per_step)
    e2e_value = job_value(world, cand_per_step, e2e_s * 1e3 / args.steps)
    peaks, which = _peaks()
    n_sm = torch.cuda.get_device_properties(local).multi_processor_count
    sm_max_mhz = float(peaks.get("sm_max_mhz", 1965.0))
    # Roofline of the scoring kernel (bound: FP32 issue).  Algorithmic work per candidate = the four
    # FP32 lane-instructions of the cost definition (fused multiply-add, maximum, addition, running
    # minimum); like the peak, every lane-instruction is counted as 2 flop.  The kernel itself executes
    # only two of them per candidate (the maximum and the addition are taken once per (call, decode
    # instance) after the reduction over the prefill instances): frac_executed counts those two only.
    score_ms, score_n = kt["scoring"]
    score_avg_ms = score_ms / max(score_n, 1)
    lane_rate = chunk * P * D / (score_avg_ms * 1e-3)              # candidates per second of one launch
    peak = 2.0 * n_sm * FP32_LANES_PER_SM * sm_max_mhz * 1e6 / 1e12
    achieved = 2.0 * ALGO_LANE_OPS_PER_CANDIDATE * lane_rate / 1e12
    rates, rate_ms = hx.hx_measure_fp32_rates(h, sptr)             # register-only loops, each longer than a millisecond
    peak_measured = 2.0 * rates["fma"] / 1e12                      # every lane-instruction counted as 2 flop, like `peak`
    loop_ceiling = rates["mix"]                                    # the loop issues one instruction of the mix per candidate and lane
    roofline = {"bound": "alu", "kernel": "hx_score_kernel", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "peak_measured": peak_measured, "frac_of_peak_measured": achieved / peak_measured,
                "loop_ceiling_measured": loop_ceiling, "loop_ceiling_unit": "candidates/s",
                "frac_of_loop_ceiling": lane_rate / loop_ceiling,
                "lane_instr_per_s_measured": rates, "micro_kernel_ms": rate_ms,
                "measured_with": "hx_measure_fp32_rates: fma.rn.f32, fma.rn.f32x2, three-input min.f32 and their one-to-one "
                                 "mix in registers, CUDA events, during the clock sampling of this run",
                "frac": achieved / peak, "traffic": SCORE_DRAM_BYTES_PER_LAUNCH,
                "peak_source": "%d SMs x %d FP32 lanes x %.0f MHz x 2 flop (%s sm_max_mhz)" % (
                    n_sm, FP32_LANES_PER_SM, sm_max_mhz, which),
                "avg_launch_us": score_avg_ms * 1e3, "launches_timed": score_n,
                "lane_ops_per_candidate": ALGO_LANE_OPS_PER_CANDIDATE,
                "frac_executed": 2.0 * EXEC_LANE_OPS_PER_CANDIDATE * lane_rate / 1e12 / peak,
                "lane_ops_executed_per_candidate": EXEC_LANE_OPS_PER_CANDIDATE,
                "candidates_per_s_kernel": lane_rate,
                "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum, one launch, same workload",
                "time_share": {k: v[0] / max(inst_ms, 1e-9) for k, v in kt.items()},
                "timed_with": "%d steps enqueued call by call with event pairs around every kernel family" % n_inst}

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        n_b = 8
        n_host, all_cores = host_cores(), (os.sched_getaffinity(0) if hasattr(os, "sched_getaffinity") else None)
        core = pin_to_one_core()
        cand, dt = oracle_chunks(make_workload("sweep"), n_b, with_dag=False)
        if all_cores is not None:
            unpin(all_cores)
        cpu = {"value": cand / dt, "unit": UNIT, "cores": 1, "host_cores": n_host, "pinned_to_core": core, "kind": "oracle",
               "sample": "%d of 16 invocations (%d calls x 16384 pairs, top-4 + conflict pass), %.1f s" % (
                   n_b, n_b * chunk, dt),
               "omits": "horizons (the scores use elapsed = 0, tail = 0, H = 1; the oracle's pass over the whole "
                        "forest is timed in horizon_refinement.oracle_full_pass_ms_1_core)"}

    # side legs (oracle sample, greedy planner) are skipped together, e.g. under a profiler
    greedy = greedy_leg(with_cpu=True) if world == 1 and not args.no_cpu_baseline else None
    h2d = n_calls * 16 + (P + 2 * D) * 4 + n_chunks * D * 4
    d2h = n_calls * 8
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "sweep: %dx%d instances, %d ready calls in %d chunks of %d, top-%d lists + "
                               "capacity-conflict pass with commit, horizons over %d nodes / %d workflows" % (
                                   P, D, n_calls, n_chunks, chunk, wl.topk, wl.n_nodes, wl.n_workflows),
                   "candidates_per_step": cand_per_step, "l2": "flushed between timed steps (256 MB write)",
                   "seed": wl.seed, "score_mode": "ratio",
                   "forest": "%d workflows of 8-24 nodes (chains, fan-out/join stages, random layered DAGs), %d nodes, "
                             "%d edges" % (wl.n_workflows, wl.n_nodes, wl.n_edges)},
        "placed_fraction": {"per_invocation": [float(x) for x in placed], "mean": float(placed.mean()),
                            "what": "share of the 16,384 calls of each scheduler invocation that obtained a pair; the others "
                                    "found none of their four candidate decode instances with room"},
        "schedule_latency": {"batch_calls": chunk, "p50_us": float(np.percentile(chunk_us, 50)),
                             "p95_us": float(np.percentile(chunk_us, 95)),
                             "what": "hx_schedule_batch (scoring, top-4, conflict pass starting from the restored free KV "
                                     "tokens, commit) per ready batch, CUDA events"},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "what": "hx_schedule_sweep_host (all 16 chunks, copies on their own streams) from pinned host memory into "
                        "pinned host memory, one synchronisation per step, wall clock"},
        "gpu_launches": int(launches), "launch_mode": mode, "replay_matches_call_by_call": replay_ok,
        "ms_per_step_call_by_call_instrumented": inst_ms / n_inst,
        "kernel_ms_per_step": {k: v[0] / n_inst for k, v in kt.items()},
        "device_status": status, "roofline": roofline, "cpu_baseline": cpu, "clocks": clocks,
        "greedy_planner": greedy,
        "decode_scheduler": decode_leg() if world == 1 and not args.no_cpu_baseline else None,
        "horizon_refinement": refine_leg() if world == 1 and not args.no_cpu_baseline else None,
        "replay": replay_leg() if world == 1 and not args.no_cpu_baseline else None,
        "batch_robustness": robustness_leg() if world == 1 and not args.no_cpu_baseline else None,
    }
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def greedy_leg(with_cpu):
    """Side measurement, outside the timed region: the recomputing greedy planner (Algorithm 1,
    small queues) on the medium configuration, 4,096 ready calls x 16 x 16 pairs."""
    import torch
    import paper_2605_16637_b200 as hx
    from hx_synth import make_workload
    out = {}
    for label, scale in (("medium", 1.0), ("medium_quarter", 0.25)):
        wl = make_workload("medium", scale=scale)
        gc = hx.Cluster.from_workload(wl)
        gc.set_options(score_mode=hx.HX_MODE_COMPLETION, flags=hx.HX_FLAG_UNLOADED | hx.HX_FLAG_NO_DAG)
        cost = gc.schedule_batch(wl.node_calls)[1].cpu().numpy()
        gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
        gc.critical_path()
        gc.set_options(score_mode=hx.HX_MODE_RATIO, commit=0)
        calls = torch.from_numpy(wl.calls.view(np.uint8).reshape(-1, 16).copy()).cuda()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(5)]
        for _ in range(2):
            gc.schedule_greedy(calls)
        for a, b in ev:
            a.record(); res = gc.schedule_greedy(calls); b.record()
        torch.cuda.synchronize()
        ms = float(np.median([a.elapsed_time(b) for a, b in ev]))
        n = len(wl.calls)
        out[label] = {"calls": n, "pairs": wl.P * wl.D, "ms": ms, "placed": int((res[0] >= 0).sum().item()),
                      "us_per_iteration": 1e3 * ms / n}
        if with_cpu and label == "medium_quarter":
            from oracle import hx_oracle as ho
            orc, oc = ho.Oracle(), ho.Cluster.from_workload(wl)
            dag = orc.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
            t0 = time.perf_counter()
            orc.greedy(oc, wl.calls, wl.kv_free[wl.P:], dag=dag, node_wf=wl.node_wf, elapsed=wl.elapsed)
            out[label]["oracle_ms_1_core"] = 1e3 * (time.perf_counter() - t0)
        gc.close()
    return out


def decode_leg():
    """Side measurement, outside the timed region: the decode-stage scheduler (Section 5.4) on the decode
    pool of the medium configuration (16 instances), queue of 1,024 calls, four running calls per instance."""
    import paper_2605_16637_b200 as hx
    from hx_synth import make_decode_queue, make_workload
    from oracle import hx_oracle as ho
    wl = make_workload("medium")
    calls, lock, ready, ptr, end, tok = make_decode_queue(wl, 1024)
    gc = hx.Cluster.from_workload(wl)
    gc.set_options(score_mode=hx.HX_MODE_RATIO, flags=hx.HX_FLAG_NO_DAG, commit=0)
    gc.decode_set_running(ptr, end, tok)
    times = []
    for i in range(6):
        t0 = time.perf_counter()
        res = gc.schedule_decode(calls, lock, ready)         # synchronises
        times.append(time.perf_counter() - t0)
    orc, oc = ho.Oracle(), ho.Cluster.from_workload(wl)
    t0 = time.perf_counter()
    want = orc.decode_greedy(oc, calls, ptr, end, tok, lock, ready)
    cpu_ms = 1e3 * (time.perf_counter() - t0)
    same = bool(np.array_equal(res[0].cpu().numpy(), want[0]) and np.array_equal(res[3].cpu().numpy(), want[3]))
    gc.close()
    return {"calls": 1024, "decode_instances": wl.D, "ms_wall_incl_copies": 1e3 * float(np.median(times[1:])),
            "oracle_ms_1_core": cpu_ms, "identical_to_oracle": same}


def refine_leg():
    """Side measurement, outside the timed region: online refinement of the horizons on the forest of the
    sweep (Section 5.1).  Wall clock per call including host work and a synchronisation, median of 5;
    the oracle's full pass on one core beside it."""
    import torch
    import paper_2605_16637_b200 as hx
    from hx_synth import make_workload
    from oracle import hx_oracle as ho
    wl = make_workload("sweep")
    rng = np.random.default_rng(5)
    cost = rng.lognormal(0, 1, wl.n_nodes).astype(np.float32)
    gc = hx.Cluster.from_workload(wl)

    def wall(fn, reps=5):
        ts = []
        for _ in range(reps):
            torch.cuda.synchronize(); t0 = time.perf_counter(); fn(); torch.cuda.synchronize()
            ts.append(time.perf_counter() - t0)
        return 1e3 * float(np.median(ts))

    out = {"nodes": wl.n_nodes, "workflows": wl.n_workflows}
    out["upload_ms"] = wall(lambda: gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed), reps=3)
    out["full_pass_ms"] = wall(gc.critical_path)
    k = 1000
    ids = rng.choice(wl.n_nodes, k, replace=False).astype(np.uint32)
    out["update_1000_costs_ms"] = wall(lambda: gc.update_costs(ids, (cost[ids] * rng.uniform(0.5, 2, k)).astype(np.float32)))
    def forward():
        gc.earliest_start()
    out["forward_pass_first_ms"] = wall(forward, reps=1)
    out["forward_pass_ms"] = wall(forward)
    # 1,000 newly revealed nodes, one behind a random node of each of 1,000 workflows
    order = np.argsort(wl.node_wf, kind="stable")
    first_of = order[np.searchsorted(wl.node_wf[order], np.arange(wl.n_workflows))].astype(np.uint32)
    batches = []
    for i in range(5):
        wfs = rng.choice(wl.n_workflows, k, replace=False).astype(np.uint32)
        new = np.arange(wl.n_nodes + i * k, wl.n_nodes + (i + 1) * k, dtype=np.uint32)
        batches.append((rng.lognormal(0, 1, k).astype(np.float32), wfs, first_of[wfs], new))
    out["append_1000_nodes_ms"] = wall(lambda: gc.dag_append(*batches.pop(0)))
    # 1,000 arriving workflows (Section 5.2, first trigger): registered, then their two source calls each handed in
    state = {"n": wl.n_nodes + 5 * k, "w": wl.n_workflows}
    def arrive():
        gc.dag_append_workflows(np.zeros(k, np.float32))
        wfs = np.repeat(np.arange(state["w"], state["w"] + k, dtype=np.uint32), 2)
        gc.dag_append(rng.lognormal(0, 1, 2 * k).astype(np.float32), wfs, [], [])
        state["n"] += 2 * k; state["w"] += k
    out["arrival_1000_workflows_ms"] = wall(arrive)
    orc = ho.Oracle()
    t0 = time.perf_counter()
    orc.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
    out["oracle_full_pass_ms_1_core"] = 1e3 * (time.perf_counter() - t0)
    out["device_status"] = gc.status()
    gc.close()
    return out


def robustness_leg():
    """Side measurement, outside the timed region: one ready batch of the sweep (16,384 calls, top-4, capacity pass)
    as generated, with a tenth of the calls fitting no decode instance (priority +inf), and with a fifth of the calls
    exact duplicates of one another (equal priorities share a bin of the visiting order and are ranked against each
    other there).  CUDA events around hx_schedule_batch, median of 20."""
    import torch
    import paper_2605_16637_b200 as hx
    from hx_synth import make_workload
    wl = make_workload("sweep")
    gc = hx.Cluster.from_workload(wl)
    gc.set_options(score_mode=hx.HX_MODE_RATIO, topk=wl.topk, commit=0, flags=hx.HX_FLAG_NO_DAG)
    rng = np.random.default_rng(8)
    base = wl.calls[:wl.chunk].copy()
    infeasible = base.copy(); infeasible["prompt_tokens"][rng.random(wl.chunk) < 0.1] = 2.0e6
    dup = base.copy(); m = rng.random(wl.chunk) < 0.2
    dup["model"][m] = 0; dup["prompt_tokens"][m] = 777; dup["output_tokens"][m] = 33
    out = {}
    stream = torch.cuda.current_stream()
    for label, calls in (("as_generated", base), ("tenth_infeasible", infeasible), ("fifth_duplicates", dup)):
        dev = torch.from_numpy(calls.view(np.uint8).reshape(-1, 16).copy()).cuda()
        a = torch.empty(wl.chunk, dtype=torch.int32, device="cuda"); c = torch.empty(wl.chunk, dtype=torch.float32, device="cuda")
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
        for _ in range(3):
            hx.hx_schedule_batch(gc.h, dev.data_ptr(), wl.chunk, a.data_ptr(), c.data_ptr(), stream.cuda_stream)
        for e0, e1 in ev:
            e0.record(stream)
            hx.hx_schedule_batch(gc.h, dev.data_ptr(), wl.chunk, a.data_ptr(), c.data_ptr(), stream.cuda_stream)
            e1.record(stream)
        torch.cuda.synchronize()
        out[label] = {"batch_us": 1e3 * float(np.median([e0.elapsed_time(e1) for e0, e1 in ev])),
                      "placed": int((a >= 0).sum().item())}
    out["device_status"] = gc.status()
    gc.close()
    return out


LOADS = (4.0, 32.0, 256.0)       # offered stand-alone work per second and prefill instance (replay leg)


def replay_leg():
    """Side measurement, outside the timed region: the event-driven replay (Section 6, Section 7.3) of the
    medium configuration (512 workflows, 16 x 16 instances) at three offered loads; Req95 / Req99 and wall
    clock, and the oracle's replay of the middle load on one core beside it."""
    import paper_2605_16637_b200 as hx
    from hx_synth import make_workload
    from oracle import hx_oracle as ho
    from oracle import hx_replay as hr
    wl = make_workload("medium")
    gc = hx.Cluster.from_workload(wl)
    gc.set_options(score_mode=hx.HX_MODE_COMPLETION, flags=hx.HX_FLAG_UNLOADED | hx.HX_FLAG_NO_DAG)
    cost = gc.schedule_batch(wl.node_calls)[1].cpu().numpy()
    gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
    gc.critical_path()
    gc.set_options(score_mode=hx.HX_MODE_RATIO)
    out = {"workflows": wl.n_workflows, "calls": wl.n_nodes, "pairs": wl.P * wl.D, "loads": {}}
    rng = np.random.default_rng(6)
    u = np.sort(rng.uniform(0, 1, wl.n_workflows))
    for load in LOADS:
        arrival = u * float(cost.sum()) / (wl.P * load)
        t0 = time.perf_counter()
        r = gc.replay(wl.row_ptr, wl.col, wl.node_wf, wl.node_calls, arrival)
        dt = time.perf_counter() - t0
        out["loads"]["%.1f" % load] = {"req95": r["req95"], "req99": r["req99"], "planner_runs": r["runs"],
                                       "unplanned": r["stuck"], "wall_ms": 1e3 * dt,
                                       "us_per_planner_run": 1e6 * dt / max(r["runs"], 1)}
        if load == LOADS[1]:
            orc, oc = ho.Oracle(), ho.Cluster.from_workload(wl)
            dag = orc.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
            t0 = time.perf_counter()
            w = hr.replay(orc, oc, wl.row_ptr, wl.col, wl.node_wf, wl.n_workflows, wl.node_calls, arrival, dag)
            out["oracle_wall_ms_1_core_middle_load"] = 1e3 * (time.perf_counter() - t0)
            out["identical_to_oracle"] = bool(np.array_equal(r["fin"], w["fin"]) and r["req99"] == w["req99"])
    # the stages of a call kept apart, the decode stage scheduled, estimation error on what the schedulers see
    # (Section 7.6): Req95 / Req99 at four error levels on the heaviest of the loads above
    arrival = u * float(cost.sum()) / (wl.P * LOADS[-1])
    life = {}
    for eps in (0.0, 0.1, 0.2, 0.3):
        t0 = time.perf_counter()
        r = gc.replay_lifecycle(wl.node_calls, arrival, est_error=eps)
        dt = time.perf_counter() - t0
        life["%.1f" % eps] = {"req95": r["req95"], "req99": r["req99"], "prefill_planner_runs": r["runs"],
                              "decode_planner_runs": r["decode_runs"], "unplanned": r["stuck"], "wall_ms": 1e3 * dt,
                              "us_per_planner_run": 1e6 * dt / max(r["runs"] + r["decode_runs"], 1)}
    orc, oc = ho.Oracle(), ho.Cluster.from_workload(wl)
    dag = orc.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
    t0 = time.perf_counter()
    w = hr.replay_lifecycle(orc, oc, wl.row_ptr, wl.col, wl.node_wf, wl.n_workflows, wl.node_calls, arrival, dag, est_error=0.2)
    out["lifecycle"] = {"load": LOADS[-1], "est_error": life, "oracle_wall_ms_1_core_error_0.2": 1e3 * (time.perf_counter() - t0),
                        "identical_to_oracle_error_0.2": bool(np.array_equal(
                            gc.replay_lifecycle(wl.node_calls, arrival, est_error=0.2)["fin"], w["fin"]))}
    out["device_status"] = gc.status()
    gc.close()
    return out


def run_configs(args):
    """`--configs`: ready-batch schedule latency and horizon time on the four smaller configurations
    (the default run times the sweep).  Prints one JSON object; plain argmin, slack score, whole batch in
    one hx_schedule_batch call; CUDA events per call plus host wall clock enqueue -> synchronise."""
    import torch
    import paper_2605_16637_b200 as hx
    from hx_synth import make_workload
    from oracle import hx_oracle as ho
    torch.cuda.set_device(0)
    out = {}
    reps, warm = 200, 20
    for name in ("tiny", "medium", "large", "cp_stress"):
        wl = make_workload(name)
        gc = hx.Cluster.from_workload(wl)
        if wl.node_cost is not None:
            cost = np.asarray(wl.node_cost, np.float32)
        else:
            gc.set_options(score_mode=hx.HX_MODE_COMPLETION, flags=hx.HX_FLAG_UNLOADED | hx.HX_FLAG_NO_DAG)
            cost = gc.schedule_batch(wl.node_calls)[1].cpu().numpy()
        gc.dag_upload(wl.row_ptr, wl.col, cost, wl.node_wf, wl.elapsed)
        gc.critical_path()
        gc.set_options(score_mode=hx.HX_MODE_SLACK, alpha=wl.alpha)
        calls = torch.from_numpy(wl.calls.view(np.uint8).reshape(-1, 16).copy()).cuda()
        n = len(wl.calls)
        a = torch.empty(n, dtype=torch.int32, device="cuda"); c = torch.empty(n, dtype=torch.float32, device="cuda")
        stream = torch.cuda.current_stream(); sp = stream.cuda_stream
        def timed(fn):
            for _ in range(warm):
                fn()
            torch.cuda.synchronize()
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
            wall = []
            for e0, e1 in ev:
                t0 = time.perf_counter()
                e0.record(stream); fn(); e1.record(stream)
                stream.synchronize()
                wall.append(1e6 * (time.perf_counter() - t0))
            us = np.array([1e3 * e0.elapsed_time(e1) for e0, e1 in ev])
            return {"p50_us": float(np.percentile(us, 50)), "p95_us": float(np.percentile(us, 95)),
                    "wall_p50_us": float(np.percentile(wall, 50))}
        sched = timed(lambda: hx.hx_schedule_batch(gc.h, calls.data_ptr(), n, a.data_ptr(), c.data_ptr(), sp))
        cpath = timed(lambda: hx.hx_critical_path(gc.h, sp))
        cand = n * wl.P * wl.D
        m = min(n, 4096)                                   # bounded oracle sample
        orc, oc = ho.Oracle(), ho.Cluster.from_workload(wl)
        t0 = time.perf_counter()
        dag = orc.longest_path(wl.row_ptr, wl.col, cost, wl.node_wf, wl.n_workflows)
        t_dag = time.perf_counter() - t0
        t0 = time.perf_counter()
        orc.schedule(oc, wl.calls[:m], mode=ho.MODE_SLACK, alpha=wl.alpha, dag=dag, node_wf=wl.node_wf, elapsed=wl.elapsed)
        t_or = time.perf_counter() - t0
        out[name] = {"instances": "%dx%d" % (wl.P, wl.D), "calls": n, "candidates": cand, "nodes": int(wl.n_nodes),
                     "workflows": int(wl.n_workflows), "schedule_batch": sched,
                     "candidates_per_s": cand / (sched["p50_us"] * 1e-6), "critical_path": cpath,
                     "nodes_per_s": wl.n_nodes / (cpath["p50_us"] * 1e-6),
                     "oracle": {"schedule_candidates_per_s_1_core": m * wl.P * wl.D / t_or, "sample_calls": m,
                                "longest_path_ms_1_core": 1e3 * t_dag}}
        gc.close()
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true",
                    help="skip the side legs outside the timed region (oracle sample, greedy planner)")
    ap.add_argument("--no-graph", action="store_true", help="enqueue every step call by call instead of replaying a CUDA graph")
    ap.add_argument("--configs", action="store_true",
                    help="time the four smaller configurations instead (one JSON object)")
    args = ap.parse_args()
    if args.configs:
        run_configs(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
