/* hx.h - C ABI of the batched placement-scoring library for workflow-aware
 * scheduling on heterogeneous prefill/decode (P-D) disaggregated clusters.
 *
 * The library evaluates, on one CUDA device, every ready LLM call against every
 * (prefill instance, decode instance) pair of the cluster and picks, per call,
 * the pair with the earliest projected decode finish (paper Section 5.3); it
 * also computes the workflow horizons H_w(t) (Section 5.1) that turn a finish
 * time into the projected ratio of Eq. 2.
 *
 * Conventions
 *   - Every function returns HX_OK (0) or a negative HX_ERR_* code and never
 *     throws or aborts; hx_last_error() gives a message for the last failure.
 *   - "host" pointers are ordinary CPU memory, read or written during the call
 *     and not retained.  "device" pointers are CUDA global memory of the device
 *     that was current when the handle was created; buffers passed as device
 *     pointers stay owned by the caller and must stay alive until the work
 *     enqueued on `stream` has finished.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Unless stated otherwise a call only enqueues work and returns.
 *   - All quantities are IEEE binary32.  Times are seconds, token counts are
 *     integer-valued floats below 2^24, bandwidths and rates use decimal units.
 *   - A handle is not thread-safe; use one handle per host thread or lock.
 */
#ifndef HX_H_
#define HX_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HX_OK                0
#define HX_ERR_INVALID_ARG  (-1)   /* bad size, id out of range, non-finite or non-positive rate ... */
#define HX_ERR_CUDA         (-2)   /* a CUDA runtime call failed; message holds cudaGetErrorString */
#define HX_ERR_CYCLE        (-3)   /* the uploaded graph is not acyclic */
#define HX_ERR_NOT_READY    (-4)   /* scoring needs horizons but hx_critical_path was not enqueued */
#define HX_ERR_TIMEOUT      (-5)   /* reserved for a bounded device-side wait that runs out; no entry point of
                                      this version waits on the device, so the code is never returned */
#define HX_ERR_OOM          (-6)   /* host or device allocation failed */

/* out_cost of hx_schedule_batch (Delta = earliest projected decode finish of the call) */
#define HX_MODE_COMPLETION   0     /* (elapsed_w + Delta) + tail(node): projected workflow completion */
#define HX_MODE_SLACK        1     /* alpha * H_w - completion: slack against the scaled SLO (Eq. 1) */
#define HX_MODE_RATIO        2     /* completion / H_w; with HX_FLAG_NO_TAIL this is Eq. 2 as printed */

#define HX_FLAG_NO_DAG       1     /* ignore the DAG: elapsed = 0, tail = 0, H = 1 */
#define HX_FLAG_NO_TAIL      2     /* drop the remaining-critical-path term from the score */
#define HX_FLAG_UNLOADED     4     /* score against an idle cluster (all queue loads zero) */
#define HX_FLAG_ONE_PASS     8     /* hx_schedule_decode only: rank the queue once instead of after every assignment */

#define HX_MAX_TYPES        32     /* GPU classes */
#define HX_MAX_MODELS       32
#define HX_MAX_PREFILL    4096     /* prefill instances */
#define HX_MAX_DECODE      512     /* decode instances */
#define HX_MAX_TOPK          8
#define HX_MAX_COMMIT_CALLS 65536  /* largest batch the capacity-conflict pass accepts */

typedef struct hx_cluster hx_cluster;   /* opaque; owns every packed device table */

/* One GPU class ("instance type"): peak dense compute in TFLOP/s and memory
 * bandwidth in TB/s of one model instance (tensor parallelism folded in).
 * Inputs of the roofline-style latency estimate of Section 4.2. */
typedef struct { float peak_tflops, hbm_tbps; } hx_gpu_type;

/* One model instance of the P-D cluster (Section 4.2, "Heterogeneous resource
 * modelling").  role 0 = prefill (single-server queue), 1 = decode (batched,
 * KV-capacity bound).  load_s: seconds until a prefill instance has drained
 * its queue, or earliest time a decode instance can admit a new call.
 * kv_cap_tokens is Cap(d) of Eq. 4, kv_free_tokens the part of it not in use
 * (both ignored for prefill instances; whole numbers in [0, 2^24) for decode
 * instances, HX_ERR_INVALID_ARG otherwise). */
typedef struct {
    uint32_t type;
    uint32_t role;
    float load_s;
    float kv_cap_tokens;
    float kv_free_tokens;
} hx_instance;

/* Served model: forward FLOPs per token, bytes of weights read per pass, KV
 * bytes per token. */
typedef struct { float flops_per_token, weight_bytes, kv_bytes_per_token; } hx_model;

/* One ready LLM call (Section 7.1: calls carry input length, output length and
 * workflow identity).  node indexes the uploaded DAG (ignored with
 * HX_FLAG_NO_DAG), output_tokens is the predicted output length of Eq. 3.
 * 16 bytes, read with one 128-bit load. */
typedef struct { uint32_t node, model; float prompt_tokens, output_tokens; } hx_call;

typedef struct {
    int score_mode;   /* HX_MODE_* */
    int topk;         /* 0: plain argmin.  1..HX_MAX_TOPK: also build the top-K list and run the
                         capacity-conflict pass over the batch */
    int commit;       /* with topk > 0: write the loads consumed by the pass back into the cluster */
    int flags;        /* HX_FLAG_* */
    float alpha;      /* SLO scale of Eq. 1, used by HX_MODE_SLACK */
} hx_options;

/* Cluster-state packing (State Collector snapshot, Section 4.2 and 4.3).
 * instances: all prefill instances first, then all decode instances.
 * link_bw_gbps: host, n_instances x n_instances row-major, effective KV-transfer
 * bandwidth in GB/s from instance i to instance j; only [prefill][decode]
 * entries are read.  The tables are converted to reciprocal rates and packed
 * as structure-of-arrays binary32 on the device; the link table is stored
 * transposed, every row padded to a 16-byte boundary.
 * Errors: HX_ERR_INVALID_ARG for sizes out of range, ids out of range,
 * non-finite values, rates or bandwidths <= 0, negative loads, a prefill
 * instance listed after a decode instance, or a pool that is empty;
 * HX_ERR_OOM / HX_ERR_CUDA for allocation failures.  *out is set on success. */
int hx_cluster_create(const hx_gpu_type* gpu_types, int n_types,
                      const hx_instance* instances, int n_instances,
                      const float* link_bw_gbps,
                      const hx_model* models, int n_models,
                      hx_cluster** out);

/* Replace queue loads and free KV tokens (State Collector refresh between
 * scheduler invocations).  Each pointer is host memory or NULL (= keep):
 * qP[n_prefill], qD[n_decode], kv_free[n_decode] (finite and >= 0; kv_free
 * whole numbers below 2^24; HX_ERR_INVALID_ARG otherwise, nothing changed).
 * The copies are enqueued on `stream`; the host arrays may be reused when the
 * call returns. */
int hx_cluster_update_loads(hx_cluster* h, const float* qP, const float* qD,
                            const float* kv_free, void* stream);

/* Capacity restored between scheduler invocations (decode completions free KV
 * tokens while the scheduler is not looking): with kv_free != NULL (host,
 * n_decode whole numbers below 2^24) every capacity-conflict pass from now on
 * starts from these free KV tokens instead of the table's, exactly as if
 * hx_cluster_update_loads(h, NULL, NULL, kv_free) had been enqueued ahead of
 * every batch, but without a copy between the kernels of successive batches;
 * the table is set to the same values at once, and a committing pass still
 * writes what it leaves into the table.  NULL switches this off (enqueues
 * nothing).  Only batches with topk > 0 read free KV tokens.  The copies are
 * enqueued on `stream`; the host array may be reused when the call returns.
 * HX_ERR_INVALID_ARG for a bad value, nothing changed. */
int hx_set_kv_free_restore(hx_cluster* h, const float* kv_free, void* stream);

/* Read the current loads back (after commits).  Synchronises `stream`. */
int hx_cluster_read_loads(hx_cluster* h, float* qP, float* qD, float* kv_free, void* stream);

int hx_cluster_destroy(hx_cluster* h);

/* Upload the revealed workflow forest (Section 4.1) in successor-CSR form:
 * row_ptr[n_nodes+1], col_idx[n_edges], one cost per node in seconds, the
 * workflow of every node, and the elapsed time (t - a_w) of every workflow.
 * All arrays are host memory.  The graph is validated (monotone row_ptr,
 * columns in range, edges inside one workflow, finite non-negative costs,
 * acyclic) and levelised on the host; nodes are regrouped workflow by workflow
 * and by height for the device pass.  Synchronous.  Errors: HX_ERR_INVALID_ARG,
 * HX_ERR_CYCLE, HX_ERR_OOM, HX_ERR_CUDA.  Replaces any earlier upload. */
int hx_dag_upload(hx_cluster* h, const uint32_t* row_ptr, const uint32_t* col_idx,
                  const float* node_costs, const uint32_t* node_workflow,
                  const float* workflow_elapsed_s,
                  uint32_t n_nodes, uint32_t n_edges, uint32_t n_workflows);

/* Workflow horizons (Section 5.1, "Define online workflow horizon"; Algorithm 1,
 * horizon update): for every node cp = cost + tail, tail = max over successors
 * of cp (0 for sinks); H[w] = max over the workflow's nodes of cp.  Each sum
 * runs from the sink towards the source, so results do not depend on the
 * traversal order.  Enqueues on `stream`; independent groups of workflows may
 * run on side streams owned by the handle that fork from `stream` and join it
 * again with events before the call returns, so later work on `stream` sees
 * the results. */
int hx_critical_path(hx_cluster* h, void* stream);

/* Online horizon refinement (Section 5.1, "Define online workflow horizon": the
 * horizon is kept up to date as the workflow proceeds and cost estimates are
 * replaced by observed latencies; Algorithm 1, horizon update).
 * hx_dag_update_costs replaces the cost of n_updates nodes (host arrays: node
 * ids in the numbering of the upload, new costs in seconds; if a node is listed
 * more than once its last value counts) and recomputes cp, tail and H of the
 * workflows these nodes belong to, and of no other; the result equals a full
 * hx_critical_path over the updated costs bit for bit.  If hx_critical_path has
 * not run since the upload, only the costs are replaced.  The host arrays may
 * be reused on return; the work is enqueued on `stream`.  The first call (and
 * a call larger than any before) allocates scratch for the update lists and
 * synchronises the device while doing so.  Errors: HX_ERR_NOT_READY without an
 * upload, HX_ERR_INVALID_ARG for ids out of range or costs that are negative
 * or not finite (nothing is changed then).
 * hx_dag_update_elapsed replaces the elapsed time (t - a_w) of every workflow
 * (host array of n_workflows values), which Eq. 2 needs afresh at every
 * scheduler invocation; the structure and the horizons stay as they are. */
int hx_dag_update_costs(hx_cluster* h, const uint32_t* node_ids, const float* new_costs,
                        uint32_t n_updates, void* stream);
int hx_dag_update_elapsed(hx_cluster* h, const float* workflow_elapsed_s, void* stream);

/* Borrowed device pointers to cp[n_nodes], tail[n_nodes] (original node
 * numbering) and H[n_workflows]; valid until the next upload or destroy.
 * Any of the three output arguments may be NULL. */
int hx_get_dag_results(hx_cluster* h, const float** cp, const float** tail, const float** H);

/* Appends newly revealed nodes and edges to the uploaded forest (Section 5.1:
 * the horizon is refined as the workflow reveals more of its DAG).  The new
 * nodes take the numbers n_nodes .. n_nodes + n_new_nodes - 1 (n_nodes = the
 * count before the call); new_costs[i] and new_node_workflow[i] (an existing
 * workflow, possibly one registered by hx_dag_append_workflows) describe node
 * n_nodes + i.  Edge e runs from edge_src[e] to
 * edge_dst[e]; either end may be an old or a new node of the same workflow.
 * All arrays are host arrays, read before the call returns.  The workflows
 * touched are levelised again as a group of their own and, once horizons
 * exist, recomputed on `stream`; all other workflows keep their results
 * untouched, and the outcome equals a fresh upload of the grown graph followed
 * by hx_critical_path, bit for bit.  The call allocates device memory for the
 * regrouped workflows; when the node arrays outgrow their reserve (a quarter
 * of the uploaded size) they are reallocated, which synchronises the device
 * and moves the arrays: fetch hx_get_dag_results again after an append.  The
 * forward results are dropped; call hx_earliest_start again.
 * Errors, all leaving the forest as it was: HX_ERR_NOT_READY without an
 * upload; HX_ERR_INVALID_ARG for a NULL array, a workflow or endpoint out of
 * range, an edge across workflows, a cost that is negative or not finite;
 * HX_ERR_CYCLE when the new edges close a cycle. */
int hx_dag_append(hx_cluster* h, uint32_t n_new_nodes, const float* new_costs,
                  const uint32_t* new_node_workflow, uint32_t n_new_edges,
                  const uint32_t* edge_src, const uint32_t* edge_dst, void* stream);

/* Arrival of workflows (Section 5.2: the scheduler runs "when a workflow arrives
 * and reveals source calls"; Section 4.3: only the source calls are revealed on
 * arrival).  Registers n_new_workflows workflows numbered n_workflows ..
 * n_workflows + n_new_workflows - 1 (n_workflows = the count before the call)
 * with the elapsed times new_elapsed_s (host, or NULL = all 0) and no node yet:
 * their horizon is 0 until hx_dag_append hands in their first (source) calls,
 * which then costs what any append costs and leaves every other workflow
 * untouched.  The result equals a fresh upload of the grown forest bit for bit.
 * The horizon and elapsed-time arrays keep a reserve (a quarter of the uploaded
 * count, at least 4,096); beyond it they are reallocated, which synchronises the
 * device and moves them: fetch hx_get_dag_results again.  The forward results
 * are dropped; call hx_earliest_start again.  Later hx_dag_update_elapsed calls
 * pass one value per workflow of the grown count.  Errors (nothing changed):
 * HX_ERR_NOT_READY without an upload, HX_ERR_INVALID_ARG for an elapsed time
 * that is negative or not finite. */
int hx_dag_append_workflows(hx_cluster* h, uint32_t n_new_workflows, const float* new_elapsed_s,
                            void* stream);

/* Forward pass over the same forest (Section 4.1: a node becomes ready when
 * all its predecessors have completed): for every node v
 *   est[v] = max over predecessors u of eft[u]      (0 for a source)
 *   eft[v] = est[v] + cost[v]
 * the earliest start and finish of v measured from the start of its workflow
 * when every node takes its stand-alone cost; est[v] + cp[v] is the longest
 * path through v, so H_w - (est[v] + cp[v]) is the slack of v.  Binary32, one
 * rounded add per node, max exact.  The first call after an upload builds the
 * transposed forest on the host (O(N + E)), allocates and synchronises the
 * device; later calls only enqueue on `stream`.  hx_dag_update_costs keeps the
 * forward results current once this has been called.  Scheduling does not
 * read them.  Errors: HX_ERR_NOT_READY without an upload.
 * hx_get_earliest_results: borrowed device pointers est[n_nodes],
 * eft[n_nodes] (original node numbering), valid until the next upload or
 * destroy; either argument may be NULL. */
int hx_earliest_start(hx_cluster* h, void* stream);
int hx_get_earliest_results(hx_cluster* h, const float** est, const float** eft);

/* Prefill variant with a quadratic attention term (the roofline-style estimate of
 * Section 4.2 leaves the shape of the compute term open): with per_model[m] =
 * attention FLOPs per pair of prompt tokens of model m, the compute time of a
 * prefill becomes (n * flops_per_token + n * n * per_model[m]) / peak instead of
 * n * flops_per_token / peak.  per_model: host, n_models values, finite and
 * >= 0; all zero (the state after hx_cluster_create) is the linear model bit for
 * bit.  Takes effect for every later scoring, greedy and stand-alone-cost call. */
int hx_set_attention_flops(hx_cluster* h, const float* per_model);

/* Validates and stores the options used by later hx_schedule_batch calls. */
int hx_set_options(hx_cluster* h, const hx_options* opts);

/* Batched placement scoring (Algorithm 1, inner loop over the waiting calls;
 * Section 5.3 "Projected-risk prefill ranking" and "Joint prefill-decode
 * planning"; feasibility by Eq. 3-4).  calls: device, n_calls records, 16-byte
 * aligned.  out_assign: device int32[n_calls], pair index p * n_decode + d of
 * the pair with the earliest projected decode finish (lowest index among
 * equals), or -1 if no decode instance can hold the call.  out_cost: device
 * float[n_calls], the score selected by hx_options.score_mode.  With topk > 0
 * the call also fills the top-K list (see hx_get_topk) and runs the
 * capacity-conflict pass (one-pass ordering by the same risk score for large
 * queues, Section 5.3 last sentence, with Eq. 4 as the capacity constraint):
 * out_assign then holds the pair each call obtained, or -1 if none of its K
 * candidates had room.  The first call with topk > 0, or with a larger batch
 * than before, allocates the buffers of that pass (and synchronises the
 * device while doing so).  Needs hx_critical_path to have been enqueued since
 * the last upload unless HX_FLAG_NO_DAG is set (else HX_ERR_NOT_READY).
 * A call record whose model or node id is out of range gets assignment -1,
 * cost +inf, and raises HX_ERR_INVALID_ARG in the status word; with topk > 0
 * the same happens to a record whose prompt or output length is negative, not
 * a whole number, or sums to 2^24 or more (the capacity pass takes its decisions
 * on integer token counts).
 * n_calls = 0 is a no-op.  Enqueues on `stream`; does not synchronise. */
int hx_schedule_batch(hx_cluster* h, const hx_call* calls, int n_calls,
                      int32_t* out_assign, float* out_cost, void* stream);

/* Same operation with host buffers: copies the calls to the device, runs the
 * kernels, copies both results back and synchronises `stream`. */
int hx_schedule_batch_host(hx_cluster* h, const hx_call* calls, int n_calls,
                           int32_t* out_assign, float* out_cost, void* stream);

/* The same without the final synchronisation: the copies and kernels are only
 * enqueued on `stream`, and out_assign / out_cost hold the results once the
 * stream has reached the end of this call's work.  For successive ready batches
 * whose loads depend on one another (the commits of one batch are the snapshot
 * of the next) this lets the caller enqueue all of them and synchronise once.
 * calls, out_assign and out_cost must be page-locked host memory and stay alive
 * and untouched until then; the device staging buffers are shared by all calls
 * on the handle, so use one stream per handle. */
int hx_schedule_batch_host_async(hx_cluster* h, const hx_call* calls, int n_calls,
                                 int32_t* out_assign, float* out_cost, void* stream);

/* A whole sweep of successive ready batches from host buffers: the n_calls
 * records are handled in chunks of chunk_calls (the last one may be shorter),
 * in order, each chunk exactly as hx_schedule_batch_host_async would handle it
 * (the commits of a chunk are the snapshot of the next).  When kv_free_reset is
 * not NULL (host, n_decode values) the free KV tokens of the decode instances
 * are set to it ahead of every chunk (decode completions between two scheduler
 * invocations), as hx_cluster_update_loads(h, NULL, NULL, kv_free_reset) would
 * (done through hx_set_kv_free_restore, which is switched off again on return).
 * Unlike a loop over the per-chunk call, the records of all chunks go up on a
 * copy stream of the handle ahead of the kernels, and the results of a chunk
 * come down on a second copy stream while the next chunk is being scored; the
 * caller's `stream` carries the kernels, waits for what was on it before, and
 * ends after the last copy, so one synchronisation of `stream` covers
 * everything.  calls, out_assign, out_cost (and kv_free_reset) should be
 * page-locked for the copies to overlap, and must stay alive and untouched until
 * then.  Device staging grows to n_calls records (a synchronising allocation the
 * first time).  Errors: those of hx_schedule_batch; HX_ERR_INVALID_ARG for
 * chunk_calls < 1 or, with topk > 0, > HX_MAX_COMMIT_CALLS. */
int hx_schedule_sweep_host(hx_cluster* h, const hx_call* calls, int n_calls, int chunk_calls,
                           const float* kv_free_reset, int32_t* out_assign, float* out_cost,
                           void* stream);

/* hx_schedule_batch for callers that must not allocate.  (The paper has no
 * counterpart: this entry point exists only because of how the library is
 * embedded.)  hx_schedule_batch with topk > 0 obtains its intermediate buffers
 * with cudaMalloc on first use and whenever a batch is larger than any before.
 * Some hosts of this library cannot tolerate that: a serving process whose
 * memory pool already owns the whole device, so that a late cudaMalloc fails;
 * a latency-critical scheduling thread for which the device-wide
 * synchronisation of an allocation is a stall; code running where the CUDA
 * allocator may not be entered at all.  This variant computes the same
 * results but keeps the top-K lists, the visiting order and the bookkeeping of
 * the capacity pass in one fixed array of about 2.0 MB that is part of the
 * library image; every device that loads the library holds that array until
 * the process exits.  It calls no allocating routine.
 *   Limits: n_calls <= HX_STATIC_MAX_CALLS when topk > 0, topk <=
 * HX_STATIC_MAX_TOPK; beyond them it returns HX_ERR_INVALID_ARG with a message
 * naming the limit (with topk = 0 no intermediate buffer is needed and any
 * batch size is accepted).  Inputs, outputs, options, stream semantics and
 * error codes are those of hx_schedule_batch; hx_get_topk does not see this
 * call's lists.
 *   Set-up: the first call on a device looks up the array's device address
 * (once per device, under a lock); the first call with a given option set also
 * makes the CUDA runtime load the kernels it launches and raise their
 * shared-memory limit, which may allocate inside the driver.  Make one warm-up
 * call per option set before the phase in which nothing may allocate, and
 * before starting any stream capture.  (With kernel timing enabled the call
 * also creates CUDA events the first few times; leave timing off there.)
 *   Sharing: all handles and all calls on a device use the same array, which
 * keeps whatever the previous call left; every call rewrites all it reads, so
 * nothing needs clearing, but two calls that overlap on the GPU (different
 * streams, or different handles) race on it.  Serialise them. */
#define HX_STATIC_MAX_CALLS 16384
#define HX_STATIC_MAX_TOPK      4
int hx_schedule_batch_static(hx_cluster* h, const hx_call* calls, int n_calls,
                             int32_t* out_assign, float* out_cost, void* stream);

/* Recomputing greedy planner for small queues (Algorithm 1, the while-loop over
 * the queue snapshot; Section 5.3 "Adaptive greedy prefill assignment"): until
 * the queue is empty, every waiting call's best feasible pair, its Delta and its
 * ratio R = (elapsed_w + Delta) / H_w (Eq. 2) are projected against the simulated
 * state; the call with the largest R is taken (lower call index among equals),
 * its pair is recorded, its prefill time is added to the chosen prefill queue
 * and its m(c) = L_in + L_out tokens (Eq. 3) are taken from the free KV tokens of
 * the chosen decode instance; then it leaves the queue.  A pair is feasible when
 * m(c) <= Cap(d) (Eq. 4) and m(c) fits the free KV tokens the simulated state has
 * left on d.  A call that fits nowhere is passed over; the loop ends when no
 * waiting call fits anywhere.
 *   calls: device, n_calls records, 16-byte aligned, 1 <= n_calls <=
 * HX_GREEDY_MAX_CALLS and small enough for the whole state to fit the shared
 * memory of one SM (HX_ERR_INVALID_ARG otherwise).  out_assign: device
 * int32[n_calls], pair p * n_decode + d or -1.  out_ratio: device
 * float[n_calls], R at the moment the call was taken, +inf if never taken.
 * out_order: device int32[n_calls], out_order[i] = call taken in iteration i,
 * -1 after the last one.  Uses hx_options.flags (HX_FLAG_NO_DAG: elapsed = 0,
 * H = 1; HX_FLAG_UNLOADED is rejected) and hx_options.commit (write the
 * simulated queues and free KV tokens back into the cluster).  Needs
 * hx_critical_path unless HX_FLAG_NO_DAG is set.  Invalid model or node ids:
 * as for hx_schedule_batch.  Enqueues one kernel on `stream`. */
#define HX_GREEDY_MAX_CALLS 4096
int hx_schedule_greedy(hx_cluster* h, const hx_call* calls, int n_calls,
                       int32_t* out_assign, float* out_ratio, int32_t* out_order, void* stream);

/* hx_schedule_greedy with one more output: out_delta, device float[n_calls], the
 * projected completion Delta (seconds from now) of each call on the pair it was
 * given, i.e. the Delta inside its ratio (Eq. 2), projected against the
 * simulated state at the moment the call was taken; +inf if never taken.  May
 * be NULL, which makes the call hx_schedule_greedy. */
int hx_schedule_greedy_plan(hx_cluster* h, const hx_call* calls, int n_calls,
                            int32_t* out_assign, float* out_ratio, int32_t* out_order,
                            float* out_delta, void* stream);

/* Minimal event-driven replay around the greedy planner (Section 6: the
 * stand-alone simulator tracks every call from waiting for prefill to
 * completion; Section 7.3: Req95 / Req99).  Workflows arrive at arrival_s[w]; a
 * call becomes ready when all its predecessors have completed (Section 4.1); at
 * every event time (an arrival or a completion; equal time stamps are taken
 * together) all ready calls are planned by hx_schedule_greedy_plan in ratio mode
 * against the state of the cluster at that time, at most qmax calls per run in
 * increasing node number, run after run until every ready call was offered once.
 * State shown to the planner at time t: prefill queue max(0, busy_p - t), free KV
 * tokens Cap(d) minus the tokens (Eq. 3) of the calls planned onto d and not yet
 * complete, decode hint 0, elapsed time t - a_w.  The planner's projection is
 * taken as what happens: a planned call completes Delta after t and its prefill
 * instance is busy until t + (simulated queue after the run); the six stages of
 * a call's life are the terms inside Delta.  A call the planner passes over
 * stays ready until the next event.  Time is binary64 on the host and rounded to
 * binary32 for the planner.  The paper prints no pseudo-code of its simulator:
 * these rules are this library's reading.
 *   The forest must have been uploaded with the same row_ptr / col_idx /
 * node_workflow (host arrays, given again here) and hx_critical_path enqueued;
 * node_calls[v] (host, n_nodes records) describes node v.  Outputs (host):
 * out_fin[n_nodes] completion time of every call (+inf if never planned),
 * out_ratio[n_workflows] = (completion of the last call - arrival) / H_w,
 * out_req[2] = Req95, Req99 (the smallest scale alpha such that at least 95 % /
 * 99 % of the workflows have ratio <= alpha), out_stats[2] = planner runs, calls
 * left unplanned.  The call overwrites the cluster's loads and elapsed times,
 * uses `stream`, synchronises it once per planner run, allocates and frees its
 * device scratch, and restores hx_options on return.  Errors:
 * HX_ERR_INVALID_ARG (NULL array, qmax outside 1 .. HX_GREEDY_MAX_CALLS, a graph
 * that differs from the uploaded one in size, row bounds, successors or workflow
 * of a node, node_calls[v].node != v, a negative or non-finite arrival),
 * HX_ERR_NOT_READY without horizons, and those of the calls it makes. */
int hx_replay(hx_cluster* h, const uint32_t* row_ptr, const uint32_t* col_idx,
              const uint32_t* node_workflow, uint32_t n_nodes, uint32_t n_workflows,
              const hx_call* node_calls, const double* arrival_s, int qmax,
              double* out_fin, double* out_ratio, double* out_req, int* out_stats,
              void* stream);

/* The same replay with the stages of a call's life kept apart, the decode stage
 * scheduled, and scheduler-visible estimates that may be wrong (Section 6: the
 * simulator follows every call through waiting for prefill, prefill, KV transfer,
 * waiting for decode, decode and completion and keeps decode token-capacity
 * intervals; Section 5.2: the schedulers run when work enters a stage; Section 5.4:
 * decode scheduling with the planned instance as a lock; Section 7.6: a
 * deterministic multiplicative error on the prefill and decode estimates the
 * scheduler sees, the service durations unchanged).
 *   What happens: prefill instance p serves the calls planned onto it one at a
 * time in the order they were planned, each for its prefill time on p's class;
 * the KV cache then travels for kv_bytes / link(p, d); at its decode instance d
 * the call waits until d admits it: whenever a plan, an arrival or a completion
 * changed d's state, the waiting calls are taken in the order of the latest
 * decode plan (node number among calls of equal rank) and every one whose tokens
 * (Eq. 3) fit the tokens really free starts decoding and holds them for its
 * decode time on d's class; a call completes with its decode.
 *   What the schedulers see: all service times from the same latency model with
 * the constants of the call's model scaled by the binary32 factor 1 + est_error
 * or 1 - est_error (the sign is a fixed function of the node number); prefill
 * queue = estimated time left of the call in service (at least 0) plus the
 * estimated prefill times queued behind it; free KV tokens = Cap(d) minus the
 * tokens of every call planned onto d and not complete; decode hint 0; elapsed
 * time t - a_w; decode snapshot = every call decoding on d until its estimated
 * end (at least 1e-6 s from now).
 *   Scheduler runs: hx_schedule_greedy_plan at every event time at which calls are
 * ready (increasing node number, at most qmax per run, run after run; a call
 * passed over stays ready); hx_schedule_decode, without commit, at every event
 * time at which a KV transfer completed, over the calls waiting for decode
 * (increasing node number, the first HX_DECODE_MAX_CALLS of them).  Events with
 * equal time stamps are taken together.  Time is binary64 on the host, service
 * times are the binary32 values of hx_estimate_calls.  The paper prints no
 * pseudo-code of its simulator: these rules are this library's reading.
 *   The replay runs on the uploaded forest (including appended nodes) with
 * hx_critical_path enqueued; node_calls[v] (host) describes node v; arrival_s
 * (host) has one entry per workflow.  Outputs (host): out_fin[n_nodes],
 * out_ratio[n_workflows], out_req[2] = Req95, Req99 (Section 7.3), out_stats[3] =
 * prefill planner runs, decode planner runs, calls never planned.  The call
 * overwrites the cluster's loads, elapsed times and decode snapshot, uses
 * `stream` and synchronises it once per planner run, allocates and frees its
 * scratch, needs three times the cluster's models to fit HX_MAX_MODELS, and
 * restores hx_options on return.  Errors: HX_ERR_INVALID_ARG (NULL array, qmax
 * outside 1 .. HX_GREEDY_MAX_CALLS, est_error outside [0, 1), node_calls[v].node
 * != v, a model id out of range, a bad arrival time, too many models),
 * HX_ERR_NOT_READY without forest or horizons, and those of the calls it makes. */
int hx_replay_lifecycle(hx_cluster* h, const hx_call* node_calls, const double* arrival_s,
                        double est_error, int qmax, double* out_fin, double* out_ratio,
                        double* out_req, int* out_stats, void* stream);

/* Service-time estimates of n_calls call records (the Estimator of Section 4.2,
 * "Scheduler internals": prefill time, decode time, KV-transfer volume and decode
 * memory demand from input and output length with a roofline-style model), the
 * terms the scoring and planning kernels build their projections from.  calls:
 * device, 16-byte aligned.  Outputs, device: out_tpre and out_tdec
 * float[n_calls][n_types] (seconds on each GPU class), out_kv_bytes
 * float[n_calls] (bytes of the prompt's KV cache: the transfer takes this over the
 * link bandwidth), out_tokens float[n_calls] (m of Eq. 3).  A record with a model id
 * out of range gets +inf times and raises HX_ERR_INVALID_ARG in the status word.
 * Enqueues one kernel on `stream`. */
int hx_estimate_calls(hx_cluster* h, const hx_call* calls, int n_calls, float* out_tpre,
                      float* out_tdec, float* out_kv_bytes, float* out_tokens, void* stream);

/* Decode-stage scheduler (Section 5.4, "Decode scheduling with instance locks",
 * "Decode KV-capacity feasibility check", "Adaptive greedy decode assignment").
 * State: the decode token-capacity intervals of every decode instance
 * (Section 6), i.e. which calls hold how many KV tokens until when.
 *
 * hx_decode_set_running loads the snapshot: inst_ptr[n_decode + 1] (host, CSR
 * offsets into `running`) and one hx_kv_interval per call that is decoding now
 * (end_s: seconds from now until it finishes, finite and > 0; tokens: the KV
 * tokens it holds, a whole number; the tokens in use on one instance must stay
 * below 2^24).  An instance may have no running call.  Enqueues copies on
 * `stream`; the host arrays may be reused on return; may (re)allocate, which
 * synchronises the device.
 *
 * hx_schedule_decode plans the queue of calls whose KV cache is (or will be) on
 * the decode side.  calls: device, n_calls records (1..HX_DECODE_MAX_CALLS).
 * lock: device int32[n_calls] or NULL: -1 = free call, else the decode instance
 * the call was planned on during prefill scheduling (it cannot migrate).
 * ready_s: device float[n_calls] or NULL (= 0): time from now at which the
 * call's KV cache is on the decode side.  Until the queue is empty the most
 * urgent waiting call (largest R = (elapsed_w + Delta_D) / H_w, Eq. 2; lower index
 * among equals) is assigned: on every legal instance (its lock, or every
 * instance with m(c) <= Cap(d), Eq. 3-4) the earliest start >= ready_s is found
 * at which m(c) tokens are free for the whole decode time of the call on that
 * instance's GPU class; Delta_D is the earliest finish over those instances
 * (lower instance index among equals); the interval is added to the simulated
 * state.  out_inst: device int32[n_calls], decode instance or -1 (the call
 * exceeds Cap of every legal instance).  out_start: planned decode start.
 * out_ratio: R when taken (+inf if never).  out_order: out_order[i] = call
 * taken in iteration i, -1 after the last.  With hx_options.commit the simulated
 * intervals become the snapshot of the next call; otherwise the snapshot is
 * left as it was.  Uses HX_FLAG_NO_DAG like hx_schedule_batch.
 *   HX_FLAG_ONE_PASS selects the lightweight ordering that Section 5.4 falls back
 * to for large or special-case queues (Section 5.3, last sentence): every call
 * is scored once, R with Delta_D projected against the snapshot alone, the calls
 * are visited by decreasing score (lower index among equals), and a visited call
 * takes the instance with the earliest finish in the state that the calls
 * before it have left.  out_ratio is then the score the call was ordered by.
 * The other entry points ignore the flag.  Errors:
 * HX_ERR_NOT_READY without a snapshot or horizons; HX_ERR_INVALID_ARG for sizes
 * out of range; a record with an id out of range, a lock >= n_decode or a
 * ready time that is negative or not finite is left unassigned and raises
 * HX_ERR_INVALID_ARG in the status word.  Enqueues one kernel on `stream`. */
typedef struct { float end_s; float tokens; } hx_kv_interval;
#define HX_DECODE_MAX_CALLS 2048
int hx_decode_set_running(hx_cluster* h, const uint32_t* inst_ptr, const hx_kv_interval* running, void* stream);
int hx_schedule_decode(hx_cluster* h, const hx_call* calls, const int32_t* lock, const float* ready_s,
                       int n_calls, int32_t* out_inst, float* out_start, float* out_ratio,
                       int32_t* out_order, void* stream);

/* Borrowed device pointers to the top-K results of the last batch scored with
 * topk = K > 0: pairs int32[n_calls][K] (-1 = unused slot), costs
 * float[n_calls][K] (projected decode finish of that pair, +inf if unused),
 * prio float[n_calls] (Eq. 2 of the best pair; the pass visits calls by
 * decreasing prio).  The K entries are the K cheapest distinct decode
 * instances, each with its best prefill partner, ordered by (cost, d).
 * Any output argument may be NULL. */
int hx_get_topk(hx_cluster* h, const int32_t** pairs, const float** costs, const float** prio);

/* Device-side status word: 0 = fine, else the HX_ERR_* code a kernel raised
 * (HX_ERR_INVALID_ARG for a bad call record) in work enqueued on `stream` since
 * the previous hx_get_status.  Reads the word, clears it, and synchronises
 * `stream`, so each call reports on the batches since the one before. */
int hx_get_status(hx_cluster* h, int* status, void* stream);

/* Tracing aid (the paper reports scheduler time per invocation, Section 7.7):
 * while enabled, each kernel family the library enqueues is bracketed by a pair
 * of CUDA events on the caller's stream.  Families: 0 = scoring kernel,
 * 1 = capacity-conflict pass (all its kernels), 2 = horizon kernels.
 * hx_read_kernel_timing waits for the recorded events, writes the summed
 * device time in milliseconds and the number of bracketed enqueues per family
 * (arrays of 3) since the previous read, and resets the record. */
int hx_enable_kernel_timing(hx_cluster* h, int enable);
int hx_read_kernel_timing(hx_cluster* h, float* ms, int* launches);

/* Measurement aid for the roofline of the scoring kernel, whose bound is the issue
 * rate of the FP32 pipes (one fused multiply-add and one minimum per candidate,
 * Algorithm 1, inner loop): runs four register-only loops of at least a
 * millisecond each on `stream` and reports, in lane-instructions per second (32
 * per warp instruction), what the device sustains for [0] fma.rn.f32, [1]
 * fma.rn.f32x2, [2] three-input min.f32, [3] the one-to-one mix of [1] and [2]
 * that the candidate loop issues; ms[4] receives the device time of each timed
 * launch.  Synchronises.  Errors: HX_ERR_INVALID_ARG for NULL arguments. */
int hx_measure_fp32_rates(hx_cluster* h, double* lane_instr_per_s, float* ms, void* stream);

/* Message of the last error on this handle ("" if none); with h = NULL, the
 * message of the last failed hx_cluster_create of the calling thread. */
const char* hx_last_error(const hx_cluster* h);

/* Number of kernels this library has launched on the handle so far. */
long long hx_launch_count(const hx_cluster* h);

#ifdef __cplusplus
}
#endif
#endif /* HX_H_ */
