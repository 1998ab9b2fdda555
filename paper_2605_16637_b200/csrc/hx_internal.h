// Internal declarations shared by the translation units of libhx.so.
#ifndef HX_INTERNAL_H_
#define HX_INTERNAL_H_

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "hx.h"

// ---------------------------------------------------------------------------
// Packed cluster snapshot on the device (structure of arrays, binary32).
// invLT is the link table transposed and inverted: invLT[d * Ppad + p] =
// 1 / (GB/s of link p->d * 1e9); rows are padded with zeros to Ppad (a
// multiple of 4) so that every row starts on a 16-byte boundary.
// ---------------------------------------------------------------------------
struct HxTables {
    int G, P, D, M, Ppad;
    const float* invF;      // [G] 1 / (TFLOP/s * 1e12)
    const float* invB;      // [G] 1 / (TB/s * 1e12)
    const int* typeP;       // [Ppad]
    const int* typeD;       // [D]
    float* qP;              // [Ppad] seconds
    float* qD;              // [D]
    const float* capD;      // [D] tokens
    float* freeD;           // [D] tokens
    const float* invLT;     // [D * Ppad]
    const float* invLTt;    // same values tiled for the scoring kernel: [Ppad / 4][DpadT][4], zero padded
    int DpadT;              // decode columns of the tiled copy (hx_score_dpad(D))
    const float* phi;       // [M] flops per token
    const float* omega;     // [M] weight bytes
    const float* kappa;     // [M] KV bytes per token
};

// Per-class and per-model constants, small enough to travel with the kernel parameters.
struct HxConstTables {
    float invF[HX_MAX_TYPES], invB[HX_MAX_TYPES];
    float phi[HX_MAX_MODELS], omega[HX_MAX_MODELS], kappa[HX_MAX_MODELS];
    float psi[HX_MAX_MODELS];       // attention FLOPs per pair of prompt tokens (0 = linear prefill model)
};

// Thread-tile shape of the scoring kernel as a function of the decode pool: LD lanes of a warp
// along the decode columns, TD columns per thread; the block covers Dpad columns.
inline void hx_score_shape(int D, int* LD, int* TD, int* Dpad) {
    const int ld = D > 32 ? 8 : D > 16 ? 4 : D > 8 ? 2 : 1;
    const int td = ld == 8 ? 4 : 8;
    const int wd = ld * td;
    *LD = ld; *TD = td; *Dpad = (D + wd - 1) / wd * wd;
}

// Device view of the uploaded forest and of the horizon results.
struct HxDagView {
    const uint32_t* node_wf;   // [N] original numbering
    const float* tail;         // [N]
    const float* H;            // [W]
    const float* elapsed;      // [W]
    uint32_t n_nodes, n_workflows;
};

// Per-batch buffers of the top-K list and of the capacity-conflict pass; all
// sizes are linear in the batch.  "rank" = position of a call in visiting order.
struct HxTopkBufs {
    int K;
    int cap_calls;             // capacity (calls) of the per-call arrays
    // written by the scoring kernel, indexed by call
    int32_t* pair;             // [cap][K]
    float* cost;               // [cap][K]
    float* tpre;               // [cap][K] prefill time on the prefill instance of slot k
    uint4* dsel;               // [cap] decode instance of each slot as 8 x 16 bits, 0xFFFF = unused
    float* prio;               // [cap]
    float* mtok;               // [cap]
    // visiting order
    unsigned int* blk_lohi;    // [2 * HX_ORDER_MAXBLK] smallest / largest finite key seen by each block of the scoring kernel
    unsigned int* ghist;       // [HX_ORDER_BINS] keys per bin (zeroed by the scoring kernel), then [HX_ORDER_CALLBLK] first-key calls per block of the binning kernel
    unsigned int* oslot;       // [cap] bin << 16 | arrival number inside the bin, per call
    unsigned long long* okey;  // [cap] keys grouped by bin
    unsigned int* obase;       // [HX_ORDER_BINS + 3] bin bounds, smallest key, key-to-bin shift
    unsigned int* ocall;       // [cap] call of each rank
    int* om;                   // [cap] demand of each rank, tokens
    uint4* od;                 // [cap] same rows in visiting order, unused slots pointing at instance D
    // outcome: calls that obtained a pair, in visiting order
    unsigned int* n_acc;       // [1]
    unsigned int* acc_rk;      // [cap] call | k << 24
    int* acc_p;                // [cap] prefill instance obtained
    float* acc_t;              // [cap] prefill time added to that instance
};

// Visiting order of the capacity pass: key = bit pattern of the priority, inverted (larger priority =
// smaller key); a priority of +inf, or one that is not a number or negative, gets HX_FIRST_KEY and is
// visited first.  Bin 0 holds those keys; bins 1 .. HX_ORDER_BINS - 1 are linear in the key between the
// smallest and the largest finite key of the batch.
#define HX_ORDER_BINS 2048
#define HX_ORDER_MAXBLK 1024
#define HX_ORDER_CALLBLK 256   /* blocks of 256 calls in the largest batch (HX_MAX_COMMIT_CALLS) */
#define HX_FIRST_KEY 0x807FFFFFu
__host__ __device__ inline unsigned hx_order_key(unsigned prio_bits) {
    return prio_bits >= 0x7F800000u ? HX_FIRST_KEY : ~prio_bits;
}

struct ScoreLaunch {
    const hx_call* calls;
    int n_calls;
    int32_t* out_assign;
    float* out_cost;
    int mode, flags, K;
    float alpha;
};

// Levelised forest on the device (internal numbering: workflow by workflow,
// inside a workflow by increasing height above the sinks).
struct HxForestDev {
    uint32_t n_nodes, n_edges, n_workflows;
    const uint32_t* wf_node_start;   // [W+1] internal index of the first node of each workflow
    const uint32_t* wf_edge_start;   // [W+1] first edge of each workflow in icol
    const uint32_t* wf_seg_start;    // [W+1] first entry of each workflow in seg_off
    const uint32_t* seg_off;         // per workflow: local offsets of its levels, nlev+1 entries
    const uint32_t* irow;            // [N+1] edge offsets (global) in internal numbering
    const uint16_t* icol16;          // [E] successor as local index inside the workflow (16-bit copy)
    const uint32_t* icol32;          // [E] same, 32-bit
    const float* icost;              // [N]
    const uint32_t* perm;            // [N] internal -> original node number
    const uint32_t* wf_gid;          // [W] workflow number of the caller for H, or NULL when it is w itself
    float* cp;                       // [N] original numbering
    float* tail;                     // [N]
    float* H;                        // [W]
};

cudaError_t hx_launch_score(const HxTables& t, const HxConstTables& ct, const HxDagView& dag, const HxTopkBufs& tk,
                            const ScoreLaunch& s, int n_sm, size_t max_smem, int* status,
                            cudaStream_t stream, long long* launches);

cudaError_t hx_launch_conflict(const HxTables& t, const HxTopkBufs& tk, int n_calls, int commit,
                               int32_t* out_assign, int* status, cudaStream_t stream,
                               long long* launches, const float* free_reset = nullptr);

cudaError_t hx_launch_estimate(const HxConstTables& ct, int G, int M, const hx_call* calls, int n_calls,
                               float* tpre, float* tdec, float* kvB, float* m, int* status, cudaStream_t stream,
                               long long* launches);

// Issue rates of the instruction kinds of the candidate loop: lane-instructions per second of fma.rn.f32,
// fma.rn.f32x2, three-input min.f32 and their one-to-one mix; device time of each timed launch in ms.
cudaError_t hx_run_micro(int n_sm, float* sink, cudaStream_t stream, double* lane_instr_per_s, float* ms, long long* launches);

size_t hx_greedy_smem_bytes(const HxTables& t, int n_calls);
cudaError_t hx_launch_greedy(const HxTables& t, const HxConstTables& ct, const HxDagView& dag,
                             const hx_call* calls, int n_calls, int flags, int commit,
                             int32_t* out_assign, float* out_ratio, int32_t* out_order, float* out_delta, int* status,
                             cudaStream_t stream, long long* launches);

// Tokens in use on every decode instance as step functions of time (decode token-capacity
// intervals): instance d has K[d] breakpoints t[d * cap + k] (t = 0 first, ascending) and usage
// u[d * cap + k] on [t[k], t[k + 1]); the last segment runs to infinity.
struct HxStepFns {
    float* t;
    float* u;
    int* K;
    int cap;
};

size_t hx_decode_smem_bytes(const HxTables& t, int n_calls);
int hx_decode_replicas();      // copies of the simulated step functions the kernel may use (one per cluster block)
cudaError_t hx_launch_decode(const HxTables& t, const HxConstTables& ct, const HxDagView& dag,
                             const HxStepFns& base, const HxStepFns& work, int k_total,
                             const hx_call* calls, const int32_t* lock, const float* ready, int n_calls,
                             int flags, int commit, int32_t* out_inst, float* out_start, float* out_ratio,
                             int32_t* out_order, int* status, cudaStream_t stream, long long* launches);

// Workflow classes of the horizon pass: lists of workflow ids handled by one launch each.
struct HxCpClass {
    const uint32_t* wf_ids;    // device
    uint32_t count;
    int threads_per_wf;        // 32 (one warp) or the block size
    int wfs_per_block;
    size_t smem_per_wf;        // bytes of staging per workflow, 0 = work in global memory
};

#define HX_CP_CLASSES 6      // workflow classes of the horizon pass
#define HX_CP_SIDE 5         // side streams: every class after the first

// Side streams and events for running the independent workflow classes of one horizon pass
// next to each other (fork from / join into the caller's stream).  Zero-initialised = serial.
struct HxForkJoin {
    cudaStream_t aux[HX_CP_SIDE];
    cudaEvent_t fork, join[HX_CP_SIDE];
    int ready;
};

cudaError_t hx_launch_cpath(const HxForestDev& f, const HxCpClass* classes, int n_classes,
                            cudaStream_t stream, long long* launches, const HxForkJoin* fj = nullptr);

// Launch shape of workflow class k, by staging footprint: 0 = a quarter warp, <= 768 B, 64 per block;
// 1 = one warp, <= 3 KB, 16 per block; 2 = one warp, <= 12 KB, 8 per block; 3 = one warp, <= 48 KB, 2 per
// block (blocks of 96 KB or less can share an SM with blocks of other classes); 4 = one block,
// <= 200 KB; 5 = one block working in global memory.
inline HxCpClass hx_cpath_class_shape(int k) {
    const int tpw[HX_CP_CLASSES] = {8, 32, 32, 32, 256, 256}, per_block[HX_CP_CLASSES] = {64, 16, 8, 2, 1, 1};
    const size_t sm[HX_CP_CLASSES] = {768, 3072, 12288, 49152, 200 * 1024, 0};
    return HxCpClass{nullptr, 0, tpw[k], per_block[k], sm[k]};
}
inline int hx_cpath_class_of(size_t need_bytes, size_t n_nodes) {
    if (n_nodes > 65535) return HX_CP_CLASSES - 1;              // successor indices are 16-bit in the staged kernels
    for (int k = 0; k < HX_CP_CLASSES - 1; ++k)
        if (need_bytes <= hx_cpath_class_shape(k).smem_per_wf) return k;
    return HX_CP_CLASSES - 1;
}

// icost[idx[i]] = cost[i] (internal node numbering), ahead of a partial horizon pass.
cudaError_t hx_launch_cost_update(const HxForestDev& f, const uint32_t* idx, const float* cost, uint32_t n,
                                  cudaStream_t stream, long long* launches);

// Accessors for host code outside the file that defines the handle.
int hx_fail(hx_cluster* h, int code, const char* msg);            // records msg as the last error, returns code
void hx_cluster_shape(const hx_cluster* h, int* P, int* D, const float** capD_dev, uint32_t* n_nodes, uint32_t* n_workflows);
hx_options hx_current_options(const hx_cluster* h);
// Classes of the instances (prefill first, then decode) and the reciprocal link table, read back from the device.
int hx_cluster_tables_host(hx_cluster* h, std::vector<int>* typeP, std::vector<int>* typeD, std::vector<float>* invLT,
                           int* Ppad, int* G, int* M, cudaStream_t s);
// Successor lists of the forest as it stands (upload plus appended nodes and edges) and the workflow of every node.
void hx_forest_host(const hx_cluster* h, std::vector<uint32_t>* row, std::vector<uint32_t>* col, std::vector<uint32_t>* node_wf);
// Every model once more with its constants scaled by up and by down (models M .. 2M - 1 and 2M .. 3M - 1), until
// hx_pop_scaled_models; HX_ERR_INVALID_ARG when three times the models do not fit the table.
// hx_cluster_update_loads from ONE host array laid out like the device tables (prefill queues, decode hints, free KV
// tokens: P + 2 D values of one allocation): a single copy.
int hx_update_loads_packed(hx_cluster* h, const float* packed, cudaStream_t s);
int hx_push_scaled_models(hx_cluster* h, float up, float down);
void hx_pop_scaled_models(hx_cluster* h);

// Programmatic dependent launch: a kernel launched with hx_launch_dependent may be made resident while the
// kernel before it on the stream is still running, once every block of that kernel has called
// hx_release_dependents() or exited; it must call hx_wait_for_primary() before it touches anything the earlier
// kernel writes.  The wait returns once the earlier grid has completed and its writes are visible; launched the
// ordinary way both calls do nothing.  The attribute is kept inside a stream capture (the replayed graph gets
// programmatic edges).  Measured on the sweep step: a kernel that releases its dependents long before it ends
// slows the step down unless the dependent has real work to do ahead of its wait (the scoring kernel behind the
// capacity pass has, the binning kernel behind the scoring kernel has not: 1.72 against 1.64 ms per step), so
// only the pass releases early.
__device__ __forceinline__ void hx_wait_for_primary() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void hx_release_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
template <class... KArgs, class... Args>
inline cudaError_t hx_launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                       Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Opt a kernel in to `bytes` of dynamic shared memory, once per device and size: the attribute
// call is too slow to repeat on every launch.  `allowed` is a per-kernel table of 64 entries
// that starts at the size the kernel may use without opting in.
template <class Kernel>
inline cudaError_t hx_opt_in_smem(Kernel kernel, size_t bytes, size_t* allowed, size_t without_opt_in) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    dev &= 63;
    if (allowed[dev] < without_opt_in) allowed[dev] = without_opt_in;
    if (bytes <= allowed[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) allowed[dev] = bytes;
    return e;
}

#endif  // HX_INTERNAL_H_
