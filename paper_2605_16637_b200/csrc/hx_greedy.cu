// Recomputing greedy planner for small queues (paper Algorithm 1, the while-loop
// over the queue snapshot; Section 5.3 "Adaptive greedy prefill assignment").
//
// Until the queue is empty: project every waiting call's best feasible pair
// against the simulated state, its Delta and its ratio R = (elapsed + Delta) / H
// (Eq. 2); take the call with the largest R (lower call index among equals);
// record its pair; add its prefill time to the chosen prefill queue and take its
// m(c) = L_in + L_out KV tokens (Eq. 3) from the chosen decode instance; remove
// it.  A pair is feasible when m(c) <= Cap(d) (Eq. 4) and m(c) fits the KV tokens
// the simulated state has left on d.
//
// One persistent block holds the whole state in shared memory.  A commit touches
// one prefill queue p* and one decode instance d*, and every candidate only gets
// later or disappears; so the projection of a waiting call changes only if its
// own best pair uses p*, or uses d* and no longer fits.  Per iteration the block
// (1) re-projects exactly those calls, one warp per call with the lanes over the
// pairs, (2) reduces the largest ratio, (3) commits and lists the calls to
// re-project.  The arithmetic of a candidate is the canonical binary32 sequence
// of the scoring kernel, so the results equal the definition bit for bit.
//
// Long queues run on a thread-block cluster of kCluster blocks (one SM each): call c belongs to
// block c mod kCluster, every block keeps its own copy of the small simulated state, and per
// iteration the blocks exchange their most urgent call and the winner's commit through
// distributed shared memory with two cluster barriers.  All blocks reduce the same candidates and
// apply the same commit, so their copies stay identical and every exit is taken by all of them.
#include <cooperative_groups.h>

#include "hx_internal.h"

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
#define HX_INF __int_as_float(0x7f800000)
#define HX_NEG_INF __int_as_float(0xff800000)
constexpr int kDead = -2;          // call already taken (or rejected as invalid)
constexpr int kNoPair = -1;        // waiting, but no feasible pair: can never be taken any more

struct GreedyParams {
    HxTables t;
    HxConstTables ct;
    HxDagView dag;
    const hx_call* calls;
    int n, flags, commit;
    int32_t* out_assign;
    float* out_ratio;
    int32_t* out_order;
    float* out_delta;          // may be NULL
    int* status;
};

// CACHE: the per-class prefill and decode times, the KV bytes and the demand of every call are computed once and kept
// in shared memory ([class][call]); without it a warp recomputes them whenever it re-projects a call.
template <int NC, bool CACHE>   // NC: blocks of the cluster (1 = a plain single block)
__global__ void __launch_bounds__(kThreads, 1) hx_greedy_kernel(const __grid_constant__ GreedyParams prm) {
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ float red_v[kWarps];
    __shared__ int red_c[kWarps];
    __shared__ int s_call, s_p, s_d, s_ndirty;
    __shared__ float x_v[NC];                  // most urgent call of every block (written by its owner block)
    __shared__ int x_c[NC];
    __shared__ float x_commit[4];              // p, d (as int bits), prefill time, demand of the committed call
    const HxTables& T = prm.t;
    const int P = T.P, D = T.D, G = T.G;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int rank = 0;
    if (NC > 1) rank = (int)cg::this_cluster().block_rank();
    const int n_all = prm.n;
    const int n = (n_all - rank + NC - 1) / NC;                // calls of this block: c = li * NC + rank

    float* invL = reinterpret_cast<float*>(smem);              // [P][D]
    float* qPs = invL + (size_t)P * D;                         // [P]
    float* qDs = qPs + P;                                      // [D]
    float* capDs = qDs + D;                                    // [D]
    float* frees = capDs + D;                                  // [D]
    int* typePs = reinterpret_cast<int*>(frees + D);           // [P]
    int* typeDs = typePs + P;                                  // [D]
    float* scratch = reinterpret_cast<float*>(typeDs + D);     // [kWarps][64] per-class times of the call a warp works on
    float* cn = scratch + kWarps * 64;                         // [n] prompt tokens
    float* co = cn + n;                                        // [n] output tokens
    float* cel = co + n;                                       // [n] elapsed time of the workflow
    float* cH = cel + n;                                       // [n] horizon of the workflow
    float* cR = cH + n;                                        // [n] projected ratio, -inf if it cannot be taken
    int* cpair = reinterpret_cast<int*>(cR + n);               // [n] best pair as p << 16 | d, kNoPair, kDead
    int* cmodel = cpair + n;                                   // [n]
    float* ckv = reinterpret_cast<float*>(cmodel + n);         // [n] KV bytes of the prompt (CACHE)
    float* cmm = ckv + (CACHE ? n : 0);                        // [n] demand in tokens (CACHE)
    float* tpreC = cmm + (CACHE ? n : 0);                      // [G][n] prefill time per GPU class (CACHE)
    float* tdecC = tpreC + (CACHE ? (size_t)G * n : 0);        // [G][n] decode time per GPU class (CACHE)
    unsigned short* dirty = reinterpret_cast<unsigned short*>(tdecC + (CACHE ? (size_t)G * n : 0));   // [n] calls to re-project

    for (int i = tid; i < P * D; i += kThreads) { const int p = i / D, d = i - p * D; invL[i] = T.invLT[(size_t)d * T.Ppad + p]; }
    for (int p = tid; p < P; p += kThreads) { qPs[p] = T.qP[p]; typePs[p] = T.typeP[p]; }
    for (int d = tid; d < D; d += kThreads) { qDs[d] = T.qD[d]; capDs[d] = T.capD[d]; frees[d] = T.freeD[d]; typeDs[d] = T.typeD[d]; }
    for (int c = tid; c < n; c += kThreads) {
        const int gcall = c * NC + rank;
        const uint4 raw = __ldg(reinterpret_cast<const uint4*>(prm.calls) + gcall);
        bool bad = raw.y >= (unsigned)T.M;
        float el = 0.f, H = 1.f;
        if (!(prm.flags & HX_FLAG_NO_DAG)) {
            if (raw.x < prm.dag.n_nodes) { const uint32_t w = prm.dag.node_wf[raw.x]; el = prm.dag.elapsed[w]; H = prm.dag.H[w]; }
            else bad = true;
        }
        if (bad) atomicExch(prm.status, HX_ERR_INVALID_ARG);
        cn[c] = __uint_as_float(raw.z); co[c] = __uint_as_float(raw.w);
        cmodel[c] = bad ? 0 : (int)raw.y;
        cel[c] = el; cH[c] = H;
        cR[c] = HX_NEG_INF;
        cpair[c] = bad ? kDead : kNoPair;
        dirty[c] = (unsigned short)c;
        if (CACHE) {
            const float nt = cn[c], ot = co[c];
            const int mdl = cmodel[c];
            const float phi = prm.ct.phi[mdl], omega = prm.ct.omega[mdl], kappa = prm.ct.kappa[mdl];
            const float kvB = __fmul_rn(nt, kappa);
            const float ctx = __fmaf_rn(0.5f, __fsub_rn(ot, 1.0f), nt);
            const float step = __fmaf_rn(kappa, ctx, omega);
            ckv[c] = kvB; cmm[c] = __fadd_rn(nt, ot);
            for (int g = 0; g < G; ++g) {
                const float iF = prm.ct.invF[g], iB = prm.ct.invB[g];
                tpreC[g * n + c] = fmaxf(__fmul_rn(__fmaf_rn(__fmul_rn(nt, prm.ct.psi[mdl]), nt, __fmul_rn(nt, phi)), iF), __fmul_rn(__fadd_rn(omega, kvB), iB));
                tdecC[g * n + c] = __fmul_rn(__fmul_rn(ot, step), iB);
            }
        }
        prm.out_assign[gcall] = -1; prm.out_ratio[gcall] = HX_INF; prm.out_order[gcall] = -1;
        if (prm.out_delta) prm.out_delta[gcall] = HX_INF;
    }
    if (tid == 0) s_ndirty = n;
    __syncthreads();

    for (int it = 0; it < n_all; ++it) {
        // (1) re-project the listed calls: one warp per call, lanes over the pairs
        const int nd = s_ndirty;
        for (int i = warp; i < nd; i += kWarps) {
            const int c = dirty[i];
            if (cpair[c] == kDead) continue;                   // rejected at load time (warp-uniform)
            // per-class times of this call: tpre[g * ts], tdec[g * ts]
            const float* tpre; const float* tdec; int ts;
            float kvB, m;
            if (CACHE) {
                tpre = tpreC + c; tdec = tdecC + c; ts = n;
                kvB = ckv[c]; m = cmm[c];
            } else {
                float* wpre = scratch + warp * 64;
                float* wdec = wpre + 32;
                const float nt = cn[c], ot = co[c];
                const int mdl = cmodel[c];
                const float phi = prm.ct.phi[mdl], omega = prm.ct.omega[mdl], kappa = prm.ct.kappa[mdl];
                kvB = __fmul_rn(nt, kappa);
                const float ctx = __fmaf_rn(0.5f, __fsub_rn(ot, 1.0f), nt);
                const float step = __fmaf_rn(kappa, ctx, omega);
                m = __fadd_rn(nt, ot);
                if (lane < G) {
                    const float iF = prm.ct.invF[lane], iB = prm.ct.invB[lane];
                    wpre[lane] = fmaxf(__fmul_rn(__fmaf_rn(__fmul_rn(nt, prm.ct.psi[mdl]), nt, __fmul_rn(nt, phi)), iF), __fmul_rn(__fadd_rn(omega, kvB), iB));
                    wdec[lane] = __fmul_rn(__fmul_rn(ot, step), iB);
                }
                __syncwarp();
                tpre = wpre; tdec = wdec; ts = 1;
            }
            float best = HX_INF; int bj = 0x7fffffff;
            // a lane keeps its decode instance and walks the prefill instances, so that everything that
            // depends on d alone (room, decode time, availability) is read once per call: with D lanes per
            // prefill row when D divides 32, else with the lanes over d and every lane over all rows
            const int dlanes = (D < 32 && 32 % D == 0) ? D : 32;
            const int prow = lane / dlanes, pstep = 32 / dlanes;
            for (int d = lane - prow * dlanes; d < D; d += dlanes) {
                const bool fits = m <= capDs[d] && m <= frees[d];
                if (!fits) continue;                           // every pair on d is +inf: cannot be the minimum
                const float Dd = tdec[typeDs[d] * ts], qd = qDs[d];
                for (int p = prow; p < P; p += pstep) {
                    const float A = __fadd_rn(qPs[p], tpre[typePs[p] * ts]);
                    const float ready = __fmaf_rn(kvB, invL[p * D + d], A);
                    const float fin = __fadd_rn(fmaxf(ready, qd), Dd);
                    const int j = (p << 16) | d;
                    if (fin < best || (fin == best && j < bj)) { best = fin; bj = j; }
                }
            }
            // finish times are >= 0 or +inf, so their bit patterns order like the values: two warp-wide
            // integer minima give the smallest value and the lowest pair among the lanes that hold it
            const unsigned vmin = __reduce_min_sync(0xffffffffu, __float_as_uint(best));
            bj = (int)__reduce_min_sync(0xffffffffu, __float_as_uint(best) == vmin ? (unsigned)bj : 0x7fffffffu);
            best = __uint_as_float(vmin);
            if (lane == 0) {
                if (best < HX_INF) { cpair[c] = bj; cR[c] = __fdiv_rn(__fadd_rn(cel[c], best), cH[c]); }
                else { cpair[c] = kNoPair; cR[c] = HX_NEG_INF; }
            }
            __syncwarp();
        }
        __syncthreads();
        // (2) most urgent waiting call: largest ratio, lower call index among equals
        float rv = HX_NEG_INF; int rc = 0x7fffffff;
        for (int c = tid; c < n; c += kThreads) {
            const float r = cR[c];
            if (r > rv) { rv = r; rc = c * NC + rank; }        // ascending c: keeps the lowest index
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, rv, off);
            const int oc = __shfl_xor_sync(0xffffffffu, rc, off);
            if (ov > rv || (ov == rv && oc < rc)) { rv = ov; rc = oc; }
        }
        if (lane == 0) { red_v[warp] = rv; red_c[warp] = rc; }
        __syncthreads();
        if (warp == 0) {
            rv = red_v[lane]; rc = red_c[lane];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, rv, off);
                const int oc = __shfl_xor_sync(0xffffffffu, rc, off);
                if (ov > rv || (ov == rv && oc < rc)) { rv = ov; rc = oc; }
            }
            if (lane == 0) {
                if (NC > 1) {                                  // publish the block's candidate in every block
                    cg::cluster_group cl = cg::this_cluster();
                    for (int r = 0; r < NC; ++r) {
                        *cl.map_shared_rank(&x_v[rank], r) = rv;
                        *cl.map_shared_rank(&x_c[rank], r) = rc;
                    }
                } else {
                    x_v[0] = rv; x_c[0] = rc;
                }
            }
        }
        if (NC > 1) cg::this_cluster().sync(); else __syncthreads();      // every thread of every block
        if (warp == 0) {
            rv = lane < NC ? x_v[lane] : HX_NEG_INF;           // all blocks reduce the same list
            rc = lane < NC ? x_c[lane] : 0x7fffffff;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, rv, off);
                const int oc = __shfl_xor_sync(0xffffffffu, rc, off);
                if (ov > rv || (ov == rv && oc < rc)) { rv = ov; rc = oc; }
            }
            const bool none = rc == 0x7fffffff;
            if (lane == 0) s_call = none ? -1 : rc;            // -1: nobody left that fits anywhere
            if (lane == 0 && !none && rc % NC == rank) {
                // (3) commit by the block that owns the call
                const int li = rc / NC;
                const int bj = cpair[li], p = bj >> 16, d = bj & 0xFFFF;
                const float nt = cn[li], ot = co[li];
                const int mdl = cmodel[li];
                const float phi = prm.ct.phi[mdl], omega = prm.ct.omega[mdl], kappa = prm.ct.kappa[mdl];
                const float kvB = __fmul_rn(nt, kappa);
                const int g = typePs[p];
                const float tp = fmaxf(__fmul_rn(__fmaf_rn(__fmul_rn(nt, prm.ct.psi[mdl]), nt, __fmul_rn(nt, phi)), prm.ct.invF[g]), __fmul_rn(__fadd_rn(omega, kvB), prm.ct.invB[g]));
                const float m = __fadd_rn(nt, ot);
                prm.out_assign[rc] = p * D + d;
                prm.out_ratio[rc] = rv;
                prm.out_order[it] = rc;
                if (prm.out_delta) {
                    // Delta of the chosen pair: the projection that made the ratio, from the same state
                    const float ctx = __fmaf_rn(0.5f, __fsub_rn(ot, 1.0f), nt);
                    const float td = __fmul_rn(__fmul_rn(ot, __fmaf_rn(kappa, ctx, omega)), prm.ct.invB[typeDs[d]]);
                    const float ready = __fmaf_rn(kvB, invL[p * D + d], __fadd_rn(qPs[p], tp));
                    prm.out_delta[rc] = __fadd_rn(fmaxf(ready, qDs[d]), td);
                }
                cpair[li] = kDead; cR[li] = HX_NEG_INF;
                if (NC > 1) {
                    cg::cluster_group cl = cg::this_cluster();
                    for (int r = 0; r < NC; ++r) {
                        float* xc = cl.map_shared_rank(x_commit, r);
                        xc[0] = __int_as_float(p); xc[1] = __int_as_float(d); xc[2] = tp; xc[3] = m;
                    }
                } else {
                    x_commit[0] = __int_as_float(p); x_commit[1] = __int_as_float(d); x_commit[2] = tp; x_commit[3] = m;
                }
            }
        }
        if (NC > 1) cg::this_cluster().sync(); else __syncthreads();      // the commit has reached every block
        if (tid == 0) {
            if (s_call >= 0) {                                 // the same update in every block
                const int p = __float_as_int(x_commit[0]), d = __float_as_int(x_commit[1]);
                qPs[p] = __fadd_rn(qPs[p], x_commit[2]);
                frees[d] = __fsub_rn(frees[d], x_commit[3]);
                s_p = p; s_d = d;
            }
            s_ndirty = 0;
        }
        __syncthreads();
        if (s_call < 0) break;
        // calls whose projection the commit can have changed
        const int ps = s_p, ds = s_d;
        const float left = frees[ds];
        for (int c = tid; c < n; c += kThreads) {
            const int bj = cpair[c];
            if (bj < 0) continue;
            const bool hit = (bj >> 16) == ps || ((bj & 0xFFFF) == ds && __fadd_rn(cn[c], co[c]) > left);
            if (hit) dirty[atomicAdd(&s_ndirty, 1)] = (unsigned short)c;
        }
        __syncthreads();
    }
    if (prm.commit && rank == 0) {
        for (int p = tid; p < P; p += kThreads) T.qP[p] = qPs[p];
        for (int d = tid; d < D; d += kThreads) T.freeD[d] = frees[d];
    }
    if (NC > 1) cg::this_cluster().sync();     // no block leaves while another may still write into it
}

}  // namespace

constexpr int kCluster = 8;                    // blocks of the cluster used for long queues (portable maximum)
constexpr int kClusterFrom = 512;              // queues longer than this use the cluster

static size_t greedy_smem(const HxTables& t, int calls_per_block) {
    return ((size_t)t.P * t.D + 2 * (size_t)t.P + 5 * (size_t)t.D + kWarps * 64 + 7 * (size_t)calls_per_block) * 4 +
           (size_t)calls_per_block * 2 + 16;
}
// With the per-class times of every call kept in shared memory.
static size_t greedy_cache_smem(const HxTables& t, int calls_per_block) {
    return greedy_smem(t, calls_per_block) + (size_t)calls_per_block * (2 + 2 * (size_t)t.G) * 4;
}
static bool greedy_cache_ok(const HxTables& t, int calls_per_block) {
    return greedy_cache_smem(t, calls_per_block) <= (size_t)200 * 1024;
}

// Shared memory of one block for a queue of n_calls (the longest queue a single block must be able
// to take is kClusterFrom calls; longer ones are split over the cluster when the device can run it).
size_t hx_greedy_smem_bytes(const HxTables& t, int n_calls) {
    return greedy_smem(t, n_calls > kClusterFrom ? (n_calls + kCluster - 1) / kCluster : n_calls);
}

cudaError_t hx_launch_greedy(const HxTables& t, const HxConstTables& ct, const HxDagView& dag,
                             const hx_call* calls, int n_calls, int flags, int commit,
                             int32_t* out_assign, float* out_ratio, int32_t* out_order, float* out_delta, int* status,
                             cudaStream_t stream, long long* launches) {
    GreedyParams prm;
    prm.t = t; prm.ct = ct; prm.dag = dag; prm.calls = calls; prm.n = n_calls; prm.flags = flags; prm.commit = commit;
    prm.out_assign = out_assign; prm.out_ratio = out_ratio; prm.out_order = out_order; prm.out_delta = out_delta;
    prm.status = status;
    cudaError_t e;
    if (n_calls > kClusterFrom) {
        const int cpb = (n_calls + kCluster - 1) / kCluster;
        const bool cache = greedy_cache_ok(t, cpb);
        const size_t smem = cache ? greedy_cache_smem(t, cpb) : greedy_smem(t, cpb);
        static size_t allowed[64], allowed_c[64];
        void (*kern)(GreedyParams) = cache ? hx_greedy_kernel<kCluster, true> : hx_greedy_kernel<kCluster, false>;
        if ((e = hx_opt_in_smem(kern, smem, cache ? allowed_c : allowed, 40 * 1024)) != cudaSuccess) return e;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(kCluster); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = kCluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        int n_clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&n_clusters, kern, &cfg) == cudaSuccess && n_clusters >= 1) {
            e = cudaLaunchKernelEx(&cfg, kern, prm);
            if (e == cudaSuccess) ++*launches;
            return e;
        }
        (void)cudaGetLastError();              // the device cannot host the cluster: one block, if the queue fits
        if (greedy_smem(t, n_calls) > (size_t)227 * 1024) return cudaErrorInvalidConfiguration;
    }
    const bool cache = greedy_cache_ok(t, n_calls);
    const size_t smem = cache ? greedy_cache_smem(t, n_calls) : greedy_smem(t, n_calls);
    static size_t allowed1[64], allowed1_c[64];
    if (cache) {
        if ((e = hx_opt_in_smem(hx_greedy_kernel<1, true>, smem, allowed1_c, 40 * 1024)) != cudaSuccess) return e;
        hx_greedy_kernel<1, true><<<1, kThreads, smem, stream>>>(prm);
    } else {
        if ((e = hx_opt_in_smem(hx_greedy_kernel<1, false>, smem, allowed1, 40 * 1024)) != cudaSuccess) return e;
        hx_greedy_kernel<1, false><<<1, kThreads, smem, stream>>>(prm);
    }
    e = cudaGetLastError();
    if (e == cudaSuccess) ++*launches;
    return e;
}
