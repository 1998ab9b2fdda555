// Capacity-conflict pass over one scored batch (paper Section 5.3, last
// sentence: large queues are ordered once by the risk score instead of being
// re-planned call by call; Section 5.4 / Eq. 3-4: decode KV capacity is the
// constraint that placements compete for).
//
// Definition (sequential): visit the calls by decreasing prio (Eq. 2), lower
// call index first among equals.  A call takes the first of its K candidates
// whose decode instance still has kv_free >= m(c); that subtracts m(c) from the
// instance and adds the call's prefill time to the chosen prefill queue.
//
// Parallel form with identical results:
//  1. hx_order_bins_kernel / hx_order_rank_kernel - visiting order of the batch.
//     Calls are binned by the leading bits of the priority key (bins linear in
//     the key bits between the batch minimum and maximum); inside a bin every
//     key counts the keys that precede it.  Keys (prio, call) are unique.
//  2. hx_conflict_kernel - optimistic windows over the visiting order.  A block
//     takes the next W calls; every call picks the first candidate that fits the
//     capacities committed so far, then checks it against the demand of the
//     earlier calls of the same window that picked the same instance (ordered,
//     segmented prefix sum).  All calls before the first one whose check fails
//     have, by induction, made exactly the sequential decision: they commit, the
//     window restarts at the failing call, which now sees the reduced capacity.
//     Token counts are integer-valued and below 2^24, so the prefix sums are
//     exact and equal to the sequential subtractions.  The first call of a
//     window can never fail, so every step commits at least one call.
//  3. hx_finish_kernel - writes the obtained pairs and gathers, in visiting
//     order, (prefill instance, prefill time) of the calls that obtained one.
//  4. hx_qsum_kernel - one thread per prefill instance adds its prefill times in
//     visiting order (binary32 addition is not associative, so the order is
//     part of the definition).
#include "hx_internal.h"

namespace {

typedef unsigned long long u64;

constexpr int kBins = 2048;
constexpr int kWin = 256;          // calls per optimistic window (= block size of the pass)
constexpr int kCache = 4096;       // calls staged in shared memory ahead of the window
constexpr unsigned kNone = 0xFFu;  // no candidate taken

// Exclusive prefix sum of n counters into shared memory, by the whole block
// (blockDim a multiple of 32).  base gets n + 1 entries, tmp needs 33.
__device__ void block_exclusive_scan(const unsigned* cnt, int n, unsigned* base, unsigned* tmp) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int per = (n + nthr - 1) / nthr;
    const int lo = min(n, tid * per), hi = min(n, (tid + 1) * per);
    unsigned sum = 0;
    for (int i = lo; i < hi; ++i) sum += cnt[i];
    const int lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    unsigned x = sum;
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned y = __shfl_up_sync(0xffffffffu, x, off);
        if (lane >= off) x += y;
    }
    if (lane == 31) tmp[warp] = x;
    __syncthreads();
    if (warp == 0) {
        unsigned w = lane < nwarp ? tmp[lane] : 0;
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned y = __shfl_up_sync(0xffffffffu, w, off);
            if (lane >= off) w += y;
        }
        tmp[lane] = w;
    }
    __syncthreads();
    unsigned run = x - sum + (warp > 0 ? tmp[warp - 1] : 0);
    for (int i = lo; i < hi; ++i) { base[i] = run; run += cnt[i]; }
    if (tid == 0) base[n] = tmp[nwarp - 1];
    __syncthreads();
}

// 1a. Bin the priority keys: one block.  obase receives the kBins + 1 bin bounds, the smallest
// key and the shift that maps a key to its bin.  Each thread keeps its first kKeep keys in
// registers (one round trip to memory); the rest of a large batch is read again per pass.
constexpr int kKeep = 16;
__global__ void __launch_bounds__(1024) hx_order_bins_kernel(HxTopkBufs tk, int n) {
    __shared__ unsigned hist[kBins], base[kBins + 1], tmp[33], lohi[2];
    const int tid = threadIdx.x, nthr = blockDim.x;
    for (int i = tid; i < kBins; i += nthr) hist[i] = 0;
    if (tid == 0) { lohi[0] = 0xFFFFFFFFu; lohi[1] = 0u; }
    unsigned keep[kKeep];
#pragma unroll
    for (int u = 0; u < kKeep; ++u) {
        const int c = tid + u * nthr;
        keep[u] = c < n ? ~__float_as_uint(__ldg(tk.prio + c)) : 0u;      // larger priority = smaller key
    }
    auto key_of = [&](int u, int c) { return u < kKeep ? keep[u] : ~__float_as_uint(__ldg(tk.prio + c)); };
    __syncthreads();
    unsigned lo = 0xFFFFFFFFu, hi = 0u;
#pragma unroll
    for (int u = 0; u < kKeep; ++u) if (tid + u * nthr < n) { lo = min(lo, keep[u]); hi = max(hi, keep[u]); }
    for (int c = tid + kKeep * nthr; c < n; c += nthr) { const unsigned k = key_of(kKeep, c); lo = min(lo, k); hi = max(hi, k); }
    lo = __reduce_min_sync(0xffffffffu, lo); hi = __reduce_max_sync(0xffffffffu, hi);
    if ((tid & 31) == 0) { atomicMin(&lohi[0], lo); atomicMax(&lohi[1], hi); }
    __syncthreads();
    lo = lohi[0];
    const unsigned span = lohi[1] - lo;
    int shift = 0;
    while ((span >> shift) >= (unsigned)kBins) ++shift;
#pragma unroll
    for (int u = 0; u < kKeep; ++u) if (tid + u * nthr < n) atomicAdd(&hist[(keep[u] - lo) >> shift], 1u);
    for (int c = tid + kKeep * nthr; c < n; c += nthr) atomicAdd(&hist[(key_of(kKeep, c) - lo) >> shift], 1u);
    __syncthreads();
    block_exclusive_scan(hist, kBins, base, tmp);
    for (int i = tid; i <= kBins; i += nthr) tk.obase[i] = base[i];
    if (tid == 0) { tk.obase[kBins + 1] = lo; tk.obase[kBins + 2] = (unsigned)shift; }
    for (int i = tid; i < kBins; i += nthr) hist[i] = 0;           // now the bin cursors
    __syncthreads();
#pragma unroll
    for (int u = 0; u < kKeep; ++u) {
        const int c = tid + u * nthr;
        if (c < n) {
            const unsigned bin = (keep[u] - lo) >> shift;
            tk.okey[base[bin] + atomicAdd(&hist[bin], 1u)] = ((u64)keep[u] << 32) | (unsigned)c;
        }
    }
    for (int c = tid + kKeep * nthr; c < n; c += nthr) {
        const unsigned key = key_of(kKeep, c);
        const unsigned bin = (key - lo) >> shift;
        tk.okey[base[bin] + atomicAdd(&hist[bin], 1u)] = ((u64)key << 32) | (unsigned)c;
    }
}

// 1b. Rank inside the bins and gather the per-call data in visiting order.
__global__ void hx_order_rank_kernel(HxTopkBufs tk, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const unsigned lo = tk.obase[kBins + 1], shift = tk.obase[kBins + 2];
    const u64 key = tk.okey[i];
    const unsigned bin = ((unsigned)(key >> 32) - lo) >> shift;
    const unsigned b0 = tk.obase[bin], b1 = tk.obase[bin + 1];
    unsigned rank = b0;
    for (unsigned j = b0; j < b1; ++j) rank += __ldg(tk.okey + j) < key;
    const unsigned c = (unsigned)key;
    tk.ocall[rank] = c;
    tk.om[rank] = tk.mtok[c];
    tk.od[rank] = tk.dsel[c];
}

// 2. The pass itself: one block of kWin threads.
__global__ void __launch_bounds__(kWin) hx_conflict_kernel(HxTopkBufs tk, HxTables t, int n, int commit) {
    extern __shared__ __align__(16) unsigned sm[];
    constexpr int NW = kWin / 32;
    const int D = t.D, K = tk.K;
    uint4* cd = reinterpret_cast<uint4*>(sm);                   // [kCache] candidate instances of the staged calls
    float* cm = reinterpret_cast<float*>(cd + kCache);          // [kCache] their demands
    float* free_s = cm + kCache;                                // [D] capacity left after the commits so far
    float* wtot = free_s + D;                                   // [NW][D] demand per warp and instance
    __shared__ int first_fail;
    __shared__ unsigned wacc[NW];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int d = tid; d < D; d += kWin) free_s[d] = t.freeD[d];
    for (int i = tid; i < NW * D; i += kWin) wtot[i] = 0.f;
    if (tid == 0) first_fail = kWin;
    int pos = 0, cache_lo = -kCache;
    unsigned n_acc = 0;                                         // same value in every thread
    while (pos < n) {
        if (pos + kWin > cache_lo + kCache) {                   // stage the next calls: one round trip
            __syncthreads();
            cache_lo = pos;
#pragma unroll
            for (int u = 0; u < kCache / kWin; ++u) {
                const int i = tid + u * kWin, r = pos + i;
                cd[i] = r < n ? __ldcg(tk.od + r) : make_uint4(~0u, ~0u, ~0u, ~0u);
                cm[i] = r < n ? __ldcg(tk.om + r) : 0.f;
            }
        }
        __syncthreads();                                        // S0: staged data, capacities and zeroed totals visible
        const int r = pos + tid, ci = r - cache_lo;
        const bool active = r < n;
        const float m = cm[ci];
        // first candidate that fits the committed capacities
        unsigned kt = kNone; int dt = -1;
        if (active) {
            const uint4 row = cd[ci];
            const unsigned w[4] = {row.x, row.y, row.z, row.w};
#pragma unroll
            for (int k = HX_MAX_TOPK - 1; k >= 0; --k) {
                const unsigned d = (w[k >> 1] >> ((k & 1) * 16)) & 0xFFFFu;
                if (k < K && d != 0xFFFFu && free_s[d] >= m) { kt = k; dt = (int)d; }
            }
        }
        // demand of the earlier lanes of this warp that picked the same instance: one warp scan
        // per distinct instance
        float cum = 0.f, incl = 0.f;
        unsigned rem = __ballot_sync(0xffffffffu, dt >= 0);
        while (rem) {
            const int leader = __ffs(rem) - 1;
            const int dl = __shfl_sync(0xffffffffu, dt, leader);
            const bool mine = dt == dl;
            float x = mine ? m : 0.f;
            for (int off = 1; off < 32; off <<= 1) {
                const float y = __shfl_up_sync(0xffffffffu, x, off);
                if (lane >= off) x = __fadd_rn(x, y);
            }
            if (mine) { incl = x; cum = __fsub_rn(x, m); }
            rem &= ~__ballot_sync(0xffffffffu, mine);
        }
        const unsigned peers = __match_any_sync(0xffffffffu, dt);
        const bool last_peer = dt >= 0 && (peers >> lane) <= 1u;
        if (last_peer) wtot[warp * D + dt] = incl;              // demand of this warp on dt
        __syncthreads();                                        // S1
        float before = cum;
        if (dt >= 0) for (int w = 0; w < warp; ++w) before = __fadd_rn(before, wtot[w * D + dt]);
        if (dt >= 0 && __fadd_rn(before, m) > free_s[dt]) atomicMin(&first_fail, tid);
        __syncthreads();                                        // S2
        const int f = first_fail;                               // calls before f decided as the sequential pass would
        const bool acc = active && tid < f && dt >= 0;
        // the last committing peer of each warp subtracts the demand of its warp's committing peers
        const unsigned accm = __ballot_sync(0xffffffffu, acc);
        if (acc && (((peers & accm) >> lane) <= 1u)) atomicAdd(&free_s[dt], -incl);   // exact: integer-valued
        if (last_peer) wtot[warp * D + dt] = 0.f;
        if (lane == 0) wacc[warp] = __popc(accm);
        __syncthreads();                                        // S3
        if (tid == 0) first_fail = kWin;
        unsigned off = n_acc + __popc(accm & ((1u << lane) - 1u));
        unsigned tot = 0;
        for (int w = 0; w < NW; ++w) { const unsigned a = wacc[w]; tot += a; if (w < warp) off += a; }
        if (acc) tk.acc_rk[off] = (unsigned)r | (kt << 24);     // obtained pairs, in visiting order
        n_acc += tot;
        pos += f < kWin ? f : kWin;
    }
    __syncthreads();
    if (tid == 0) *tk.n_acc = n_acc;
    if (commit) for (int d = tid; d < D; d += kWin) t.freeD[d] = free_s[d];
}

// 3. Publish the obtained pairs; gather prefill instance and prefill time in visiting order.
__global__ void hx_finish_kernel(HxTopkBufs tk, int D, int32_t* out_assign) {
    const unsigned i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= *tk.n_acc) return;
    const unsigned rk = tk.acc_rk[i], r = rk & 0xFFFFFFu, k = rk >> 24;
    const unsigned c = tk.ocall[r];
    const int pr = tk.pair[(size_t)c * tk.K + k];
    out_assign[c] = pr;
    tk.acc_p[i] = pr / D;
    tk.acc_t[i] = tk.tpre[(size_t)c * tk.K + k];
}

// 4. Prefill queues: thread p adds, in visiting order, the prefill times of the calls that obtained p.
__global__ void hx_qsum_kernel(HxTopkBufs tk, HxTables t) {
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned na = *tk.n_acc;
    float q = p < t.P ? t.qP[p] : 0.f;
#pragma unroll 8
    for (unsigned i = 0; i < na; ++i) {
        const int pi = __ldg(tk.acc_p + i);
        const float ti = __ldg(tk.acc_t + i);
        if (pi == p) q = __fadd_rn(q, ti);
    }
    if (p < t.P) t.qP[p] = q;
}

}  // namespace

cudaError_t hx_launch_conflict(const HxTables& t, const HxTopkBufs& tk, int n_calls, int commit,
                               int32_t* out_assign, int* status, cudaStream_t stream,
                               long long* launches) {
    (void)status;
    const int D = t.D, P = t.P;
    hx_order_bins_kernel<<<1, 1024, 0, stream>>>(tk, n_calls);
    hx_order_rank_kernel<<<(n_calls + 127) / 128, 128, 0, stream>>>(tk, n_calls);
    const size_t smC = (size_t)kCache * 20 + (size_t)(D + (kWin / 32) * D) * 4;
    if (smC > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(hx_conflict_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smC);
        if (e != cudaSuccess) return e;
    }
    hx_conflict_kernel<<<1, kWin, smC, stream>>>(tk, t, n_calls, commit);
    hx_finish_kernel<<<(n_calls + 255) / 256, 256, 0, stream>>>(tk, D, out_assign);
    *launches += 4;
    if (commit) {
        hx_qsum_kernel<<<(P + 31) / 32, 32, 0, stream>>>(tk, t);
        *launches += 1;
    }
    return cudaGetLastError();
}
