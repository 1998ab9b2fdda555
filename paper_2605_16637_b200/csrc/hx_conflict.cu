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
// Parallel form with identical results: the only shared state a decision reads
// is the free capacity of one decode instance, so every decode instance is
// owned by one thread that walks, in visiting order, the list of (call, k)
// slots naming it.  A slot (c, k) can be decided as soon as call c is known to
// have failed on its candidates 0..k-1; until then the owner waits, and since
// the most urgent undecided call is always at the head of the list of the
// instance it is pending on, some thread can always advance.  Prefill queues
// are updated afterwards by summing, per prefill instance, the prefill times of
// the calls it obtained in visiting order (binary32 addition is not
// associative, so the order is part of the definition).
//
// Ordering without a global sort: slots are bucketed per decode instance
// (counting pass fused into the scoring kernel, scatter here), and each bucket
// is ordered by counting, for every entry, the entries of the same bucket that
// precede it; keys (prio, call) are unique inside a bucket.
#include "hx_internal.h"

namespace {

typedef unsigned long long u64;

__device__ __forceinline__ u64 key_of(unsigned hi, unsigned lo) { return ((u64)hi << 32) | lo; }

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

// Scatter every valid (call, k) slot into the segment of its decode instance.
__global__ void hx_dscatter_kernel(HxTopkBufs tk, int n_calls, int D) {
    extern __shared__ unsigned sm[];
    unsigned* base = sm;            // D + 1
    unsigned* tmp = sm + D + 1;     // 33
    block_exclusive_scan(tk.dcount, D, base, tmp);
    const int K = tk.K;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_calls * K; i += gridDim.x * blockDim.x) {
        const int pr = tk.pair[i];
        if (pr < 0) continue;
        const int c = i / K, k = i - c * K, d = pr % D;
        const unsigned pos = base[d] + atomicAdd(&tk.dcursor[d], 1u);
        tk.dflat[pos] = make_uint4(~__float_as_uint(tk.prio[c]), (unsigned)c, (unsigned)k, __float_as_uint(tk.mtok[c]));
    }
}

// Order every decode segment: position = number of entries of the segment with a smaller key.
__global__ void hx_drank_kernel(HxTopkBufs tk, int D) {
    extern __shared__ unsigned sm[];
    unsigned* base = sm;
    unsigned* tmp = sm + D + 1;
    block_exclusive_scan(tk.dcount, D, base, tmp);
    const unsigned total = base[D];
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        int lo = 0, hi = D;                       // segment d with base[d] <= i < base[d + 1]
        while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (base[mid] <= i) lo = mid; else hi = mid; }
        const unsigned b0 = base[lo], b1 = base[lo + 1];
        const uint4 me = tk.dflat[i];
        const u64 key = key_of(me.x, me.y);
        unsigned rank = 0;
        for (unsigned j = b0; j < b1; ++j) {
            const uint2 o = __ldg(reinterpret_cast<const uint2*>(tk.dflat + j));
            rank += key_of(o.x, o.y) < key;
        }
        tk.dsorted[b0 + rank] = make_uint2(me.y | (me.z << 24), me.w);
    }
}

// One thread per decode instance walks its ordered slot list.  state[c] holds
// the index of the candidate call c is pending on, or 0xFF once it has a pair.
// A wait never blocks: a thread that cannot decide its head slot simply retries
// in the next round, and the number of rounds is bounded.
__global__ void hx_conflict_kernel(HxTopkBufs tk, HxTables t, int n_calls, int commit,
                                   int32_t* out_assign, int* status, int max_rounds) {
    extern __shared__ unsigned sm[];
    const int D = t.D, K = tk.K;
    unsigned* base = sm;                                        // D + 1
    unsigned* tmp = sm + D + 1;                                 // 33
    volatile unsigned char* state = reinterpret_cast<volatile unsigned char*>(sm + D + 1 + 33);
    block_exclusive_scan(tk.dcount, D, base, tmp);
    for (int c = threadIdx.x; c < n_calls; c += blockDim.x) state[c] = 0;
    __syncthreads();
    const int d = threadIdx.x;
    const bool own = d < D;
    unsigned pos = own ? base[d] : 0;
    const unsigned end = own ? base[d + 1] : 0;
    float free_tok = own ? t.freeD[d] : 0.f;
    int rounds = 0;
    for (;;) {
        // take every decidable slot at the head of the list, stop at the first undecidable one
        while (pos < end) {
            const uint2 e = tk.dsorted[pos];
            const unsigned c = e.x & 0xFFFFFFu, k = e.x >> 24;
            const unsigned s = state[c];
            if (s < k) break;                                   // call still pending on an earlier candidate
            if (s == k) {
                const float m = __uint_as_float(e.y);
                if (free_tok >= m) {
                    free_tok = __fsub_rn(free_tok, m);
                    const int pr = tk.pair[(size_t)c * K + k];
                    out_assign[c] = pr;
                    const int p = pr / D;
                    atomicAdd(&tk.pcount[p], 1u);
                    const unsigned a = atomicAdd(tk.n_acc, 1u);
                    tk.accflat[a] = make_uint4(~__float_as_uint(tk.prio[c]), c, (unsigned)p,
                                               __float_as_uint(tk.tpre[(size_t)c * K + k]));
                    state[c] = 0xFF;
                } else {
                    state[c] = (unsigned char)(k + 1);
                }
            }
            ++pos;
        }
        const int done = pos >= end;
        if (__syncthreads_and(done)) break;
        if (++rounds > max_rounds) {                            // cannot happen for a consistent list
            if (threadIdx.x == 0) atomicExch(status, HX_ERR_TIMEOUT);
            break;
        }
    }
    if (own && commit) t.freeD[d] = free_tok;
}

// Bucket the obtained pairs per prefill instance.
__global__ void hx_pscatter_kernel(HxTopkBufs tk, int P) {
    extern __shared__ unsigned sm[];
    unsigned* base = sm;
    unsigned* tmp = sm + P + 1;
    block_exclusive_scan(tk.pcount, P, base, tmp);
    const unsigned total = *tk.n_acc;
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const uint4 e = tk.accflat[i];
        const unsigned pos = base[e.z] + atomicAdd(&tk.pcursor[e.z], 1u);
        tk.pseg[pos] = e;
    }
}

// Order each prefill bucket by visiting order and add the prefill times to the
// queue in that order.
__global__ void hx_qupdate_kernel(HxTopkBufs tk, HxTables t, int P) {
    extern __shared__ unsigned sm[];
    unsigned* base = sm;
    unsigned* tmp = sm + P + 1;
    block_exclusive_scan(tk.pcount, P, base, tmp);
    for (int p = blockIdx.x; p < P; p += gridDim.x) {
        const unsigned b0 = base[p], b1 = base[p + 1];
        for (unsigned i = b0 + threadIdx.x; i < b1; i += blockDim.x) {
            const uint4 me = tk.pseg[i];
            const u64 key = key_of(me.x, me.y);
            unsigned rank = 0;
            for (unsigned j = b0; j < b1; ++j) {
                const uint2 o = __ldg(reinterpret_cast<const uint2*>(tk.pseg + j));
                rank += key_of(o.x, o.y) < key;
            }
            tk.psorted[b0 + rank] = __uint_as_float(me.w);
        }
        __syncthreads();
        if (threadIdx.x == 0 && b1 > b0) {
            float q = t.qP[p];
            for (unsigned i = b0; i < b1; ++i) q = __fadd_rn(q, __ldcg(&tk.psorted[i]));
            t.qP[p] = q;
        }
        __syncthreads();
    }
}

}  // namespace

cudaError_t hx_launch_conflict(const HxTables& t, const HxTopkBufs& tk, int n_calls, int commit,
                               int32_t* out_assign, int* status, cudaStream_t stream,
                               long long* launches) {
    const int D = t.D, P = t.P;
    const size_t smD = (size_t)(D + 1 + 33) * 4, smP = (size_t)(P + 1 + 33) * 4;
    const int nslots = n_calls * tk.K;
    int grid = (nslots + 255) / 256; if (grid > 592) grid = 592;
    hx_dscatter_kernel<<<grid, 256, smD, stream>>>(tk, n_calls, D);
    hx_drank_kernel<<<grid, 256, smD, stream>>>(tk, D);
    const int cthreads = (D + 31) / 32 * 32;
    const size_t smC = smD + (size_t)((n_calls + 15) / 16 * 16);
    if (smC > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(hx_conflict_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smC);
        if (e != cudaSuccess) return e;
    }
    // every round decides at least one slot, so n_calls * K + 2 rounds always suffice
    hx_conflict_kernel<<<1, cthreads, smC, stream>>>(tk, t, n_calls, commit, out_assign, status, nslots + 2);
    *launches += 3;
    if (commit) {
        int gp = (n_calls + 255) / 256; if (gp > 592) gp = 592;
        hx_pscatter_kernel<<<gp, 256, smP, stream>>>(tk, P);
        hx_qupdate_kernel<<<P < 592 ? P : 592, 128, smP, stream>>>(tk, t, P);
        *launches += 2;
    }
    return cudaGetLastError();
}
