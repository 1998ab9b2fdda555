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
//  1. hx_order_hist_kernel / hx_order_scatter_kernel / hx_order_rank_kernel -
//     visiting order of the batch, three short grids.  Calls are binned by the
//     leading bits of the priority key (bins linear in the key bits between the
//     batch minimum and maximum, which the scoring kernel left behind per block;
//     priorities of +inf have a bin of their own, filled in call order, so that
//     calls that fit nowhere neither stretch the range nor need ranking); inside
//     every other bin a key counts the keys that precede it.  Keys (prio, call) are unique.
//  2. hx_conflict_kernel - optimistic windows over the visiting order.  A warp
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
//
#include <type_traits>

#include "hx_internal.h"

namespace {

typedef unsigned long long u64;

constexpr int kBins = HX_ORDER_BINS;
constexpr unsigned kNone = 0xFFu;  // no candidate taken
constexpr int kTailLen = 8192;     // obtained pairs handled per round of the fused tail
constexpr int kTailMaxP = 512;     // largest prefill pool the fused tail handles

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

// 1a. Bin the priority keys (grid of 256-thread blocks, one call per thread).  The scoring kernel left the
// key range of each of its blocks behind and cleared the bin counters; every block here reduces those ranges
// to the range of the batch, and every call draws its arrival number inside its bin from the global counter.
constexpr int kOrdThreads = 256;
__device__ __forceinline__ unsigned bin_of(unsigned key, unsigned lo, unsigned shift) {
    return key == HX_FIRST_KEY ? 0u : 1u + ((key - lo) >> shift);
}
__global__ void __launch_bounds__(kOrdThreads) hx_order_hist_kernel(HxTopkBufs tk, int n) {
    __shared__ unsigned lohi[2], wfirst[kOrdThreads / 32];
    const int tid = threadIdx.x;
    if (tid == 0) { lohi[0] = 0xFFFFFFFFu; lohi[1] = 0u; }
    __syncthreads();
    hx_wait_for_primary();                                        // the scoring kernel's key ranges, priorities and cleared counters
    unsigned lo = 0xFFFFFFFFu, hi = 0u;
    for (int b = tid; b < HX_ORDER_MAXBLK; b += kOrdThreads) {
        lo = min(lo, __ldcg(tk.blk_lohi + b)); hi = max(hi, __ldcg(tk.blk_lohi + HX_ORDER_MAXBLK + b));
    }
    lo = __reduce_min_sync(0xffffffffu, lo); hi = __reduce_max_sync(0xffffffffu, hi);
    if ((tid & 31) == 0) { atomicMin(&lohi[0], lo); atomicMax(&lohi[1], hi); }
    __syncthreads();
    lo = lohi[0];
    const unsigned span = lohi[1] >= lo ? lohi[1] - lo : 0u;      // no finite key at all: nothing lands in bins 1 ..
    unsigned shift = 0;
    while ((span >> shift) >= (unsigned)(kBins - 1)) ++shift;
    if (blockIdx.x == 0 && tid == 0) { tk.obase[kBins + 1] = lo; tk.obase[kBins + 2] = shift; }
    // Calls with the first key (all equal, so their order is the call order) take their place by counting: a
    // stable number inside the block here, the blocks before this one in the scatter step.  Every other call
    // draws an arrival number inside its bin.
    const int c = blockIdx.x * kOrdThreads + tid;
    const unsigned key = c < n ? hx_order_key(__float_as_uint(__ldcg(tk.prio + c))) : 0u;
    const bool first = c < n && key == HX_FIRST_KEY;
    const unsigned vote = __ballot_sync(0xffffffffu, first);
    if ((tid & 31) == 0) wfirst[tid >> 5] = __popc(vote);
    __syncthreads();
    unsigned before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < kOrdThreads / 32; ++w) { before += w < (tid >> 5) ? wfirst[w] : 0u; total += wfirst[w]; }
    if (tid == 0) { tk.ghist[kBins + blockIdx.x] = total; if (total) atomicAdd(tk.ghist, total); }
    if (c >= n) return;
    if (first) { tk.oslot[c] = before + __popc(vote & ((1u << (tid & 31)) - 1u)); return; }
    const unsigned bin = bin_of(key, lo, shift);
    tk.oslot[c] = (bin << 16) | atomicAdd(tk.ghist + bin, 1u);
}

// 1b. Every block turns the bin counters into bin bounds (the same 2,048-entry scan in every block is cheaper
// than one more launch) and moves its calls' keys to their place in bin order.
__global__ void __launch_bounds__(kOrdThreads) hx_order_scatter_kernel(HxTopkBufs tk, int n) {
    __shared__ unsigned hist[kBins], base[kBins + 1], tmp[33];
    const int tid = threadIdx.x;
    hx_wait_for_primary();                                        // the complete bin counters
    for (int i = tid; i < kBins; i += kOrdThreads) hist[i] = __ldcg(tk.ghist + i);
    __syncthreads();
    block_exclusive_scan(hist, kBins, base, tmp);
    if (blockIdx.x == 0) for (int i = tid; i <= kBins; i += kOrdThreads) tk.obase[i] = base[i];
    // first-key calls of the blocks before this one (at most 256 blocks: one counter per thread)
    unsigned mine = tid < (int)blockIdx.x ? __ldcg(tk.ghist + kBins + tid) : 0u;
    mine = __reduce_add_sync(0xffffffffu, mine);
    if ((tid & 31) == 0) tmp[tid >> 5] = mine;
    __syncthreads();
    unsigned first_before = 0;
#pragma unroll
    for (int w = 0; w < kOrdThreads / 32; ++w) first_before += tmp[w];
    const int c = blockIdx.x * kOrdThreads + tid;
    if (c >= n) return;
    const unsigned bs = __ldcg(tk.oslot + c);
    const unsigned key = hx_order_key(__float_as_uint(__ldcg(tk.prio + c)));
    const unsigned at = key == HX_FIRST_KEY ? first_before + bs : base[bs >> 16] + (bs & 0xFFFFu);
    tk.okey[at] = ((u64)key << 32) | (unsigned)c;
}

// 1c. Rank inside the bins and gather the per-call data in visiting order.  One key per thread; the block
// brings the keys of all bins that its threads belong to (one contiguous stretch) through shared memory, a
// tile at a time, and every thread counts the smaller keys of its own bin among them: a crowded bin (many
// equal priorities) then costs one shared-memory load per comparison instead of a trip to L2.
constexpr int kRankThreads = 128, kRankTile = 512;
__global__ void __launch_bounds__(kRankThreads) hx_order_rank_kernel(HxTopkBufs tk, int n, unsigned D) {
    __shared__ u64 tile[kRankTile];
    __shared__ unsigned range[2];
    const int tid = threadIdx.x;
    const int i = blockIdx.x * kRankThreads + tid;
    hx_wait_for_primary();                                        // every key is in its bin
    const bool valid = i < n;
    const unsigned lo = tk.obase[kBins + 1], shift = tk.obase[kBins + 2];
    const u64 key = valid ? tk.okey[i] : 0ull;
    const unsigned bin = valid ? bin_of((unsigned)(key >> 32), lo, shift) : 0u;
    // the first bin arrived in call order: nothing to count there
    const unsigned b0 = bin ? tk.obase[bin] : (unsigned)i, b1 = bin ? tk.obase[bin + 1] : (unsigned)i;
    if (tid == 0) range[0] = b0;                                  // bins ascend with the position: the first thread has the lowest
    if (i == min(n, (int)(blockIdx.x + 1) * kRankThreads) - 1) range[1] = b1;   // ... and the last valid one the highest
    __syncthreads();
    const unsigned u0 = range[0], u1 = range[1];
    unsigned rank = b0;
    for (unsigned t0 = u0; t0 < u1; t0 += kRankTile) {
        const unsigned len = min((unsigned)kRankTile, u1 - t0);
        if (t0 != u0) __syncthreads();                            // the previous tile has been read
        for (unsigned j = tid; j < len; j += kRankThreads) tile[j] = __ldcg(tk.okey + t0 + j);
        __syncthreads();
        const unsigned a = max(b0, t0), e = min(b1, t0 + len);
#pragma unroll 4
        for (unsigned j = a; j < e; ++j) rank += tile[j - t0] < key;
    }
    if (!valid) return;
    const unsigned c = (unsigned)key;
    tk.ocall[rank] = c;
    tk.om[rank] = __float2int_ru(tk.mtok[c]);                   // token counts are whole numbers below 2^24
    // candidate instances, 16 bits each; an unused slot (0xFFFF) points at instance D, which never has room
    const uint4 r = tk.dsel[c];
    const unsigned w[4] = {r.x, r.y, r.z, r.w};
    unsigned o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) o[q] = min(w[q] & 0xFFFFu, D) | (min(w[q] >> 16, D) << 16);
    tk.od[rank] = make_uint4(o[0], o[1], o[2], o[3]);
}

// Publishes the obtained pairs and adds the prefill times to the prefill queues in visiting order (NT
// threads).  The list of obtained pairs holds call | k << 24.  It is taken in rounds of kTailLen entries; a
// round is split by prefill instance with a stable counting sort (per-warp groups by match, per-warp
// counts, offsets), then one thread per instance adds its run one after the other (binary32 addition is
// not associative: the order is part of the definition).  pbuf [kTailLen] u16, tbuf and sorted [kTailLen]
// f32, tail_i [(4 + NT / 32) * P] ints.
template <int NT>
__device__ __forceinline__ void publish_and_sum(const HxTopkBufs& tk, const HxTables& t, unsigned n_acc, int commit,
                                                int32_t* out_assign, unsigned short* pbuf, float* tbuf,
                                                float* sorted, int* tail_i) {
    constexpr int NW = NT / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int P = t.P, D = t.D;
    float* qsum = reinterpret_cast<float*>(tail_i);                         // [P]
    int* hist = tail_i + P;                                                 // [P]
    int* off0 = hist + P;                                                   // [P] start of the run of p in `sorted`
    int* off = off0 + P;                                                    // [P] next free slot of the run
    int* wcnt = off + P;                                                    // [NW][P], zero between uses
    for (int p = tid; p < P; p += NT) qsum[p] = t.qP[p];
    for (int i = tid; i < NW * P; i += NT) wcnt[i] = 0;
    for (unsigned r0 = 0; r0 < n_acc; r0 += kTailLen) {
        const int len = (int)min((unsigned)kTailLen, n_acc - r0);
        for (int p = tid; p < P; p += NT) hist[p] = 0;
        __syncthreads();
        // dependent gathers per entry (list -> [call ->] pair, prefill time): eight entries in flight per thread
        for (int i0 = tid; i0 < len; i0 += 8 * NT) {
            unsigned rk[8], c[8]; int pr[8]; float tp[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) rk[u] = i0 + u * NT < len ? __ldcg(tk.acc_rk + r0 + i0 + u * NT) : 0u;
#pragma unroll
            for (int u = 0; u < 8; ++u) c[u] = rk[u] & 0xFFFFFFu;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const size_t o = (size_t)c[u] * tk.K + (rk[u] >> 24);
                const bool ok = i0 + u * NT < len;
                pr[u] = ok ? __ldcg(tk.pair + o) : 0;
                tp[u] = ok ? __ldcg(tk.tpre + o) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = i0 + u * NT;
                if (i < len) {
                    out_assign[c[u]] = pr[u];
                    const int p = pr[u] / D;
                    pbuf[i] = (unsigned short)p;
                    tbuf[i] = tp[u];
                    atomicAdd(&hist[p], 1);
                }
            }
        }
        __syncthreads();
        if (warp == 0) {                                        // exclusive prefix of the histogram
            int run = 0;
            for (int p0 = 0; p0 < P; p0 += 32) {
                const int p = p0 + lane;
                const int h = p < P ? hist[p] : 0;
                int x = h;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, x, o); if (lane >= o) x += y; }
                if (p < P) { off0[p] = run + x - h; off[p] = run + x - h; }
                run += __shfl_sync(0xffffffffu, x, 31);
            }
        }
        __syncthreads();
        for (int ch = 0; ch < len; ch += NT) {
            const int i = ch + tid;
            const bool valid = i < len;
            const int p = valid ? (int)pbuf[i] : -1 - lane;
            const unsigned peers = __match_any_sync(0xffffffffu, p);
            const int rank = __popc(peers & ((1u << lane) - 1u));
            const bool leader = valid && rank == 0;
            if (leader) wcnt[warp * P + p] = __popc(peers);
            __syncthreads();
            int before = 0, total = 0;
            if (valid) {
#pragma unroll 8
                for (int w = 0; w < NW; ++w) { const int cw = wcnt[w * P + p]; total += cw; before += w < warp ? cw : 0; }
                sorted[off[p] + before + rank] = tbuf[i];
            }
            __syncthreads();
            if (leader) {
                if (before == 0) off[p] += total;               // first warp of this chunk that holds p
                wcnt[warp * P + p] = 0;
            }
            __syncthreads();
        }
        for (int p = tid; p < P; p += NT) {
            const int a = off0[p], b = a + hist[p];
            float q = qsum[p];
#pragma unroll 8
            for (int j = a; j < b; ++j) q = __fadd_rn(q, sorted[j]);
            qsum[p] = q;
        }
        __syncthreads();
    }
    if (commit) for (int p = tid; p < P; p += NT) t.qP[p] = qsum[p];
}

// 2. The pass itself: one block of kPassThreads threads.  Capacities and demands are handled as
// integers (token counts are whole numbers below 2^24).  The visiting order is staged kPassThreads
// ranks at a time by the whole block: calls none of whose candidates fits the capacities committed
// so far can never obtain a pair (capacity only shrinks) and are dropped, in parallel, so that only
// calls that may still be placed reach the sequential part.  That part is run by ONE warp, in
// optimistic windows of 32 staged calls, with warp shuffles and votes only: a window step costs a
// few hundred cycles, where a step of a block-wide window costs a chain of block barriers.
constexpr int kPassThreads = 1024;
constexpr int kRing = 2048;        // staged calls waiting for the window warp (at most kDrain + kPassThreads)
constexpr int kDrain = 96;         // the windows run once this many calls are staged (or the order is exhausted)
template <int KT>   // candidate slots examined per call: K rounded up to 1, 2, 4 or 8
__global__ void __launch_bounds__(kPassThreads, 1) hx_conflict_kernel(HxTopkBufs tk, HxTables t, int n, int commit,
                                                                      int fused_tail, int32_t* out_assign,
                                                                      const float* free_reset) {
    extern __shared__ __align__(16) unsigned sm[];
    constexpr int NW = kPassThreads / 32;
    static_assert(NW == 32, "the staging step keeps one warp total per lane");
    const int D = t.D;
    // candidate instances of a staged call, 16 bits each; an unused slot points at instance D, which never has room
    using Row = typename std::conditional<(KT > 4), uint4, uint2>::type;
    Row* cd = reinterpret_cast<Row*>(sm);                       // [kRing] candidate instances of the staged calls
    int* cm = reinterpret_cast<int*>(cd + kRing);               // [kRing] their demands
    int* cr = cm + kRing;                                       // [kRing] their call numbers
    int* free_s = cr + kRing;                                   // [D + 1] capacity left after the commits so far
    __shared__ int wsum[NW];
    __shared__ unsigned n_acc_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned lt = (1u << lane) - 1u;
    // the scoring kernel of the next batch may take the other SMs and do the part of its set-up that reads
    // nothing a kernel writes; it waits for this grid before it goes on, and releases its own dependents after
    hx_release_dependents();
    // free KV tokens the pass starts from: the table's, or the values the capacity is restored to ahead of every
    // batch (neither is written by a kernel that may still run: the same grid of the batch before wrote the table)
    const float* free0 = free_reset ? free_reset : t.freeD;
    for (int d = tid; d <= D; d += kPassThreads) free_s[d] = d < D ? __float2int_rd(free0[d]) : -1;
    hx_wait_for_primary();                                      // the visiting order
    __syncthreads();
    auto narrow = [&](const uint4& r) {                         // the slots this instantiation examines
        Row out;
        out.x = r.x; out.y = r.y;
        if constexpr (KT > 4) { out.z = r.z; out.w = r.w; }
        return out;
    };
    auto any_fit = [&](const Row& row, int m) {                  // does any candidate still have room?
        unsigned w[4] = {row.x, row.y, 0u, 0u};
        if constexpr (KT > 4) { w[2] = row.z; w[3] = row.w; }
        int best = -1;
#pragma unroll
        for (int k = 0; k < KT; ++k) best = max(best, free_s[(k & 1) ? w[k >> 1] >> 16 : w[k >> 1] & 0xFFFFu]);
        return best >= m;
    };
    auto first_fit = [&](const Row& row, int m, unsigned& kt, int& dt, int& fr_t) {
        unsigned w[4] = {row.x, row.y, 0u, 0u};
        if constexpr (KT > 4) { w[2] = row.z; w[3] = row.w; }
        int fr[KT]; unsigned dk[KT];
#pragma unroll
        for (int k = 0; k < KT; ++k) {
            dk[k] = (k & 1) ? w[k >> 1] >> 16 : w[k >> 1] & 0xFFFFu;
            fr[k] = free_s[dk[k]];
        }
        kt = kNone; dt = -1; fr_t = 0;
#pragma unroll
        for (int k = KT - 1; k >= 0; --k)
            if (fr[k] >= m) { kt = k; dt = (int)dk[k]; fr_t = fr[k]; }
    };
    // rank scan + tid is in flight two staging steps ahead of its use (a staging step without windows
    // in between is shorter than a round trip to the L2)
    uint4 nrow, nrow2; int nm, nm2; unsigned ncall, ncall2;
    auto fetch = [&](int from, uint4& row, int& m, unsigned& call) {
        const int r = from + tid;
        row = r < n ? __ldcg(tk.od + r) : make_uint4(~0u, ~0u, ~0u, ~0u);
        m = r < n ? __ldcg(tk.om + r) : 0;
        call = r < n ? __ldcg(tk.ocall + r) : 0u;
    };
    fetch(0, nrow, nm, ncall);
    fetch(kPassThreads, nrow2, nm2, ncall2);
    unsigned n_acc = 0;                                         // kept by warp 0 (the same in its 32 lanes)
    unsigned count = 0;                                         // staged calls, the same in every thread
    for (int scan = 0; scan < n; scan += kPassThreads) {
        const Row row = narrow(nrow);
        const int mm = nm;
        const unsigned call = ncall;
        nrow = nrow2; nm = nm2; ncall = ncall2;
        fetch(scan + 2 * kPassThreads, nrow2, nm2, ncall2);
        const bool live = scan + tid < n && any_fit(row, mm);
        const unsigned lm = __ballot_sync(0xffffffffu, live);   // ordered compaction behind the staged calls
        if (lane == 0) wsum[warp] = __popc(lm);
        __syncthreads();
        unsigned wx = (unsigned)wsum[lane];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned y = __shfl_up_sync(0xffffffffu, wx, off);
            if (lane >= off) wx += y;
        }
        const unsigned total = __shfl_sync(0xffffffffu, wx, 31);
        const unsigned before = __shfl_sync(0xffffffffu, wx, warp) - (unsigned)__popc(lm);
        if (live) {
            const unsigned o = count + before + __popc(lm & lt);
            cd[o] = row; cm[o] = mm; cr[o] = (int)call;
        }
        count += total;
        const bool drain = count >= (unsigned)kDrain || scan + kPassThreads >= n;
        __syncthreads();
        if (!drain) continue;
        // One warp walks the staged calls in windows of 32: every lane picks the first candidate that fits the
        // committed capacities.  A lane whose pick no longer fits after the lower lanes that picked the same
        // instance has failed; every lane before the lowest failing lane has taken the decision of the
        // sequential pass and commits; the window restarts at the failing lane, which then sees the reduced
        // capacity.  Lane 0 always fits its pick, so every step advances.
        if (warp == 0) {
            unsigned pos = 0;
            while (pos < count) {
                const unsigned i = pos + lane;
                int m = 0, dt = -1, fr = 0; unsigned kt = kNone;
                if (i < count) { m = cm[i]; first_fit(cd[i], m, kt, dt, fr); }
                const unsigned picked = __ballot_sync(0xffffffffu, dt >= 0);
                if (picked == 0u) { pos += 32; continue; }      // nothing here fits any more
                // A pick can only fail if its instance has less room than the whole window asks for (S): all other
                // picks are safe whatever the lower lanes took.  Instances short of S are resolved one by one: total
                // demand of the lanes that picked it and, if that overflows, an ordered prefix sum to find the
                // first lane that no longer fits.
                const int S = __reduce_add_sync(0xffffffffu, dt >= 0 ? m : 0);
                unsigned f = 32, gm = 0; int v = 0;
                for (unsigned rem = __ballot_sync(0xffffffffu, dt >= 0 && fr < S); rem;) {
                    const int leader = __ffs(rem) - 1;
                    const int d0 = __shfl_sync(0xffffffffu, dt, leader);
                    const int room = __shfl_sync(0xffffffffu, fr, leader);
                    const bool mine = dt == d0;
                    const unsigned g = __ballot_sync(0xffffffffu, mine);
                    if (__reduce_add_sync(0xffffffffu, mine ? m : 0) > room) {
                        int x = mine ? m : 0;
#pragma unroll
                        for (int off = 1; off < 32; off <<= 1) {
                            const int y = __shfl_up_sync(0xffffffffu, x, off);
                            if (lane >= off) x += y;
                        }
                        if (mine) { v = x; gm = g; }
                        const unsigned fail = __ballot_sync(0xffffffffu, mine && x > room);
                        f = min(f, (unsigned)(__ffs(fail) - 1));     // lane 0 never fails
                    }
                    rem &= ~g;
                }
                const bool acc = dt >= 0 && (unsigned)lane < f;
                const unsigned accm = __ballot_sync(0xffffffffu, acc);
                if (acc) {
                    if (gm == 0u) atomicSub(&free_s[dt], m);                              // the whole group fits
                    else if (((gm & accm) >> lane) == 1u) free_s[dt] = fr - v;            // last committing lane of an overflowing group
                }
                if (acc) tk.acc_rk[n_acc + __popc(accm & lt)] = (unsigned)cr[i] | (kt << 24);   // obtained pairs, in visiting order
                n_acc += __popc(accm);
                pos += f;
                __syncwarp();
            }
        }
        count = 0;
        __syncthreads();
    }
    if (tid == 0) { *tk.n_acc = n_acc; n_acc_s = n_acc; }
    __syncthreads();
    n_acc = n_acc_s;
    if (commit) for (int d = tid; d < D; d += kPassThreads) t.freeD[d] = __int2float_rn(free_s[d]);
    if (!fused_tail) return;

    // ---- tail (prefill pools of up to kTailMaxP instances): publish the obtained pairs and add the
    // prefill times to the prefill queues in visiting order, without leaving the block (acc_rk was
    // written by this block: visible after the barrier above).
    unsigned short* pbuf = reinterpret_cast<unsigned short*>(sm);           // [kTailLen]
    float* tbuf = reinterpret_cast<float*>(pbuf + kTailLen);                // [kTailLen]
    float* sorted = tbuf + kTailLen;                                        // [kTailLen]
    publish_and_sum<kPassThreads>(tk, t, n_acc, commit, out_assign, pbuf, tbuf, sorted,
                                         reinterpret_cast<int*>(sorted + kTailLen));
}

// 3. Publish the obtained pairs; gather prefill instance and prefill time in visiting order.
__global__ void hx_finish_kernel(HxTopkBufs tk, int D, int32_t* out_assign) {
    const unsigned i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= *tk.n_acc) return;
    const unsigned rk = tk.acc_rk[i], c = rk & 0xFFFFFFu, k = rk >> 24;
    const int pr = tk.pair[(size_t)c * tk.K + k];
    out_assign[c] = pr;
    tk.acc_p[i] = pr / D;
    tk.acc_t[i] = tk.tpre[(size_t)c * tk.K + k];
}

// 4. Prefill queues: warp p adds, in visiting order, the prefill times of the calls that obtained p.
// The block stages the list in shared memory chunk by chunk; each warp compacts the entries of
// its instance (ballot prefix keeps the order) and one lane adds them one after the other.
constexpr int kQChunk = 1024, kQWarps = 8;
__global__ void __launch_bounds__(32 * kQWarps) hx_qsum_kernel(HxTopkBufs tk, HxTables t) {
    __shared__ int sp[kQChunk];
    __shared__ float st[kQChunk];
    __shared__ float mine[kQWarps][kQChunk];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int p = blockIdx.x * kQWarps + warp;
    const unsigned na = *tk.n_acc;
    float q = p < t.P ? t.qP[p] : 0.f;
    for (unsigned c0 = 0; c0 < na; c0 += kQChunk) {
        const unsigned len = min((unsigned)kQChunk, na - c0);
        __syncthreads();
        for (unsigned i = threadIdx.x; i < len; i += blockDim.x) { sp[i] = __ldg(tk.acc_p + c0 + i); st[i] = __ldg(tk.acc_t + c0 + i); }
        __syncthreads();
        unsigned cnt = 0;
        for (unsigned i0 = 0; i0 < len; i0 += 32) {
            const unsigned i = i0 + lane;
            const bool hit = i < len && sp[i] == p;
            const unsigned b = __ballot_sync(0xffffffffu, hit);
            if (hit) mine[warp][cnt + __popc(b & ((1u << lane) - 1u))] = st[i];
            cnt += __popc(b);
        }
        __syncwarp();
        if (lane == 0) {
#pragma unroll 8
            for (unsigned i = 0; i < cnt; ++i) q = __fadd_rn(q, mine[warp][i]);
        }
        __syncwarp();
    }
    if (lane == 0 && p < t.P) t.qP[p] = q;
}


}  // namespace

cudaError_t hx_launch_conflict(const HxTables& t, const HxTopkBufs& tk, int n_calls, int commit,
                               int32_t* out_assign, int* status, cudaStream_t stream,
                               long long* launches, const float* free_reset) {
    (void)status;
    const int D = t.D, P = t.P;
    const int nb = (n_calls + kOrdThreads - 1) / kOrdThreads;
    // every kernel of the pass is made ready while the one before it drains (released when its blocks exit);
    // each waits for its predecessor before reading what that one wrote
    cudaError_t e = hx_launch_dependent(hx_order_hist_kernel, dim3(nb), dim3(kOrdThreads), 0, stream, tk, n_calls);
    if (e == cudaSuccess) e = hx_launch_dependent(hx_order_scatter_kernel, dim3(nb), dim3(kOrdThreads), 0, stream, tk, n_calls);
    if (e == cudaSuccess) e = hx_launch_dependent(hx_order_rank_kernel, dim3((n_calls + kRankThreads - 1) / kRankThreads), dim3(kRankThreads), 0, stream, tk, n_calls, (unsigned)D);
    if (e != cudaSuccess) return e;
    const int fused = P <= kTailMaxP;                               // pairs published and queues summed inside the pass
    const size_t smRing = (size_t)kRing * 24 + (size_t)(D + 1) * 4;
    const size_t smTail = fused ? (size_t)kTailLen * 10 + (size_t)(4 + kPassThreads / 32) * P * 4 : 0;
    const size_t smC = smRing > smTail ? smRing : smTail;
    auto pass = tk.K <= 1 ? hx_conflict_kernel<1> : tk.K <= 2 ? hx_conflict_kernel<2>
              : tk.K <= 4 ? hx_conflict_kernel<4> : hx_conflict_kernel<8>;
    static size_t allowed_pass[4][64];
    e = hx_opt_in_smem(pass, smC, allowed_pass[tk.K <= 1 ? 0 : tk.K <= 2 ? 1 : tk.K <= 4 ? 2 : 3], 40 * 1024);
    if (e != cudaSuccess) return e;
    e = hx_launch_dependent(pass, dim3(1), dim3(kPassThreads), smC, stream, tk, t, n_calls, commit, fused, out_assign, free_reset);
    if (e != cudaSuccess) return e;
    *launches += 4;
    if (!fused) {
        hx_finish_kernel<<<(n_calls + 255) / 256, 256, 0, stream>>>(tk, D, out_assign);
        *launches += 1;
        if (commit) {
            hx_qsum_kernel<<<(P + kQWarps - 1) / kQWarps, 32 * kQWarps, 0, stream>>>(tk, t);
            *launches += 1;
        }
    }
    return cudaGetLastError();
}
