// Decode-stage scheduler (paper Section 5.4, "Decode scheduling with instance
// locks", "Adaptive greedy decode assignment"; Section 6 names the state it
// works on: decode token-capacity intervals).
//
// Calls whose KV cache has arrived wait for decode admission.  Until the queue
// is empty: for every waiting call find, on each legal decode instance (its
// lock if it has one, else every instance with m(c) <= Cap(d), Eq. 3-4), the
// earliest start >= ready at which m(c) tokens are free for the whole decode;
// its Delta_D is the earliest projected finish over those instances, its ratio
// R = (elapsed + Delta_D) / H (Eq. 2); the call with the largest R (lower index
// among equals) is assigned, its interval is added to the chosen instance.
// With HX_FLAG_ONE_PASS (the lightweight ordering Section 5.4 falls back to,
// Section 5.3 last sentence) R keeps the value of the first projection, against
// the snapshot alone: the same loop then visits the calls in the order of that
// score, each placed by its projection against the state left by the calls
// before it.
//
// Tokens in use on an instance are a step function of time: breakpoints
// t[0] = 0 < t[1] < ... and usage u[k] on [t[k], t[k+1]); the last segment runs
// to infinity.  A search walks the segments from the one that holds the ready
// time: a segment without room moves the candidate start to its end, and the
// candidate is accepted once a segment ends at or after candidate + duration.
// One persistent block; one warp projects one call with the lanes over the
// instances (two or four warps share a call when few calls are listed); adding
// an interval only delays starts on that instance, so only
// calls whose best instance it was are projected again.
//
// Long queues run on a thread-block cluster: call c belongs to block c mod kCluster, every block
// keeps its own copy of the step functions, and per iteration every block writes its most urgent call
// with its interval into all blocks through distributed shared memory, behind one cluster barrier (two
// sets of slots used in turn); all blocks reduce the same candidates and insert the same interval, so the copies stay identical and
// every exit is taken by all blocks.
#include <cooperative_groups.h>

#include "hx_internal.h"

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
#define HX_INF __int_as_float(0x7f800000)
#define HX_NEG_INF __int_as_float(0xff800000)
constexpr int kDead = -2, kNoInst = -1;

struct DecodeParams {
    HxTables t;
    HxConstTables ct;
    HxDagView dag;
    HxStepFns base, work;      // usage step functions: snapshot and simulated state
    const hx_call* calls;
    const int32_t* lock;
    const float* ready;
    int n, flags, commit;
    int pool_T;                // entries of the shared-memory pool of breakpoints (POOL variant)
    int32_t* out_inst;
    float* out_start;
    float* out_ratio;
    int32_t* out_order;
    int* status;
};

// Segment index holding x in t[0..K): the largest k with t[k] <= x.  Executed by one warp: up to 1,024
// breakpoints in two rounds (every lane samples the start of one stretch, then the lanes share the stretch that
// holds x), longer arrays 32 breakpoints at a time.
__device__ __forceinline__ int warp_find_segment(const float* t, int K, float x, int lane) {
    if (K <= 1024) {
        const int stride = (K + 31) >> 5;
        const int s = lane * stride;
        const int b = __popc(__ballot_sync(0xffffffffu, s < K && t[s] <= x)) - 1;     // t[0] = 0 <= x always
        const int i = b * stride + lane;
        return b * stride + __popc(__ballot_sync(0xffffffffu, lane < stride && i < K && t[i] <= x)) - 1;
    }
    int cnt = 0;
    for (int i0 = 0; i0 < K; i0 += 32) {
        const int i = i0 + lane;
        cnt += __popc(__ballot_sync(0xffffffffu, i < K && t[i] <= x));
    }
    return cnt - 1;
}

// Make x a breakpoint of instance arrays (t, u, K); returns its index.  One warp.
__device__ int warp_cut(float* t, float* u, int& K, float x, int lane) {
    const int k = warp_find_segment(t, K, x, lane);
    if (t[k] == x) return k;
    // shift (k, K) up by one, from the top, a warp-wide chunk at a time
    for (int hi = K; hi > k + 1; hi -= 32) {
        const int i = hi - 1 - lane;                    // hi-1, hi-2, ... > k
        float tv = 0.f, uv = 0.f;
        const bool mv = i > k;
        if (mv) { tv = t[i]; uv = u[i]; }
        __syncwarp();
        if (mv) { t[i + 1] = tv; u[i + 1] = uv; }
        __syncwarp();
    }
    if (lane == 0) { t[k + 1] = x; u[k + 1] = u[k]; }
    __syncwarp();
    ++K;
    return k + 1;
}

// POOL: the step functions of all instances live in one shared-memory pool (their total length is bounded by
// the snapshot plus two breakpoints per queued call, whatever the split between instances); an instance whose
// region is full makes warp 0 lay the regions out again in the second half of the pool.  Without POOL every
// block works on its own copy in global memory, each instance with room for the worst case.
template <int NC, bool POOL>   // NC: blocks of the cluster (1 = a plain single block)
__global__ void __launch_bounds__(kThreads, 1) hx_decode_kernel(const __grid_constant__ DecodeParams prm) {
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ float red_v[kWarps];
    __shared__ int red_c[kWarps];
    __shared__ int s_ndirty, s_cur, s_full;
    __shared__ float part_v[kWarps], part_s[kWarps];   // partial projections of warps that share a call
    __shared__ int part_d[kWarps];
    // most urgent call of every block with its interval: ratio, call, instance (int bits), start, finish, demand;
    // written by the owner block into every block, two sets used in turn by the iterations
    __shared__ float x_cand[2][NC][6];
    const HxTables& T = prm.t;
    const int D = T.D;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cap = prm.work.cap;
    int rank = 0;
    if (NC > 1) rank = (int)cg::this_cluster().block_rank();
    const int n_all = prm.n;
    const int n = (n_all - rank + NC - 1) / NC;                // calls of this block: c = li * NC + rank
    float* const wt = prm.work.t + (size_t)rank * D * cap;      // this block's copy of the step functions
    float* const wu = prm.work.u + (size_t)rank * D * cap;

    float* capDs = reinterpret_cast<float*>(smem);              // [D]
    int* typeDs = reinterpret_cast<int*>(capDs + D);            // [D]
    int* Ks = typeDs + D;                                       // [D] breakpoints per instance
    float* umax = reinterpret_cast<float*>(Ks + D);             // [D] largest usage of any segment of the instance
    float* cn = umax + D;                                       // [n]
    float* co = cn + n;
    float* cel = co + n;
    float* cH = cel + n;
    float* cready = cH + n;
    float* cR = cready + n;                                     // projected ratio, -inf if it cannot be taken
    float* cstart = cR + n;
    float* cfin = cstart + n;
    int* cbest = reinterpret_cast<int*>(cfin + n);              // best instance, kNoInst, kDead
    int* clock_ = cbest + n;                                    // lock (-1 = free)
    int* cmodel = clock_ + n;
    unsigned short* dirty = reinterpret_cast<unsigned short*>(cmodel + n);
    const int PT = prm.pool_T;
    int* roff = reinterpret_cast<int*>(dirty + ((n + 1) & ~1));  // [D+1] regions of the pool (POOL)
    int* roff2 = roff + D + 1;                                    // [D+1] the next layout while regions move
    float* pool_t = reinterpret_cast<float*>(roff2 + D + 1);     // [2][PT] breakpoints, two halves
    float* pool_u = pool_t + 2 * (size_t)PT;                    // [2][PT] usage
    // step function of instance d in the simulated state
    auto seg_t = [&](int d) -> float* { return POOL ? pool_t + (size_t)s_cur * PT + roff[d] : wt + (size_t)d * cap; };
    auto seg_u = [&](int d) -> float* { return POOL ? pool_u + (size_t)s_cur * PT + roff[d] : wu + (size_t)d * cap; };

    for (int d = tid; d < D; d += kThreads) {
        capDs[d] = T.capD[d]; typeDs[d] = T.typeD[d];
        Ks[d] = prm.base.K[d];
    }
    if (tid == 0) { s_cur = 0; s_full = 0; }
    __syncthreads();
    if (POOL && tid == 0) {                                     // every instance its breakpoints plus an equal share of the rest
        int sum = 0;
        for (int d = 0; d < D; ++d) sum += Ks[d];
        const int share = max(0, (PT - sum) / D);
        int o = 0;
        for (int d = 0; d < D; ++d) { roff[d] = o; o += Ks[d] + share; }
        roff[D] = o;
    }
    __syncthreads();
    for (int d = warp; d < D; d += kWarps) {                    // simulated state starts as the snapshot
        float* tt = seg_t(d); float* uu = seg_u(d);
        float mx = 0.f;
        for (int i = lane; i < Ks[d]; i += 32) {
            tt[i] = prm.base.t[(size_t)d * prm.base.cap + i];
            const float uv = prm.base.u[(size_t)d * prm.base.cap + i];
            uu[i] = uv; mx = fmaxf(mx, uv);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (lane == 0) umax[d] = mx;
    }
    for (int c = tid; c < n; c += kThreads) {
        const int gcall = c * NC + rank;
        const uint4 raw = __ldg(reinterpret_cast<const uint4*>(prm.calls) + gcall);
        bool bad = raw.y >= (unsigned)T.M;
        float el = 0.f, H = 1.f;
        if (!(prm.flags & HX_FLAG_NO_DAG)) {
            if (raw.x < prm.dag.n_nodes) { const uint32_t w = prm.dag.node_wf[raw.x]; el = prm.dag.elapsed[w]; H = prm.dag.H[w]; }
            else bad = true;
        }
        const int lk = prm.lock ? prm.lock[gcall] : -1;
        const float rd = prm.ready ? prm.ready[gcall] : 0.f;
        if (lk >= D || !(rd >= 0.f) || rd == HX_INF) bad = true;
        if (bad) atomicExch(prm.status, HX_ERR_INVALID_ARG);
        cn[c] = __uint_as_float(raw.z); co[c] = __uint_as_float(raw.w);
        cmodel[c] = bad ? 0 : (int)raw.y;
        cel[c] = el; cH[c] = H; cready[c] = rd; clock_[c] = lk < 0 ? -1 : lk;
        cR[c] = HX_NEG_INF; cstart[c] = HX_INF; cfin[c] = HX_INF;
        cbest[c] = bad ? kDead : kNoInst;
        dirty[c] = (unsigned short)c;
        prm.out_inst[gcall] = -1; prm.out_start[gcall] = HX_INF; prm.out_ratio[gcall] = HX_INF; prm.out_order[gcall] = -1;
    }
    if (tid == 0) s_ndirty = n;
    __syncthreads();

    int it = 0;
    // result of a projection: instance, start, finish and ratio of call c (no instance: it can never be taken)
    auto record = [&](int c, float best, float bs, int bd) {
        if (bd != 0x7fffffff) {
            cbest[c] = bd; cstart[c] = bs; cfin[c] = best;
            // one-pass ordering: the score of the first projection (against the snapshot) stays
            if (it == 0 || !(prm.flags & HX_FLAG_ONE_PASS)) cR[c] = __fdiv_rn(__fadd_rn(cel[c], best), cH[c]);
        } else { cbest[c] = kNoInst; cR[c] = HX_NEG_INF; }
    };
    for (; it < n_all; ++it) {
        // (1) project the listed calls: one warp per call, lanes over the decode instances
        const int nd = s_ndirty;
        // few listed calls: two or four warps share a call, each walking a part of its instances; the parts are
        // put together after the barrier
        const int split = nd * 4 <= kWarps ? 4 : nd * 2 <= kWarps ? 2 : 1;
        for (int w = warp; w < nd * split; w += kWarps) {
            const int i = w / split, part = w - i * split;
            const int c = dirty[i];
            if (cbest[c] == kDead) continue;
            const float nt = cn[c], ot = co[c];
            const int mdl = cmodel[c];
            const float omega = prm.ct.omega[mdl], kappa = prm.ct.kappa[mdl];
            const float ctx = __fmaf_rn(0.5f, __fsub_rn(ot, 1.0f), nt);
            const float step = __fmaf_rn(kappa, ctx, omega);
            const float m = __fadd_rn(nt, ot);
            const float rd = cready[c];
            const int lk = clock_[c];
            float best = HX_INF, bs = 0.f; int bd = 0x7fffffff;
            for (int d0 = 0; d0 < D; d0 += 32) {
                const int d = d0 + lane;
                bool walk = false; float tau = 0.f;
                if (d < D && !((lk >= 0 && lk != d) || !(m <= capDs[d]))) {
                    tau = __fmul_rn(__fmul_rn(ot, step), prm.ct.invB[typeDs[d]]);
                    if (__fadd_rn(umax[d], m) <= capDs[d]) {
                        // room in every segment (token counts are whole numbers, so the sum is exact): the walk
                        // would accept the ready time itself
                        const float fin = __fadd_rn(rd, tau);
                        if (part == 0 && fin < best) { best = fin; bs = rd; bd = d; }
                    } else {
                        walk = true;
                    }
                }
                // the instances that have to be walked, one after the other, the warp on 32 segments at a time:
                // the sequential walk stops at the first segment that either has no room (the candidate start moves
                // to the end of the run of such segments) or ends at or after candidate + duration (accepted)
                unsigned todo = __ballot_sync(0xffffffffu, walk);
                for (int turn = 0; todo; ++turn) {
                    const int src = __ffs(todo) - 1;
                    todo &= todo - 1;
                    if (turn % split != part) continue;           // another warp's instance
                    const int dd = d0 + src;
                    const float tau_d = __shfl_sync(0xffffffffu, tau, src);
                    const float* tt = seg_t(dd);
                    const float* uu = seg_u(dd);
                    const int K = Ks[dd];
                    const float capd = capDs[dd];
                    int k = warp_find_segment(tt, K, rd, lane);           // segment that holds the ready time
                    float cand = rd, fin = HX_INF;
                    for (;;) {
                        const int i = k + lane;
                        const bool in = i < K;
                        const float end_i = (in && i + 1 < K) ? tt[i + 1] : HX_INF;
                        const bool viol = in && __fadd_rn(uu[i], m) > capd;
                        const float f = __fadd_rn(cand, tau_d);
                        const bool acc = in && !viol && end_i >= f;
                        const unsigned mv = __ballot_sync(0xffffffffu, viol), ma = __ballot_sync(0xffffffffu, acc);
                        const int fv = mv ? __ffs(mv) - 1 : 32, fa = ma ? __ffs(ma) - 1 : 32;
                        if (fa < fv) { fin = f; break; }
                        if (fv == 32) {                                   // no decision among these 32 segments
                            k += 32;
                            if (k >= K) break;                            // not reached: the last segment ends at +inf
                            continue;
                        }
                        const unsigned rest = ~(mv >> fv);                // zero bits: the run of full segments goes on
                        const int len = rest ? __ffs(rest) - 1 : 32 - fv;
                        const int last = fv + len - 1;
                        if (k + last + 1 >= K) break;                     // the last segment has no room: no start at all
                        cand = __shfl_sync(0xffffffffu, end_i, last);
                        k += last + 1;
                    }
                    if (lane == src && fin < best) { best = fin; bs = cand; bd = dd; }   // ascending d per lane: lowest d kept
                }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, best, off);
                const float os = __shfl_xor_sync(0xffffffffu, bs, off);
                const int od = __shfl_xor_sync(0xffffffffu, bd, off);
                if (ov < best || (ov == best && od < bd)) { best = ov; bs = os; bd = od; }
            }
            if (lane == 0) {
                if (split > 1) { part_v[w] = best; part_s[w] = bs; part_d[w] = bd; }
                else record(c, best, bs, bd);
            }
        }
        __syncthreads();
        if (split > 1) {
            if (tid < nd && cbest[dirty[tid]] != kDead) {
                float best = HX_INF, bs = 0.f; int bd = 0x7fffffff;
                for (int k = 0; k < split; ++k) {
                    const float ov = part_v[tid * split + k]; const int od = part_d[tid * split + k];
                    if (ov < best || (ov == best && od < bd)) { best = ov; bs = part_s[tid * split + k]; bd = od; }
                }
                record(dirty[tid], best, bs, bd);
            }
            __syncthreads();
        }
        // (2) most urgent waiting call of this block
        float rv = HX_NEG_INF; int rc = 0x7fffffff;
        for (int c = tid; c < n; c += kThreads) {
            const float r = cR[c];
            if (r > rv) { rv = r; rc = c * NC + rank; }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, rv, off);
            const int oc = __shfl_xor_sync(0xffffffffu, rc, off);
            if (ov > rv || (ov == rv && oc < rc)) { rv = ov; rc = oc; }
        }
        if (lane == 0) { red_v[warp] = rv; red_c[warp] = rc; }
        __syncthreads();
        float (*xc)[6] = x_cand[it & 1];
        if (warp == 0) {
            rv = red_v[lane]; rc = red_c[lane];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, rv, off);
                const int oc = __shfl_xor_sync(0xffffffffu, rc, off);
                if (ov > rv || (ov == rv && oc < rc)) { rv = ov; rc = oc; }
            }
            if (lane == 0) {
                // the block's candidate with its interval (instance, start, finish, demand), published in every block
                float cand[6] = {rv, __int_as_float(rc), 0.f, 0.f, 0.f, 0.f};
                if (rc != 0x7fffffff) {
                    const int li = rc / NC;
                    cand[2] = __int_as_float(cbest[li]); cand[3] = cstart[li]; cand[4] = cfin[li];
                    cand[5] = __fadd_rn(cn[li], co[li]);
                }
                if (NC > 1) {
                    cg::cluster_group cl = cg::this_cluster();
                    for (int r = 0; r < NC; ++r) {
                        float* dst = cl.map_shared_rank(&xc[rank][0], r);
#pragma unroll
                        for (int k = 0; k < 6; ++k) dst[k] = cand[k];
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < 6; ++k) xc[0][k] = cand[k];
                }
                s_ndirty = 0;                                  // the list of this iteration has been read by everybody
            }
        }
        // one barrier per iteration: a block that runs ahead writes the other set of candidates, and cannot get
        // past the next barrier before every block has read this one
        if (NC > 1) cg::this_cluster().sync(); else __syncthreads();      // every thread of every block
        // every warp of every block reduces the same list: nothing to hand round inside the block
        rv = lane < NC ? xc[lane][0] : HX_NEG_INF;
        rc = lane < NC ? __float_as_int(xc[lane][1]) : 0x7fffffff;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, rv, off);
            const int oc = __shfl_xor_sync(0xffffffffu, rc, off);
            if (ov > rv || (ov == rv && oc < rc)) { rv = ov; rc = oc; }
        }
        if (rc == 0x7fffffff) break;                            // nobody left that fits anywhere: all blocks leave
        const float* win = xc[rc % NC];
        const int ds = __float_as_int(win[2]);
        if (warp == 0) {
            // (3) commit (warp 0 of every block): add the interval [start, finish) with m tokens to the block's copy
            const int d = ds;
            const float st = win[3], en = win[4], m = win[5];
            if (lane == 0 && rc % NC == rank) {                 // the block that owns the call records the result
                const int li = rc / NC;
                prm.out_inst[rc] = d; prm.out_start[rc] = st; prm.out_ratio[rc] = rv; prm.out_order[it] = rc;
                cbest[li] = kDead; cR[li] = HX_NEG_INF;
            }
            int K = Ks[d];
            bool room = POOL ? K + 2 <= roff[d + 1] - roff[d] : K + 2 <= cap;
            if (POOL && !room) {
                // lay the regions out again in the other half, after two entries set aside for this commit
                if (lane == 0) {
                    int sum = 0;
                    for (int e = 0; e < D; ++e) sum += Ks[e];
                    const int free_now = PT - sum - 2;
                    if (free_now >= 0) {
                        // half of what is free goes to the instance that ran full (it is the popular one and
                        // would be back soon with an equal share), the rest is split evenly
                        const int mine = free_now / 2, share = (free_now - mine) / D;
                        int o = 0;
                        for (int e = 0; e < D; ++e) { roff2[e] = o; o += Ks[e] + share + (e == d ? 2 + mine : 0); }
                        roff2[D] = o;
                    } else {
                        roff2[D] = -1;                       // the pool itself is full: the host sized it too small
                    }
                }
                __syncwarp();
                if (roff2[D] >= 0) {
                    const int cur = s_cur;
                    for (int e = 0; e < D; ++e) {
                        const float* ot = pool_t + (size_t)cur * PT + roff[e];
                        const float* ou = pool_u + (size_t)cur * PT + roff[e];
                        float* nt2 = pool_t + (size_t)(cur ^ 1) * PT + roff2[e];
                        float* nu2 = pool_u + (size_t)(cur ^ 1) * PT + roff2[e];
                        for (int i = lane; i < Ks[e]; i += 32) { nt2[i] = ot[i]; nu2[i] = ou[i]; }
                    }
                    __syncwarp();
                    for (int e = lane; e <= D; e += 32) roff[e] = roff2[e];
                    if (lane == 0) s_cur = cur ^ 1;
                    __syncwarp();
                    room = true;
                }
            }
            float* tt = seg_t(d);
            float* uu = seg_u(d);
            __syncwarp();
            if (!room) {                                    // cannot happen with the capacity the host sizes
                if (lane == 0) { atomicExch(prm.status, HX_ERR_INVALID_ARG); s_full = 1; }
            } else {
                const int a = warp_cut(tt, uu, K, st, lane);
                const int b = warp_cut(tt, uu, K, en, lane);
                float mx = 0.f;
                for (int k = a + lane; k < b; k += 32) { const float uv = __fadd_rn(uu[k], m); uu[k] = uv; mx = fmaxf(mx, uv); }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                if (lane == 0) { Ks[d] = K; umax[d] = fmaxf(umax[d], mx); }
            }
        } else {
            // meanwhile the other warps list the calls whose best instance gets the interval (a call that is being
            // taken right now may be listed: the projection skips it)
            for (int c = tid - 32; c < n; c += kThreads - 32)
                if (cbest[c] == ds) dirty[atomicAdd(&s_ndirty, 1)] = (unsigned short)c;
        }
        __syncthreads();
        if (s_full) break;                                      // an instance's region ran full (same in every block)
    }
    if (prm.commit && rank == 0) {                              // the simulated state becomes the snapshot
        __syncthreads();
        for (int d = warp; d < D; d += kWarps) {
            const int K = min(Ks[d], prm.base.cap);
            const float* tt = seg_t(d); const float* uu = seg_u(d);
            for (int i = lane; i < K; i += 32) {
                prm.base.t[(size_t)d * prm.base.cap + i] = tt[i];
                prm.base.u[(size_t)d * prm.base.cap + i] = uu[i];
            }
            if (lane == 0) prm.base.K[d] = K;
        }
    }
    if (NC > 1) cg::this_cluster().sync();     // no block leaves while another may still write into it
}

}  // namespace

constexpr int kCluster = 8;                    // blocks of the cluster used for long queues
constexpr int kClusterFrom = 256;              // queues longer than this use the cluster

static size_t decode_smem(const HxTables& t, int calls_per_block) {
    return (4 * (size_t)t.D + 11 * (size_t)calls_per_block) * 4 + (size_t)calls_per_block * 2 + 16;
}
// With the pool of breakpoints behind the per-call state: two layouts of pool_T entries, times and usage.
static size_t decode_pool_smem(const HxTables& t, int calls_per_block, int pool_T) {
    return decode_smem(t, calls_per_block) + 4 + 2 * ((size_t)t.D + 1) * 4 + 4 * (size_t)pool_T * 4;
}

size_t hx_decode_smem_bytes(const HxTables& t, int n_calls) { return decode_smem(t, n_calls); }

int hx_decode_replicas() { return kCluster; }

template <int NC, bool POOL>
static cudaError_t launch_variant(const DecodeParams& prm, size_t smem, cudaStream_t stream, bool* launched) {
    static size_t allowed[64];
    *launched = false;
    cudaError_t e = hx_opt_in_smem(hx_decode_kernel<NC, POOL>, smem, allowed, 40 * 1024);
    if (e != cudaSuccess) return e;
    if (NC == 1) {
        hx_decode_kernel<NC, POOL><<<1, kThreads, smem, stream>>>(prm);
        *launched = true;
        return cudaGetLastError();
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(NC); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = NC; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&n_clusters, hx_decode_kernel<NC, POOL>, &cfg) != cudaSuccess || n_clusters < 1) {
        (void)cudaGetLastError();              // the device cannot host the cluster: the caller falls back to one block
        return cudaSuccess;
    }
    *launched = true;
    return cudaLaunchKernelEx(&cfg, hx_decode_kernel<NC, POOL>, prm);
}

cudaError_t hx_launch_decode(const HxTables& t, const HxConstTables& ct, const HxDagView& dag,
                             const HxStepFns& base, const HxStepFns& work, int k_total,
                             const hx_call* calls, const int32_t* lock, const float* ready, int n_calls,
                             int flags, int commit, int32_t* out_inst, float* out_start, float* out_ratio,
                             int32_t* out_order, int* status, cudaStream_t stream, long long* launches) {
    DecodeParams prm;
    prm.t = t; prm.ct = ct; prm.dag = dag; prm.base = base; prm.work = work;
    prm.calls = calls; prm.lock = lock; prm.ready = ready; prm.n = n_calls; prm.flags = flags; prm.commit = commit;
    prm.out_inst = out_inst; prm.out_start = out_start; prm.out_ratio = out_ratio; prm.out_order = out_order;
    prm.status = status;
    // all breakpoints the run can create: those of the snapshot, two per queued call, some slack per instance
    const long long pool = (long long)k_total + 2LL * n_calls + 4LL * t.D;
    const size_t kPoolLimit = 200 * 1024;
    cudaError_t e;
    bool launched = false;
    if (n_calls > kClusterFrom) {
        const int cpb = (n_calls + kCluster - 1) / kCluster;
        if (pool < (1 << 24) && decode_pool_smem(t, cpb, (int)pool) <= kPoolLimit) {
            prm.pool_T = (int)pool;
            e = launch_variant<kCluster, true>(prm, decode_pool_smem(t, cpb, (int)pool), stream, &launched);
        } else {
            prm.pool_T = 0;
            e = launch_variant<kCluster, false>(prm, decode_smem(t, cpb), stream, &launched);
        }
        if (e != cudaSuccess) return e;
        if (launched) { ++*launches; return cudaSuccess; }
    }
    if (pool < (1 << 24) && decode_pool_smem(t, n_calls, (int)pool) <= kPoolLimit) {
        prm.pool_T = (int)pool;
        e = launch_variant<1, true>(prm, decode_pool_smem(t, n_calls, (int)pool), stream, &launched);
    } else {
        prm.pool_T = 0;
        e = launch_variant<1, false>(prm, decode_smem(t, n_calls), stream, &launched);
    }
    if (e == cudaSuccess) ++*launches;
    return e;
}
