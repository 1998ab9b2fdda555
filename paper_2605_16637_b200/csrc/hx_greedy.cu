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
// Where shared memory allows, every call also keeps, per prefill instance p, the
// earliest finish over the decode instances and where it is reached.  Such a row
// stays right until a commit lands on p (a version counter per prefill instance
// tells) or its decode instance no longer has room for the call (room only
// shrinks, so the test at the time of use is exact); a re-projection recomputes
// the rows that are not, D candidates each, and takes the minimum over the rows
// instead of walking all P x D pairs: three block-wide passes over the listed
// calls (find the rows, recompute them with four lanes each, reduce).
//
// Long queues run on a thread-block cluster of kCluster blocks (one SM each): call c belongs to
// block c mod kCluster, every block keeps its own copy of the small simulated state, and per
// iteration every block writes its most urgent call, with what its commit would change, into all
// blocks through distributed shared memory, behind one cluster barrier (two sets of slots used in
// turn).  All blocks reduce the same candidates and apply the same commit, so their copies stay
// identical and every exit is taken by all of them.
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
constexpr int kItemCap = 4096;         // rows recomputed per slice of the re-projection
constexpr unsigned kNoRow = 0xFFFFu;   // no decode instance has room for the call (row of a prefill instance)

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

// MODE >= 1 (CACHE): the per-class prefill and decode times, the KV bytes and the demand of every call are computed
// once and kept in shared memory ([class][call]); without it a warp recomputes them whenever it re-projects a call.
// MODE 2 (ROWS): the per-prefill-instance minima of every call are kept as well.
template <int NC, int MODE>     // NC: blocks of the cluster (1 = a plain single block)
__global__ void __launch_bounds__(kThreads, 1) hx_greedy_kernel(const __grid_constant__ GreedyParams prm) {
    extern __shared__ __align__(16) unsigned char smem[];
    constexpr bool CACHE = MODE >= 1, ROWS = MODE == 2;
    __shared__ float red_v[kWarps];
    __shared__ int red_c[kWarps];
    __shared__ int s_call, s_p, s_d, s_ndirty, s_nitems;
    // most urgent call of every block with what its commit would change: ratio, call, p, d (int bits), prefill
    // time, demand; written by the owner block into every block, two sets used in turn by the iterations
    __shared__ float x_cand[2][NC][6];
    const HxTables& T = prm.t;
    const int P = T.P, D = T.D, G = T.G;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int rank = 0;
    if (NC > 1) rank = (int)cg::this_cluster().block_rank();
    const int n_all = prm.n;
    const int n = (n_all - rank + NC - 1) / NC;                // calls of this block: c = li * NC + rank

    float* invL = reinterpret_cast<float*>(smem);              // [P][D]; [D][P] with ROWS
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
    const int nst = n | 1;                                     // odd stride: the classes of one call lie in different banks
    float* tpreC = cmm + (CACHE ? n : 0);                      // [G][nst] prefill time per GPU class (CACHE)
    float* tdecC = tpreC + (CACHE ? (size_t)G * nst : 0);      // [G][nst] decode time per GPU class (CACHE)
    float* rowmin = tdecC + (CACHE ? (size_t)G * nst : 0);     // [P][n] earliest finish of the call on prefill instance p (ROWS)
    unsigned* items = reinterpret_cast<unsigned*>(rowmin + (ROWS ? (size_t)n * P : 0));   // [kItemCap] rows to compute again: call << 16 | p
    unsigned short* rowarg = reinterpret_cast<unsigned short*>(items + (ROWS ? kItemCap : 0));   // [P][n] its decode instance, kNoRow = none
    unsigned short* rowver = rowarg + (ROWS ? (size_t)n * P : 0);   // [P][n] version of p the row was computed at
    unsigned short* verP = rowver + (ROWS ? (size_t)n * P : 0);     // [P] commits on p so far (at most one per call: no wrap)
    unsigned short* dirty = verP + (ROWS ? ((P + 1) & ~1) : 0);     // [n] calls to re-project

    for (int i = tid; i < P * D; i += kThreads) { const int p = i / D, d = i - p * D; invL[ROWS ? d * P + p : i] = T.invLT[(size_t)d * T.Ppad + p]; }
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
                tpreC[g * nst + c] = fmaxf(__fmul_rn(__fmaf_rn(__fmul_rn(nt, prm.ct.psi[mdl]), nt, __fmul_rn(nt, phi)), iF), __fmul_rn(__fadd_rn(omega, kvB), iB));
                tdecC[g * nst + c] = __fmul_rn(__fmul_rn(ot, step), iB);
            }
        }
        prm.out_assign[gcall] = -1; prm.out_ratio[gcall] = HX_INF; prm.out_order[gcall] = -1;
        if (prm.out_delta) prm.out_delta[gcall] = HX_INF;
    }
    if (ROWS) {
        for (int p = tid; p < P; p += kThreads) verP[p] = 0;
        for (int i = tid; i < n * P; i += kThreads) rowver[i] = 0xFFFFu;      // no row computed yet
    }
    if (tid == 0) s_ndirty = n;
    __syncthreads();

    for (int it = 0; it < n_all; ++it) {
        // (1) re-project the listed calls: one warp per call, lanes over the pairs
        const int nd = s_ndirty;
        if (ROWS) {
            // the listed calls in slices whose rows fit the item list
            const int slice = max(1, kItemCap / P);
            for (int s0 = 0; s0 < nd; s0 += slice) {
                const int cnt = min(slice, nd - s0);
                if (tid == 0) s_nitems = 0;
                __syncthreads();
                // (1a) which rows of which calls are no longer right: one thread per (call, prefill instance)
                const int total = cnt * P;
                auto check = [&](int t, unsigned& item) {      // is row t / cnt of listed call t % cnt no longer right?
                    if (t >= total) return false;
                    const int p = t / cnt, c = dirty[s0 + t - p * cnt];
                    if (cpair[c] == kDead) return false;       // rejected at load time
                    item = ((unsigned)c << 16) | (unsigned)p;
                    if (rowver[p * n + c] != verP[p]) return true;              // never computed, or a commit on p since
                    const unsigned rd = rowarg[p * n + c];
                    return rd != kNoRow && !(cmm[c] <= frees[rd]);
                };
                for (int t0 = warp * 32; t0 < total; t0 += 2 * kThreads) {     // two rows per thread: their loads overlap
                    unsigned item0 = 0, item1 = 0;
                    const bool st0 = check(t0 + lane, item0), st1 = check(t0 + kThreads + lane, item1);
                    const unsigned v0 = __ballot_sync(0xffffffffu, st0), v1 = __ballot_sync(0xffffffffu, st1);
                    int base = 0;
                    if (lane == 0 && (v0 | v1)) base = atomicAdd(&s_nitems, __popc(v0) + __popc(v1));
                    base = __shfl_sync(0xffffffffu, base, 0);
                    const unsigned below = (1u << lane) - 1u;
                    if (st0) items[base + __popc(v0 & below)] = item0;
                    if (st1) items[base + __popc(v0) + __popc(v1 & below)] = item1;
                }
                __syncthreads();
                // (1b) those rows again: four lanes per row, each over a quarter of the decode instances (everything
                // that depends on d alone is read by all rows alike; the link table is stored [d][p] here)
                const int nitems = s_nitems;
                const int ql = lane & 3;
                for (int b0 = warp * 8; b0 < nitems; b0 += kWarps * 8) {
                    const int ix = b0 + (lane >> 2);
                    const bool live = ix < nitems;
                    const unsigned item = live ? items[ix] : 0u;
                    const int c = item >> 16, pp = item & 0xFFFFu;
                    const float kvB = ckv[c], m = cmm[c];
                    const float A = __fadd_rn(qPs[pp], tpreC[typePs[pp] * nst + c]);
                    float fb = HX_INF; unsigned db = kNoRow;
#pragma unroll 4
                    for (int d = ql; d < D; d += 4) {                              // no branch: the loads of several d overlap
                        const bool fits = m <= capDs[d] && m <= frees[d];
                        const float ready = __fmaf_rn(kvB, invL[d * P + pp], A);
                        const float fin = fits ? __fadd_rn(fmaxf(ready, qDs[d]), tdecC[typeDs[d] * nst + c]) : HX_INF;
                        if (fin < fb) { fb = fin; db = (unsigned)d; }              // ascending d: keeps the lowest
                    }
#pragma unroll
                    for (int off = 2; off > 0; off >>= 1) {                       // stays inside the four lanes
                        const float of = __shfl_xor_sync(0xffffffffu, fb, off);
                        const unsigned od = __shfl_xor_sync(0xffffffffu, db, off);
                        if (of < fb || (of == fb && od < db)) { fb = of; db = od; }
                    }
                    if (live && ql == 0) {
                        rowmin[pp * n + c] = fb; rowarg[pp * n + c] = (unsigned short)db; rowver[pp * n + c] = verP[pp];
                    }
                }
                __syncthreads();
                // (1c) the earliest finish over the rows: one thread per call, lowest p among equals
                for (int i = tid; i < cnt; i += kThreads) {
                    const int c = dirty[s0 + i];
                    if (cpair[c] == kDead) continue;
                    float best = HX_INF; int bj = 0;
#pragma unroll 4
                    for (int p = 0; p < P; ++p) {
                        const float v = rowmin[p * n + c];
                        const int a = rowarg[p * n + c];
                        if (v < best) { best = v; bj = (p << 16) | a; }
                    }
                    if (best < HX_INF) { cpair[c] = bj; cR[c] = __fdiv_rn(__fadd_rn(cel[c], best), cH[c]); }
                    else { cpair[c] = kNoPair; cR[c] = HX_NEG_INF; }
                }
            }
        }
        for (int i = warp; !ROWS && i < nd; i += kWarps) {
            const int c = dirty[i];
            if (cpair[c] == kDead) continue;                   // rejected at load time (warp-uniform)
            float best = HX_INF; int bj = 0x7fffffff;
            {
                // per-class times of this call: tpre[g * ts], tdec[g * ts]
                const float* tpre; const float* tdec; int ts;
                float kvB, m;
                if (CACHE) {
                    tpre = tpreC + c; tdec = tdecC + c; ts = nst;
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
                // the block's candidate and what its commit would change, published in every block
                float cand[6] = {rv, __int_as_float(rc), 0.f, 0.f, 0.f, 0.f};
                if (rc != 0x7fffffff) {
                    const int li = rc / NC;
                    const int bj = cpair[li], p = bj >> 16, d = bj & 0xFFFF;
                    const float nt = cn[li], ot = co[li];
                    const int mdl = cmodel[li];
                    const float phi = prm.ct.phi[mdl], omega = prm.ct.omega[mdl], kappa = prm.ct.kappa[mdl];
                    const float kvB = __fmul_rn(nt, kappa);
                    const int g = typePs[p];
                    const float tp = fmaxf(__fmul_rn(__fmaf_rn(__fmul_rn(nt, prm.ct.psi[mdl]), nt, __fmul_rn(nt, phi)), prm.ct.invF[g]), __fmul_rn(__fadd_rn(omega, kvB), prm.ct.invB[g]));
                    cand[2] = __int_as_float(p); cand[3] = __int_as_float(d); cand[4] = tp; cand[5] = __fadd_rn(nt, ot);
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
            }
        }
        // one barrier per iteration: a block that runs ahead writes the other set of candidates, and cannot get
        // past the next barrier before every block has read this one
        if (NC > 1) cg::this_cluster().sync(); else __syncthreads();      // every thread of every block
        if (warp == 0) {
            rv = lane < NC ? xc[lane][0] : HX_NEG_INF;         // all blocks reduce the same list
            rc = lane < NC ? __float_as_int(xc[lane][1]) : 0x7fffffff;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, rv, off);
                const int oc = __shfl_xor_sync(0xffffffffu, rc, off);
                if (ov > rv || (ov == rv && oc < rc)) { rv = ov; rc = oc; }
            }
            if (lane == 0) {
                const bool none = rc == 0x7fffffff;            // nobody left that fits anywhere
                s_call = none ? -1 : rc;
                s_ndirty = 0;
                if (!none) {
                    // (3) commit: the same update in every block; the block that owns the call records it
                    const float* w = xc[rc % NC];
                    const int p = __float_as_int(w[2]), d = __float_as_int(w[3]);
                    const float tp = w[4], m = w[5];
                    if (rc % NC == rank) {
                        const int li = rc / NC;
                        prm.out_assign[rc] = p * D + d;
                        prm.out_ratio[rc] = rv;
                        prm.out_order[it] = rc;
                        if (prm.out_delta) {
                            // Delta of the chosen pair: the projection that made the ratio, from the same state
                            const float nt = cn[li], ot = co[li];
                            const int mdl = cmodel[li];
                            const float omega = prm.ct.omega[mdl], kappa = prm.ct.kappa[mdl];
                            const float ctx = __fmaf_rn(0.5f, __fsub_rn(ot, 1.0f), nt);
                            const float td = __fmul_rn(__fmul_rn(ot, __fmaf_rn(kappa, ctx, omega)), prm.ct.invB[typeDs[d]]);
                            const float ready = __fmaf_rn(__fmul_rn(nt, kappa), invL[ROWS ? d * P + p : p * D + d], __fadd_rn(qPs[p], tp));
                            prm.out_delta[rc] = __fadd_rn(fmaxf(ready, qDs[d]), td);
                        }
                        cpair[li] = kDead; cR[li] = HX_NEG_INF;
                    }
                    qPs[p] = __fadd_rn(qPs[p], tp);
                    frees[d] = __fsub_rn(frees[d], m);
                    if (ROWS) verP[p] = (unsigned short)(verP[p] + 1);
                    s_p = p; s_d = d;
                }
            }
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
    return greedy_smem(t, calls_per_block) + ((size_t)calls_per_block * 2 + 2 * (size_t)t.G * (calls_per_block | 1)) * 4;
}
// ... and the per-prefill-instance minima of every call (value, decode instance, version) plus the versions.
static size_t greedy_rows_smem(const HxTables& t, int calls_per_block) {
    return greedy_cache_smem(t, calls_per_block) + (size_t)calls_per_block * t.P * 8 + (size_t)kItemCap * 4 + ((size_t)t.P + 2) * 2;
}
// 0: the bare state, 1: with the per-class times, 2: with the row minima as well
static int greedy_mode(const HxTables& t, int calls_per_block) {
    const size_t limit = (size_t)200 * 1024;
    return greedy_rows_smem(t, calls_per_block) <= limit ? 2 : greedy_cache_smem(t, calls_per_block) <= limit ? 1 : 0;
}
static size_t greedy_mode_smem(const HxTables& t, int calls_per_block, int mode) {
    return mode == 2 ? greedy_rows_smem(t, calls_per_block) : mode == 1 ? greedy_cache_smem(t, calls_per_block) : greedy_smem(t, calls_per_block);
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
    typedef void (*Kern)(GreedyParams);
    if (n_calls > kClusterFrom) {
        const int cpb = (n_calls + kCluster - 1) / kCluster;
        const int mode = greedy_mode(t, cpb);
        const size_t smem = greedy_mode_smem(t, cpb, mode);
        static size_t allowed[3][64];
        const Kern kerns[3] = {hx_greedy_kernel<kCluster, 0>, hx_greedy_kernel<kCluster, 1>, hx_greedy_kernel<kCluster, 2>};
        const Kern kern = kerns[mode];
        if ((e = hx_opt_in_smem(kern, smem, allowed[mode], 40 * 1024)) != cudaSuccess) return e;
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
    const int mode = greedy_mode(t, n_calls);
    const size_t smem = greedy_mode_smem(t, n_calls, mode);
    static size_t allowed1[3][64];
    const Kern kerns1[3] = {hx_greedy_kernel<1, 0>, hx_greedy_kernel<1, 1>, hx_greedy_kernel<1, 2>};
    if ((e = hx_opt_in_smem(kerns1[mode], smem, allowed1[mode], 40 * 1024)) != cudaSuccess) return e;
    kerns1[mode]<<<1, kThreads, smem, stream>>>(prm);
    e = cudaGetLastError();
    if (e == cudaSuccess) ++*launches;
    return e;
}
