// Batched placement scoring (paper Algorithm 1, inner loop over the waiting
// calls; Section 5.3 "Projected-risk prefill ranking" and "Joint prefill-decode
// planning"; feasibility by Eq. 3-4; score by Eq. 2).
//
// For call c and pair (p, d):
//   ready(c,p,d) = fma(kvB_c, invL[p][d], A_c[p])        A_c[p] = qP[p] + tpre_c[typeP[p]]
//   fin(c,p,d)   = max(ready, qD[d]) + Dd_c[d]           Dd_c[d] = m_c <= capD[d] ? tdec_c[typeD[d]] : +inf
// and the call goes to the pair with the smallest fin, lowest p*D+d among equals.
//
// x -> max(x, qD) + Dd is non-decreasing in x also after rounding (max is exact,
// round-to-nearest addition is monotone), therefore
//   min_p fin(c,p,d) = max(min_p ready(c,p,d), qD[d]) + Dd_c[d]        bit for bit.
// The hot loop therefore only does one fused multiply-add and one minimum per
// candidate: a (calls x decode) register tile of running minima with the prefill
// index as the reduction dimension, operands staged in shared memory: the link
// table transposed (rows = decode instances, contiguous in p) and the per-call
// prefill-finish rows A.  Two consecutive p are processed by one packed
// fma.rn.f32x2 and folded into the running minimum by one three-input min.
// The clamp, the decode term, the selection over d and the recovery of the
// prefill index (a rescan of one row of P candidates for the few selected d)
// run once per (call, d) or per call.
#include "hx_internal.h"

namespace {

typedef unsigned long long u64;

struct ScoreParams {
    HxTables t;
    HxConstTables ct;
    HxDagView dag;
    HxTopkBufs tk;
    ScoreLaunch s;
    int* status;
    int WDn, WCn;        // warps along decode columns / along calls
    int TCB;             // calls per block tile
    int nTiles;
    int Dpad;            // decode columns covered by the block (multiple of 8*LD)
    int PC;              // prefill chunk length (multiple of 4)
    int nChunks;
    int FS;              // row stride of the per-call finish times (Dpad + 4)
    int AS, LS;          // strides, in 16-byte units, between consecutive p / 4 of the A and link tiles
    int offA, offF, offCall, offInst;   // byte offsets into dynamic shared memory (LT at 0)
    int offItem;         // selected (call, slot) entries waiting for their prefill index, 0 = recovery inside the selection loop
    int resident;        // whole link table and the A tile stay in shared memory for the index recovery
};

__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c) {
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ float min3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ u64 pack2(float lo, float hi) {
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(u64 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}

#define HX_INF __int_as_float(0x7f800000)
#define HX_NONE 0x7fffffff

// Smallest (value, column) pair of the row that is lexicographically greater
// than (pv, pd); (+inf, HX_NONE) if there is none.  Executed by an aligned
// group of four lanes (gmask); the result is the same on all four.
__device__ __forceinline__ void group_next(const float* frow, int nq, int t, unsigned gmask,
                                           float pv, int pd, float& bv, int& bd) {
    bv = HX_INF; bd = HX_NONE;
    for (int q = t; q < nq; q += 4) {
        const float4 f = *reinterpret_cast<const float4*>(frow + 4 * q);
        const float v[4] = {f.x, f.y, f.z, f.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int d = 4 * q + u;
            const bool after = (v[u] > pv) || (v[u] == pv && d > pd);
            if (after && v[u] < bv) { bv = v[u]; bd = d; }
        }
    }
#pragma unroll
    for (int off = 1; off <= 2; off <<= 1) {
        const float ov = __shfl_xor_sync(gmask, bv, off);
        const int od = __shfl_xor_sync(gmask, bd, off);
        if (ov < bv || (ov == bv && od < bd)) { bv = ov; bd = od; }
    }
}

// Lowest prefill index whose candidate on decode column d finishes exactly at v.
__device__ __forceinline__ int group_rescan(const HxTables& T, const float* qPs, const int* typePs,
                                            const float* tpre_c, int tstride, float kvB, float qd, float Dd,
                                            int d, float v, int t, unsigned gmask) {
    int best = HX_NONE;
    const float4* lrow = reinterpret_cast<const float4*>(T.invLT + (size_t)d * T.Ppad);
    const int nq = T.Ppad >> 2;
    for (int q = t; q < nq; q += 4) {
        const float4 l4 = __ldg(lrow + q);
        const float l[4] = {l4.x, l4.y, l4.z, l4.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int p = 4 * q + u;
            const float A = __fadd_rn(qPs[p], tpre_c[typePs[p] * tstride]);
            const float r = __fmaf_rn(kvB, l[u], A);
            const float f = __fadd_rn(fmaxf(r, qd), Dd);
            if (f == v && p < best) best = p;
        }
    }
#pragma unroll
    for (int off = 1; off <= 2; off <<= 1) best = min(best, __shfl_xor_sync(gmask, best, off));
    return best;
}

// Minimum of a row together with its lowest column and the number of columns attaining it.
__device__ __forceinline__ void group_min(const float* frow, int nq, int t, unsigned gmask,
                                          float& bv, int& bd, int& cnt) {
    bv = HX_INF; bd = HX_NONE; cnt = 0;
    for (int q = t; q < nq; q += 4) {
        const float4 f = *reinterpret_cast<const float4*>(frow + 4 * q);
        const float v[4] = {f.x, f.y, f.z, f.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (v[u] < bv) { bv = v[u]; bd = 4 * q + u; cnt = 1; }
            else if (v[u] == bv && bd != HX_NONE) ++cnt;
        }
    }
#pragma unroll
    for (int off = 1; off <= 2; off <<= 1) {
        const float ov = __shfl_xor_sync(gmask, bv, off);
        const int od = __shfl_xor_sync(gmask, bd, off);
        const int oc = __shfl_xor_sync(gmask, cnt, off);
        if (ov < bv) { bv = ov; bd = od; cnt = oc; }
        else if (ov == bv) { bd = min(bd, od); cnt += oc; }
    }
}

// Lowest prefill index p with fin(c, p, d[k]) == v[k] for up to NK decode columns of one call at
// once (k < n), both operands resident in shared memory as [p / 4][row] 16-byte units.  The four
// lanes of the group take the units q = t, t + 4, ... in ascending order and stop as soon as every
// column is resolved.  A candidate can only reach the minimum v if its ready time is at most
// v - Dd plus the rounding slack of the final addition (ulp(v) / 2 each for the subtraction here
// and the addition there, covered by v * 2^-21): that test costs one packed FMA pair, two minima
// and a compare per unit, and only units passing it are evaluated exactly.
template <int NK>
__device__ __forceinline__ void group_rescan_multi(const float* a_c, int astride, const float* lts, int lstride,
                                                   int nq, float kvB, const int* d, const float* qd,
                                                   const float* Dd, const float* v, int n, int t,
                                                   unsigned gmask, int* best) {
    const u64 kk2 = pack2(kvB, kvB);
    float thr[NK];
#pragma unroll
    for (int k = 0; k < NK; ++k) {
        best[k] = HX_NONE;
        thr[k] = k < n ? __fadd_rn(__fsub_rn(v[k], Dd[k]), __fmul_rn(v[k], 4.76837158203125e-07f)) : -1.0f;
    }
    unsigned pending = (1u << n) - 1u;                     // the same in the four lanes
    const int nsteps = (nq + 3) >> 2;
    for (int s = 0; s < nsteps && pending; ++s) {
        const int q = 4 * s + t;
        const bool valid = q < nq;
        ulonglong2 a = make_ulonglong2(pack2(HX_INF, HX_INF), pack2(HX_INF, HX_INF));
        if (valid) a = *reinterpret_cast<const ulonglong2*>(a_c + (size_t)q * astride);
        int cand[NK];
        bool any = false;
#pragma unroll
        for (int k = 0; k < NK; ++k) {
            cand[k] = HX_NONE;
            if (valid && ((pending >> k) & 1u)) {            // pending only has bits below n
                const ulonglong2 l = *reinterpret_cast<const ulonglong2*>(lts + (size_t)q * lstride + 4 * d[k]);
                float r[4];
                unpack2(fma2(kk2, l.x, a.x), r[0], r[1]);
                unpack2(fma2(kk2, l.y, a.y), r[2], r[3]);
                if (fminf(min3(r[0], r[1], r[2]), r[3]) <= thr[k]) {
#pragma unroll
                    for (int u = 3; u >= 0; --u)
                        if (__fadd_rn(fmaxf(r[u], qd[k]), Dd[k]) == v[k]) cand[k] = 4 * q + u;
                    any |= cand[k] != HX_NONE;
                }
            }
        }
        if (__ballot_sync(gmask, any) & gmask) {
#pragma unroll
            for (int k = 0; k < NK; ++k) {
                int c = cand[k];
                c = min(c, __shfl_xor_sync(gmask, c, 1));
                c = min(c, __shfl_xor_sync(gmask, c, 2));
                if (c != HX_NONE && ((pending >> k) & 1u)) { best[k] = c; pending &= ~(1u << k); }
            }
        }
    }
}

// Thread tile: TC calls x TD decode columns.  A warp spans LD lanes along d and 32 / LD along
// the calls; lanes interleave their rows so that the rows one instruction touches start in
// different shared-memory banks.
template <int TC, int TD, int LD>
__global__ void __launch_bounds__(TD == 4 ? 512 : 256, 1) hx_score_kernel(const __grid_constant__ ScoreParams prm) {
    extern __shared__ __align__(16) unsigned char smem[];
    constexpr int LC = 32 / LD;
    const HxTables& T = prm.t;
    const int G = T.G, P = T.P, D = T.D, Ppad = T.Ppad;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int wd = warp % prm.WDn, wc = warp / prm.WDn;
    const int dg = lane % LD, cg = lane / LD;
    const int FS = prm.FS, PC = prm.PC, TCB = prm.TCB, Dpad = prm.Dpad, AS = prm.AS, LS = prm.LS;
    const bool unloaded = prm.s.flags & HX_FLAG_UNLOADED;
    const bool resident = prm.resident;

    // operand tiles are stored [p / 4][row] as 16-byte units: for a fixed p the rows a warp
    // reads are contiguous (no bank conflicts, no padding) and their offsets are compile-time
    float* LTs = reinterpret_cast<float*>(smem);                  // [PC/4][LS][4], Dpad of LS used
    float* As = reinterpret_cast<float*>(smem + prm.offA);        // [PC/4][AS][4], TCB of AS used
    float* Fs = reinterpret_cast<float*>(smem + prm.offF);        // [TCB][FS] (may alias As)
    float* kvBs = reinterpret_cast<float*>(smem + prm.offCall);   // [TCB]
    float* mtoks = kvBs + TCB;                                    // [TCB]
    float* tpres = mtoks + TCB;                                   // [G][TCB]
    float* tdecs = tpres + TCB * G;                               // [G][TCB]
    unsigned* nodeS = reinterpret_cast<unsigned*>(tdecs + TCB * G);   // [TCB] DAG node of the call
    unsigned* wfS = nodeS + TCB;                                  // [TCB] its workflow
    float* qPs = reinterpret_cast<float*>(smem + prm.offInst);    // [Ppad]
    int* typePs = reinterpret_cast<int*>(qPs + Ppad);             // [Ppad]
    float* qDs = reinterpret_cast<float*>(typePs + Ppad);         // [Dpad]
    float* capDs = qDs + Dpad;                                    // [Dpad]
    int* typeDs = reinterpret_cast<int*>(capDs + Dpad);           // [Dpad]
    int* itemD = reinterpret_cast<int*>(smem + prm.offItem);      // [TCB * K] decode column of the entry, -1 = unused slot
    float* itemV = reinterpret_cast<float*>(itemD + TCB * HX_MAX_TOPK);   // [TCB * K] its finish time
    const bool deferred = prm.offItem != 0;                       // top-K lists with the operands resident: see below

    // visiting order of the capacity pass: this kernel clears the bin counters and leaves the smallest and
    // the largest finite priority key of every block's calls behind (no state survives from earlier batches)
    unsigned key_lo = 0xFFFFFFFFu, key_hi = 0u;
    __shared__ unsigned key_lohi[2];
    if (tid == 0) { key_lohi[0] = 0xFFFFFFFFu; key_lohi[1] = 0u; }
    // Launched as a programmatic dependent, this kernel may become resident while the kernel before it on the
    // stream (the capacity pass of the previous batch) still runs.  Everything up to sync_with_stream() reads
    // only what no kernel writes (call records, instance classes and capacities, link table, model constants)
    // and writes only shared memory; the prefill queues, the free KV tokens and every buffer of the top-K
    // lists are touched after it.  The kernels behind this one are released when a block is through (not
    // earlier: blocks of the binning kernel that become resident beside this one have nothing to do before their
    // wait and measurably slow the step down), so none of them can overtake the previous batch either.
    bool synced = false;
    auto sync_with_stream = [&] {
        if (synced) return;
        synced = true;
        hx_wait_for_primary();
        if (prm.s.K > 0)
            for (int i = blockIdx.x * nthr + tid; i < HX_ORDER_BINS; i += gridDim.x * nthr) prm.tk.ghist[i] = 0u;
        for (int p = tid; p < Ppad; p += nthr) qPs[p] = p < P ? (unloaded ? 0.0f : T.qP[p]) : HX_INF;
    };
    // the call records of the first tile come from DRAM: request them before anything else
    const bool with_dag = !(prm.s.flags & HX_FLAG_NO_DAG);
    uint4 pre[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int idx = tid + k * nthr, c = idx / G;
        const int gc = blockIdx.x * TCB + c;
        pre[k] = make_uint4(0u, 0u, 0u, 0u);
        if (idx < TCB * G && gc < prm.s.n_calls) pre[k] = __ldg(reinterpret_cast<const uint4*>(prm.s.calls) + gc);
    }
    // instance tables; padded prefill slots can never win, padded decode columns are infeasible
    for (int p = tid; p < Ppad; p += nthr) typePs[p] = p < P ? T.typeP[p] : 0;
    for (int d = tid; d < Dpad; d += nthr) {
        qDs[d] = d < D ? (unloaded ? 0.0f : T.qD[d]) : 0.0f;
        capDs[d] = d < D ? T.capD[d] : -1.0f;
        typeDs[d] = d < D ? T.typeD[d] : 0;
    }
    // asynchronous copies (no register staging) from the tiled copy of the link table: consecutive
    // threads copy consecutive 16-byte units; the wait is just before the barrier that precedes the first use
    auto load_LT = [&](int pc0) {
        const int nq = PC >> 2, q0 = pc0 >> 2, nq_all = Ppad >> 2;
        const int dq = nthr / Dpad, dd = nthr - dq * Dpad;
        int q = tid / Dpad, d = tid - q * Dpad;
        for (int idx = tid; idx < Dpad * nq; idx += nthr) {
            float* dst = LTs + 4 * (q * LS + d);
            if (q0 + q < nq_all) {
                const unsigned sa = (unsigned)__cvta_generic_to_shared(dst);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(sa), "l"(T.invLTt + 4 * ((size_t)(q0 + q) * Dpad + d)) : "memory");
            } else {
                *reinterpret_cast<float4*>(dst) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            q += dq; d += dd;
            if (d >= Dpad) { d -= Dpad; ++q; }
        }
    };
    auto lt_wait = [] { asm volatile("cp.async.wait_all;" ::: "memory"); };
    if (prm.nChunks == 1) load_LT(0);

    for (int tile = blockIdx.x; tile < prm.nTiles; tile += gridDim.x) {
        const int c0 = tile * TCB;
        const int nvalid = min(TCB, prm.s.n_calls - c0);

        // per-call service times on every GPU class (roofline-style estimate, Section 4.2):
        // one thread per (call, class)
        int k_it = 0;
        for (int idx = tid; idx < TCB * G; idx += nthr, ++k_it) {
            const int c = idx / G, g = idx - c * G;
            float n = 1.f, o = 1.f, phi = 0.f, omega = 0.f, kappa = 0.f, psi = 0.f;
            if (c < nvalid) {
                uint4 raw;
                if (tile == (int)blockIdx.x && k_it < 2) raw = k_it == 0 ? pre[0] : pre[1];
                else raw = __ldg(reinterpret_cast<const uint4*>(prm.s.calls) + c0 + c);
                if (g == 0) nodeS[c] = raw.x;
                n = __uint_as_float(raw.z); o = __uint_as_float(raw.w);
                if (raw.y < (unsigned)T.M) { phi = prm.ct.phi[raw.y]; omega = prm.ct.omega[raw.y]; kappa = prm.ct.kappa[raw.y]; psi = prm.ct.psi[raw.y]; }
            }
            const float kvB = __fmul_rn(n, kappa);
            const float ctx = __fmaf_rn(0.5f, __fsub_rn(o, 1.0f), n);
            const float step = __fmaf_rn(kappa, ctx, omega);
            const float iF = prm.ct.invF[g], iB = prm.ct.invB[g];
            const float flops = __fmaf_rn(__fmul_rn(n, psi), n, __fmul_rn(n, phi));   // exactly n * phi when psi = 0
            tpres[g * TCB + c] = fmaxf(__fmul_rn(flops, iF), __fmul_rn(__fadd_rn(omega, kvB), iB));
            tdecs[g * TCB + c] = __fmul_rn(__fmul_rn(o, step), iB);
            if (g == 0) { kvBs[c] = kvB; mtoks[c] = __fadd_rn(n, o); }
        }
        sync_with_stream();
        lt_wait();
        __syncthreads();

        // workflow of the call: requested now, parked behind the A tile, so that the score at the end
        // of the tile finds it in shared memory and its three gathers in L2
        unsigned my_node = 0xFFFFFFFFu, my_wf = 0xFFFFFFFFu;
        const bool one_pass = TCB <= nthr;                    // one call per thread; else a plain loop
        if (with_dag && one_pass && tid < nvalid) {
            my_node = nodeS[tid];
            if (my_node < prm.dag.n_nodes) my_wf = __ldg(prm.dag.node_wf + my_node);
        }
        if (with_dag && !one_pass)
            for (int c = tid; c < nvalid; c += nthr) {
                const unsigned nd = nodeS[c];
                wfS[c] = nd < prm.dag.n_nodes ? __ldg(prm.dag.node_wf + nd) : 0xFFFFFFFFu;
            }

        float acc[TC][TD];
#pragma unroll
        for (int i = 0; i < TC; ++i)
#pragma unroll
            for (int j = 0; j < TD; ++j) acc[i][j] = HX_INF;
        u64 kk[TC];
#pragma unroll
        for (int i = 0; i < TC; ++i) {
            const float k = kvBs[wc * (TC * LC) + cg + LC * i];
            kk[i] = pack2(k, k);
        }
        for (int ch = 0; ch < prm.nChunks; ++ch) {
            const int pc0 = ch * PC;
            if (prm.nChunks > 1) load_LT(pc0);
            {   // prefill finish times A[c][p] of this chunk: a thread keeps the queue loads and classes
                // of one p / 4 in registers and walks over the calls, 16 lanes along the calls
                const int nq = PC >> 2;
                const int cl = tid & 15, qs = tid >> 4, nqs = nthr >> 4;
                for (int q = qs; q < nq; q += nqs) {
                    const int p = pc0 + 4 * q;
                    float4 qp = make_float4(HX_INF, HX_INF, HX_INF, HX_INF);
                    int4 ty = make_int4(0, 0, 0, 0);
                    if (p < Ppad) {                           // Ppad is a multiple of 4: whole unit or nothing
                        qp = *reinterpret_cast<const float4*>(qPs + p);
                        ty = *reinterpret_cast<const int4*>(typePs + p);
                    }
                    const float* t0 = tpres + ty.x * TCB; const float* t1 = tpres + ty.y * TCB;
                    const float* t2 = tpres + ty.z * TCB; const float* t3 = tpres + ty.w * TCB;
                    for (int c = cl; c < TCB; c += 16)
                        *reinterpret_cast<float4*>(As + 4 * (q * AS + c)) =
                            make_float4(__fadd_rn(qp.x, t0[c]), __fadd_rn(qp.y, t1[c]), __fadd_rn(qp.z, t2[c]), __fadd_rn(qp.w, t3[c]));
                }
            }
            if (ch == 0 && with_dag && one_pass && tid < nvalid) {
                wfS[tid] = my_wf;
                if (my_wf != 0xFFFFFFFFu) {
                    asm volatile("prefetch.global.L2 [%0];" :: "l"(prm.dag.elapsed + my_wf));
                    asm volatile("prefetch.global.L2 [%0];" :: "l"(prm.dag.H + my_wf));
                    asm volatile("prefetch.global.L2 [%0];" :: "l"(prm.dag.tail + my_node));
                }
            }
            lt_wait();
            __syncthreads();
            const ulonglong2* ap = reinterpret_cast<const ulonglong2*>(As) + wc * (TC * LC) + cg;
            const ulonglong2* lp = reinterpret_cast<const ulonglong2*>(LTs) + wd * (TD * LD) + dg;
#pragma unroll 2
            for (int q = 0; q < (PC >> 2); ++q) {
                ulonglong2 a[TC], l[TD];
#pragma unroll
                for (int i = 0; i < TC; ++i) a[i] = ap[i * LC];
#pragma unroll
                for (int j = 0; j < TD; ++j) l[j] = lp[j * LD];
                ap += AS; lp += LS;
#pragma unroll
                for (int i = 0; i < TC; ++i)
#pragma unroll
                    for (int j = 0; j < TD; ++j) {
                        float r0, r1, r2, r3;
                        unpack2(fma2(kk[i], l[j].x, a[i].x), r0, r1);
                        unpack2(fma2(kk[i], l[j].y, a[i].y), r2, r3);
                        acc[i][j] = min3(min3(acc[i][j], r0, r1), r2, r3);
                    }
            }
            if (prm.nChunks > 1 || !resident) __syncthreads();
        }

        // clamp to the decode admission time and add the decode term; park the
        // per-(call, d) finish times in shared memory
        float mt[TC];
#pragma unroll
        for (int i = 0; i < TC; ++i) mt[i] = mtoks[wc * (TC * LC) + cg + LC * i];
#pragma unroll
        for (int j = 0; j < TD; ++j) {
            const int d = wd * (TD * LD) + dg + LD * j;
            const float qd = qDs[d], cap = capDs[d];
            const int ty = typeDs[d];
#pragma unroll
            for (int i = 0; i < TC; ++i) {
                const int c = wc * (TC * LC) + cg + LC * i;
                const float Dd = (mt[i] <= cap) ? tdecs[ty * TCB + c] : HX_INF;
                Fs[c * FS + d] = __fadd_rn(fmaxf(acc[i][j], qd), Dd);
            }
        }
        __syncthreads();

        // selection over d, prefill index recovery and per-call score: four lanes per call
        const int K = prm.s.K;
        const int ngroups = nthr >> 2, gid = tid >> 2, t = tid & 3;
        const unsigned gmask = 0xFu << (lane & 28);       // groups of one warp may leave the loops at different times
        for (int cb = 0; cb < TCB; cb += ngroups) {
            const int c = cb + gid;
            const bool live = c < nvalid;                 // uniform inside the group
            const int cs = live ? c : 0;
            const float* frow = Fs + cs * FS;
            const float kvB = kvBs[cs], m = mtoks[cs];
            const float* tpre_c = tpres + cs;                 // class g at tpre_c[g * TCB]
            // prefill index of n (<= NK) selected columns: lowest p whose candidate finishes exactly at v[k]
            auto recover = [&](auto nk_tag, const int* dk, const float* vk, int n, int* pk) {
                constexpr int NK = decltype(nk_tag)::value;
                float qd[NK], Dd[NK]; int dd[NK];
#pragma unroll
                for (int k = 0; k < NK; ++k) {
                    dd[k] = k < n ? dk[k] : 0;
                    qd[k] = qDs[dd[k]];
                    Dd[k] = (m <= capDs[dd[k]]) ? tdecs[typeDs[dd[k]] * TCB + cs] : HX_INF;
                }
                if (resident) {
                    group_rescan_multi<NK>(As + 4 * cs, 4 * AS, LTs, 4 * LS, Ppad >> 2, kvB, dd, qd, Dd, vk, n, t, gmask, pk);
                } else {
#pragma unroll
                    for (int k = 0; k < NK; ++k)
                        pk[k] = k < n ? group_rescan(T, qPs, typePs, tpre_c, TCB, kvB, qd[k], Dd[k], dd[k], vk[k], t, gmask) : HX_NONE;
                }
            };
            struct One { enum { value = 1 }; }; struct Four { enum { value = 4 }; };
            float v0 = HX_INF; int jbest = HX_NONE;
            int sel_pair[HX_MAX_TOPK], sel_d[HX_MAX_TOPK]; float sel_cost[HX_MAX_TOPK], sel_tpre[HX_MAX_TOPK];
#pragma unroll
            for (int k = 0; k < HX_MAX_TOPK; ++k) { sel_pair[k] = -1; sel_d[k] = 0; sel_cost[k] = HX_INF; sel_tpre[k] = 0.f; }
            if (K == 0) {
                // plain argmin: lowest p * D + d among all pairs attaining the minimum
                int d0, ntie;
                group_min(frow, Dpad >> 2, t, gmask, v0, d0, ntie);
                if (d0 != HX_NONE) {
                    int p0;
                    recover(One{}, &d0, &v0, 1, &p0);
                    jbest = p0 * D + d0;
                    float pv = v0; int pd = d0;
                    for (int r = 1; r < ntie; ++r) {      // exact ties across decode instances
                        float v; int d;
                        group_next(frow, Dpad >> 2, t, gmask, pv, pd, v, d);
                        recover(One{}, &d, &v, 1, &p0);
                        jbest = min(jbest, p0 * D + d);
                        pv = v; pd = d;
                    }
                }
            } else {
                int nsel = 0;
                if (Dpad <= 128) {
                    // a lane owns every fourth 16-byte unit of the row and keeps the minimum of each unit in
                    // a register; a round takes the smallest (finish, d) left, and only its owner re-reads
                    // that unit (the taken entry is overwritten with +inf in shared memory)
                    float um[8];
                    float* fr = Fs + cs * FS;
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int q = t + 4 * it;
                        float4 f4 = make_float4(HX_INF, HX_INF, HX_INF, HX_INF);
                        if (4 * q < Dpad) f4 = *reinterpret_cast<const float4*>(fr + 4 * q);
                        um[it] = fminf(min3(f4.x, f4.y, f4.z), f4.w);
                    }
                    for (int k = 0; k < (live ? K : 0); ++k) {     // a group without a call must not write the row
                        float v = um[0]; int bi = 0;
#pragma unroll
                        for (int it = 1; it < 8; ++it)
                            if (um[it] < v) { v = um[it]; bi = it; }
                        // position inside the unit: lowest of its four columns holding v
                        const int qb = t + 4 * bi;            // a unit beyond Dpad has minimum +inf and is never read
                        float4 f4 = make_float4(HX_INF, HX_INF, HX_INF, HX_INF);
                        if (v < HX_INF) f4 = *reinterpret_cast<const float4*>(fr + 4 * qb);
                        const int u = f4.x == v ? 0 : f4.y == v ? 1 : f4.z == v ? 2 : 3;
                        int d = v < HX_INF ? 4 * qb + u : HX_NONE;
                        const int myd = d;
#pragma unroll
                        for (int off = 1; off <= 2; off <<= 1) {
                            const float ov = __shfl_xor_sync(gmask, v, off);
                            const int od = __shfl_xor_sync(gmask, d, off);
                            if (ov < v || (ov == v && od < d)) { v = ov; d = od; }
                        }
                        if (d == HX_NONE) break;              // nothing (feasible) left
                        if (d == myd) {                       // owner: retire the entry, refresh the unit minimum
                            fr[d] = HX_INF;
                            const float a = u == 0 ? HX_INF : f4.x, b = u == 1 ? HX_INF : f4.y;
                            const float c2 = u == 2 ? HX_INF : f4.z, e = u == 3 ? HX_INF : f4.w;
                            const float nu = fminf(min3(a, b, c2), e);
#pragma unroll
                            for (int it = 0; it < 8; ++it) um[it] = it == bi ? nu : um[it];
                        }
#pragma unroll
                        for (int k2 = 0; k2 < HX_MAX_TOPK; ++k2)
                            if (k2 == k) { sel_d[k2] = d; sel_cost[k2] = v; }
                        nsel = k + 1;
                    }
                } else {
                    float pv = -1.0f; int pd = -1;
                    for (int k = 0; k < K; ++k) {
                        float v; int d;
                        group_next(frow, Dpad >> 2, t, gmask, pv, pd, v, d);
                        if (d == HX_NONE) break;              // nothing (feasible) left
#pragma unroll
                        for (int k2 = 0; k2 < HX_MAX_TOPK; ++k2)
                            if (k2 == k) { sel_d[k2] = d; sel_cost[k2] = v; }
                        nsel = k + 1;
                        pv = v; pd = d;
                    }
                }
                if (nsel > 0) v0 = sel_cost[0];
#pragma unroll
                for (int k0 = 0; k0 < HX_MAX_TOPK; k0 += 4) {
                    if (k0 < nsel && !deferred) {             // uniform inside the group
                        int pk[4];
                        recover(Four{}, &sel_d[k0], &sel_cost[k0], min(4, nsel - k0), pk);
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            if (k0 + k < nsel) { sel_pair[k0 + k] = pk[k] * D + sel_d[k0 + k]; sel_tpre[k0 + k] = tpre_c[typePs[pk[k]] * TCB]; }
                    }
                }
            }
            if (live && t == 0) {
                const int gc = c0 + c;
                const uint4 raw = __ldg(reinterpret_cast<const uint4*>(prm.s.calls) + gc);
                float elapsed = 0.f, tail = 0.f, H = 1.f;
                bool bad = raw.y >= (unsigned)T.M;
                if (K > 0) {
                    // the capacity pass decides on integers: token counts must be whole and their sum below 2^24
                    const float n = __uint_as_float(raw.z), o = __uint_as_float(raw.w);
                    bad |= !(n >= 0.f && o >= 0.f && n == floorf(n) && o == floorf(o) && __fadd_rn(n, o) < 16777216.0f);
                }
                if (!(prm.s.flags & HX_FLAG_NO_DAG)) {
                    if (raw.x < prm.dag.n_nodes) {
                        const uint32_t w = wfS[c];
                        elapsed = prm.dag.elapsed[w];
                        H = prm.dag.H[w];
                        if (!(prm.s.flags & HX_FLAG_NO_TAIL)) tail = prm.dag.tail[raw.x];
                    } else {
                        bad = true;
                    }
                }
                if (bad) { atomicExch(prm.status, HX_ERR_INVALID_ARG); v0 = HX_INF; jbest = HX_NONE; }
                const float comp = __fadd_rn(__fadd_rn(elapsed, v0), tail);
                float score = comp;
                if (prm.s.mode == HX_MODE_SLACK) score = __fsub_rn(__fmul_rn(prm.s.alpha, H), comp);
                else if (prm.s.mode == HX_MODE_RATIO) score = __fdiv_rn(comp, H);
                if (bad) score = HX_INF;
                prm.s.out_cost[gc] = score;
                if (K == 0) {
                    prm.s.out_assign[gc] = (jbest == HX_NONE) ? -1 : jbest;
                } else {
                    prm.s.out_assign[gc] = -1;            // filled in by the capacity-conflict pass
                    const float prio = __fdiv_rn(__fadd_rn(elapsed, v0), H);  // Eq. 2
                    prm.tk.prio[gc] = prio;
                    const unsigned key = hx_order_key(__float_as_uint(prio));
                    if (key != HX_FIRST_KEY) { key_lo = min(key_lo, key); key_hi = max(key_hi, key); }
                    prm.tk.mtok[gc] = m;
                    unsigned dw[4] = {~0u, ~0u, ~0u, ~0u};          // decode instances of the slots, 8 x 16 bits
#pragma unroll
                    for (int k = 0; k < HX_MAX_TOPK; ++k) {
                        if (k >= K) break;
                        const bool used = !bad && (deferred ? sel_cost[k] < HX_INF : sel_pair[k] >= 0);
                        if (deferred) {                       // pair and prefill time follow once the prefill index is known
                            itemD[c * K + k] = used ? sel_d[k] : -1;
                            itemV[c * K + k] = sel_cost[k];
                        } else {
                            prm.tk.pair[(size_t)gc * K + k] = used ? sel_pair[k] : -1;
                            prm.tk.tpre[(size_t)gc * K + k] = sel_tpre[k];
                        }
                        prm.tk.cost[(size_t)gc * K + k] = bad ? HX_INF : sel_cost[k];
                        dw[k >> 1] = (dw[k >> 1] & ~(0xFFFFu << ((k & 1) * 16))) | ((used ? (unsigned)sel_d[k] : 0xFFFFu) << ((k & 1) * 16));
                    }
                    prm.tk.dsel[gc] = make_uint4(dw[0], dw[1], dw[2], dw[3]);
                }
            }
        }
        if (deferred) {
            // Prefill index of every selected entry, one thread per entry (call c, column d, finish time v): the thread
            // walks the call's prefill-finish row against the link-table row of d in 16-byte units (one packed FMA pair,
            // two minima and a compare per unit; exact evaluation only where the ready time can reach v - Dd within the
            // rounding slack of the last addition) and stops at the first unit that holds a match.
            __syncthreads();
            const int nItems = nvalid * K, nq = Ppad >> 2;
            for (int item = tid; item < nItems; item += nthr) {
                const int d = itemD[item];
                const int c = item / K;
                int best = HX_NONE;
                if (d >= 0) {
                    const float v = itemV[item], kvB = kvBs[c], qd = qDs[d];
                    const float Dd = (mtoks[c] <= capDs[d]) ? tdecs[typeDs[d] * TCB + c] : HX_INF;
                    const float thr = __fadd_rn(__fsub_rn(v, Dd), __fmul_rn(v, 4.76837158203125e-07f));
                    const u64 kk2 = pack2(kvB, kvB);
                    const ulonglong2* ap = reinterpret_cast<const ulonglong2*>(As) + c;
                    const ulonglong2* lp = reinterpret_cast<const ulonglong2*>(LTs) + d;
                    for (int q0 = 0; q0 < nq && best == HX_NONE; q0 += 4) {
#pragma unroll
                        for (int u4 = 3; u4 >= 0; --u4) {
                            const int q = q0 + u4;
                            if (q >= nq) continue;
                            const ulonglong2 a = ap[(size_t)q * AS], l = lp[(size_t)q * LS];
                            float r[4];
                            unpack2(fma2(kk2, l.x, a.x), r[0], r[1]);
                            unpack2(fma2(kk2, l.y, a.y), r[2], r[3]);
                            if (fminf(min3(r[0], r[1], r[2]), r[3]) <= thr) {
#pragma unroll
                                for (int u = 3; u >= 0; --u)
                                    if (__fadd_rn(fmaxf(r[u], qd), Dd) == v) best = 4 * q + u;
                            }
                        }
                    }
                }
                const size_t o = (size_t)(c0 + c) * K + (item - c * K);
                const bool ok = best != HX_NONE;
                prm.tk.pair[o] = ok ? best * D + d : -1;
                prm.tk.tpre[o] = ok ? tpres[typePs[best] * TCB + c] : 0.f;
            }
        }
        __syncthreads();
    }
    sync_with_stream();                                           // a block without a tile
    hx_release_dependents();                                      // the first kernel of the capacity pass may get ready now
    if (prm.s.K > 0) {
        key_lo = __reduce_min_sync(0xffffffffu, key_lo); key_hi = __reduce_max_sync(0xffffffffu, key_hi);
        if (lane == 0) { atomicMin(&key_lohi[0], key_lo); atomicMax(&key_lohi[1], key_hi); }
        __syncthreads();
        // every slot of the table gets some block's values: the reader need not know the grid size
        for (int b = blockIdx.x + tid * gridDim.x; b < HX_ORDER_MAXBLK; b += nthr * gridDim.x) {
            prm.tk.blk_lohi[b] = key_lohi[0];
            prm.tk.blk_lohi[HX_ORDER_MAXBLK + b] = key_lohi[1];
        }
    }
}

template <int TC, int TD, int LD>
cudaError_t launch_one(const ScoreParams& prm, int grid, int threads, size_t smem, cudaStream_t stream) {
    static size_t allowed[64];
    cudaError_t e = hx_opt_in_smem(hx_score_kernel<TC, TD, LD>, smem, allowed, 0);
    if (e != cudaSuccess) return e;
    return hx_launch_dependent(hx_score_kernel<TC, TD, LD>, dim3(grid), dim3(threads), smem, stream, prm);
}

inline int round_up(int a, int b) { return (a + b - 1) / b * b; }

}  // namespace

cudaError_t hx_launch_score(const HxTables& t, const HxConstTables& ct, const HxDagView& dag, const HxTopkBufs& tk,
                            const ScoreLaunch& s, int n_sm, size_t max_smem, int* status,
                            cudaStream_t stream, long long* launches) {
    ScoreParams prm;
    prm.t = t; prm.ct = ct; prm.dag = dag; prm.tk = tk; prm.s = s; prm.status = status;
    const int D = t.D, C = s.n_calls;
    // wide decode pools: 16 warps with 4-column thread tiles; narrow ones: 8 warps, 8 columns
    int LD, TD, Dpad;
    hx_score_shape(D, &LD, &TD, &Dpad);
    if (Dpad != t.DpadT) return cudaErrorInvalidConfiguration;     // the tiled link table was packed for this shape
    const int max_warps = LD == 8 ? 16 : 8;
    const int LC = 32 / LD, WD = TD * LD;
    prm.WDn = Dpad / WD;
    prm.Dpad = Dpad;
    int WCn = prm.WDn >= max_warps ? 1 : max_warps / prm.WDn;
    int TC = 8;
    if (LD == 8) {
        // warps along calls: fewer when the batch is too small to fill the SMs
        while (WCn > 1 && (C + WCn * 4 * LC - 1) / (WCn * 4 * LC) < n_sm) WCn >>= 1;
        // thread tile height: spread the calls evenly over the SMs (a fixed height would leave SMs
        // idle whenever the batch is not a multiple of n_sm * rows * height calls)
        const int per_sm = (C + n_sm - 1) / n_sm;
        const int rows = WCn * LC;
        const int tiles_per_sm = (per_sm + 8 * rows - 1) / (8 * rows);
        TC = (per_sm + tiles_per_sm * rows - 1) / (tiles_per_sm * rows);
        TC = TC < 4 ? 4 : (TC > 8 ? 8 : TC);
    } else {
        // narrow decode pools: the candidate loop is short, latency decides.  Keep all warps of the
        // block (they hide the latency of the prologue and of the selection) and shrink the thread
        // tile instead, until the batch gives every SM a block or the tile is one call high.
        while (TC > 1 && (C + WCn * TC * LC - 1) / (WCn * TC * LC) < n_sm) TC >>= 1;
    }
    prm.WCn = WCn;
    prm.TCB = WCn * TC * LC;
    prm.nTiles = (C + prm.TCB - 1) / prm.TCB;
    prm.FS = prm.Dpad + 8;     // rows 8 banks apart: the clamp phase stores four rows x eight columns per warp
    // strides of the operand tiles: 2 (mod 8) 16-byte units, so that the four lanes of a selection
    // group, which read four consecutive p / 4 of one row, fall into different bank groups
    auto pad_stride = [](int n) { return n + ((2 - n) % 8 + 8) % 8; };
    prm.AS = pad_stride(prm.TCB);
    prm.LS = pad_stride(prm.Dpad);
    const int G = t.G;
    const size_t callB = round_up(prm.TCB * (4 + 2 * G) * 4, 16);
    const size_t instB = round_up((2 * t.Ppad + 3 * prm.Dpad) * 4, 16);
    if (callB + instB + 4096 > max_smem) return cudaErrorInvalidConfiguration;
    const size_t budget = max_smem - callB - instB - 64;
    const size_t f_rows = (size_t)prm.TCB * prm.FS * 4;
    // first choice: whole link table, A tile and finish times side by side
    int PC = t.Ppad;
    prm.resident = ((size_t)(prm.LS + prm.AS) * PC * 4 + f_rows <= budget) ? 1 : 0;
    if (!prm.resident) {
        // otherwise chunk the prefill dimension; the finish times reuse the A tile
        for (;;) {
            const size_t a_rows = (size_t)prm.AS * PC * 4;
            if ((size_t)prm.LS * PC * 4 + (a_rows > f_rows ? a_rows : f_rows) <= budget || PC <= 4) break;
            PC = round_up(PC / 2, 4);
        }
    }
    prm.PC = PC;
    prm.nChunks = (t.Ppad + PC - 1) / PC;
    const size_t ltB = (size_t)prm.LS * PC * 4;
    const size_t aB = (size_t)prm.AS * PC * 4;
    prm.offA = (int)ltB;
    if (prm.resident) { prm.offF = prm.offA + (int)aB; prm.offCall = prm.offF + round_up((int)f_rows, 16); }
    else { prm.offF = prm.offA; prm.offCall = prm.offA + (int)(aB > f_rows ? aB : round_up((int)f_rows, 16)); }
    prm.offInst = prm.offCall + (int)callB;
    size_t smem = prm.offInst + instB;
    prm.offItem = 0;
    const size_t itemB = (size_t)prm.TCB * HX_MAX_TOPK * 8;
    if (prm.resident && s.K > 0 && smem + itemB <= max_smem) { prm.offItem = (int)smem; smem += itemB; }
    if (smem > max_smem) return cudaErrorInvalidConfiguration;
    const int threads = 32 * prm.WDn * prm.WCn;
    const int grid = prm.nTiles < n_sm ? prm.nTiles : n_sm;
    cudaError_t e;
#define HX_CASE(tc, td, ld) if (TC == tc && TD == td && LD == ld) e = launch_one<tc, td, ld>(prm, grid, threads, smem, stream); else
    HX_CASE(8, 4, 8) HX_CASE(7, 4, 8) HX_CASE(6, 4, 8) HX_CASE(5, 4, 8) HX_CASE(4, 4, 8)
    HX_CASE(8, 8, 4) HX_CASE(8, 8, 2) HX_CASE(8, 8, 1) HX_CASE(4, 8, 4) HX_CASE(4, 8, 2) HX_CASE(4, 8, 1)
    HX_CASE(2, 8, 4) HX_CASE(2, 8, 2) HX_CASE(2, 8, 1) HX_CASE(1, 8, 4) HX_CASE(1, 8, 2) HX_CASE(1, 8, 1)
    e = cudaErrorInvalidConfiguration;
#undef HX_CASE
    if (e == cudaSuccess) ++*launches;
    return e;
}
