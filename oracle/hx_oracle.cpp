// CPU oracle for batched placement scoring and workflow horizons.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, single-threaded
// definition that the CUDA library is checked against.  It shares no code,
// header, table or helper with the CUDA path and must never be called from it.
// Build with:  g++ -O2 -ffp-contract=off -std=c++17 -shared -fPIC
// (-ffp-contract=off: every rounding below is written out; the compiler must
// not fuse a multiply and an add on its own).
//
// What the paper fixes and what it leaves open
//   * Horizon H_w(t) = stand-alone completion time of the revealed sub-DAG
//     (Section 5.1, "Define online workflow horizon").  With one cost per node
//     this is the longest node-weighted path: orc_longest_path.     [pinned]
//   * Projected ratio R = ((t - a_w) + Delta) / H_w(t)  (Eq. 2).      [pinned]
//   * Decode demand m = L_in + L_out and feasibility m <= Cap(d)
//     (Eq. 3, Eq. 4).                                                [pinned]
//   * A call goes to the prefill/decode pair with the earliest projected
//     decode finish (Section 5.3, "Adaptive greedy prefill assignment");
//     Delta is built from waiting time, prefill time, KV-transfer latency and
//     the earliest decode finish on the candidate decode instance
//     (Section 5.1 and 5.3).                                          [pinned]
//   * The paper names a "roofline-style" latency model (Section 4.2,
//     Section 6) but prints no formula and no worked example.  The formulas in
//     latency_terms() are this project's reading of that sentence.  They are
//     pinned to hand-computed values of that reading, not to the paper:
//     PARITY UNPINNED for the constants and the exact shape of the prefill,
//     decode and transfer terms.
//   * Large queues use a one-pass ordering by the same risk score
//     (Section 5.3 last sentence, Section 5.4); the top-K list and the
//     capacity-conflict pass below are this project's reading of that
//     sentence together with Eq. 4.                    [pinned as defined]
//
// All placement arithmetic is IEEE binary32 in the order written here, because
// a float comparison decides an integer (the chosen pair, the priority order)
// and both sides must take that decision in the same precision.  The *_f64
// twin evaluates the same model in double, in textbook form, to measure how far
// the binary32 sequence is from the real-number value.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>
#include <algorithm>

extern "C" {

struct OrcCluster {
    int32_t G, P, D, M;
    const float* peak_tflops;   // [G]
    const float* hbm_tbps;      // [G]
    const uint32_t* typeP;      // [P]
    const uint32_t* typeD;      // [D]
    const float* qP;            // [P] seconds until prefill instance p is free
    const float* qD;            // [D] earliest time decode instance d can admit
    const float* capD;          // [D] KV capacity in tokens (Eq. 4)
    const float* link_gbps;     // [P*D] effective bandwidth prefill p -> decode d
    const float* flops_per_token;   // [M]
    const float* weight_bytes;      // [M]
    const float* kv_bytes_per_token;// [M]
    const float* attn_flops_per_token2;   // [M] or NULL: attention FLOPs per pair of prompt tokens (prefill variant)
};

struct OrcCall { uint32_t node, model; float prompt_tokens, output_tokens; };

struct OrcDag {                 // results of orc_longest_path, consumed by the scorer
    const uint32_t* node_wf;    // [N]
    const float* tail;          // [N]
    const float* H;             // [W]
    const float* elapsed;       // [W]
};

enum { ORC_MODE_COMPLETION = 0, ORC_MODE_SLACK = 1, ORC_MODE_RATIO = 2 };
enum { ORC_FLAG_NO_DAG = 1, ORC_FLAG_NO_TAIL = 2, ORC_FLAG_UNLOADED = 4 };

}  // extern "C"

namespace {

const float INF = std::numeric_limits<float>::infinity();

// Per-call, per-GPU-class service times (reading of the "roofline-style model",
// Section 4.2 "Scheduler internals").
//   prefill  = max(compute time, memory time) of one pass over the prompt
//   decode   = output tokens x (weights + KV of the average context) / HBM bandwidth
struct Terms { float kvB, m; std::vector<float> tpre, tdec; };

void latency_terms(const OrcCluster& cl, const OrcCall& c, Terms& t) {
    const float n = c.prompt_tokens, o = c.output_tokens;
    const float phi = cl.flops_per_token[c.model];
    const float omega = cl.weight_bytes[c.model];
    const float kappa = cl.kv_bytes_per_token[c.model];
    const float psi = cl.attn_flops_per_token2 ? cl.attn_flops_per_token2[c.model] : 0.0f;
    t.kvB = n * kappa;                                  // KV bytes of the prompt
    t.m = n + o;                                        // Eq. 3
    t.tpre.resize(cl.G);
    t.tdec.resize(cl.G);
    const float ctx = std::fmaf(0.5f, o - 1.0f, n);     // average context length while decoding
    const float step = std::fmaf(kappa, ctx, omega);    // bytes read per decode step
    for (int g = 0; g < cl.G; ++g) {
        const float invF = 1.0f / (cl.peak_tflops[g] * 1e12f);
        const float invB = 1.0f / (cl.hbm_tbps[g] * 1e12f);
        // variant with a quadratic attention term: prefill FLOPs = n * phi + n * n * psi (psi = 0 without it)
        const float flops = std::fmaf(n * psi, n, n * phi);         // exactly n * phi when psi = 0
        const float pf = flops * invF;
        const float pm = (omega + t.kvB) * invB;
        t.tpre[g] = std::fmax(pf, pm);
        t.tdec[g] = (o * step) * invB;
    }
}

// Projected decode finish of call c on pair (p, d), measured from now
// (Section 5.3: prefill finish, plus transfer latency, then the earliest decode
// finish given the decode availability hint; Eq. 4 masks infeasible instances).
float candidate_fin(const OrcCluster& cl, const Terms& t, int p, int d, bool unloaded) {
    const float qp = unloaded ? 0.0f : cl.qP[p];
    const float qd = unloaded ? 0.0f : cl.qD[d];
    const float invL = 1.0f / (cl.link_gbps[(size_t)p * cl.D + d] * 1e9f);
    const float A = qp + t.tpre[cl.typeP[p]];                   // prefill finish
    const float ready = std::fmaf(t.kvB, invL, A);              // KV arrives at d
    const float start = std::fmax(ready, qd);                   // decode admission
    const float Dd = (t.m <= cl.capD[d]) ? t.tdec[cl.typeD[d]] : INF;   // Eq. 4
    return start + Dd;
}

struct DagView { float elapsed, tail, H; };

DagView dag_view(const OrcDag* dag, const OrcCall& c, int flags) {
    DagView v{0.0f, 0.0f, 1.0f};
    if (!(flags & ORC_FLAG_NO_DAG) && dag) {
        const uint32_t w = dag->node_wf[c.node];
        v.elapsed = dag->elapsed[w];
        v.tail = dag->tail[c.node];
        v.H = dag->H[w];
    }
    return v;
}

}  // namespace

extern "C" {

// fin[c][p][d] for every candidate.
int orc_fin_all(const OrcCluster* cl, const OrcCall* calls, int C, int flags, float* fin) {
    Terms t;
    for (int c = 0; c < C; ++c) {
        latency_terms(*cl, calls[c], t);
        for (int p = 0; p < cl->P; ++p)
            for (int d = 0; d < cl->D; ++d)
                fin[((size_t)c * cl->P + p) * cl->D + d] =
                    candidate_fin(*cl, t, p, d, flags & ORC_FLAG_UNLOADED);
    }
    return 0;
}

// Per-class service times of each call: tpre[c][g], tdec[c][g], kvB[c], m[c].
int orc_terms(const OrcCluster* cl, const OrcCall* calls, int C,
              float* tpre, float* tdec, float* kvB, float* m) {
    Terms t;
    for (int c = 0; c < C; ++c) {
        latency_terms(*cl, calls[c], t);
        for (int g = 0; g < cl->G; ++g) { tpre[(size_t)c * cl->G + g] = t.tpre[g]; tdec[(size_t)c * cl->G + g] = t.tdec[g]; }
        kvB[c] = t.kvB; m[c] = t.m;
    }
    return 0;
}

// Placement of every call against the snapshot: earliest projected decode
// finish over all pairs, lowest pair index p*D+d on ties; -1 / +inf when no
// decode instance can hold the call.  out_cost follows the score mode:
//   completion = (elapsed + Delta) + tail          (projected workflow completion)
//   slack      = alpha * H - completion
//   ratio      = completion / H        (Eq. 2 when ORC_FLAG_NO_TAIL drops the tail)
int orc_schedule(const OrcCluster* cl, const OrcDag* dag, const OrcCall* calls, int C,
                 int mode, float alpha, int flags,
                 int32_t* out_assign, float* out_cost, float* out_delta) {
    Terms t;
    for (int c = 0; c < C; ++c) {
        latency_terms(*cl, calls[c], t);
        float best = INF; int32_t arg = -1;
        for (int p = 0; p < cl->P; ++p)
            for (int d = 0; d < cl->D; ++d) {
                const float f = candidate_fin(*cl, t, p, d, flags & ORC_FLAG_UNLOADED);
                if (f < best) { best = f; arg = p * cl->D + d; }
            }
        const DagView v = dag_view(dag, calls[c], flags);
        const float tail = (flags & ORC_FLAG_NO_TAIL) ? 0.0f : v.tail;
        const float comp = (v.elapsed + best) + tail;
        float score = comp;
        if (mode == ORC_MODE_SLACK) { const float slo = alpha * v.H; score = slo - comp; }
        else if (mode == ORC_MODE_RATIO) score = comp / v.H;
        out_assign[c] = arg;
        out_cost[c] = score;
        if (out_delta) out_delta[c] = best;
    }
    return 0;
}

// For every call: its K cheapest distinct decode instances, each with its best
// prefill partner (lowest p on ties), ordered by (cost, d).  Unused slots hold
// pair -1, cost +inf.  prio = (elapsed + Delta*) / H (Eq. 2), m = Eq. 3 demand,
// tpre_sel[c][k] = prefill time of call c on the prefill instance of slot k.
int orc_topk(const OrcCluster* cl, const OrcDag* dag, const OrcCall* calls, int C, int K, int flags,
             int32_t* pair, float* cost, float* prio, float* m, float* tpre_sel) {
    Terms t;
    std::vector<float> bestd(cl->D);
    std::vector<int> bestp(cl->D);
    std::vector<char> used(cl->D);
    for (int c = 0; c < C; ++c) {
        latency_terms(*cl, calls[c], t);
        for (int d = 0; d < cl->D; ++d) {
            bestd[d] = INF; bestp[d] = -1; used[d] = 0;
            for (int p = 0; p < cl->P; ++p) {
                const float f = candidate_fin(*cl, t, p, d, flags & ORC_FLAG_UNLOADED);
                if (f < bestd[d]) { bestd[d] = f; bestp[d] = p; }
            }
        }
        float delta = INF;
        for (int k = 0; k < K; ++k) {
            int arg = -1; float b = INF;
            for (int d = 0; d < cl->D; ++d)
                if (!used[d] && bestd[d] < b) { b = bestd[d]; arg = d; }
            const size_t o = (size_t)c * K + k;
            if (arg < 0) { pair[o] = -1; cost[o] = INF; tpre_sel[o] = 0.0f; continue; }
            used[arg] = 1;
            pair[o] = bestp[arg] * cl->D + arg;
            cost[o] = b;
            tpre_sel[o] = t.tpre[cl->typeP[bestp[arg]]];
            if (k == 0) delta = b;
        }
        const DagView v = dag_view(dag, calls[c], flags);
        prio[c] = (v.elapsed + delta) / v.H;
        m[c] = t.m;
    }
    return 0;
}

// Capacity-conflict pass over one chunk.  Calls are visited by decreasing prio
// (lower call index first among equals).  A call takes the first of its K
// candidates whose decode instance still has free KV tokens for it; that
// consumes the tokens and lengthens the chosen prefill queue by the call's
// prefill time.  A call none of whose candidates fits stays unplaced (-1).
// freeD[D] and qP[P] are updated in place.
int orc_conflict(int C, int K, int D, const int32_t* pair, const float* prio, const float* m,
                 const float* tpre_sel, float* freeD, float* qP, int32_t* assign) {
    std::vector<int> order(C);
    for (int c = 0; c < C; ++c) order[c] = c;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return prio[a] > prio[b]; });
    for (int i = 0; i < C; ++i) {
        const int c = order[i];
        assign[c] = -1;
        for (int k = 0; k < K; ++k) {
            const int32_t j = pair[(size_t)c * K + k];
            if (j < 0) continue;
            const int d = j % D, p = j / D;
            if (freeD[d] >= m[c]) {
                freeD[d] = freeD[d] - m[c];
                qP[p] = qP[p] + tpre_sel[(size_t)c * K + k];
                assign[c] = j;
                break;
            }
        }
    }
    return 0;
}

// Recomputing greedy planner for small queues (Algorithm 1, the while-loop over
// the queue snapshot; Section 5.3 "Adaptive greedy prefill assignment").
// Until the queue is empty: for every waiting call project its best feasible
// placement against the simulated state, its Delta and its ratio R (Eq. 2);
// take the call with the largest R (lower call index among equals); record its
// pair; update the simulated state; remove the call.
// Simulated state: the chosen prefill queue grows by the call's prefill time,
// the chosen decode instance loses m(c) free KV tokens; qD is left as it is.
// A pair is feasible when m(c) <= Cap(d) (Eq. 4) and m(c) <= free KV tokens of
// d in the simulated state.  A call without a feasible pair is passed over; the
// loop ends when no waiting call has one (the state never improves).
// Outputs: assign[c] pair or -1, ratio[c] = R at the moment of selection (+inf
// if never placed), order[i] = call taken in iteration i (-1 past the end);
// qP[P] and freeD[D] are updated in place; delta[c] (may be NULL) = the Delta
// inside ratio[c], +inf if never placed.  Returns the number of placed calls.
int orc_greedy(const OrcCluster* cl, const OrcDag* dag, const OrcCall* calls, int C, int flags,
               float* qP, float* freeD, int32_t* assign, float* ratio, int32_t* order, float* delta_out) {
    OrcCluster sim = *cl;
    sim.qP = qP;                                        // candidate_fin reads the simulated queues
    std::vector<char> waiting(C, 1);
    std::vector<Terms> terms(C);
    for (int c = 0; c < C; ++c) {
        latency_terms(*cl, calls[c], terms[c]); assign[c] = -1; ratio[c] = INF; order[c] = -1;
        if (delta_out) delta_out[c] = INF;
    }
    int placed = 0;
    for (int it = 0; it < C; ++it) {
        int best_c = -1, best_j = -1; float best_R = -INF, best_delta = INF;
        for (int c = 0; c < C; ++c) {
            if (!waiting[c]) continue;
            const Terms& t = terms[c];
            float delta = INF; int arg = -1;
            for (int p = 0; p < cl->P; ++p)
                for (int d = 0; d < cl->D; ++d) {
                    if (!(t.m <= freeD[d])) continue;           // KV tokens left in the simulated state
                    const float f = candidate_fin(sim, t, p, d, false);
                    if (f < delta) { delta = f; arg = p * cl->D + d; }
                }
            if (arg < 0) continue;
            const DagView v = dag_view(dag, calls[c], flags);
            const float R = (v.elapsed + delta) / v.H;          // Eq. 2
            if (R > best_R) { best_R = R; best_c = c; best_j = arg; best_delta = delta; }
        }
        if (best_c < 0) break;
        const int p = best_j / cl->D, d = best_j % cl->D;
        assign[best_c] = best_j; ratio[best_c] = best_R; order[it] = best_c;
        if (delta_out) delta_out[best_c] = best_delta;
        qP[p] = qP[p] + terms[best_c].tpre[cl->typeP[p]];
        freeD[d] = freeD[d] - terms[best_c].m;
        waiting[best_c] = 0;
        ++placed;
    }
    return placed;
}

// Decode-stage scheduler (Section 5.4): calls whose KV cache has arrived wait for
// decode admission.  Ranking by the projected ratio (Eq. 2), feasibility by the
// decode KV capacity (Eq. 3-4), now over time: every decode instance carries its
// token-capacity intervals (Section 6: "decode token-capacity intervals"), i.e.
// which calls hold how many KV tokens until when.
// "Adaptive greedy decode assignment": repeatedly take the most urgent waiting
// call, find the earliest capacity-feasible start on every legal instance,
// assign it to the instance with the earliest projected finish, and add its
// interval to the simulated state.  A call locked to an instance (chosen during
// prefill planning) may only go there; a free call may go to any instance that
// can ever hold it (m <= Cap).
//
// Usage of instance d over time is a step function: breakpoints t[0] = 0 < t[1] <
// ... and tokens in use u[k] on [t[k], t[k+1]) (the last segment runs to +inf).
// Earliest feasible start of a call with demand m, duration tau, ready at r:
// walk the segments from the one holding r; a segment with u[k] + m > Cap pushes
// the candidate start to its end; the candidate is accepted as soon as a segment
// ends at or after candidate + tau (binary32 addition) without such a push.
struct StepFn { std::vector<float> t, u; };     // t.size() == u.size() >= 1, t[0] == 0

static float earliest_start(const StepFn& f, float cap, float m, float tau, float ready, float* finish) {
    size_t k = 0;
    while (k + 1 < f.t.size() && f.t[k + 1] <= ready) ++k;      // segment that holds the ready time
    float cand = ready;
    for (;; ++k) {
        const float seg_end = (k + 1 < f.t.size()) ? f.t[k + 1] : INF;
        if (f.u[k] + m > cap) { cand = seg_end; continue; }       // no room here: not before this segment ends
        const float fin = cand + tau;
        if (seg_end >= fin) { *finish = fin; return cand; }
    }
}

static void add_interval(StepFn& f, float s, float e, float m) {
    auto cut = [&](float x) {                                     // make x a breakpoint; returns its index
        size_t k = 0;
        while (k + 1 < f.t.size() && f.t[k + 1] <= x) ++k;
        if (f.t[k] == x) return k;
        f.t.insert(f.t.begin() + k + 1, x);
        f.u.insert(f.u.begin() + k + 1, f.u[k]);
        return k + 1;
    };
    const size_t a = cut(s), b = cut(e);
    for (size_t k = a; k < b; ++k) f.u[k] = f.u[k] + m;
}

// run_ptr[D+1], run_start[] (NULL = all 0), run_end[], run_tok[]: intervals already on each instance
// (calls decoding now hold run_tok tokens from 0 until run_end seconds from now; intervals planned
// earlier may start later).  lock[c] = -1 or a decode instance; ready[c] = time the
// KV cache of c is on the decode side.  Outputs: inst[c] (-1 if it fits nowhere), start[c],
// ratio[c] = R at selection, order[i]; returns the number of placed calls.
int orc_decode_greedy(const OrcCluster* cl, const OrcDag* dag, const OrcCall* calls, int C, int flags,
                      const uint32_t* run_ptr, const float* run_start, const float* run_end, const float* run_tok,
                      const int32_t* lock, const float* ready,
                      int32_t* inst, float* start, float* ratio, int32_t* order) {
    const int D = cl->D;
    std::vector<StepFn> fn(D);
    for (int d = 0; d < D; ++d) {
        fn[d].t.assign(1, 0.0f); fn[d].u.assign(1, 0.0f);
        for (uint32_t i = run_ptr[d]; i < run_ptr[d + 1]; ++i)
            add_interval(fn[d], run_start ? run_start[i] : 0.0f, run_end[i], run_tok[i]);
    }
    std::vector<Terms> terms(C);
    std::vector<char> waiting(C, 1);
    for (int c = 0; c < C; ++c) { latency_terms(*cl, calls[c], terms[c]); inst[c] = -1; start[c] = INF; ratio[c] = INF; order[c] = -1; }
    int placed = 0;
    for (int it = 0; it < C; ++it) {
        int best_c = -1, best_d = -1; float best_R = -INF, best_s = 0.0f, best_f = 0.0f;
        for (int c = 0; c < C; ++c) {
            if (!waiting[c]) continue;
            const Terms& t = terms[c];
            float fin = INF, st = 0.0f; int arg = -1;
            for (int d = 0; d < D; ++d) {
                if (lock[c] >= 0 && lock[c] != d) continue;     // locked calls do not migrate
                if (!(t.m <= cl->capD[d])) continue;            // Eq. 4
                float f;
                const float s = earliest_start(fn[d], cl->capD[d], t.m, t.tdec[cl->typeD[d]], ready[c], &f);
                if (f < fin) { fin = f; st = s; arg = d; }
            }
            if (arg < 0) continue;
            const DagView v = dag_view(dag, calls[c], flags);
            const float R = (v.elapsed + fin) / v.H;            // Eq. 2 with Delta_D = projected decode finish
            if (R > best_R) { best_R = R; best_c = c; best_d = arg; best_s = st; best_f = fin; }
        }
        if (best_c < 0) break;
        add_interval(fn[best_d], best_s, best_f, terms[best_c].m);
        inst[best_c] = best_d; start[best_c] = best_s; ratio[best_c] = best_R; order[it] = best_c;
        waiting[best_c] = 0;
        ++placed;
    }
    return placed;
}

// One-pass ordering for the decode stage (Section 5.4: queues that are large, or
// a special case, fall back to the lightweight ordering of Section 5.3, last
// sentence: one pass in the order of the risk score instead of re-planning after
// every assignment).  Reading taken here: the score is the ratio of Eq. 2 with
// Delta_D projected against the snapshot alone, as if no other queued call were
// there; the calls are visited once by decreasing score (lower index first among
// equals); a visited call is projected against the state that the calls before it
// have left and takes the instance with the earliest finish, as in the greedy
// form.  Arguments and outputs as orc_decode_greedy; ratio[c] is the score the
// call was ordered by.
int orc_decode_onepass(const OrcCluster* cl, const OrcDag* dag, const OrcCall* calls, int C, int flags,
                       const uint32_t* run_ptr, const float* run_start, const float* run_end, const float* run_tok,
                       const int32_t* lock, const float* ready,
                       int32_t* inst, float* start, float* ratio, int32_t* order) {
    const int D = cl->D;
    std::vector<StepFn> fn(D);
    for (int d = 0; d < D; ++d) {
        fn[d].t.assign(1, 0.0f); fn[d].u.assign(1, 0.0f);
        for (uint32_t i = run_ptr[d]; i < run_ptr[d + 1]; ++i)
            add_interval(fn[d], run_start ? run_start[i] : 0.0f, run_end[i], run_tok[i]);
    }
    std::vector<Terms> terms(C);
    for (int c = 0; c < C; ++c) { latency_terms(*cl, calls[c], terms[c]); inst[c] = -1; start[c] = INF; ratio[c] = INF; order[c] = -1; }
    // earliest finish of call c over its legal instances in the current state
    auto project = [&](int c, float* st, float* fin) {
        const Terms& t = terms[c];
        int arg = -1; *fin = INF; *st = 0.0f;
        for (int d = 0; d < D; ++d) {
            if (lock[c] >= 0 && lock[c] != d) continue;
            if (!(t.m <= cl->capD[d])) continue;                    // Eq. 4
            float f;
            const float s = earliest_start(fn[d], cl->capD[d], t.m, t.tdec[cl->typeD[d]], ready[c], &f);
            if (f < *fin) { *fin = f; *st = s; arg = d; }
        }
        return arg;
    };
    std::vector<int> visit;
    std::vector<float> score(C, -INF);
    for (int c = 0; c < C; ++c) {
        float st, fin;
        if (project(c, &st, &fin) < 0) continue;                    // fits no instance: never visited
        const DagView v = dag_view(dag, calls[c], flags);
        score[c] = (v.elapsed + fin) / v.H;                         // Eq. 2 against the snapshot
        visit.push_back(c);
    }
    std::stable_sort(visit.begin(), visit.end(), [&](int a, int b) { return score[a] > score[b]; });
    int placed = 0;
    for (int c : visit) {
        float st, fin;
        const int d = project(c, &st, &fin);
        if (d < 0) continue;
        add_interval(fn[d], st, fin, terms[c].m);
        inst[c] = d; start[c] = st; ratio[c] = score[c]; order[placed++] = c;
    }
    return placed;
}

// Longest node-weighted path to a sink, per node, over a successor-CSR DAG:
//   tail[v] = max over successors u of cp[u]   (0 without successors)
//   cp[v]   = cost[v] + tail[v]
//   H[w]    = max over nodes v of workflow w of cp[v]
// Nodes are visited in reverse topological order (Kahn), so every sum runs from
// the sink towards the source.  Returns -1 if the graph has a cycle.
int orc_longest_path(const uint32_t* row_ptr, const uint32_t* col, const float* cost,
                     const uint32_t* node_wf, uint32_t N, uint32_t W,
                     float* cp, float* tail, float* H) {
    std::vector<uint32_t> indeg(N, 0), topo;
    topo.reserve(N);
    for (uint32_t v = 0; v < N; ++v)
        for (uint32_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) ++indeg[col[e]];
    for (uint32_t v = 0; v < N; ++v) if (indeg[v] == 0) topo.push_back(v);
    for (size_t i = 0; i < topo.size(); ++i) {
        const uint32_t v = topo[i];
        for (uint32_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e)
            if (--indeg[col[e]] == 0) topo.push_back(col[e]);
    }
    if (topo.size() != N) return -1;
    for (uint32_t w = 0; w < W; ++w) H[w] = 0.0f;
    for (size_t i = N; i-- > 0;) {
        const uint32_t v = topo[i];
        float t = 0.0f;
        for (uint32_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) t = std::fmax(t, cp[col[e]]);
        tail[v] = t;
        cp[v] = cost[v] + t;
        H[node_wf[v]] = std::fmax(H[node_wf[v]], cp[v]);
    }
    return 0;
}

// Earliest start and finish of every node when each node takes its cost and
// starts as soon as all its predecessors have finished (Section 4.1: a node is
// ready when all predecessors have completed):
//   est[v] = max over predecessors u of eft[u]   (0 without predecessors)
//   eft[v] = est[v] + cost[v]
// Nodes are visited in topological order (Kahn) and each finished node pushes
// its finish time to its successors, so every sum runs from the source towards
// the sink.  Returns -1 if the graph has a cycle.
int orc_earliest_start(const uint32_t* row_ptr, const uint32_t* col, const float* cost,
                       uint32_t N, float* est, float* eft) {
    std::vector<uint32_t> indeg(N, 0), ready;
    ready.reserve(N);
    for (uint32_t v = 0; v < N; ++v)
        for (uint32_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) ++indeg[col[e]];
    for (uint32_t v = 0; v < N; ++v) { est[v] = 0.0f; if (indeg[v] == 0) ready.push_back(v); }
    for (size_t i = 0; i < ready.size(); ++i) {
        const uint32_t v = ready[i];
        eft[v] = est[v] + cost[v];
        for (uint32_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) {
            const uint32_t u = col[e];
            est[u] = std::fmax(est[u], eft[v]);
            if (--indeg[u] == 0) ready.push_back(u);
        }
    }
    return ready.size() == N ? 0 : -1;
}

// Double-precision twin of orc_fin_all in textbook form (units converted first,
// plain divisions), to measure the rounding error of the binary32 sequence.
int orc_fin_all_f64(const OrcCluster* cl, const OrcCall* calls, int C, int flags, double* fin) {
    for (int c = 0; c < C; ++c) {
        const double n = calls[c].prompt_tokens, o = calls[c].output_tokens;
        const double phi = cl->flops_per_token[calls[c].model];
        const double omega = cl->weight_bytes[calls[c].model];
        const double kappa = cl->kv_bytes_per_token[calls[c].model];
        for (int p = 0; p < cl->P; ++p)
            for (int d = 0; d < cl->D; ++d) {
                const int gp = cl->typeP[p], gd = cl->typeD[d];
                const double F = cl->peak_tflops[gp] * 1e12, Bp = cl->hbm_tbps[gp] * 1e12;
                const double Bd = cl->hbm_tbps[gd] * 1e12;
                const double L = cl->link_gbps[(size_t)p * cl->D + d] * 1e9;
                const double qp = (flags & ORC_FLAG_UNLOADED) ? 0.0 : cl->qP[p];
                const double qd = (flags & ORC_FLAG_UNLOADED) ? 0.0 : cl->qD[d];
                const double psi = cl->attn_flops_per_token2 ? cl->attn_flops_per_token2[calls[c].model] : 0.0;
                const double tpre = std::max((n * phi + n * n * psi) / F, (omega + n * kappa) / Bp);
                const double tdec = o * (omega + kappa * (n + 0.5 * (o - 1.0))) / Bd;
                const double ready = qp + tpre + n * kappa / L;
                const double start = std::max(ready, qd);
                fin[((size_t)c * cl->P + p) * cl->D + d] =
                    (n + o <= cl->capD[d]) ? start + tdec : std::numeric_limits<double>::infinity();
            }
    }
    return 0;
}

}  // extern "C"
