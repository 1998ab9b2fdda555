// Event-driven replay around the greedy planner (hx_replay in hx.h): host control
// flow only.  Every planning decision is taken by hx_schedule_greedy_plan on the
// device; this file keeps the clock, the event queue and the state that is shown
// to the planner at each event time.
#include <algorithm>
#include <cmath>
#include <queue>
#include <set>
#include <tuple>

#include "hx_internal.h"

namespace {

struct Event {
    double t; int kind; uint32_t id;           // kind 0: workflow arrives, 1: call completes
    bool operator>(const Event& o) const { return std::tie(t, kind, id) > std::tie(o.t, o.kind, o.id); }
};

struct Hold { double end; int d; double tokens; };

struct Buffers {                               // device scratch and page-locked staging of one replay, freed on every way out
    hx_call* calls = nullptr; int32_t* assign = nullptr; float* ratio = nullptr; int32_t* order = nullptr;
    float* delta = nullptr;
    unsigned char* pinned = nullptr;
    ~Buffers() {
        cudaFree(calls); cudaFree(assign); cudaFree(ratio); cudaFree(order);   // delta lies behind assign
        cudaFreeHost(pinned);
    }
};

double order_statistic(std::vector<double> r, double q) {
    std::sort(r.begin(), r.end());
    const long k = std::max(0L, (long)std::ceil(q * (double)r.size()) - 1);
    return r[(size_t)k];
}

}  // namespace

extern "C" int hx_replay(hx_cluster* h, const uint32_t* row_ptr, const uint32_t* col_idx,
                         const uint32_t* node_workflow, uint32_t n_nodes, uint32_t n_workflows,
                         const hx_call* node_calls, const double* arrival_s, int qmax,
                         double* out_fin, double* out_ratio, double* out_req, int* out_stats, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (!row_ptr || !node_workflow || !node_calls || !arrival_s || !out_fin || !out_ratio || !out_req || !out_stats)
        return hx_fail(h, HX_ERR_INVALID_ARG, "NULL array");
    if (qmax < 1 || qmax > HX_GREEDY_MAX_CALLS) return hx_fail(h, HX_ERR_INVALID_ARG, "qmax must be 1 .. HX_GREEDY_MAX_CALLS");
    const uint32_t N = n_nodes, W = n_workflows;
    int P = 0, D = 0;
    const float* d_cap = nullptr;
    uint32_t up_nodes = 0, up_workflows = 0;
    hx_cluster_shape(h, &P, &D, &d_cap, &up_nodes, &up_workflows);
    if (up_nodes != N || up_workflows != W) return hx_fail(h, HX_ERR_INVALID_ARG, "the graph given is not the uploaded one (sizes differ)");
    {   // the arrays given again must describe the forest the horizons were computed on: nothing below indexes with
        // a value that has not been checked against the library's own copy
        std::vector<uint32_t> row, col, nwf;
        hx_forest_host(h, &row, &col, &nwf);
        bool same = row_ptr[0] == 0;
        for (uint32_t v = 0; v < N && same; ++v)
            same = row_ptr[v + 1] == row[v + 1] && node_workflow[v] == nwf[v];     // equal row bounds: every index below is in range
        if (same && !col.empty() && !col_idx) same = false;
        std::vector<uint32_t> a, b;
        for (uint32_t v = 0; v < N && same; ++v) {
            a.assign(col_idx + row[v], col_idx + row[v + 1]); b.assign(col.begin() + row[v], col.begin() + row[v + 1]);
            std::sort(a.begin(), a.end()); std::sort(b.begin(), b.end());
            same = a == b;
        }
        if (!same) return hx_fail(h, HX_ERR_INVALID_ARG, "the graph given is not the uploaded one");
    }
    const float *d_cp = nullptr, *d_tail = nullptr, *d_H = nullptr;
    int rc = hx_get_dag_results(h, &d_cp, &d_tail, &d_H);
    if (rc != HX_OK) return rc;
    for (uint32_t w = 0; w < W; ++w)
        if (!(arrival_s[w] >= 0.0) || !std::isfinite(arrival_s[w])) return hx_fail(h, HX_ERR_INVALID_ARG, "arrival times must be finite and >= 0");
    for (uint32_t v = 0; v < N; ++v)
        if (node_workflow[v] >= W || node_calls[v].node != v) return hx_fail(h, HX_ERR_INVALID_ARG, "node_calls[v] must describe node v of an existing workflow");

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<float> cap(D), H(W);
    if (cudaMemcpyAsync(cap.data(), d_cap, D * sizeof(float), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaMemcpyAsync(H.data(), d_H, W * sizeof(float), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
        return hx_fail(h, HX_ERR_CUDA, "reading capacities and horizons");
    Buffers b;
    // pairs and projected completions side by side: one copy brings a plan back
    if (cudaMalloc(&b.calls, (size_t)qmax * sizeof(hx_call)) != cudaSuccess || cudaMalloc(&b.assign, (size_t)qmax * 8) != cudaSuccess ||
        cudaMalloc(&b.ratio, (size_t)qmax * 4) != cudaSuccess || cudaMalloc(&b.order, (size_t)qmax * 4) != cudaSuccess)
        return hx_fail(h, HX_ERR_OOM, "replay scratch");
    b.delta = reinterpret_cast<float*>(b.assign + qmax);

    std::vector<uint32_t> left(N, 0);
    for (uint32_t e = 0; e < row_ptr[N]; ++e) ++left[col_idx[e]];
    std::vector<std::vector<uint32_t>> sources(W);
    for (uint32_t v = 0; v < N; ++v) if (left[v] == 0) sources[node_workflow[v]].push_back(v);
    std::priority_queue<Event, std::vector<Event>, std::greater<Event>> events;
    for (uint32_t w = 0; w < W; ++w) events.push(Event{arrival_s[w], 0, w});
    std::vector<double> busy(P, 0.0), used(D);
    std::vector<Hold> holds;
    std::set<uint32_t> ready;                   // ordered: calls are offered in increasing node number
    // staging in page-locked memory: the copies of a planner run are asynchronous and cost one synchronisation
    const size_t n_f32 = 2 * (size_t)P + 2 * (size_t)D + W + qmax;
    if (cudaHostAlloc(&b.pinned, (size_t)qmax * sizeof(hx_call) + n_f32 * 4 + (size_t)qmax * 4, cudaHostAllocDefault) != cudaSuccess)
        return hx_fail(h, HX_ERR_OOM, "replay staging");
    hx_call* chunk = reinterpret_cast<hx_call*>(b.pinned);
    // queue loads, decode hints and free tokens in the order of the device tables (one copy refreshes all three),
    // pairs and completions in the order of the device results
    float* qP = reinterpret_cast<float*>(chunk + qmax);
    float *qD = qP + P, *kv_free = qD + D, *qP2 = kv_free + D, *elapsed = qP2 + P;
    int32_t* assign = reinterpret_cast<int32_t*>(elapsed + W);
    float* delta = reinterpret_cast<float*>(assign + qmax);
    for (int d = 0; d < D; ++d) qD[d] = 0.0f;
    std::vector<uint32_t> offered;
    std::vector<char> touched(P);
    for (uint32_t v = 0; v < N; ++v) out_fin[v] = INFINITY;
    int runs = 0;
    const hx_options saved = hx_current_options(h);
    hx_options plan = saved;
    plan.score_mode = HX_MODE_RATIO; plan.commit = 1; plan.topk = 0;
    plan.flags = saved.flags & ~(HX_FLAG_NO_DAG | HX_FLAG_UNLOADED);
    if ((rc = hx_set_options(h, &plan)) != HX_OK) return rc;
    auto leave = [&](int code) { hx_set_options(h, &saved); return code; };

    while (!events.empty()) {
        const double t = events.top().t;
        while (!events.empty() && events.top().t == t) {
            const Event ev = events.top(); events.pop();
            if (ev.kind == 0) {
                for (uint32_t v : sources[ev.id]) ready.insert(v);
            } else {
                for (uint32_t e = row_ptr[ev.id]; e < row_ptr[ev.id + 1]; ++e)
                    if (--left[col_idx[e]] == 0) ready.insert(col_idx[e]);
            }
        }
        offered.assign(ready.begin(), ready.end());
        for (size_t o = 0; o < offered.size(); o += (size_t)qmax) {
            const int n = (int)std::min<size_t>(qmax, offered.size() - o);
            // the state of the cluster at time t, rounded to binary32 for the planner
            for (int p = 0; p < P; ++p) qP[p] = (float)std::max(0.0, busy[p] - t);
            std::fill(used.begin(), used.end(), 0.0);
            for (const Hold& hd : holds) if (hd.end > t) used[hd.d] += hd.tokens;
            for (int d = 0; d < D; ++d) kv_free[d] = (float)((double)cap[d] - used[d]);
            for (uint32_t w = 0; w < W; ++w) elapsed[w] = (float)std::max(0.0, t - arrival_s[w]);
            for (int i = 0; i < n; ++i) chunk[i] = node_calls[offered[o + i]];
            if ((rc = hx_update_loads_packed(h, qP, s)) != HX_OK) return leave(rc);
            if ((rc = hx_dag_update_elapsed(h, elapsed, stream)) != HX_OK) return leave(rc);
            if (cudaMemcpyAsync(b.calls, chunk, (size_t)n * sizeof(hx_call), cudaMemcpyHostToDevice, s) != cudaSuccess)
                return leave(hx_fail(h, HX_ERR_CUDA, "copying the ready calls"));
            if ((rc = hx_schedule_greedy_plan(h, b.calls, n, b.assign, b.ratio, b.order, b.delta, stream)) != HX_OK) return leave(rc);
            if (cudaMemcpyAsync(assign, b.assign, (size_t)qmax * 8, cudaMemcpyDeviceToHost, s) != cudaSuccess)
                return leave(hx_fail(h, HX_ERR_CUDA, "reading the plan"));
            if ((rc = hx_cluster_read_loads(h, qP2, nullptr, nullptr, stream)) != HX_OK) return leave(rc);   // synchronises
            ++runs;
            std::fill(touched.begin(), touched.end(), 0);
            for (int i = 0; i < n; ++i) {
                if (assign[i] < 0) continue;
                const uint32_t v = offered[o + i];
                const int p = assign[i] / D, d = assign[i] % D;
                out_fin[v] = t + (double)delta[i];
                events.push(Event{out_fin[v], 1, v});
                holds.push_back(Hold{out_fin[v], d, (double)(node_calls[v].prompt_tokens + node_calls[v].output_tokens)});
                ready.erase(v);
                touched[p] = 1;
            }
            for (int p = 0; p < P; ++p) if (touched[p]) busy[p] = t + (double)qP2[p];
        }
        holds.erase(std::remove_if(holds.begin(), holds.end(), [&](const Hold& hd) { return !(hd.end > t); }), holds.end());
    }
    std::vector<double> done(W, -INFINITY), ratio(W);
    for (uint32_t v = 0; v < N; ++v) done[node_workflow[v]] = std::max(done[node_workflow[v]], out_fin[v]);
    for (uint32_t w = 0; w < W; ++w) out_ratio[w] = ratio[w] = (done[w] - arrival_s[w]) / (double)H[w];
    out_req[0] = W ? order_statistic(ratio, 0.95) : 0.0;
    out_req[1] = W ? order_statistic(ratio, 0.99) : 0.0;
    out_stats[0] = runs; out_stats[1] = (int)ready.size();
    return leave(HX_OK);
}

// ---------------------------------------------------------------------------
// hx_replay_lifecycle: the stages of a call's life kept apart, the decode stage
// scheduled, estimates that may differ from the service a call gets.
// ---------------------------------------------------------------------------
namespace {

struct LifeBuffers {                           // device scratch and page-locked staging, freed on every way out
    std::vector<void*> dev; void* pinned = nullptr;
    template <class T> bool alloc(T** p, size_t n) {
        void* q = nullptr;
        if (cudaMalloc(&q, std::max<size_t>(n, 1) * sizeof(T)) != cudaSuccess) return false;
        dev.push_back(q); *p = static_cast<T*>(q); return true;
    }
    ~LifeBuffers() { for (void* q : dev) cudaFree(q); cudaFreeHost(pinned); }
};

struct ModelGuard { hx_cluster* h; ~ModelGuard() { hx_pop_scaled_models(h); } };

inline int error_sign(uint32_t v) { return ((v * 2654435761u) >> 31) & 1u ? 1 : -1; }

constexpr double kTinyS = 1e-6;                // estimated time left of a call that outlives its estimate

}  // namespace

extern "C" int hx_replay_lifecycle(hx_cluster* h, const hx_call* node_calls, const double* arrival_s, double est_error,
                                   int qmax, double* out_fin, double* out_ratio, double* out_req, int* out_stats,
                                   void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (!node_calls || !arrival_s || !out_fin || !out_ratio || !out_req || !out_stats) return hx_fail(h, HX_ERR_INVALID_ARG, "NULL array");
    if (qmax < 1 || qmax > HX_GREEDY_MAX_CALLS) return hx_fail(h, HX_ERR_INVALID_ARG, "qmax must be 1 .. HX_GREEDY_MAX_CALLS");
    if (!(est_error >= 0.0) || !(est_error < 1.0)) return hx_fail(h, HX_ERR_INVALID_ARG, "est_error must be in [0, 1)");
    int P = 0, D = 0;
    const float* d_cap = nullptr;
    uint32_t N = 0, W = 0;
    hx_cluster_shape(h, &P, &D, &d_cap, &N, &W);
    if (N == 0) return hx_fail(h, HX_ERR_NOT_READY, "no forest uploaded");
    const float *d_cp = nullptr, *d_tail = nullptr, *d_H = nullptr;
    int rc = hx_get_dag_results(h, &d_cp, &d_tail, &d_H);
    if (rc != HX_OK) return rc;
    std::vector<uint32_t> row, col, node_wf;
    hx_forest_host(h, &row, &col, &node_wf);
    for (uint32_t w = 0; w < W; ++w)
        if (!(arrival_s[w] >= 0.0) || !std::isfinite(arrival_s[w])) return hx_fail(h, HX_ERR_INVALID_ARG, "arrival times must be finite and >= 0");
    for (uint32_t v = 0; v < N; ++v)
        if (node_calls[v].node != v) return hx_fail(h, HX_ERR_INVALID_ARG, "node_calls[v] must describe node v");

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<int> typeP, typeD; std::vector<float> invLT;
    int Ppad = 0, G = 0, M = 0;
    if ((rc = hx_cluster_tables_host(h, &typeP, &typeD, &invLT, &Ppad, &G, &M, s)) != HX_OK) return rc;
    for (uint32_t v = 0; v < N; ++v)
        if (node_calls[v].model >= (uint32_t)M) return hx_fail(h, HX_ERR_INVALID_ARG, "model id out of range");
    std::vector<float> cap(D), H(W);
    if (cudaMemcpyAsync(cap.data(), d_cap, D * sizeof(float), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaMemcpyAsync(H.data(), d_H, W * sizeof(float), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
        return hx_fail(h, HX_ERR_CUDA, "reading capacities and horizons");

    // what the schedulers see: every call refers to a copy of its model with the constants scaled by 1 + eps or 1 - eps
    if ((rc = hx_push_scaled_models(h, (float)(1.0 + est_error), (float)(1.0 - est_error))) != HX_OK) return rc;
    ModelGuard models{h};
    std::vector<hx_call> seen(node_calls, node_calls + N);
    for (uint32_t v = 0; v < N; ++v) seen[v].model += error_sign(v) > 0 ? (uint32_t)M : 2u * (uint32_t)M;

    const int dmax = HX_DECODE_MAX_CALLS;
    LifeBuffers b;
    hx_call *d_all = nullptr, *d_calls = nullptr, *d_dcalls = nullptr;
    float *d_tp = nullptr, *d_td = nullptr, *d_kv = nullptr, *d_m = nullptr, *d_ratio = nullptr, *d_dstart = nullptr, *d_dratio = nullptr;
    int32_t *d_assign = nullptr, *d_order = nullptr, *d_lock = nullptr, *d_dinst = nullptr, *d_dorder = nullptr;
    if (!b.alloc(&d_all, N) || !b.alloc(&d_tp, (size_t)N * G) || !b.alloc(&d_td, (size_t)N * G) || !b.alloc(&d_kv, N) || !b.alloc(&d_m, N) ||
        !b.alloc(&d_calls, qmax) || !b.alloc(&d_assign, 2 * (size_t)qmax) || !b.alloc(&d_ratio, qmax) ||
        !b.alloc(&d_dcalls, dmax) || !b.alloc(&d_lock, dmax) || !b.alloc(&d_dinst, dmax) || !b.alloc(&d_dstart, dmax) ||
        !b.alloc(&d_dratio, dmax) || !b.alloc(&d_dorder, dmax))
        return hx_fail(h, HX_ERR_OOM, "replay scratch");
    d_order = d_assign + qmax;                 // pairs and order side by side: one copy brings a plan back
    // service times from the library's own estimator: the real ones and the ones the schedulers believe
    std::vector<float> tpre((size_t)N * G), tdec((size_t)N * G), tpre_s((size_t)N * G), tdec_s((size_t)N * G), kvB(N), m_tok(N);
    for (int pass = 0; pass < 2; ++pass) {
        const hx_call* src = pass == 0 ? node_calls : seen.data();
        std::vector<float>& tp = pass == 0 ? tpre : tpre_s; std::vector<float>& td = pass == 0 ? tdec : tdec_s;
        if (cudaMemcpyAsync(d_all, src, (size_t)N * sizeof(hx_call), cudaMemcpyHostToDevice, s) != cudaSuccess)
            return hx_fail(h, HX_ERR_CUDA, "copying the call records");
        if ((rc = hx_estimate_calls(h, d_all, (int)N, d_tp, d_td, d_kv, d_m, stream)) != HX_OK) return rc;
        if (cudaMemcpyAsync(tp.data(), d_tp, tp.size() * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaMemcpyAsync(td.data(), d_td, td.size() * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            (pass == 0 && (cudaMemcpyAsync(kvB.data(), d_kv, (size_t)N * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||      // the KV bytes that really travel
                           cudaMemcpyAsync(m_tok.data(), d_m, (size_t)N * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess)) ||
            cudaStreamSynchronize(s) != cudaSuccess)
            return hx_fail(h, HX_ERR_CUDA, "reading the service times");
    }

    const size_t n_f32 = (size_t)P + 2 * (size_t)D + W;
    const size_t pin_bytes = (size_t)qmax * sizeof(hx_call) + (size_t)dmax * sizeof(hx_call) + n_f32 * 4 +
                             2 * (size_t)qmax * 4 + 2 * (size_t)dmax * 4;
    if (cudaHostAlloc(&b.pinned, pin_bytes, cudaHostAllocDefault) != cudaSuccess) return hx_fail(h, HX_ERR_OOM, "replay staging");
    hx_call* chunk = static_cast<hx_call*>(b.pinned);
    hx_call* dchunk = chunk + qmax;
    float* qP = reinterpret_cast<float*>(dchunk + dmax);
    float *qD = qP + P, *kv_free = qD + D, *elapsed = kv_free + D;
    int32_t* assign = reinterpret_cast<int32_t*>(elapsed + W);
    int32_t *order = assign + qmax, *lock = order + qmax, *dorder = lock + dmax;
    for (int d = 0; d < D; ++d) qD[d] = 0.0f;

    std::vector<uint32_t> left(N, 0);
    for (uint32_t e = 0; e < (uint32_t)col.size(); ++e) ++left[col[e]];
    std::vector<std::vector<uint32_t>> sources(W);
    for (uint32_t v = 0; v < N; ++v) if (left[v] == 0) sources[node_wf[v]].push_back(v);
    std::priority_queue<Event, std::vector<Event>, std::greater<Event>> events;   // kinds: 0 arrival, 1 prefill done, 2 transfer done, 3 decode done
    for (uint32_t w = 0; w < W; ++w) events.push(Event{arrival_s[w], 0, w});
    std::vector<std::vector<uint32_t>> queue(P), waiting(D);
    std::vector<int64_t> serving(P, -1); std::vector<double> serve_start(P, 0.0);
    std::vector<std::set<uint32_t>> running(D);
    std::vector<double> dstart(N, INFINITY), free_act(D), reserved(D, 0.0), dprio(N, INFINITY);
    std::vector<int32_t> pair(N, -1);
    for (int d = 0; d < D; ++d) free_act[d] = (double)cap[d];
    std::set<uint32_t> ready;
    std::vector<uint32_t> offered, wait_all;
    std::vector<uint32_t> run_ptr((size_t)D + 1);
    std::vector<hx_kv_interval> run;
    for (uint32_t v = 0; v < N; ++v) out_fin[v] = INFINITY;
    int runs = 0, decode_runs = 0;
    const hx_options saved = hx_current_options(h);
    hx_options plan = saved;
    plan.score_mode = HX_MODE_RATIO; plan.commit = 0; plan.topk = 0;
    plan.flags = saved.flags & ~(HX_FLAG_NO_DAG | HX_FLAG_UNLOADED);
    if ((rc = hx_set_options(h, &plan)) != HX_OK) return rc;
    auto leave = [&](int code) { hx_set_options(h, &saved); return code; };

    while (!events.empty()) {
        const double t = events.top().t;
        bool arrived = false;
        while (!events.empty() && events.top().t == t) {
            const Event ev = events.top(); events.pop();
            const uint32_t x = ev.id;
            if (ev.kind == 0) {
                for (uint32_t v : sources[x]) ready.insert(v);
            } else if (ev.kind == 1) {
                const int p = pair[x] / D, d = pair[x] % D;
                serving[p] = -1;
                events.push(Event{t + (double)(kvB[x] * invLT[(size_t)d * Ppad + p]), 2, x});
            } else if (ev.kind == 2) {
                waiting[pair[x] % D].push_back(x);
                arrived = true;
            } else {
                const int d = pair[x] % D;
                running[d].erase(x);
                free_act[d] += (double)m_tok[x]; reserved[d] -= (double)m_tok[x];
                out_fin[x] = t;
                for (uint32_t e = row[x]; e < row[x + 1]; ++e)
                    if (--left[col[e]] == 0) ready.insert(col[e]);
            }
        }
        for (uint32_t w = 0; w < W; ++w) elapsed[w] = (float)std::max(0.0, t - arrival_s[w]);
        bool elapsed_sent = false;
        // prefill stage: the recomputing greedy over the ready calls
        offered.assign(ready.begin(), ready.end());
        for (size_t o = 0; o < offered.size(); o += (size_t)qmax) {
            const int n = (int)std::min<size_t>(qmax, offered.size() - o);
            for (int p = 0; p < P; ++p) {
                double q = 0.0;
                if (serving[p] >= 0) q = std::max(0.0, serve_start[p] + (double)tpre_s[(size_t)serving[p] * G + typeP[p]] - t);
                for (uint32_t c : queue[p]) q += (double)tpre_s[(size_t)c * G + typeP[p]];
                qP[p] = (float)q;
            }
            for (int d = 0; d < D; ++d) kv_free[d] = (float)((double)cap[d] - reserved[d]);
            for (int i = 0; i < n; ++i) chunk[i] = seen[offered[o + i]];
            if ((rc = hx_update_loads_packed(h, qP, s)) != HX_OK) return leave(rc);
            if (!elapsed_sent) { if ((rc = hx_dag_update_elapsed(h, elapsed, stream)) != HX_OK) return leave(rc); elapsed_sent = true; }
            if (cudaMemcpyAsync(d_calls, chunk, (size_t)n * sizeof(hx_call), cudaMemcpyHostToDevice, s) != cudaSuccess)
                return leave(hx_fail(h, HX_ERR_CUDA, "copying the ready calls"));
            if ((rc = hx_schedule_greedy_plan(h, d_calls, n, d_assign, d_ratio, d_order, nullptr, stream)) != HX_OK) return leave(rc);
            if (cudaMemcpyAsync(assign, d_assign, (size_t)qmax * 8, cudaMemcpyDeviceToHost, s) != cudaSuccess ||   // pairs and order, side by side
                cudaStreamSynchronize(s) != cudaSuccess)
                return leave(hx_fail(h, HX_ERR_CUDA, "reading the plan"));
            ++runs;
            for (int i = 0; i < n && order[i] >= 0; ++i) {         // in the order the planner took them
                const uint32_t v = offered[o + order[i]];
                const int a = assign[order[i]];
                pair[v] = a;
                queue[a / D].push_back(v);
                reserved[a % D] += (double)m_tok[v];
                ready.erase(v);
            }
        }
        // decode stage: a plan over everything that waits for decode, the planned instance as the lock
        if (arrived) {
            wait_all.clear();
            for (int d = 0; d < D; ++d) wait_all.insert(wait_all.end(), waiting[d].begin(), waiting[d].end());
            std::sort(wait_all.begin(), wait_all.end());
            if (wait_all.size() > (size_t)dmax) wait_all.resize(dmax);
            run.clear();
            for (int d = 0; d < D; ++d) {
                run_ptr[d] = (uint32_t)run.size();
                for (uint32_t c : running[d])
                    run.push_back(hx_kv_interval{(float)std::max(dstart[c] + (double)tdec_s[(size_t)c * G + typeD[d]] - t, kTinyS), m_tok[c]});
            }
            run_ptr[D] = (uint32_t)run.size();
            const int n = (int)wait_all.size();
            for (int i = 0; i < n; ++i) { dchunk[i] = seen[wait_all[i]]; lock[i] = pair[wait_all[i]] % D; }
            if (!elapsed_sent) { if ((rc = hx_dag_update_elapsed(h, elapsed, stream)) != HX_OK) return leave(rc); elapsed_sent = true; }
            if ((rc = hx_decode_set_running(h, run_ptr.data(), run.data(), stream)) != HX_OK) return leave(rc);
            if (cudaMemcpyAsync(d_dcalls, dchunk, (size_t)n * sizeof(hx_call), cudaMemcpyHostToDevice, s) != cudaSuccess ||
                cudaMemcpyAsync(d_lock, lock, (size_t)n * 4, cudaMemcpyHostToDevice, s) != cudaSuccess)
                return leave(hx_fail(h, HX_ERR_CUDA, "copying the decode queue"));
            if ((rc = hx_schedule_decode(h, d_dcalls, d_lock, nullptr, n, d_dinst, d_dstart, d_dratio, d_dorder, stream)) != HX_OK) return leave(rc);
            if (cudaMemcpyAsync(dorder, d_dorder, (size_t)n * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
                cudaStreamSynchronize(s) != cudaSuccess)
                return leave(hx_fail(h, HX_ERR_CUDA, "reading the decode plan"));
            ++decode_runs;
            for (uint32_t v : wait_all) dprio[v] = INFINITY;
            for (int i = 0; i < n && dorder[i] >= 0; ++i) dprio[wait_all[dorder[i]]] = (double)i;
        }
        // admission in plan order on the tokens really free, then the prefill instances take their next call
        for (int d = 0; d < D; ++d) {
            std::vector<uint32_t>& wq = waiting[d];
            std::sort(wq.begin(), wq.end(), [&](uint32_t a, uint32_t c) { return std::make_pair(dprio[a], a) < std::make_pair(dprio[c], c); });
            size_t keep = 0;
            for (uint32_t v : wq) {
                if ((double)m_tok[v] <= free_act[d]) {
                    free_act[d] -= (double)m_tok[v]; running[d].insert(v); dstart[v] = t;
                    events.push(Event{t + (double)tdec[(size_t)v * G + typeD[d]], 3, v});
                } else {
                    wq[keep++] = v;
                }
            }
            wq.resize(keep);
        }
        for (int p = 0; p < P; ++p)
            if (serving[p] < 0 && !queue[p].empty()) {
                const uint32_t c = queue[p].front(); queue[p].erase(queue[p].begin());
                serving[p] = c; serve_start[p] = t;
                events.push(Event{t + (double)tpre[(size_t)c * G + typeP[p]], 1, c});
            }
    }
    std::vector<double> done(W, -INFINITY), ratio(W);
    for (uint32_t v = 0; v < N; ++v) done[node_wf[v]] = std::max(done[node_wf[v]], out_fin[v]);
    for (uint32_t w = 0; w < W; ++w) out_ratio[w] = ratio[w] = (done[w] - arrival_s[w]) / (double)H[w];
    out_req[0] = W ? order_statistic(ratio, 0.95) : 0.0;
    out_req[1] = W ? order_statistic(ratio, 0.99) : 0.0;
    out_stats[0] = runs; out_stats[1] = decode_runs; out_stats[2] = (int)ready.size();
    return leave(HX_OK);
}
