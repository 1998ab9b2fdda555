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
        cudaFree(calls); cudaFree(assign); cudaFree(ratio); cudaFree(order); cudaFree(delta);
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
    if (!row_ptr || !node_workflow || !node_calls || !arrival_s || !out_fin || !out_ratio || !out_req || !out_stats ||
        (row_ptr[n_nodes] && !col_idx))
        return hx_fail(h, HX_ERR_INVALID_ARG, "NULL array");
    if (qmax < 1 || qmax > HX_GREEDY_MAX_CALLS) return hx_fail(h, HX_ERR_INVALID_ARG, "qmax must be 1 .. HX_GREEDY_MAX_CALLS");
    const uint32_t N = n_nodes, W = n_workflows;
    int P = 0, D = 0;
    const float* d_cap = nullptr;
    uint32_t up_nodes = 0, up_workflows = 0;
    hx_cluster_shape(h, &P, &D, &d_cap, &up_nodes, &up_workflows);
    if (up_nodes != N || up_workflows != W) return hx_fail(h, HX_ERR_INVALID_ARG, "the graph given is not the uploaded one (sizes differ)");
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
    if (cudaMalloc(&b.calls, (size_t)qmax * sizeof(hx_call)) != cudaSuccess || cudaMalloc(&b.assign, (size_t)qmax * 4) != cudaSuccess ||
        cudaMalloc(&b.ratio, (size_t)qmax * 4) != cudaSuccess || cudaMalloc(&b.order, (size_t)qmax * 4) != cudaSuccess ||
        cudaMalloc(&b.delta, (size_t)qmax * 4) != cudaSuccess)
        return hx_fail(h, HX_ERR_OOM, "replay scratch");

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
    float* qP = reinterpret_cast<float*>(chunk + qmax);
    float *qP2 = qP + P, *qD = qP2 + P, *kv_free = qD + D, *elapsed = kv_free + D, *delta = elapsed + W;
    int32_t* assign = reinterpret_cast<int32_t*>(delta + qmax);
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
            if ((rc = hx_cluster_update_loads(h, qP, qD, kv_free, stream)) != HX_OK) return leave(rc);
            if ((rc = hx_dag_update_elapsed(h, elapsed, stream)) != HX_OK) return leave(rc);
            if (cudaMemcpyAsync(b.calls, chunk, (size_t)n * sizeof(hx_call), cudaMemcpyHostToDevice, s) != cudaSuccess)
                return leave(hx_fail(h, HX_ERR_CUDA, "copying the ready calls"));
            if ((rc = hx_schedule_greedy_plan(h, b.calls, n, b.assign, b.ratio, b.order, b.delta, stream)) != HX_OK) return leave(rc);
            if (cudaMemcpyAsync(assign, b.assign, (size_t)n * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
                cudaMemcpyAsync(delta, b.delta, (size_t)n * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess)
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
