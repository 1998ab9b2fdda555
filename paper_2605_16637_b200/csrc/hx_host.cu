// Host side of libhx.so: handle, validation, cluster-state packing, forest
// levelisation and the C ABI declared in hx.h.  No arithmetic of the method
// runs here except the one-time conversion of rates to reciprocal rates.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <system_error>
#include <thread>
#include <unordered_map>

#include "hx_internal.h"

// A group of workflows levelised together: the upload is part 0, every append adds one that takes
// over the workflows it touched.  The class lists on the device are mirrored here so that a workflow
// can be taken out of its list with one 4-byte copy.
struct ForestPart {
    HxForestDev f{};
    std::vector<void*> allocs;
    std::vector<uint32_t> ids[HX_CP_CLASSES];   // workflows (numbering of this part) per class
    uint32_t* d_ids[HX_CP_CLASSES] = {};
    std::vector<uint32_t> pos;                  // workflow -> position in its class list
    std::vector<uint8_t> wf_class;              // workflow -> class
    uint32_t live = 0;                          // workflows this part still owns
    void classes(std::vector<HxCpClass>* out) const {
        out->clear();
        for (int k = 0; k < HX_CP_CLASSES; ++k) {
            if (ids[k].empty()) continue;
            HxCpClass c = hx_cpath_class_shape(k);
            c.wf_ids = d_ids[k]; c.count = (uint32_t)ids[k].size();
            out->push_back(c);
        }
    }
    // Workflow l now belongs to another part: the last entry of its list takes its place.  The device
    // lists follow at the next flush().
    std::vector<uint32_t> changed[HX_CP_CLASSES];
    void drop(uint32_t l) {
        const int k = wf_class[l];
        std::vector<uint32_t>& v = ids[k];
        const uint32_t p = pos[l], last = v.back();
        v[p] = last; pos[last] = p; v.pop_back(); pos[l] = ~0u; --live;
        changed[k].push_back(p);
    }
    cudaError_t flush(cudaStream_t s) {
        cudaError_t e = cudaSuccess;
        for (int k = 0; k < HX_CP_CLASSES && e == cudaSuccess; ++k) {
            const std::vector<uint32_t>& v = ids[k];
            if (changed[k].size() > 8) {             // one copy of the whole list beats many 4-byte copies
                if (!v.empty()) e = cudaMemcpyAsync(d_ids[k], v.data(), v.size() * sizeof(uint32_t), cudaMemcpyHostToDevice, s);
            } else {
                for (uint32_t p : changed[k])
                    if (p < v.size() && e == cudaSuccess)
                        e = cudaMemcpyAsync(d_ids[k] + p, &v[p], sizeof(uint32_t), cudaMemcpyHostToDevice, s);
            }
            changed[k].clear();
        }
        return e;
    }
};

struct hx_cluster {
    int device = 0, n_sm = 0;
    size_t max_smem = 0;
    int G = 0, P = 0, D = 0, M = 0, Ppad = 0;
    std::vector<void*> allocs;          // cluster tables, freed at destroy
    std::vector<void*> dag_allocs;      // forest, freed at the next upload
    std::vector<void*> tk_allocs;       // top-K / conflict-pass buffers
    HxTables tab{};
    HxConstTables ctab{};
    int* status = nullptr;
    // forest
    bool dag_uploaded = false, cp_ready = false;
    std::vector<ForestPart> parts;      // part 0: the upload; later ones: workflows rebuilt by hx_dag_append
    uint32_t N = 0, E = 0, W = 0;       // current size of the forest
    size_t capN = 0;                    // room in cp, tail and node_wf
    size_t capW = 0;                    // room in H and the elapsed times
    std::vector<void*> wf_allocs;       // H, elapsed: regrown when arriving workflows outgrow them
    std::vector<void*> node_allocs;     // cp, tail, node_wf: regrown when appended nodes outgrow them
    float *g_cp = nullptr, *g_tail = nullptr, *g_H = nullptr;
    uint32_t* d_node_wf = nullptr;
    float* d_elapsed = nullptr;
    HxForkJoin fj{};                    // side streams of the horizon pass, created with the first upload
    // host state for incremental refinement: node -> index inside the owning part, node -> workflow,
    // workflow -> owning part and its number there; appended nodes and edges on top of the uploaded CSR
    std::vector<uint32_t> h_inv, h_node_wf, h_wf_part, h_wf_local, h_base_perm, h_base_wns, h_local;
    std::vector<float> h_elapsed;
    std::unordered_map<uint32_t, std::vector<uint32_t>> extra_succ, extra_nodes;
    // forward pass (earliest start): the same kernels on the transposed forest, built on first use
    std::vector<uint32_t> h_row, h_col; std::vector<float> h_cost;
    std::vector<void*> fwd_allocs;
    HxForestDev fwd{};
    std::vector<HxCpClass> fwd_classes;
    std::vector<uint32_t> h_fwd_inv; std::vector<uint8_t> h_fwd_wf_class;
    bool fwd_built = false, est_ready = false;
    std::vector<void*> upd_allocs;      // scratch of hx_dag_update_costs, grown on demand
    uint32_t* d_upd_idx = nullptr; float* d_upd_cost = nullptr; uint32_t* d_upd_wf = nullptr;
    size_t upd_cap = 0, upd_wf_cap = 0;
    // decode-stage scheduler: usage step functions (snapshot and simulated state)
    std::vector<void*> dec_allocs;
    HxStepFns dec_base{}, dec_work{};
    int dec_k_bound = 0;                // upper bound on the breakpoints of any instance in the snapshot
    long long dec_k_total = 0;          // upper bound on the breakpoints of all instances together
    bool dec_ready = false;
    // top-K
    HxTopkBufs tk{};
    // staging for the host-buffer entry point
    hx_call* st_calls = nullptr; int32_t* st_assign = nullptr; float* st_cost = nullptr; int st_cap = 0;
    float* d_free_reset = nullptr;      // [D] free KV tokens every capacity pass starts from while free_reset_on
    bool free_reset_on = false;
    // copy streams and events of hx_schedule_sweep_host, created on first use
    cudaStream_t sw_in = nullptr, sw_out = nullptr;
    std::vector<cudaEvent_t> sw_ev;
    int M_base = 0;                     // models before hx_push_scaled_models (0 = nothing pushed)
    hx_options opts{HX_MODE_COMPLETION, 0, 0, 0, 1.5f};
    std::string err;
    long long launches = 0;
    // optional per-kernel-family device timing
    struct Span { int family; cudaEvent_t a, b; };
    bool timing = false;
    std::vector<Span> spans;            // recorded since the last read
    std::vector<Span> spare;            // events ready for reuse
};

namespace {

thread_local std::string g_create_err;

int fail(hx_cluster* h, int code, const std::string& msg) {
    if (h) h->err = msg; else g_create_err = msg;
    return code;
}
int fail_cuda(hx_cluster* h, cudaError_t e, const char* what) {
    return fail(h, e == cudaErrorMemoryAllocation ? HX_ERR_OOM : HX_ERR_CUDA,
                std::string(what) + ": " + cudaGetErrorString(e));
}

struct DeviceGuard {
    int prev = -1; bool changed = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) { cudaSetDevice(dev); changed = true; }
    }
    ~DeviceGuard() { if (changed) cudaSetDevice(prev); }
};

template <class T>
cudaError_t dev_alloc(std::vector<void*>& pool, T** out, size_t count) {
    void* p = nullptr;
    cudaError_t e = cudaMalloc(&p, std::max<size_t>(count, 1) * sizeof(T));
    if (e != cudaSuccess) { *out = nullptr; return e; }
    pool.push_back(p);
    *out = static_cast<T*>(p);
    return cudaSuccess;
}
template <class T>
cudaError_t dev_upload(std::vector<void*>& pool, T** out, const std::vector<T>& src) {
    cudaError_t e = dev_alloc(pool, out, src.size());
    if (e != cudaSuccess) return e;
    if (src.empty()) return cudaSuccess;
    return cudaMemcpy(*out, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice);
}
void free_pool(std::vector<void*>& pool) {
    for (void* p : pool) cudaFree(p);
    pool.clear();
}

bool good_rate(float x) { return std::isfinite(x) && x > 0.0f; }
bool good_load(float x) { return std::isfinite(x) && x >= 0.0f; }
// KV token counts are whole numbers below 2^24: sums and differences of such values are exact in
// binary32, which the capacity pass relies on when it takes its decisions on integers.
bool good_tokens(float x) { return std::isfinite(x) && x >= 0.0f && x < 16777216.0f && x == std::floor(x); }

#define HX_TRY(call, what) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return fail_cuda(h, e_, what); } while (0)

// Brackets the launches of one kernel family with events while timing is enabled.
struct SpanGuard {
    hx_cluster* h; cudaStream_t s; hx_cluster::Span sp{}; bool on = false;
    SpanGuard(hx_cluster* h_, int family, cudaStream_t s_) : h(h_), s(s_) {
        if (!h->timing) return;
        if (!h->spare.empty()) { sp = h->spare.back(); h->spare.pop_back(); }
        else if (cudaEventCreate(&sp.a) != cudaSuccess || cudaEventCreate(&sp.b) != cudaSuccess) return;
        sp.family = family;
        on = cudaEventRecord(sp.a, s) == cudaSuccess;
    }
    ~SpanGuard() {
        if (!on) return;
        cudaEventRecord(sp.b, s);
        h->spans.push_back(sp);
    }
};

int ensure_topk(hx_cluster* h, int n_calls, int K) {
    if (h->tk.cap_calls >= n_calls && h->tk.K == K) return HX_OK;
    cudaDeviceSynchronize();
    free_pool(h->tk_allocs);
    h->tk = HxTopkBufs{};
    HxTopkBufs b{};
    b.K = K;
    const size_t cap = (size_t)std::max(n_calls, 16384);
    HX_TRY(dev_alloc(h->tk_allocs, &b.pair, cap * K), "alloc top-K");
    HX_TRY(dev_alloc(h->tk_allocs, &b.cost, cap * K), "alloc top-K");
    HX_TRY(dev_alloc(h->tk_allocs, &b.tpre, cap * K), "alloc top-K");
    HX_TRY(dev_alloc(h->tk_allocs, &b.dsel, cap), "alloc top-K");
    HX_TRY(dev_alloc(h->tk_allocs, &b.prio, cap), "alloc top-K");
    HX_TRY(dev_alloc(h->tk_allocs, &b.mtok, cap), "alloc top-K");
    HX_TRY(dev_alloc(h->tk_allocs, &b.blk_lohi, (size_t)2 * HX_ORDER_MAXBLK), "alloc order");
    HX_TRY(dev_alloc(h->tk_allocs, &b.ghist, (size_t)HX_ORDER_BINS + HX_ORDER_CALLBLK), "alloc order");
    HX_TRY(dev_alloc(h->tk_allocs, &b.oslot, cap), "alloc order");
    HX_TRY(dev_alloc(h->tk_allocs, &b.okey, cap), "alloc order");
    HX_TRY(dev_alloc(h->tk_allocs, &b.obase, (size_t)HX_ORDER_BINS + 3), "alloc order");
    HX_TRY(dev_alloc(h->tk_allocs, &b.ocall, cap), "alloc order");
    HX_TRY(dev_alloc(h->tk_allocs, &b.om, cap), "alloc order");
    HX_TRY(dev_alloc(h->tk_allocs, &b.od, cap), "alloc order");
    HX_TRY(dev_alloc(h->tk_allocs, &b.n_acc, (size_t)1), "alloc outcome");
    HX_TRY(dev_alloc(h->tk_allocs, &b.acc_rk, cap), "alloc outcome");
    HX_TRY(dev_alloc(h->tk_allocs, &b.acc_p, cap), "alloc outcome");
    HX_TRY(dev_alloc(h->tk_allocs, &b.acc_t, cap), "alloc outcome");
    b.cap_calls = (int)cap;
    h->tk = b;
    return HX_OK;
}


// A forest regrouped for the horizon kernels: workflow by workflow, inside a workflow level by level
// (level = height above the sinks), successors as local indices.
struct HostForest {
    uint32_t N = 0, E = 0, W = 0;
    std::vector<uint32_t> perm, inv, wf_node_start, wf_edge_start, wf_seg_start, seg_off, irow, icol32;
    std::vector<uint16_t> icol16;
    std::vector<float> icost;
    std::vector<uint32_t> ids[HX_CP_CLASSES];
    std::vector<uint8_t> wf_class;
};

// Classes of the horizon pass by staging footprint; largest workflows first inside a class, so that the long
// ones do not start last.
void classify_workflows(HostForest* out) {
    HostForest& hf = *out;
    const uint32_t W = hf.W;
    const auto& wf_node_start = hf.wf_node_start;
    hf.wf_class.assign(W, 0);
    for (auto& v : hf.ids) v.clear();
    for (uint32_t w = 0; w < W; ++w) {
        const size_t n = wf_node_start[w + 1] - wf_node_start[w], e = hf.wf_edge_start[w + 1] - hf.wf_edge_start[w];
        const size_t nlev = hf.wf_seg_start[w + 1] - hf.wf_seg_start[w] - 1;
        const size_t need = 4 * (3 * n + 1) + 4 * (nlev + 1) + 2 * e + 16;
        const int k = hx_cpath_class_of(need, n);
        hf.ids[k].push_back(w);
        hf.wf_class[w] = (uint8_t)k;
    }
    for (auto& v : hf.ids)
        std::stable_sort(v.begin(), v.end(), [&](uint32_t a, uint32_t b) {
            return wf_node_start[a + 1] - wf_node_start[a] > wf_node_start[b + 1] - wf_node_start[b]; });
}

// The regrouping of prepare_forest for a forest whose nodes are listed workflow by workflow: every workflow is a
// contiguous range of nodes with all its edges inside (the caller checked that no edge crosses workflows), so
// the topological order, the heights and the ordering by (height, node number) are taken range by range on
// arrays that stay in the cache.  Same result as the general path; false when a workflow has a cycle.
bool regroup_workflow_by_workflow(const uint32_t* row_ptr, const uint32_t* col_idx, const float* node_costs,
                                  const uint32_t* node_workflow, uint32_t N, uint32_t E, uint32_t W, HostForest* out) {
    HostForest& hf = *out;
    auto& wns = hf.wf_node_start;
    wns.assign((size_t)W + 1, 0);
    for (uint32_t v = 0; v < N; ++v) ++wns[node_workflow[v] + 1];
    for (uint32_t w = 0; w < W; ++w) wns[w + 1] += wns[w];
    hf.perm.resize(N); hf.inv.resize(N);
    hf.irow.resize((size_t)N + 1); hf.icol32.resize(E); hf.icol16.assign((size_t)E + 2, 0);   // two spare entries: slices are copied as 32-bit words
    hf.icost.resize(N);
    hf.wf_seg_start.assign((size_t)W + 1, 0); hf.wf_edge_start.assign((size_t)W + 1, 0);
    // Workflows are independent and every output position is known from the node and edge ranges, except the
    // level boundaries, which each worker collects for its stretch of workflows and which are joined afterwards.
    const unsigned hw = std::thread::hardware_concurrency();
    const uint32_t n_workers = N < 65536 ? 1u : std::max(1u, std::min({hw ? hw : 1u, 8u, W}));
    std::vector<std::vector<uint32_t>> seg_part(n_workers), seg_count(n_workers);
    std::vector<char> failed(n_workers, 0);
    auto work = [&](uint32_t k) {
        const uint32_t w0 = (uint32_t)((uint64_t)W * k / n_workers), w1 = (uint32_t)((uint64_t)W * (k + 1) / n_workers);
        std::vector<uint32_t> indeg, topo, hgt, order, cnt;
        auto& segs = seg_part[k]; auto& nseg = seg_count[k];
        segs.reserve((size_t)(wns[w1] - wns[w0]) + (w1 - w0)); nseg.reserve(w1 - w0);
        for (uint32_t w = w0; w < w1; ++w) {
            const uint32_t ns = wns[w], n = wns[w + 1] - ns;
            if (indeg.size() < n) { indeg.resize(n); topo.resize(n); hgt.resize(n); order.resize(n); }
            std::fill(indeg.begin(), indeg.begin() + n, 0u);
            for (uint32_t e = row_ptr[ns]; e < row_ptr[ns + n]; ++e) ++indeg[col_idx[e] - ns];
            uint32_t nt = 0;
            for (uint32_t i = 0; i < n; ++i) if (indeg[i] == 0) topo[nt++] = i;
            for (uint32_t i = 0; i < nt; ++i) {
                const uint32_t v = ns + topo[i];
                for (uint32_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) if (--indeg[col_idx[e] - ns] == 0) topo[nt++] = col_idx[e] - ns;
            }
            if (nt != n) { failed[k] = 1; return; }
            uint32_t max_h = 0;
            for (uint32_t i = n; i-- > 0;) {
                const uint32_t l = topo[i], v = ns + l;
                uint32_t hh = 0;
                for (uint32_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) hh = std::max(hh, hgt[col_idx[e] - ns] + 1);
                hgt[l] = hh; max_h = std::max(max_h, hh);
            }
            cnt.assign((size_t)max_h + 2, 0);          // stable counting sort by height: node number decides among equals
            for (uint32_t i = 0; i < n; ++i) ++cnt[hgt[i] + 1];
            for (size_t i = 1; i < cnt.size(); ++i) cnt[i] += cnt[i - 1];
            for (uint32_t i = 0; i < n; ++i) order[cnt[hgt[i]]++] = i;
            const size_t seg0 = segs.size();
            segs.push_back(0);
            for (uint32_t j = 0; j < n; ++j) {
                hf.perm[ns + j] = ns + order[j]; hf.inv[ns + order[j]] = ns + j;
                if (j + 1 == n || hgt[order[j + 1]] != hgt[order[j]]) segs.push_back(j + 1);
            }
            nseg.push_back((uint32_t)(segs.size() - seg0));
            uint32_t o = row_ptr[ns];                  // the edges of a workflow keep their stretch of the edge array
            hf.wf_edge_start[w] = o;
            for (uint32_t j = 0; j < n; ++j) {
                const uint32_t v = ns + order[j];
                hf.icost[ns + j] = node_costs[v];
                hf.irow[ns + j] = o;
                for (uint32_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e, ++o) {
                    const uint32_t local = hf.inv[col_idx[e]] - ns;
                    hf.icol32[o] = local; hf.icol16[o] = (uint16_t)local;
                }
            }
        }
    };
    if (n_workers == 1) {
        work(0);
    } else {
        std::vector<std::thread> pool;
        uint32_t started = 1;                          // stretches that have a thread of their own (0 runs here)
        try {
            for (; started < n_workers; ++started) pool.emplace_back(work, started);
        } catch (const std::system_error&) {}          // no more threads to be had: this one takes the rest
        work(0);
        for (uint32_t k = started; k < n_workers; ++k) work(k);
        for (auto& th : pool) th.join();
    }
    for (char f : failed) if (f) return false;
    size_t off = 0;
    uint32_t w = 0;
    for (uint32_t k = 0; k < n_workers; ++k)
        for (uint32_t c : seg_count[k]) { hf.wf_seg_start[w++] = (uint32_t)off; off += c; }
    hf.seg_off.resize(off);
    off = 0;
    for (uint32_t k = 0; k < n_workers; ++k) { std::copy(seg_part[k].begin(), seg_part[k].end(), hf.seg_off.begin() + off); off += seg_part[k].size(); }
    const uint32_t o = E;
    hf.irow[N] = o;
    hf.wf_seg_start[W] = (uint32_t)hf.seg_off.size();
    hf.wf_edge_start[W] = o;
    return true;
}

// Host part of an upload; false when the graph has a cycle.  The arrays were validated by the caller.
bool prepare_forest(const uint32_t* row_ptr, const uint32_t* col_idx, const float* node_costs,
                    const uint32_t* node_workflow, uint32_t N, uint32_t E, uint32_t W, HostForest* out) {
    HostForest& hf = *out;
    hf.N = N; hf.E = E; hf.W = W;
    bool grouped = true;                               // nodes listed workflow by workflow (the usual case)?
    for (uint32_t v = 1; v < N && grouped; ++v) grouped = node_workflow[v] >= node_workflow[v - 1];
    if (grouped) {
        if (!regroup_workflow_by_workflow(row_ptr, col_idx, node_costs, node_workflow, N, E, W, &hf)) return false;
        classify_workflows(&hf);
        return true;
    }
    std::vector<uint32_t> indeg(N, 0);
    for (uint32_t e = 0; e < E; ++e) ++indeg[col_idx[e]];
    // topological order (cycle check), then height above the sinks
    std::vector<uint32_t> topo; topo.reserve(N);
    for (uint32_t v = 0; v < N; ++v) if (indeg[v] == 0) topo.push_back(v);
    for (size_t i = 0; i < topo.size(); ++i) {
        const uint32_t v = topo[i];
        for (uint32_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) if (--indeg[col_idx[e]] == 0) topo.push_back(col_idx[e]);
    }
    if (topo.size() != N) return false;
    std::vector<uint32_t> height(N, 0);
    uint32_t max_h = 0;
    for (size_t i = N; i-- > 0;) {
        const uint32_t v = topo[i];
        uint32_t hh = 0;
        for (uint32_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) hh = std::max(hh, height[col_idx[e]] + 1);
        height[v] = hh; max_h = std::max(max_h, hh);
    }
    // regroup: workflow by workflow, inside a workflow by height (two stable counting sorts)
    std::vector<uint32_t> by_h(N);
    auto& perm = hf.perm; auto& inv = hf.inv;
    perm.assign(N, 0); inv.assign(N, 0);
    {
        std::vector<uint32_t> cnt((size_t)max_h + 2, 0);
        for (uint32_t v = 0; v < N; ++v) ++cnt[height[v] + 1];
        for (size_t i = 1; i < cnt.size(); ++i) cnt[i] += cnt[i - 1];
        for (uint32_t v = 0; v < N; ++v) by_h[cnt[height[v]]++] = v;
    }
    auto& wf_node_start = hf.wf_node_start;
    wf_node_start.assign((size_t)W + 1, 0);
    for (uint32_t v = 0; v < N; ++v) ++wf_node_start[node_workflow[v] + 1];
    for (uint32_t w = 0; w < W; ++w) wf_node_start[w + 1] += wf_node_start[w];
    {
        std::vector<uint32_t> cur(wf_node_start.begin(), wf_node_start.end() - 1);
        for (uint32_t i = 0; i < N; ++i) { const uint32_t v = by_h[i]; perm[cur[node_workflow[v]]++] = v; }
    }
    for (uint32_t i = 0; i < N; ++i) inv[perm[i]] = i;
    auto& wf_seg_start = hf.wf_seg_start; auto& seg_off = hf.seg_off;
    wf_seg_start.assign((size_t)W + 1, 0); seg_off.clear();
    seg_off.reserve((size_t)N + W);
    for (uint32_t w = 0; w < W; ++w) {
        wf_seg_start[w] = (uint32_t)seg_off.size();
        const uint32_t ns = wf_node_start[w], ne = wf_node_start[w + 1];
        seg_off.push_back(0);
        for (uint32_t i = ns; i < ne; ++i)
            if (i + 1 == ne || height[perm[i + 1]] != height[perm[i]]) seg_off.push_back(i + 1 - ns);
    }
    wf_seg_start[W] = (uint32_t)seg_off.size();
    auto& irow = hf.irow; auto& icol32 = hf.icol32; auto& wf_edge_start = hf.wf_edge_start;
    irow.assign((size_t)N + 1, 0); icol32.assign(E, 0); wf_edge_start.assign((size_t)W + 1, 0);
    auto& icol16 = hf.icol16; auto& icost = hf.icost;
    icol16.assign((size_t)E + 2, 0);                   // two spare entries: slices are copied as 32-bit words
    icost.assign(N, 0.0f);
    for (uint32_t i = 0; i < N; ++i) {
        const uint32_t v = perm[i], ns = wf_node_start[node_workflow[v]];
        icost[i] = node_costs[v];
        uint32_t o = irow[i];
        for (uint32_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e, ++o) {
            const uint32_t local = inv[col_idx[e]] - ns;
            icol32[o] = local; icol16[o] = (uint16_t)local;
        }
        irow[i + 1] = o;
    }
    for (uint32_t w = 0; w <= W; ++w) wf_edge_start[w] = irow[wf_node_start[w]];

    classify_workflows(&hf);
    return true;
}

// Device part of an upload into part->allocs.  part->f.cp, .tail and .H are set by the caller.  With
// `node_gid` / `wf_gid` the forest is a slice of a larger one: results go to those node and workflow numbers.
int upload_forest(hx_cluster* h, const HostForest& hf, ForestPart* part,
                  const std::vector<uint32_t>* node_gid = nullptr, const std::vector<uint32_t>* wf_gid = nullptr) {
    HxForestDev* f = &part->f;
    f->n_nodes = hf.N; f->n_edges = hf.E; f->n_workflows = hf.W;
    // one allocation and one copy for the whole part: sections packed on 256-byte boundaries
    std::vector<unsigned char> blob;
    {   // room for every section at once: growing section by section would copy the blob again and again
        size_t words = hf.wf_node_start.size() + hf.wf_edge_start.size() + hf.wf_seg_start.size() + hf.seg_off.size() +
                       hf.irow.size() + hf.icol32.size() + hf.icost.size() + hf.perm.size() + (wf_gid ? wf_gid->size() : 0);
        for (int k = 0; k < HX_CP_CLASSES; ++k) words += hf.ids[k].size();
        blob.reserve(words * 4 + hf.icol16.size() * 2 + 256 * (10 + HX_CP_CLASSES));
    }
    auto put = [&](const void* src, size_t bytes) {
        const size_t off = (blob.size() + 255) & ~size_t(255);
        blob.resize(off + bytes);
        if (bytes) std::memcpy(blob.data() + off, src, bytes);
        return off;
    };
    auto put_u32 = [&](const std::vector<uint32_t>& v) { return put(v.data(), v.size() * sizeof(uint32_t)); };
    const size_t o_wns = put_u32(hf.wf_node_start), o_wes = put_u32(hf.wf_edge_start), o_wss = put_u32(hf.wf_seg_start);
    const size_t o_seg = put_u32(hf.seg_off), o_irow = put_u32(hf.irow), o_icol32 = put_u32(hf.icol32);
    const size_t o_icol16 = put(hf.icol16.data(), hf.icol16.size() * sizeof(uint16_t));
    const size_t o_icost = put(hf.icost.data(), hf.icost.size() * sizeof(float));
    size_t o_perm;
    if (node_gid) {
        std::vector<uint32_t> perm(hf.perm.size());
        for (size_t i = 0; i < perm.size(); ++i) perm[i] = (*node_gid)[hf.perm[i]];
        o_perm = put_u32(perm);
    } else {
        o_perm = put_u32(hf.perm);
    }
    const size_t o_gid = wf_gid ? put_u32(*wf_gid) : 0;
    size_t o_ids[HX_CP_CLASSES];
    for (int k = 0; k < HX_CP_CLASSES; ++k) o_ids[k] = put_u32(hf.ids[k]);
    unsigned char* base = nullptr;
    HX_TRY(dev_alloc(part->allocs, &base, blob.size()), "alloc forest");
    HX_TRY(cudaMemcpy(base, blob.data(), blob.size(), cudaMemcpyHostToDevice), "upload forest");
    auto u32 = [&](size_t off) { return reinterpret_cast<uint32_t*>(base + off); };
    f->wf_node_start = u32(o_wns); f->wf_edge_start = u32(o_wes); f->wf_seg_start = u32(o_wss);
    f->seg_off = u32(o_seg); f->irow = u32(o_irow); f->icol32 = u32(o_icol32);
    f->icol16 = reinterpret_cast<uint16_t*>(base + o_icol16);
    f->icost = reinterpret_cast<float*>(base + o_icost);
    f->perm = u32(o_perm);
    f->wf_gid = wf_gid ? u32(o_gid) : nullptr;
    part->wf_class = hf.wf_class;
    part->pos.assign(hf.W, 0);
    part->live = hf.W;
    for (int k = 0; k < HX_CP_CLASSES; ++k) {
        part->ids[k] = hf.ids[k];
        part->d_ids[k] = hf.ids[k].empty() ? nullptr : u32(o_ids[k]);
        for (size_t i = 0; i < hf.ids[k].size(); ++i) part->pos[hf.ids[k][i]] = (uint32_t)i;
    }
    return HX_OK;
}

// Successors of node v in the current graph: its row of the uploaded CSR plus appended edges.
template <class Fn>
void for_each_successor(const hx_cluster* h, uint32_t v, Fn fn) {
    if ((size_t)v + 1 < h->h_row.size())
        for (uint32_t e = h->h_row[v]; e < h->h_row[v + 1]; ++e) fn(h->h_col[e]);
    auto it = h->extra_succ.find(v);
    if (it != h->extra_succ.end()) for (uint32_t u : it->second) fn(u);
}

}  // namespace

int hx_fail(hx_cluster* h, int code, const char* msg) { return fail(h, code, msg); }
void hx_cluster_shape(const hx_cluster* h, int* P, int* D, const float** capD_dev, uint32_t* n_nodes, uint32_t* n_workflows) {
    *P = h->P; *D = h->D; *capD_dev = h->tab.capD;
    *n_nodes = h->dag_uploaded ? h->N : 0; *n_workflows = h->dag_uploaded ? h->W : 0;
}
hx_options hx_current_options(const hx_cluster* h) { return h->opts; }

int hx_update_loads_packed(hx_cluster* h, const float* packed, cudaStream_t s) {
    const size_t n = (size_t)h->P + 2 * (size_t)h->D;
    for (size_t i = 0; i < n; ++i) {
        if (!good_load(packed[i])) return fail(h, HX_ERR_INVALID_ARG, "loads must be finite and >= 0");
        if (i >= (size_t)h->P + h->D && !good_tokens(packed[i]))
            return fail(h, HX_ERR_INVALID_ARG, "free KV tokens must be whole numbers in [0, 2^24)");
    }
    DeviceGuard guard(h->device);
    HX_TRY(cudaMemcpyAsync(h->tab.qP, packed, n * sizeof(float), cudaMemcpyHostToDevice, s), "cudaMemcpyAsync(loads)");
    return HX_OK;
}

int hx_cluster_tables_host(hx_cluster* h, std::vector<int>* typeP, std::vector<int>* typeD, std::vector<float>* invLT,
                           int* Ppad, int* G, int* M, cudaStream_t s) {
    typeP->resize(h->Ppad); typeD->resize(h->D); invLT->resize((size_t)h->D * h->Ppad);
    *Ppad = h->Ppad; *G = h->G; *M = h->M;
    HX_TRY(cudaMemcpyAsync(typeP->data(), h->tab.typeP, typeP->size() * sizeof(int), cudaMemcpyDeviceToHost, s), "reading the cluster tables");
    HX_TRY(cudaMemcpyAsync(typeD->data(), h->tab.typeD, typeD->size() * sizeof(int), cudaMemcpyDeviceToHost, s), "reading the cluster tables");
    HX_TRY(cudaMemcpyAsync(invLT->data(), h->tab.invLT, invLT->size() * sizeof(float), cudaMemcpyDeviceToHost, s), "reading the cluster tables");
    HX_TRY(cudaStreamSynchronize(s), "cudaStreamSynchronize");
    return HX_OK;
}

void hx_forest_host(const hx_cluster* h, std::vector<uint32_t>* row, std::vector<uint32_t>* col, std::vector<uint32_t>* node_wf) {
    const uint32_t N = h->N;
    row->assign((size_t)N + 1, 0); col->clear(); col->reserve(h->E);
    for (uint32_t v = 0; v < N; ++v) {
        for_each_successor(h, v, [&](uint32_t u) { col->push_back(u); });
        (*row)[v + 1] = (uint32_t)col->size();
    }
    *node_wf = h->h_node_wf;
}

int hx_push_scaled_models(hx_cluster* h, float up, float down) {
    if (h->M_base) return fail(h, HX_ERR_INVALID_ARG, "scaled models are already in place");
    const int M = h->M;
    if (3 * M > HX_MAX_MODELS) return fail(h, HX_ERR_INVALID_ARG, "three times the models do not fit the model table");
    const float f[2] = {up, down};
    for (int k = 0; k < 2; ++k)
        for (int m = 0; m < M; ++m) {
            const int o = (k + 1) * M + m;
            h->ctab.phi[o] = h->ctab.phi[m] * f[k]; h->ctab.omega[o] = h->ctab.omega[m] * f[k];
            h->ctab.kappa[o] = h->ctab.kappa[m] * f[k]; h->ctab.psi[o] = h->ctab.psi[m] * f[k];
        }
    h->M_base = M; h->M = 3 * M; h->tab.M = 3 * M;
    return HX_OK;
}

void hx_pop_scaled_models(hx_cluster* h) {
    if (!h->M_base) return;
    h->M = h->M_base; h->tab.M = h->M_base; h->M_base = 0;
}

extern "C" {

int hx_cluster_create(const hx_gpu_type* gpu_types, int n_types, const hx_instance* instances,
                      int n_instances, const float* link_bw_gbps, const hx_model* models,
                      int n_models, hx_cluster** out) {
    if (!out) return fail(nullptr, HX_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (!gpu_types || !instances || !link_bw_gbps || !models)
        return fail(nullptr, HX_ERR_INVALID_ARG, "NULL table");
    if (n_types < 1 || n_types > HX_MAX_TYPES) return fail(nullptr, HX_ERR_INVALID_ARG, "n_types out of range");
    if (n_models < 1 || n_models > HX_MAX_MODELS) return fail(nullptr, HX_ERR_INVALID_ARG, "n_models out of range");
    if (n_instances < 2) return fail(nullptr, HX_ERR_INVALID_ARG, "need at least one prefill and one decode instance");
    int P = 0;
    while (P < n_instances && instances[P].role == 0) ++P;
    const int D = n_instances - P;
    for (int i = P; i < n_instances; ++i)
        if (instances[i].role != 1)
            return fail(nullptr, HX_ERR_INVALID_ARG, "instances must list all prefill (role 0) then all decode (role 1)");
    if (P < 1 || D < 1) return fail(nullptr, HX_ERR_INVALID_ARG, "empty prefill or decode pool");
    if (P > HX_MAX_PREFILL || D > HX_MAX_DECODE) return fail(nullptr, HX_ERR_INVALID_ARG, "pool larger than supported");
    for (int g = 0; g < n_types; ++g)
        if (!good_rate(gpu_types[g].peak_tflops) || !good_rate(gpu_types[g].hbm_tbps))
            return fail(nullptr, HX_ERR_INVALID_ARG, "GPU type rates must be finite and > 0");
    for (int m = 0; m < n_models; ++m)
        if (!good_load(models[m].flops_per_token) || !good_load(models[m].weight_bytes) ||
            !good_load(models[m].kv_bytes_per_token))
            return fail(nullptr, HX_ERR_INVALID_ARG, "model constants must be finite and >= 0");
    for (int i = 0; i < n_instances; ++i) {
        if (instances[i].type >= (uint32_t)n_types) return fail(nullptr, HX_ERR_INVALID_ARG, "instance type out of range");
        if (!good_load(instances[i].load_s)) return fail(nullptr, HX_ERR_INVALID_ARG, "instance load must be finite and >= 0");
        if (i >= P && (!good_tokens(instances[i].kv_cap_tokens) || !good_tokens(instances[i].kv_free_tokens)))
            return fail(nullptr, HX_ERR_INVALID_ARG, "KV capacities and free KV tokens must be whole numbers in [0, 2^24)");
    }
    for (int p = 0; p < P; ++p)
        for (int d = 0; d < D; ++d)
            if (!good_rate(link_bw_gbps[(size_t)p * n_instances + P + d]))
                return fail(nullptr, HX_ERR_INVALID_ARG, "link bandwidth must be finite and > 0");

    hx_cluster* h = new (std::nothrow) hx_cluster();
    if (!h) return fail(nullptr, HX_ERR_OOM, "out of host memory");
    auto bail = [&](int code) { g_create_err = h->err; free_pool(h->allocs); delete h; return code; };
    cudaError_t e = cudaGetDevice(&h->device);
    if (e != cudaSuccess) return bail(fail_cuda(h, e, "cudaGetDevice"));
    int v = 0;
    if ((e = cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, h->device)) != cudaSuccess)
        return bail(fail_cuda(h, e, "cudaDeviceGetAttribute"));
    h->n_sm = v;
    if ((e = cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, h->device)) != cudaSuccess)
        return bail(fail_cuda(h, e, "cudaDeviceGetAttribute"));
    h->max_smem = (size_t)v;

    h->G = n_types; h->P = P; h->D = D; h->M = n_models; h->Ppad = (P + 3) / 4 * 4;
    std::vector<float> invF(n_types), invB(n_types), qP(h->Ppad, 0.f), qD(D), capD(D), freeD(D);
    std::vector<float> phi(n_models), omega(n_models), kappa(n_models), invLT((size_t)D * h->Ppad, 0.f);
    std::vector<int> typeP(h->Ppad, 0), typeD(D);
    for (int g = 0; g < n_types; ++g) {
        invF[g] = 1.0f / (gpu_types[g].peak_tflops * 1e12f);
        invB[g] = 1.0f / (gpu_types[g].hbm_tbps * 1e12f);
    }
    for (int p = 0; p < P; ++p) { typeP[p] = (int)instances[p].type; qP[p] = instances[p].load_s; }
    for (int d = 0; d < D; ++d) {
        const hx_instance& in = instances[P + d];
        typeD[d] = (int)in.type; qD[d] = in.load_s; capD[d] = in.kv_cap_tokens; freeD[d] = in.kv_free_tokens;
    }
    for (int m = 0; m < n_models; ++m) {
        phi[m] = models[m].flops_per_token; omega[m] = models[m].weight_bytes; kappa[m] = models[m].kv_bytes_per_token;
    }
    for (int p = 0; p < P; ++p)
        for (int d = 0; d < D; ++d)
            invLT[(size_t)d * h->Ppad + p] = 1.0f / (link_bw_gbps[(size_t)p * n_instances + P + d] * 1e9f);

    // the same reciprocal link table in the tile order of the scoring kernel
    int ld_, td_, dpadT;
    hx_score_shape(D, &ld_, &td_, &dpadT);
    std::vector<float> invLTt((size_t)h->Ppad * dpadT, 0.f);
    for (int p = 0; p < P; ++p)
        for (int d = 0; d < D; ++d)
            invLTt[((size_t)(p >> 2) * dpadT + d) * 4 + (p & 3)] = invLT[(size_t)d * h->Ppad + p];
    for (int g = 0; g < n_types; ++g) { h->ctab.invF[g] = invF[g]; h->ctab.invB[g] = invB[g]; }
    for (int m = 0; m < n_models; ++m) { h->ctab.phi[m] = phi[m]; h->ctab.omega[m] = omega[m]; h->ctab.kappa[m] = kappa[m]; }

    float *d_invF, *d_invB, *d_qP, *d_qD, *d_capD, *d_freeD, *d_invLT, *d_invLTt, *d_phi, *d_omega, *d_kappa;
    int *d_typeP, *d_typeD;
    bool ok = true; cudaError_t first = cudaSuccess;
    auto up = [&](cudaError_t r) { if (r != cudaSuccess && ok) { ok = false; first = r; } };
    up(dev_upload(h->allocs, &d_invF, invF)); up(dev_upload(h->allocs, &d_invB, invB));
    {   // prefill queues, decode hints and free KV tokens side by side: a refresh of all three is one copy
        std::vector<float> loads;
        loads.insert(loads.end(), qP.begin(), qP.begin() + P);
        loads.insert(loads.end(), qD.begin(), qD.begin() + D);
        loads.insert(loads.end(), freeD.begin(), freeD.begin() + D);
        up(dev_upload(h->allocs, &d_qP, loads));
        d_qD = d_qP + P; d_freeD = d_qD + D;
    }
    up(dev_upload(h->allocs, &d_capD, capD));
    up(dev_upload(h->allocs, &d_invLT, invLT)); up(dev_upload(h->allocs, &d_invLTt, invLTt));
    up(dev_upload(h->allocs, &d_phi, phi));
    up(dev_upload(h->allocs, &d_omega, omega)); up(dev_upload(h->allocs, &d_kappa, kappa));
    up(dev_upload(h->allocs, &d_typeP, typeP)); up(dev_upload(h->allocs, &d_typeD, typeD));
    up(dev_alloc(h->allocs, &h->status, 2));                // status word, and a sink for the issue-rate kernels
    up(dev_alloc(h->allocs, &h->d_free_reset, (size_t)D));
    if (ok) up(cudaMemset(h->status, 0, 2 * sizeof(int)));
    if (!ok) return bail(fail_cuda(h, first, "uploading cluster tables"));
    h->tab = HxTables{n_types, P, D, n_models, h->Ppad, d_invF, d_invB, d_typeP, d_typeD, d_qP, d_qD,
                      d_capD, d_freeD, d_invLT, d_invLTt, dpadT, d_phi, d_omega, d_kappa};
    *out = h;
    return HX_OK;
}

int hx_cluster_update_loads(hx_cluster* h, const float* qP, const float* qD, const float* kv_free, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const float* src[3] = {qP, qD, kv_free};
    float* dst[3] = {h->tab.qP, h->tab.qD, h->tab.freeD};
    const int n[3] = {h->P, h->D, h->D};
    for (int k = 0; k < 3; ++k) {
        if (!src[k]) continue;
        for (int i = 0; i < n[k]; ++i) {
            if (!good_load(src[k][i])) return fail(h, HX_ERR_INVALID_ARG, "loads must be finite and >= 0");
            if (k == 2 && !good_tokens(src[k][i]))
                return fail(h, HX_ERR_INVALID_ARG, "free KV tokens must be whole numbers in [0, 2^24)");
        }
    }
    for (int k = 0; k < 3; ++k)
        if (src[k])
            HX_TRY(cudaMemcpyAsync(dst[k], src[k], n[k] * sizeof(float), cudaMemcpyHostToDevice, s), "cudaMemcpyAsync(loads)");
    return HX_OK;
}

int hx_set_kv_free_restore(hx_cluster* h, const float* kv_free, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (!kv_free) { h->free_reset_on = false; return HX_OK; }
    for (int d = 0; d < h->D; ++d)
        if (!good_tokens(kv_free[d])) return fail(h, HX_ERR_INVALID_ARG, "free KV tokens must be whole numbers in [0, 2^24)");
    DeviceGuard guard(h->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    HX_TRY(cudaMemcpyAsync(h->d_free_reset, kv_free, h->D * sizeof(float), cudaMemcpyHostToDevice, s), "cudaMemcpyAsync(kv_free)");
    // the table holds the same values until a pass commits: what a read-back shows without a commit
    HX_TRY(cudaMemcpyAsync(h->tab.freeD, h->d_free_reset, h->D * sizeof(float), cudaMemcpyDeviceToDevice, s), "cudaMemcpyAsync(kv_free)");
    h->free_reset_on = true;
    return HX_OK;
}

int hx_cluster_read_loads(hx_cluster* h, float* qP, float* qD, float* kv_free, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (qP) HX_TRY(cudaMemcpyAsync(qP, h->tab.qP, h->P * sizeof(float), cudaMemcpyDeviceToHost, s), "cudaMemcpyAsync(qP)");
    if (qD) HX_TRY(cudaMemcpyAsync(qD, h->tab.qD, h->D * sizeof(float), cudaMemcpyDeviceToHost, s), "cudaMemcpyAsync(qD)");
    if (kv_free) HX_TRY(cudaMemcpyAsync(kv_free, h->tab.freeD, h->D * sizeof(float), cudaMemcpyDeviceToHost, s), "cudaMemcpyAsync(kv_free)");
    HX_TRY(cudaStreamSynchronize(s), "cudaStreamSynchronize");
    return HX_OK;
}

int hx_cluster_destroy(hx_cluster* h) {
    if (!h) return HX_OK;
    DeviceGuard guard(h->device);
    cudaDeviceSynchronize();
    for (auto& p : h->parts) free_pool(p.allocs);
    free_pool(h->node_allocs); free_pool(h->wf_allocs);
    free_pool(h->allocs); free_pool(h->dag_allocs); free_pool(h->fwd_allocs); free_pool(h->tk_allocs); free_pool(h->upd_allocs); free_pool(h->dec_allocs);
    if (h->st_calls) cudaFree(h->st_calls);
    if (h->st_assign) cudaFree(h->st_assign);
    if (h->st_cost) cudaFree(h->st_cost);
    if (h->fj.ready) {
        for (int i = 0; i < HX_CP_SIDE; ++i) { cudaStreamDestroy(h->fj.aux[i]); cudaEventDestroy(h->fj.join[i]); }
        cudaEventDestroy(h->fj.fork);
    }
    for (cudaEvent_t e : h->sw_ev) cudaEventDestroy(e);
    if (h->sw_in) cudaStreamDestroy(h->sw_in);
    if (h->sw_out) cudaStreamDestroy(h->sw_out);
    for (auto* v : {&h->spans, &h->spare})
        for (auto& sp : *v) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
    delete h;
    return HX_OK;
}

int hx_dag_upload(hx_cluster* h, const uint32_t* row_ptr, const uint32_t* col_idx, const float* node_costs,
                  const uint32_t* node_workflow, const float* workflow_elapsed_s,
                  uint32_t n_nodes, uint32_t n_edges, uint32_t n_workflows) {
    if (!h) return HX_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    const uint32_t N = n_nodes, E = n_edges, W = n_workflows;
    if (!row_ptr || !node_costs || !node_workflow || !workflow_elapsed_s || (E && !col_idx))
        return fail(h, HX_ERR_INVALID_ARG, "NULL array");
    if (W == 0 || N == 0) return fail(h, HX_ERR_INVALID_ARG, "empty forest");
    if (row_ptr[0] != 0 || row_ptr[N] != E) return fail(h, HX_ERR_INVALID_ARG, "row_ptr does not span the edge array");
    for (uint32_t v = 0; v < N; ++v) {
        if (row_ptr[v + 1] < row_ptr[v]) return fail(h, HX_ERR_INVALID_ARG, "row_ptr is not monotone");
        if (node_workflow[v] >= W) return fail(h, HX_ERR_INVALID_ARG, "workflow id out of range");
        if (!good_load(node_costs[v])) return fail(h, HX_ERR_INVALID_ARG, "node costs must be finite and >= 0");
    }
    for (uint32_t w = 0; w < W; ++w)
        if (!good_load(workflow_elapsed_s[w])) return fail(h, HX_ERR_INVALID_ARG, "elapsed times must be finite and >= 0");
    for (uint32_t v = 0; v < N; ++v)
        for (uint32_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) {
            const uint32_t u = col_idx[e];
            if (u >= N) return fail(h, HX_ERR_INVALID_ARG, "edge target out of range");
            if (node_workflow[u] != node_workflow[v]) return fail(h, HX_ERR_INVALID_ARG, "edge crosses workflows");
        }
    HostForest hf;
    if (!prepare_forest(row_ptr, col_idx, node_costs, node_workflow, N, E, W, &hf))
        return fail(h, HX_ERR_CYCLE, "the graph has a cycle");

    cudaDeviceSynchronize();
    for (auto& p : h->parts) free_pool(p.allocs);
    h->parts.clear();
    free_pool(h->dag_allocs);
    free_pool(h->node_allocs);
    free_pool(h->fwd_allocs);
    h->dag_uploaded = false; h->cp_ready = false;
    h->fwd_built = false; h->est_ready = false; h->fwd_classes.clear();
    free_pool(h->wf_allocs);
    h->N = h->E = h->W = 0; h->capN = 0; h->capW = 0;
    // results and the node -> workflow map keep room for nodes appended later
    const size_t cap = (size_t)N + std::max<size_t>(N / 4, 4096);
    HX_TRY(dev_alloc(h->node_allocs, &h->g_cp, cap), "alloc cp");
    HX_TRY(dev_alloc(h->node_allocs, &h->g_tail, cap), "alloc tail");
    HX_TRY(dev_alloc(h->node_allocs, &h->d_node_wf, cap), "alloc node_workflow");
    const size_t capW = (size_t)W + std::max<size_t>(W / 4, 4096);   // room for workflows that arrive later
    HX_TRY(dev_alloc(h->wf_allocs, &h->g_H, capW), "alloc H");
    HX_TRY(cudaMemcpy(h->d_node_wf, node_workflow, (size_t)N * sizeof(uint32_t), cudaMemcpyHostToDevice), "upload node_workflow");
    std::vector<float> el(workflow_elapsed_s, workflow_elapsed_s + W);
    HX_TRY(dev_alloc(h->wf_allocs, &h->d_elapsed, capW), "alloc elapsed");
    HX_TRY(cudaMemcpy(h->d_elapsed, el.data(), (size_t)W * sizeof(float), cudaMemcpyHostToDevice), "upload elapsed");
    h->parts.emplace_back();
    ForestPart& base = h->parts.back();
    base.f.cp = h->g_cp; base.f.tail = h->g_tail; base.f.H = h->g_H;
    if (int rc = upload_forest(h, hf, &base)) return rc;
    if (!h->fj.ready) {
        bool ok = cudaEventCreateWithFlags(&h->fj.fork, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < HX_CP_SIDE && ok; ++i)
            ok = cudaStreamCreateWithFlags(&h->fj.aux[i], cudaStreamNonBlocking) == cudaSuccess &&
                 cudaEventCreateWithFlags(&h->fj.join[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return fail(h, HX_ERR_CUDA, "creating the side streams of the horizon pass");
        h->fj.ready = 1;
    }
    h->N = N; h->E = E; h->W = W; h->capN = cap; h->capW = capW;
    h->h_inv = std::move(hf.inv);
    h->h_node_wf.assign(node_workflow, node_workflow + N);
    h->h_wf_part.assign(W, 0);
    h->h_wf_local.resize(W);
    for (uint32_t w = 0; w < W; ++w) h->h_wf_local[w] = w;
    // host copy of the graph: appended nodes and the forward pass rebuild slices of it
    h->h_row.assign(row_ptr, row_ptr + N + 1);
    h->h_col.assign(col_idx, col_idx + E);
    h->h_cost.assign(node_costs, node_costs + N);
    h->h_elapsed = std::move(el);
    h->h_base_perm = std::move(hf.perm);
    h->h_base_wns = std::move(hf.wf_node_start);
    h->extra_succ.clear(); h->extra_nodes.clear();
    h->h_local.assign(N, ~0u);
    h->dag_uploaded = true;
    return HX_OK;
}

// One horizon pass over every live workflow of every part.
static int launch_all_parts(hx_cluster* h, cudaStream_t s) {
    std::vector<HxCpClass> cls;
    for (auto& p : h->parts) {
        if (!p.live) continue;
        p.classes(&cls);
        HX_TRY(hx_launch_cpath(p.f, cls.data(), (int)cls.size(), s, &h->launches, &h->fj), "horizon kernels");
    }
    return HX_OK;
}

int hx_critical_path(hx_cluster* h, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (!h->dag_uploaded) return fail(h, HX_ERR_NOT_READY, "no forest uploaded");
    DeviceGuard guard(h->device);
    {
        SpanGuard span(h, 2, static_cast<cudaStream_t>(stream));
        if (int rc = launch_all_parts(h, static_cast<cudaStream_t>(stream))) return rc;
    }
    h->cp_ready = true;
    return HX_OK;
}

int hx_dag_update_elapsed(hx_cluster* h, const float* workflow_elapsed_s, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (!h->dag_uploaded) return fail(h, HX_ERR_NOT_READY, "no forest uploaded");
    if (!workflow_elapsed_s) return fail(h, HX_ERR_INVALID_ARG, "NULL array");
    const uint32_t W = h->W;
    for (uint32_t w = 0; w < W; ++w)
        if (!good_load(workflow_elapsed_s[w])) return fail(h, HX_ERR_INVALID_ARG, "elapsed times must be finite and >= 0");
    DeviceGuard guard(h->device);
    HX_TRY(cudaMemcpyAsync(h->d_elapsed, workflow_elapsed_s, (size_t)W * sizeof(float), cudaMemcpyHostToDevice,
                           static_cast<cudaStream_t>(stream)), "cudaMemcpyAsync(elapsed)");
    h->h_elapsed.assign(workflow_elapsed_s, workflow_elapsed_s + W);
    return HX_OK;
}

int hx_dag_update_costs(hx_cluster* h, const uint32_t* node_ids, const float* new_costs, uint32_t n_updates,
                        void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (!h->dag_uploaded) return fail(h, HX_ERR_NOT_READY, "no forest uploaded");
    if (n_updates == 0) return HX_OK;
    if (!node_ids || !new_costs) return fail(h, HX_ERR_INVALID_ARG, "NULL array");
    const uint32_t N = h->N;
    for (uint32_t i = 0; i < n_updates; ++i) {
        if (node_ids[i] >= N) return fail(h, HX_ERR_INVALID_ARG, "node id out of range");
        if (!good_load(new_costs[i])) return fail(h, HX_ERR_INVALID_ARG, "node costs must be finite and >= 0");
    }
    // the last value given for a node wins; the workflows touched are recomputed, nothing else.
    // Nodes are grouped by the part that owns their workflow; the transposed forest is one more group.
    struct Group { const HxForestDev* f; std::vector<uint32_t> idx; std::vector<float> val; std::vector<uint32_t> dirty[HX_CP_CLASSES]; };
    const bool fwd = h->fwd_built;
    std::vector<Group> groups(h->parts.size() + 1);
    for (size_t q = 0; q < h->parts.size(); ++q) groups[q].f = &h->parts[q].f;
    Group& gf = groups.back();
    gf.f = &h->fwd;
    {
        std::vector<uint32_t> order(n_updates);
        for (uint32_t i = 0; i < n_updates; ++i) order[i] = i;
        std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return node_ids[a] < node_ids[b]; });
        std::vector<uint32_t> wfs;
        for (uint32_t i = 0; i < n_updates; ++i) {
            if (i + 1 < n_updates && node_ids[order[i + 1]] == node_ids[order[i]]) continue;
            const uint32_t v = node_ids[order[i]], w = h->h_node_wf[v];
            const float c = new_costs[order[i]];
            Group& g = groups[h->h_wf_part[w]];
            g.idx.push_back(h->h_inv[v]); g.val.push_back(c);
            if (fwd) { gf.idx.push_back(h->h_fwd_inv[v]); gf.val.push_back(c); }
            wfs.push_back(w);
            h->h_cost[v] = c;
        }
        std::sort(wfs.begin(), wfs.end());
        wfs.erase(std::unique(wfs.begin(), wfs.end()), wfs.end());
        for (uint32_t w : wfs) {
            const uint32_t q = h->h_wf_part[w], l = h->h_wf_local[w];
            groups[q].dirty[h->parts[q].wf_class[l]].push_back(l);
            if (fwd) gf.dirty[h->h_fwd_wf_class[w]].push_back(w);
        }
    }
    DeviceGuard guard(h->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    size_t n_idx = 0, n_wf = 0;
    for (auto& g : groups) { n_idx += g.idx.size(); for (auto& v : g.dirty) n_wf += v.size(); }
    if (n_idx > h->upd_cap || n_wf > h->upd_wf_cap) {
        cudaDeviceSynchronize();
        free_pool(h->upd_allocs);
        h->upd_cap = std::max<size_t>(n_idx, 4096); h->upd_wf_cap = std::max<size_t>(n_wf, 4096);
        HX_TRY(dev_alloc(h->upd_allocs, &h->d_upd_idx, h->upd_cap), "alloc update scratch");
        HX_TRY(dev_alloc(h->upd_allocs, &h->d_upd_cost, h->upd_cap), "alloc update scratch");
        HX_TRY(dev_alloc(h->upd_allocs, &h->d_upd_wf, h->upd_wf_cap), "alloc update scratch");
    }
    // pageable host memory: every copy below has read its vector by the time it returns
    SpanGuard span(h, 2, s);
    size_t off = 0, woff = 0;
    std::vector<HxCpClass> part;
    for (size_t q = 0; q < groups.size(); ++q) {
        Group& g = groups[q];
        if (g.idx.empty()) continue;
        const bool is_fwd = q + 1 == groups.size();
        HX_TRY(cudaMemcpyAsync(h->d_upd_idx + off, g.idx.data(), g.idx.size() * sizeof(uint32_t), cudaMemcpyHostToDevice, s), "copy updates");
        HX_TRY(cudaMemcpyAsync(h->d_upd_cost + off, g.val.data(), g.val.size() * sizeof(float), cudaMemcpyHostToDevice, s), "copy updates");
        HX_TRY(hx_launch_cost_update(*g.f, h->d_upd_idx + off, h->d_upd_cost + off, (uint32_t)g.idx.size(), s, &h->launches), "cost update kernel");
        off += g.idx.size();
        part.clear();
        for (int k = 0; k < HX_CP_CLASSES; ++k) {
            if (g.dirty[k].empty()) continue;
            HX_TRY(cudaMemcpyAsync(h->d_upd_wf + woff, g.dirty[k].data(), g.dirty[k].size() * sizeof(uint32_t),
                                   cudaMemcpyHostToDevice, s), "copy dirty workflows");
            HxCpClass c = hx_cpath_class_shape(k);
            c.wf_ids = h->d_upd_wf + woff; c.count = (uint32_t)g.dirty[k].size();
            part.push_back(c);
            woff += g.dirty[k].size();
        }
        if (is_fwd ? h->est_ready : h->cp_ready)
            HX_TRY(hx_launch_cpath(*g.f, part.data(), (int)part.size(), s, &h->launches, &h->fj), "horizon kernels");
    }
    return HX_OK;
}

int hx_get_dag_results(hx_cluster* h, const float** cp, const float** tail, const float** H) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (!h->dag_uploaded) return fail(h, HX_ERR_NOT_READY, "no forest uploaded");
    if (cp) *cp = h->g_cp;
    if (tail) *tail = h->g_tail;
    if (H) *H = h->g_H;
    return HX_OK;
}

// Builds the transposed forest (every edge reversed) for the forward pass.
static int build_forward_forest(hx_cluster* h) {
    const uint32_t N = h->N, E = h->E, W = h->W;
    std::vector<uint32_t> trow((size_t)N + 1, 0), tcol(E);
    for (uint32_t v = 0; v < N; ++v) for_each_successor(h, v, [&](uint32_t u) { ++trow[u + 1]; });
    for (uint32_t v = 0; v < N; ++v) trow[v + 1] += trow[v];
    {
        std::vector<uint32_t> cur(trow.begin(), trow.end() - 1);
        for (uint32_t v = 0; v < N; ++v) for_each_successor(h, v, [&](uint32_t u) { tcol[cur[u]++] = v; });
    }
    HostForest hf;
    if (!prepare_forest(trow.data(), tcol.data(), h->h_cost.data(), h->h_node_wf.data(), N, E, W, &hf))
        return fail(h, HX_ERR_CYCLE, "the graph has a cycle");
    cudaDeviceSynchronize();
    free_pool(h->fwd_allocs);
    h->fwd_built = false; h->est_ready = false;
    ForestPart tmp;
    HX_TRY(dev_alloc(h->fwd_allocs, &tmp.f.cp, N), "alloc earliest finish");
    HX_TRY(dev_alloc(h->fwd_allocs, &tmp.f.tail, N), "alloc earliest start");
    HX_TRY(dev_alloc(h->fwd_allocs, &tmp.f.H, W), "alloc forward horizon");
    const int rc = upload_forest(h, hf, &tmp);
    h->fwd_allocs.insert(h->fwd_allocs.end(), tmp.allocs.begin(), tmp.allocs.end());
    tmp.allocs.clear();
    if (rc) return rc;
    h->fwd = tmp.f;
    tmp.classes(&h->fwd_classes);
    h->h_fwd_inv = std::move(hf.inv);
    h->h_fwd_wf_class = std::move(hf.wf_class);
    h->fwd_built = true;
    return HX_OK;
}

int hx_earliest_start(hx_cluster* h, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (!h->dag_uploaded) return fail(h, HX_ERR_NOT_READY, "no forest uploaded");
    DeviceGuard guard(h->device);
    if (!h->fwd_built)
        if (int rc = build_forward_forest(h)) return rc;
    {
        SpanGuard span(h, 2, static_cast<cudaStream_t>(stream));
        HX_TRY(hx_launch_cpath(h->fwd, h->fwd_classes.data(), (int)h->fwd_classes.size(),
                               static_cast<cudaStream_t>(stream), &h->launches, &h->fj), "forward pass kernels");
    }
    h->est_ready = true;
    return HX_OK;
}

int hx_get_earliest_results(hx_cluster* h, const float** est, const float** eft) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (!h->fwd_built) return fail(h, HX_ERR_NOT_READY, "no forward pass yet: call hx_earliest_start");
    if (est) *est = h->fwd.tail;
    if (eft) *eft = h->fwd.cp;
    return HX_OK;
}

// Too many parts make a full pass a long chain of small launches: regroup the whole graph as one upload.
static const size_t kMaxParts = 64;
static int rebuild_as_one_part(hx_cluster* h, cudaStream_t s) {
    const uint32_t N = h->N, E = h->E, W = h->W;
    std::vector<uint32_t> row((size_t)N + 1, 0), col;
    col.reserve(E);
    for (uint32_t v = 0; v < N; ++v) {
        for_each_successor(h, v, [&](uint32_t u) { col.push_back(u); });
        row[v + 1] = (uint32_t)col.size();
    }
    const std::vector<float> cost = h->h_cost, el = h->h_elapsed;      // the upload replaces the members
    const std::vector<uint32_t> nwf = h->h_node_wf;
    const bool had_cp = h->cp_ready;
    int rc = hx_dag_upload(h, row.data(), col.data(), cost.data(), nwf.data(), el.data(), N, E, W);
    if (rc == HX_OK && had_cp) rc = hx_critical_path(h, s);
    return rc;
}

// Room for `need` nodes in cp, tail and the node -> workflow map; the arrays move when they grow.
static int reserve_nodes(hx_cluster* h, size_t need) {
    if (need <= h->capN) return HX_OK;
    const size_t cap = std::max(need, 2 * h->capN);
    std::vector<void*> fresh;
    float *cp, *tail; uint32_t* nwf;
    cudaError_t e = dev_alloc(fresh, &cp, cap);
    if (e == cudaSuccess) e = dev_alloc(fresh, &tail, cap);
    if (e == cudaSuccess) e = dev_alloc(fresh, &nwf, cap);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(cp, h->g_cp, (size_t)h->N * sizeof(float), cudaMemcpyDeviceToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(tail, h->g_tail, (size_t)h->N * sizeof(float), cudaMemcpyDeviceToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(nwf, h->d_node_wf, (size_t)h->N * sizeof(uint32_t), cudaMemcpyDeviceToDevice);
    if (e != cudaSuccess) { free_pool(fresh); return fail_cuda(h, e, "growing the node arrays"); }
    free_pool(h->node_allocs);
    h->node_allocs = fresh;
    h->g_cp = cp; h->g_tail = tail; h->d_node_wf = nwf; h->capN = cap;
    for (auto& p : h->parts) { p.f.cp = cp; p.f.tail = tail; }
    return HX_OK;
}

int hx_dag_append(hx_cluster* h, uint32_t n_new_nodes, const float* new_costs, const uint32_t* new_node_workflow,
                  uint32_t n_new_edges, const uint32_t* edge_src, const uint32_t* edge_dst, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (!h->dag_uploaded) return fail(h, HX_ERR_NOT_READY, "no forest uploaded");
    if (n_new_nodes == 0 && n_new_edges == 0) return HX_OK;
    if ((n_new_nodes && (!new_costs || !new_node_workflow)) || (n_new_edges && (!edge_src || !edge_dst)))
        return fail(h, HX_ERR_INVALID_ARG, "NULL array");
    const uint32_t N0 = h->N, W = h->W;
    if ((uint64_t)N0 + n_new_nodes > 0xFFFFFFF0ull || (uint64_t)h->E + n_new_edges > 0xFFFFFFF0ull)
        return fail(h, HX_ERR_INVALID_ARG, "more than 2^32 nodes or edges");
    const uint32_t N1 = N0 + n_new_nodes;
    auto wf_of = [&](uint32_t v) { return v < N0 ? h->h_node_wf[v] : new_node_workflow[v - N0]; };
    for (uint32_t i = 0; i < n_new_nodes; ++i) {
        if (new_node_workflow[i] >= W) return fail(h, HX_ERR_INVALID_ARG, "workflow id out of range");
        if (!good_load(new_costs[i])) return fail(h, HX_ERR_INVALID_ARG, "node costs must be finite and >= 0");
    }
    for (uint32_t e = 0; e < n_new_edges; ++e) {
        if (edge_src[e] >= N1 || edge_dst[e] >= N1) return fail(h, HX_ERR_INVALID_ARG, "edge endpoint out of range");
        if (wf_of(edge_src[e]) != wf_of(edge_dst[e])) return fail(h, HX_ERR_INVALID_ARG, "edge crosses workflows");
    }
    // workflows touched, in increasing order: they are rebuilt as one new part
    std::vector<uint32_t> touched;
    for (uint32_t i = 0; i < n_new_nodes; ++i) touched.push_back(new_node_workflow[i]);
    for (uint32_t e = 0; e < n_new_edges; ++e) touched.push_back(wf_of(edge_src[e]));
    std::sort(touched.begin(), touched.end());
    touched.erase(std::unique(touched.begin(), touched.end()), touched.end());
    // nodes of those workflows: uploaded ones, ones appended earlier, new ones
    std::vector<uint32_t> gid, lwf;                      // local node -> node number, local node -> local workflow
    // node number -> local node: a table over all nodes that is kept between calls; the entries set
    // here are cleared again on every way out
    struct LocalTable {
        std::vector<uint32_t>& t; const std::vector<uint32_t>& used;
        ~LocalTable() { for (uint32_t v : used) t[v] = ~0u; }
        uint32_t at(uint32_t v) const { return t[v]; }
    };
    h->h_local.resize(N1, ~0u);
    LocalTable local{h->h_local, gid};
    std::vector<std::vector<uint32_t>> fresh(touched.size());
    for (uint32_t i = 0; i < n_new_nodes; ++i) {
        const size_t j = std::lower_bound(touched.begin(), touched.end(), new_node_workflow[i]) - touched.begin();
        fresh[j].push_back(N0 + i);
    }
    for (size_t j = 0; j < touched.size(); ++j) {
        const uint32_t w = touched[j];
        auto add = [&](uint32_t v) { h->h_local[v] = (uint32_t)gid.size(); gid.push_back(v); lwf.push_back((uint32_t)j); };
        for (uint32_t i = h->h_base_wns[w]; i < h->h_base_wns[w + 1]; ++i) add(h->h_base_perm[i]);
        auto it = h->extra_nodes.find(w);
        if (it != h->extra_nodes.end()) for (uint32_t v : it->second) add(v);
        for (uint32_t v : fresh[j]) add(v);
    }
    const uint32_t n = (uint32_t)gid.size();
    // their edges: old ones, then the new ones
    std::vector<std::vector<uint32_t>> extra(n);
    for (uint32_t e = 0; e < n_new_edges; ++e) extra[local.at(edge_src[e])].push_back(local.at(edge_dst[e]));
    std::vector<uint32_t> row((size_t)n + 1, 0), col;
    std::vector<float> cost(n);
    for (uint32_t i = 0; i < n; ++i) {
        const uint32_t v = gid[i];
        cost[i] = v < N0 ? h->h_cost[v] : new_costs[v - N0];
        if (v < N0) for_each_successor(h, v, [&](uint32_t u) { col.push_back(local.at(u)); });
        for (uint32_t u : extra[i]) col.push_back(u);
        row[i + 1] = (uint32_t)col.size();
    }
    HostForest hf;
    if (!prepare_forest(row.data(), col.data(), cost.data(), lwf.data(), n, (uint32_t)col.size(), (uint32_t)touched.size(), &hf))
        return fail(h, HX_ERR_CYCLE, "the new edges close a cycle");     // nothing has changed so far

    DeviceGuard guard(h->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (int rc = reserve_nodes(h, N1)) return rc;
    // a free slot, else a new one
    size_t q = 1;
    while (q < h->parts.size() && (h->parts[q].live || !h->parts[q].allocs.empty())) ++q;
    if (q >= h->parts.size()) h->parts.emplace_back();
    {
        ForestPart fresh_part;
        fresh_part.f.cp = h->g_cp; fresh_part.f.tail = h->g_tail; fresh_part.f.H = h->g_H;
        int rc = upload_forest(h, hf, &fresh_part, &gid, &touched);
        if (!rc && n_new_nodes) {
            const cudaError_t e = cudaMemcpyAsync(h->d_node_wf + N0, new_node_workflow, (size_t)n_new_nodes * sizeof(uint32_t),
                                                  cudaMemcpyHostToDevice, s);
            if (e != cudaSuccess) rc = fail_cuda(h, e, "copy node_workflow");
        }
        if (rc) { free_pool(fresh_part.allocs); return rc; }
        h->parts[q] = std::move(fresh_part);
    }
    // from here on nothing fails: commit the host state
    h->h_node_wf.insert(h->h_node_wf.end(), new_node_workflow, new_node_workflow + n_new_nodes);
    h->h_cost.insert(h->h_cost.end(), new_costs, new_costs + n_new_nodes);
    h->h_inv.resize(N1);
    for (uint32_t i = 0; i < n; ++i) h->h_inv[gid[i]] = hf.inv[i];
    for (size_t j = 0; j < touched.size(); ++j) {
        const uint32_t w = touched[j];
        if (h->h_wf_part[w] != ~0u) h->parts[h->h_wf_part[w]].drop(h->h_wf_local[w]);   // ~0u: arrived without nodes so far
        h->h_wf_part[w] = (uint32_t)q; h->h_wf_local[w] = (uint32_t)j;
        if (!fresh[j].empty()) {
            auto& v = h->extra_nodes[w];
            v.insert(v.end(), fresh[j].begin(), fresh[j].end());
        }
    }
    for (uint32_t e = 0; e < n_new_edges; ++e) h->extra_succ[edge_src[e]].push_back(edge_dst[e]);
    h->N = N1; h->E += n_new_edges;
    for (auto& p : h->parts)
        if (p.live) HX_TRY(p.flush(s), "updating the class lists");
    // parts that own nothing any more give their memory back (cudaFree waits for the work in flight)
    for (size_t i = 1; i < h->parts.size(); ++i)
        if (!h->parts[i].live && !h->parts[i].allocs.empty()) { free_pool(h->parts[i].allocs); h->parts[i] = ForestPart{}; }
    h->fwd_built = false; h->est_ready = false;          // the transposed forest is rebuilt at the next forward pass
    size_t n_live = 0;
    for (auto& p : h->parts) n_live += p.live != 0;
    if (n_live > kMaxParts) return rebuild_as_one_part(h, s);
    if (h->cp_ready) {
        SpanGuard span(h, 2, s);
        std::vector<HxCpClass> cls;
        h->parts[q].classes(&cls);
        HX_TRY(hx_launch_cpath(h->parts[q].f, cls.data(), (int)cls.size(), s, &h->launches, &h->fj), "horizon kernels");
    }
    return HX_OK;
}

int hx_dag_append_workflows(hx_cluster* h, uint32_t n_new_workflows, const float* new_elapsed_s, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (!h->dag_uploaded) return fail(h, HX_ERR_NOT_READY, "no forest uploaded");
    if (n_new_workflows == 0) return HX_OK;
    if ((uint64_t)h->W + n_new_workflows > 0xFFFFFFF0ull) return fail(h, HX_ERR_INVALID_ARG, "more than 2^32 workflows");
    if (new_elapsed_s)
        for (uint32_t i = 0; i < n_new_workflows; ++i)
            if (!good_load(new_elapsed_s[i])) return fail(h, HX_ERR_INVALID_ARG, "elapsed times must be finite and >= 0");
    DeviceGuard guard(h->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint32_t W0 = h->W, W1 = W0 + n_new_workflows;
    if (W1 > h->capW) {                                   // H and the elapsed times move to larger arrays
        const size_t cap = std::max<size_t>(W1, 2 * h->capW);
        std::vector<void*> fresh;
        float *H, *el;
        cudaError_t e = dev_alloc(fresh, &H, cap);
        if (e == cudaSuccess) e = dev_alloc(fresh, &el, cap);
        if (e == cudaSuccess) e = cudaDeviceSynchronize();
        if (e == cudaSuccess) e = cudaMemcpy(H, h->g_H, (size_t)W0 * sizeof(float), cudaMemcpyDeviceToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(el, h->d_elapsed, (size_t)W0 * sizeof(float), cudaMemcpyDeviceToDevice);
        if (e != cudaSuccess) { free_pool(fresh); return fail_cuda(h, e, "growing the workflow arrays"); }
        free_pool(h->wf_allocs);
        h->wf_allocs = fresh;
        h->g_H = H; h->d_elapsed = el; h->capW = cap;
        for (auto& p : h->parts) p.f.H = H;
    }
    std::vector<float> el(n_new_workflows, 0.0f);
    if (new_elapsed_s) el.assign(new_elapsed_s, new_elapsed_s + n_new_workflows);
    HX_TRY(cudaMemsetAsync(h->g_H + W0, 0, (size_t)n_new_workflows * sizeof(float), s), "clearing the new horizons");
    HX_TRY(cudaMemcpyAsync(h->d_elapsed + W0, el.data(), el.size() * sizeof(float), cudaMemcpyHostToDevice, s), "copy elapsed");
    h->h_elapsed.insert(h->h_elapsed.end(), el.begin(), el.end());
    h->h_wf_part.resize(W1, ~0u);                          // no part owns them until their first nodes arrive
    h->h_wf_local.resize(W1, 0u);
    h->h_base_wns.resize((size_t)W1 + 1, h->h_base_wns.back());   // no node of the upload belongs to them
    h->W = W1;
    h->fwd_built = false; h->est_ready = false;            // the transposed forest is rebuilt at the next forward pass
    return HX_OK;
}

int hx_set_attention_flops(hx_cluster* h, const float* per_model) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (!per_model) return fail(h, HX_ERR_INVALID_ARG, "NULL array");
    for (int m = 0; m < h->M; ++m)
        if (!good_load(per_model[m])) return fail(h, HX_ERR_INVALID_ARG, "attention FLOPs must be finite and >= 0");
    for (int m = 0; m < h->M; ++m) h->ctab.psi[m] = per_model[m];     // travels with the kernel parameters
    return HX_OK;
}

int hx_set_options(hx_cluster* h, const hx_options* o) {
    if (!h || !o) return HX_ERR_INVALID_ARG;
    if (o->score_mode < HX_MODE_COMPLETION || o->score_mode > HX_MODE_RATIO) return fail(h, HX_ERR_INVALID_ARG, "unknown score mode");
    if (o->topk < 0 || o->topk > HX_MAX_TOPK) return fail(h, HX_ERR_INVALID_ARG, "topk out of range");
    if (o->flags & ~(HX_FLAG_NO_DAG | HX_FLAG_NO_TAIL | HX_FLAG_UNLOADED | HX_FLAG_ONE_PASS)) return fail(h, HX_ERR_INVALID_ARG, "unknown flag");
    if (!std::isfinite(o->alpha) || o->alpha <= 0.f) return fail(h, HX_ERR_INVALID_ARG, "alpha must be finite and > 0");
    h->opts = *o;
    return HX_OK;
}

int hx_schedule_batch(hx_cluster* h, const hx_call* calls, int n_calls, int32_t* out_assign,
                      float* out_cost, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (n_calls < 0) return fail(h, HX_ERR_INVALID_ARG, "negative n_calls");
    if (n_calls == 0) return HX_OK;
    if (!calls || !out_assign || !out_cost) return fail(h, HX_ERR_INVALID_ARG, "NULL buffer");
    if (reinterpret_cast<uintptr_t>(calls) % 16) return fail(h, HX_ERR_INVALID_ARG, "calls must be 16-byte aligned");
    const hx_options& o = h->opts;
    if (!(o.flags & HX_FLAG_NO_DAG) && !(h->dag_uploaded && h->cp_ready))
        return fail(h, HX_ERR_NOT_READY, "horizons not computed: call hx_dag_upload and hx_critical_path, or set HX_FLAG_NO_DAG");
    if (o.topk > 0 && n_calls > HX_MAX_COMMIT_CALLS)
        return fail(h, HX_ERR_INVALID_ARG, "batch too large for the capacity-conflict pass; split it into chunks");
    DeviceGuard guard(h->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (o.topk > 0) {
        int rc = ensure_topk(h, n_calls, o.topk);
        if (rc != HX_OK) return rc;
    }
    HxDagView dag{};
    if (!(o.flags & HX_FLAG_NO_DAG))
        dag = HxDagView{h->d_node_wf, h->g_tail, h->g_H, h->d_elapsed, h->N, h->W};
    HxTopkBufs tk = h->tk;
    tk.K = o.topk;
    ScoreLaunch sl{calls, n_calls, out_assign, out_cost, o.score_mode, o.flags, o.topk, o.alpha};
    {
        SpanGuard span(h, 0, s);
        HX_TRY(hx_launch_score(h->tab, h->ctab, dag, tk, sl, h->n_sm, h->max_smem, h->status, s, &h->launches), "scoring kernel");
    }
    if (o.topk > 0) {
        SpanGuard span(h, 1, s);
        HX_TRY(hx_launch_conflict(h->tab, tk, n_calls, o.commit, out_assign, h->status, s, &h->launches,
                                  h->free_reset_on ? h->d_free_reset : nullptr), "conflict pass");
    }
    return HX_OK;
}

// Device staging of the host-buffer entry points: room for n_calls records and results.
static int reserve_staging(hx_cluster* h, int n_calls) {
    if (h->st_cap >= n_calls) return HX_OK;
    cudaDeviceSynchronize();
    if (h->st_calls) cudaFree(h->st_calls);
    if (h->st_assign) cudaFree(h->st_assign);
    if (h->st_cost) cudaFree(h->st_cost);
    h->st_calls = nullptr; h->st_assign = nullptr; h->st_cost = nullptr; h->st_cap = 0;
    const size_t cap = (size_t)std::max(n_calls, 16384);
    HX_TRY(cudaMalloc(&h->st_calls, cap * sizeof(hx_call)), "alloc staging");
    HX_TRY(cudaMalloc(&h->st_assign, cap * sizeof(int32_t)), "alloc staging");
    HX_TRY(cudaMalloc(&h->st_cost, cap * sizeof(float)), "alloc staging");
    h->st_cap = (int)cap;
    return HX_OK;
}

static int schedule_batch_host_impl(hx_cluster* h, const hx_call* calls, int n_calls, int32_t* out_assign,
                                    float* out_cost, void* stream, bool sync) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (n_calls < 0) return fail(h, HX_ERR_INVALID_ARG, "negative n_calls");
    if (n_calls == 0) return HX_OK;
    if (!calls || !out_assign || !out_cost) return fail(h, HX_ERR_INVALID_ARG, "NULL buffer");
    DeviceGuard guard(h->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (int rc = reserve_staging(h, n_calls)) return rc;
    HX_TRY(cudaMemcpyAsync(h->st_calls, calls, (size_t)n_calls * sizeof(hx_call), cudaMemcpyHostToDevice, s), "copy calls");
    int rc = hx_schedule_batch(h, h->st_calls, n_calls, h->st_assign, h->st_cost, stream);
    if (rc != HX_OK) return rc;
    HX_TRY(cudaMemcpyAsync(out_assign, h->st_assign, (size_t)n_calls * sizeof(int32_t), cudaMemcpyDeviceToHost, s), "copy assign");
    HX_TRY(cudaMemcpyAsync(out_cost, h->st_cost, (size_t)n_calls * sizeof(float), cudaMemcpyDeviceToHost, s), "copy cost");
    if (sync) HX_TRY(cudaStreamSynchronize(s), "cudaStreamSynchronize");
    return HX_OK;
}

int hx_schedule_batch_host(hx_cluster* h, const hx_call* calls, int n_calls, int32_t* out_assign,
                           float* out_cost, void* stream) {
    return schedule_batch_host_impl(h, calls, n_calls, out_assign, out_cost, stream, true);
}

int hx_schedule_batch_host_async(hx_cluster* h, const hx_call* calls, int n_calls, int32_t* out_assign,
                                 float* out_cost, void* stream) {
    return schedule_batch_host_impl(h, calls, n_calls, out_assign, out_cost, stream, false);
}

int hx_schedule_sweep_host(hx_cluster* h, const hx_call* calls, int n_calls, int chunk_calls,
                           const float* kv_free_reset, int32_t* out_assign, float* out_cost, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (n_calls < 0 || chunk_calls < 1) return fail(h, HX_ERR_INVALID_ARG, "n_calls must be >= 0 and chunk_calls >= 1");
    if (n_calls == 0) return HX_OK;
    if (!calls || !out_assign || !out_cost) return fail(h, HX_ERR_INVALID_ARG, "NULL buffer");
    if (h->opts.topk > 0 && chunk_calls > HX_MAX_COMMIT_CALLS)
        return fail(h, HX_ERR_INVALID_ARG, "chunk too large for the capacity-conflict pass");
    if (kv_free_reset)
        for (int d = 0; d < h->D; ++d)
            if (!good_tokens(kv_free_reset[d]))
                return fail(h, HX_ERR_INVALID_ARG, "free KV tokens must be whole numbers in [0, 2^24)");
    DeviceGuard guard(h->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (int rc = reserve_staging(h, n_calls)) return rc;
    const int n_chunks = (n_calls + chunk_calls - 1) / chunk_calls;
    if (!h->sw_in) {
        HX_TRY(cudaStreamCreateWithFlags(&h->sw_in, cudaStreamNonBlocking), "creating the copy streams");
        HX_TRY(cudaStreamCreateWithFlags(&h->sw_out, cudaStreamNonBlocking), "creating the copy streams");
    }
    while (h->sw_ev.size() < 2 * (size_t)n_chunks + 2) {
        cudaEvent_t e;
        HX_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming), "creating events");
        h->sw_ev.push_back(e);
    }
    cudaEvent_t ev_start = h->sw_ev[0], ev_done = h->sw_ev[1];
    // whatever is already on the caller's stream comes first
    HX_TRY(cudaEventRecord(ev_start, s), "event");
    HX_TRY(cudaStreamWaitEvent(h->sw_in, ev_start, 0), "event");
    HX_TRY(cudaStreamWaitEvent(h->sw_out, ev_start, 0), "event");
    // the free KV tokens every chunk starts from: one copy, then every capacity pass reads them itself (a copy ahead
    // of every chunk would sit between the pass of one chunk and the scoring kernel of the next)
    if (kv_free_reset)
        if (int rc = hx_set_kv_free_restore(h, kv_free_reset, stream)) return rc;
    struct RestoreOff {                                  // the values given here hold for this sweep only
        hx_cluster* h; bool mine;
        ~RestoreOff() { if (mine) h->free_reset_on = false; }
    } restore_off{h, kv_free_reset != nullptr};
    // every chunk's records go up on their own stream, ahead of the kernels that need them
    for (int c = 0; c < n_chunks; ++c) {
        const size_t o = (size_t)c * chunk_calls, n = std::min<size_t>(chunk_calls, (size_t)n_calls - o);
        HX_TRY(cudaMemcpyAsync(h->st_calls + o, calls + o, n * sizeof(hx_call), cudaMemcpyHostToDevice, h->sw_in), "copy calls");
        HX_TRY(cudaEventRecord(h->sw_ev[2 + c], h->sw_in), "event");
    }
    for (int c = 0; c < n_chunks; ++c) {
        const size_t o = (size_t)c * chunk_calls, n = std::min<size_t>(chunk_calls, (size_t)n_calls - o);
        HX_TRY(cudaStreamWaitEvent(s, h->sw_ev[2 + c], 0), "event");
        const int rc = hx_schedule_batch(h, h->st_calls + o, (int)n, h->st_assign + o, h->st_cost + o, stream);
        if (rc != HX_OK) {                               // leave no stream waiting on work that will never come
            cudaEventRecord(ev_done, h->sw_out); cudaStreamWaitEvent(s, ev_done, 0);
            return rc;
        }
        // results go down on their own stream as soon as the chunk's kernels are through
        cudaEvent_t ev_k = h->sw_ev[2 + n_chunks + c];
        HX_TRY(cudaEventRecord(ev_k, s), "event");
        HX_TRY(cudaStreamWaitEvent(h->sw_out, ev_k, 0), "event");
        HX_TRY(cudaMemcpyAsync(out_assign + o, h->st_assign + o, n * sizeof(int32_t), cudaMemcpyDeviceToHost, h->sw_out), "copy assign");
        HX_TRY(cudaMemcpyAsync(out_cost + o, h->st_cost + o, n * sizeof(float), cudaMemcpyDeviceToHost, h->sw_out), "copy cost");
    }
    HX_TRY(cudaEventRecord(ev_done, h->sw_out), "event");
    HX_TRY(cudaStreamWaitEvent(s, ev_done, 0), "event");         // the caller's stream ends after the last copy
    return HX_OK;
}


// ---------------------------------------------------------------------------
// hx_schedule_batch_static: the same batch operation with every intermediate
// buffer in a fixed device array that is part of the library image.
// ---------------------------------------------------------------------------
namespace {

constexpr size_t kStaticAlign = 256;
constexpr size_t static_round(size_t b) { return (b + kStaticAlign - 1) / kStaticAlign * kStaticAlign; }
constexpr size_t kSC = HX_STATIC_MAX_CALLS, kSK = HX_STATIC_MAX_TOPK;
constexpr size_t kStaticBytes =
    3 * static_round(kSC * kSK * 4) +     // pair, cost, tpre
    2 * static_round(kSC * 16) +          // dsel, od
    4 * static_round(kSC * 4) +           // prio, mtok, ocall, om
    static_round(kSC * 8) +               // okey
    static_round((HX_ORDER_BINS + 3) * 4) +   // obase
    static_round(2 * HX_ORDER_MAXBLK * 4) +   // blk_lohi
    static_round((HX_ORDER_BINS + HX_ORDER_CALLBLK) * 4) +  // ghist
    static_round(kSC * 4) +               // oslot
    static_round(4) +                     // n_acc
    3 * static_round(kSC * 4);            // acc_rk, acc_p, acc_t

// Held by every device that loads the library, until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

std::mutex g_static_mu;
unsigned char* g_static_base[64] = {};    // device address of the array, per device ordinal

}  // namespace

int hx_schedule_batch_static(hx_cluster* h, const hx_call* calls, int n_calls, int32_t* out_assign,
                             float* out_cost, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (n_calls < 0) return fail(h, HX_ERR_INVALID_ARG, "negative n_calls");
    if (n_calls == 0) return HX_OK;
    if (!calls || !out_assign || !out_cost) return fail(h, HX_ERR_INVALID_ARG, "NULL buffer");
    if (reinterpret_cast<uintptr_t>(calls) % 16) return fail(h, HX_ERR_INVALID_ARG, "calls must be 16-byte aligned");
    const hx_options& o = h->opts;
    if (!(o.flags & HX_FLAG_NO_DAG) && !(h->dag_uploaded && h->cp_ready))
        return fail(h, HX_ERR_NOT_READY, "horizons not computed: call hx_dag_upload and hx_critical_path, or set HX_FLAG_NO_DAG");
    if (o.topk > 0 && n_calls > HX_STATIC_MAX_CALLS)
        return fail(h, HX_ERR_INVALID_ARG, "hx_schedule_batch_static: more than HX_STATIC_MAX_CALLS (16384) calls in one batch; "
                                           "split the batch or use hx_schedule_batch");
    if (o.topk > HX_STATIC_MAX_TOPK)
        return fail(h, HX_ERR_INVALID_ARG, "hx_schedule_batch_static: topk above HX_STATIC_MAX_TOPK (4); use hx_schedule_batch");
    if (h->device < 0 || h->device >= 64) return fail(h, HX_ERR_INVALID_ARG, "device ordinal out of range");
    DeviceGuard guard(h->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned char* base = nullptr;
    {
        // the array's name is only a host-side handle: ask the runtime for its address on this device, once
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (!g_static_base[h->device]) {
            void* p = nullptr;
            HX_TRY(cudaGetSymbolAddress(&p, g_static_scratch), "cudaGetSymbolAddress(static scratch)");
            g_static_base[h->device] = static_cast<unsigned char*>(p);
        }
        base = g_static_base[h->device];
    }
    HxTopkBufs b{};
    b.K = o.topk;
    b.cap_calls = HX_STATIC_MAX_CALLS;
    size_t off = 0;
    auto carve = [&](size_t bytes) { unsigned char* p = base + off; off += static_round(bytes); return p; };
    b.pair = reinterpret_cast<int32_t*>(carve(kSC * kSK * 4));
    b.cost = reinterpret_cast<float*>(carve(kSC * kSK * 4));
    b.tpre = reinterpret_cast<float*>(carve(kSC * kSK * 4));
    b.dsel = reinterpret_cast<uint4*>(carve(kSC * 16));
    b.od = reinterpret_cast<uint4*>(carve(kSC * 16));
    b.prio = reinterpret_cast<float*>(carve(kSC * 4));
    b.mtok = reinterpret_cast<float*>(carve(kSC * 4));
    b.ocall = reinterpret_cast<unsigned int*>(carve(kSC * 4));
    b.om = reinterpret_cast<int*>(carve(kSC * 4));
    b.okey = reinterpret_cast<unsigned long long*>(carve(kSC * 8));
    b.obase = reinterpret_cast<unsigned int*>(carve((HX_ORDER_BINS + 3) * 4));
    b.blk_lohi = reinterpret_cast<unsigned int*>(carve(2 * HX_ORDER_MAXBLK * 4));
    b.ghist = reinterpret_cast<unsigned int*>(carve((HX_ORDER_BINS + HX_ORDER_CALLBLK) * 4));
    b.oslot = reinterpret_cast<unsigned int*>(carve(kSC * 4));
    b.n_acc = reinterpret_cast<unsigned int*>(carve(4));
    b.acc_rk = reinterpret_cast<unsigned int*>(carve(kSC * 4));
    b.acc_p = reinterpret_cast<int*>(carve(kSC * 4));
    b.acc_t = reinterpret_cast<float*>(carve(kSC * 4));
    if (off != kStaticBytes) return fail(h, HX_ERR_INVALID_ARG, "internal: static scratch layout mismatch");
    HxDagView dag{};
    if (!(o.flags & HX_FLAG_NO_DAG))
        dag = HxDagView{h->d_node_wf, h->g_tail, h->g_H, h->d_elapsed, h->N, h->W};
    ScoreLaunch sl{calls, n_calls, out_assign, out_cost, o.score_mode, o.flags, o.topk, o.alpha};
    {
        SpanGuard span(h, 0, s);
        HX_TRY(hx_launch_score(h->tab, h->ctab, dag, b, sl, h->n_sm, h->max_smem, h->status, s, &h->launches), "scoring kernel");
    }
    if (o.topk > 0) {
        SpanGuard span(h, 1, s);
        HX_TRY(hx_launch_conflict(h->tab, b, n_calls, o.commit, out_assign, h->status, s, &h->launches,
                                  h->free_reset_on ? h->d_free_reset : nullptr), "conflict pass");
    }
    return HX_OK;
}

int hx_schedule_greedy(hx_cluster* h, const hx_call* calls, int n_calls, int32_t* out_assign,
                       float* out_ratio, int32_t* out_order, void* stream) {
    return hx_schedule_greedy_plan(h, calls, n_calls, out_assign, out_ratio, out_order, nullptr, stream);
}

int hx_schedule_greedy_plan(hx_cluster* h, const hx_call* calls, int n_calls, int32_t* out_assign,
                            float* out_ratio, int32_t* out_order, float* out_delta, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (n_calls < 0) return fail(h, HX_ERR_INVALID_ARG, "negative n_calls");
    if (n_calls == 0) return HX_OK;
    if (!calls || !out_assign || !out_ratio || !out_order) return fail(h, HX_ERR_INVALID_ARG, "NULL buffer");
    if (reinterpret_cast<uintptr_t>(calls) % 16) return fail(h, HX_ERR_INVALID_ARG, "calls must be 16-byte aligned");
    const hx_options& o = h->opts;
    if (o.flags & HX_FLAG_UNLOADED) return fail(h, HX_ERR_INVALID_ARG, "hx_schedule_greedy plans against the loaded cluster: clear HX_FLAG_UNLOADED");
    if (!(o.flags & HX_FLAG_NO_DAG) && !(h->dag_uploaded && h->cp_ready))
        return fail(h, HX_ERR_NOT_READY, "horizons not computed: call hx_dag_upload and hx_critical_path, or set HX_FLAG_NO_DAG");
    if (n_calls > HX_GREEDY_MAX_CALLS)
        return fail(h, HX_ERR_INVALID_ARG, "hx_schedule_greedy: more than HX_GREEDY_MAX_CALLS (4096) calls; use hx_schedule_batch with topk > 0 for large queues");
    if (hx_greedy_smem_bytes(h->tab, n_calls) > h->max_smem)
        return fail(h, HX_ERR_INVALID_ARG, "hx_schedule_greedy: cluster tables and queue do not fit the shared memory of one SM");
    DeviceGuard guard(h->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    HxDagView dag{};
    if (!(o.flags & HX_FLAG_NO_DAG))
        dag = HxDagView{h->d_node_wf, h->g_tail, h->g_H, h->d_elapsed, h->N, h->W};
    {
        SpanGuard span(h, 0, s);
        HX_TRY(hx_launch_greedy(h->tab, h->ctab, dag, calls, n_calls, o.flags, o.commit, out_assign, out_ratio,
                                out_order, out_delta, h->status, s, &h->launches), "greedy planner kernel");
    }
    return HX_OK;
}

namespace {

// (Re)allocates the step-function arrays with room for `cap` breakpoints per instance; the
// snapshot is carried over when keep is set.
int decode_reserve(hx_cluster* h, int cap, bool keep) {
    if (h->dec_base.cap >= cap) return HX_OK;
    const int D = h->D;
    cudaDeviceSynchronize();
    std::vector<void*> fresh;
    HxStepFns b{}, w{};
    b.cap = w.cap = cap;
    HX_TRY(dev_alloc(fresh, &b.t, (size_t)D * cap), "alloc decode intervals");
    HX_TRY(dev_alloc(fresh, &b.u, (size_t)D * cap), "alloc decode intervals");
    HX_TRY(dev_alloc(fresh, &b.K, (size_t)D), "alloc decode intervals");
    HX_TRY(dev_alloc(fresh, &w.t, (size_t)hx_decode_replicas() * D * cap), "alloc decode intervals");
    HX_TRY(dev_alloc(fresh, &w.u, (size_t)hx_decode_replicas() * D * cap), "alloc decode intervals");
    w.K = b.K;
    if (keep && h->dec_base.cap > 0) {
        const size_t ow = (size_t)h->dec_base.cap * sizeof(float);
        HX_TRY(cudaMemcpy2D(b.t, (size_t)cap * sizeof(float), h->dec_base.t, ow, ow, D, cudaMemcpyDeviceToDevice), "copy decode intervals");
        HX_TRY(cudaMemcpy2D(b.u, (size_t)cap * sizeof(float), h->dec_base.u, ow, ow, D, cudaMemcpyDeviceToDevice), "copy decode intervals");
        HX_TRY(cudaMemcpy(b.K, h->dec_base.K, (size_t)D * sizeof(int), cudaMemcpyDeviceToDevice), "copy decode intervals");
    }
    free_pool(h->dec_allocs);
    h->dec_allocs = fresh;
    h->dec_base = b; h->dec_work = w;
    return HX_OK;
}

}  // namespace

int hx_decode_set_running(hx_cluster* h, const uint32_t* inst_ptr, const hx_kv_interval* running, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (!inst_ptr) return fail(h, HX_ERR_INVALID_ARG, "NULL array");
    const int D = h->D;
    if (inst_ptr[0] != 0) return fail(h, HX_ERR_INVALID_ARG, "inst_ptr must start at 0");
    for (int d = 0; d < D; ++d)
        if (inst_ptr[d + 1] < inst_ptr[d]) return fail(h, HX_ERR_INVALID_ARG, "inst_ptr is not monotone");
    const uint32_t total = inst_ptr[D];
    if (total && !running) return fail(h, HX_ERR_INVALID_ARG, "NULL array");
    int maxK = 1;
    for (uint32_t i = 0; i < total; ++i) {
        if (!(std::isfinite(running[i].end_s) && running[i].end_s > 0.0f))
            return fail(h, HX_ERR_INVALID_ARG, "a running call must end at a finite time > 0");
        if (!good_load(running[i].tokens) || running[i].tokens >= 16777216.0f || running[i].tokens != std::floor(running[i].tokens))
            return fail(h, HX_ERR_INVALID_ARG, "tokens of a running call must be a whole number below 2^24");
    }
    for (int d = 0; d < D; ++d) maxK = std::max<int>(maxK, (int)(inst_ptr[d + 1] - inst_ptr[d]) + 1);
    DeviceGuard guard(h->device);
    int rc = decode_reserve(h, std::max(maxK + 2, 64), false);
    if (rc != HX_OK) return rc;
    // step function of every instance: usage until the next call ends (token counts are whole
    // numbers, so the sums are exact in any order)
    const int cap = h->dec_base.cap;
    std::vector<float> t((size_t)D * cap, 0.f), u((size_t)D * cap, 0.f);
    std::vector<int> K(D, 1);
    for (int d = 0; d < D; ++d) {
        std::vector<std::pair<float, float>> ev;
        for (uint32_t i = inst_ptr[d]; i < inst_ptr[d + 1]; ++i) ev.emplace_back(running[i].end_s, running[i].tokens);
        std::sort(ev.begin(), ev.end());
        float held = 0.f;
        for (auto& e : ev) held += e.second;
        if (held >= 16777216.0f) return fail(h, HX_ERR_INVALID_ARG, "tokens in use on an instance must stay below 2^24");
        float* td = &t[(size_t)d * cap]; float* ud = &u[(size_t)d * cap];
        int k = 0;
        td[0] = 0.f; ud[0] = held;
        for (size_t i = 0; i < ev.size(); ++i) {
            held -= ev[i].second;
            if (i + 1 < ev.size() && ev[i + 1].first == ev[i].first) continue;     // calls ending together
            ++k; td[k] = ev[i].first; ud[k] = held;
        }
        K[d] = k + 1;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    HX_TRY(cudaMemcpyAsync(h->dec_base.t, t.data(), t.size() * sizeof(float), cudaMemcpyHostToDevice, s), "copy decode intervals");
    HX_TRY(cudaMemcpyAsync(h->dec_base.u, u.data(), u.size() * sizeof(float), cudaMemcpyHostToDevice, s), "copy decode intervals");
    HX_TRY(cudaMemcpyAsync(h->dec_base.K, K.data(), K.size() * sizeof(int), cudaMemcpyHostToDevice, s), "copy decode intervals");
    h->dec_k_bound = maxK;
    h->dec_k_total = 0;
    for (int d = 0; d < D; ++d) h->dec_k_total += K[d];
    h->dec_ready = true;
    return HX_OK;
}

int hx_schedule_decode(hx_cluster* h, const hx_call* calls, const int32_t* lock, const float* ready_s, int n_calls,
                       int32_t* out_inst, float* out_start, float* out_ratio, int32_t* out_order, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (n_calls < 0) return fail(h, HX_ERR_INVALID_ARG, "negative n_calls");
    if (n_calls == 0) return HX_OK;
    if (!calls || !out_inst || !out_start || !out_ratio || !out_order) return fail(h, HX_ERR_INVALID_ARG, "NULL buffer");
    if (reinterpret_cast<uintptr_t>(calls) % 16) return fail(h, HX_ERR_INVALID_ARG, "calls must be 16-byte aligned");
    if (!h->dec_ready) return fail(h, HX_ERR_NOT_READY, "no decode intervals: call hx_decode_set_running first (it may list no running call)");
    const hx_options& o = h->opts;
    if (!(o.flags & HX_FLAG_NO_DAG) && !(h->dag_uploaded && h->cp_ready))
        return fail(h, HX_ERR_NOT_READY, "horizons not computed: call hx_dag_upload and hx_critical_path, or set HX_FLAG_NO_DAG");
    if (n_calls > HX_DECODE_MAX_CALLS)
        return fail(h, HX_ERR_INVALID_ARG, "hx_schedule_decode: more than HX_DECODE_MAX_CALLS (2048) calls in the decode queue");
    if (hx_decode_smem_bytes(h->tab, n_calls) > h->max_smem)
        return fail(h, HX_ERR_INVALID_ARG, "hx_schedule_decode: queue does not fit the shared memory of one SM");
    DeviceGuard guard(h->device);
    int rc = decode_reserve(h, h->dec_k_bound + 2 * n_calls + 2, true);
    if (rc != HX_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    HxDagView dag{};
    if (!(o.flags & HX_FLAG_NO_DAG))
        dag = HxDagView{h->d_node_wf, h->g_tail, h->g_H, h->d_elapsed, h->N, h->W};
    {
        SpanGuard span(h, 0, s);
        HX_TRY(hx_launch_decode(h->tab, h->ctab, dag, h->dec_base, h->dec_work,
                                (int)std::min<long long>(h->dec_k_total, 1 << 30), calls, lock, ready_s, n_calls, o.flags,
                                o.commit, out_inst, out_start, out_ratio, out_order, h->status, s, &h->launches),
               "decode scheduler kernel");
    }
    if (o.commit) { h->dec_k_bound += 2 * n_calls; h->dec_k_total += 2LL * n_calls; }
    return HX_OK;
}

int hx_estimate_calls(hx_cluster* h, const hx_call* calls, int n_calls, float* out_tpre, float* out_tdec,
                      float* out_kv_bytes, float* out_tokens, void* stream) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (n_calls < 0) return fail(h, HX_ERR_INVALID_ARG, "negative n_calls");
    if (n_calls == 0) return HX_OK;
    if (!calls || !out_tpre || !out_tdec || !out_kv_bytes || !out_tokens) return fail(h, HX_ERR_INVALID_ARG, "NULL buffer");
    if (reinterpret_cast<uintptr_t>(calls) % 16) return fail(h, HX_ERR_INVALID_ARG, "calls must be 16-byte aligned");
    DeviceGuard guard(h->device);
    HX_TRY(hx_launch_estimate(h->ctab, h->G, h->M, calls, n_calls, out_tpre, out_tdec, out_kv_bytes, out_tokens, h->status,
                              static_cast<cudaStream_t>(stream), &h->launches), "estimate kernel");
    return HX_OK;
}

int hx_get_topk(hx_cluster* h, const int32_t** pairs, const float** costs, const float** prio) {
    if (!h) return HX_ERR_INVALID_ARG;
    if (h->tk.cap_calls == 0) return fail(h, HX_ERR_NOT_READY, "no batch has been scored with topk > 0");
    if (pairs) *pairs = h->tk.pair;
    if (costs) *costs = h->tk.cost;
    if (prio) *prio = h->tk.prio;
    return HX_OK;
}

int hx_get_status(hx_cluster* h, int* status, void* stream) {
    if (!h || !status) return HX_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    HX_TRY(cudaMemcpyAsync(status, h->status, sizeof(int), cudaMemcpyDeviceToHost, s), "read status");
    HX_TRY(cudaMemsetAsync(h->status, 0, sizeof(int), s), "clear status");      // read and clear: the next read covers later work only
    HX_TRY(cudaStreamSynchronize(s), "cudaStreamSynchronize");
    return HX_OK;
}

int hx_measure_fp32_rates(hx_cluster* h, double* lane_instr_per_s, float* ms, void* stream) {
    if (!h || !lane_instr_per_s || !ms) return HX_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    // the status word doubles as the never-written sink of the loops (they store only if a sum hits one exact value)
    HX_TRY(hx_run_micro(h->n_sm, reinterpret_cast<float*>(h->status + 1), static_cast<cudaStream_t>(stream), lane_instr_per_s, ms,
                        &h->launches), "issue-rate kernels");
    return HX_OK;
}

int hx_enable_kernel_timing(hx_cluster* h, int enable) {
    if (!h) return HX_ERR_INVALID_ARG;
    h->timing = enable != 0;
    return HX_OK;
}

int hx_read_kernel_timing(hx_cluster* h, float* ms, int* launches) {
    if (!h || !ms || !launches) return HX_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    for (int k = 0; k < 3; ++k) { ms[k] = 0.f; launches[k] = 0; }
    for (auto& sp : h->spans) {
        HX_TRY(cudaEventSynchronize(sp.b), "cudaEventSynchronize");
        float t = 0.f;
        HX_TRY(cudaEventElapsedTime(&t, sp.a, sp.b), "cudaEventElapsedTime");
        ms[sp.family] += t; ++launches[sp.family];
        h->spare.push_back(sp);
    }
    h->spans.clear();
    return HX_OK;
}

const char* hx_last_error(const hx_cluster* h) { return h ? h->err.c_str() : g_create_err.c_str(); }

long long hx_launch_count(const hx_cluster* h) { return h ? h->launches : 0; }

}  // extern "C"
