// Workflow horizons: longest node-weighted path to a sink for every node of the
// revealed forest (paper Section 5.1, "Define online workflow horizon";
// Algorithm 1, horizon update).
//
//   tail[v] = max over successors u of cp[u]      (0 for a sink)
//   cp[v]   = cost[v] + tail[v]
//   H[w]    = max over the nodes of workflow w of cp[v]
//
// Workflows are independent components, so no grid-wide level barrier is
// needed: one group of threads (a warp, or a whole block for big workflows)
// walks all levels of one workflow.  The host has regrouped the nodes workflow
// by workflow and by height above the sinks, so the frontier segment of a level
// is a contiguous index range: the group stages the workflow's slice of the CSR
// arrays in shared memory with coalesced loads, sweeps the levels there with a
// group barrier between levels, and writes cp/tail back once.  max is exact and
// every node does exactly one addition, so the result is independent of the
// order in which a level is processed.
#include "hx_internal.h"

namespace {

// GW = lanes of the group that owns one workflow: 8 (a quarter of a warp), 32 (a warp) or 0 (the
// whole block).  Small workflows have one to eight nodes per level: with a quarter warp per workflow
// a warp instruction serves four workflows instead of one.
template <int GW>
__device__ __forceinline__ unsigned group_mask() {
    return GW == 8 ? 0xFFu << (threadIdx.x & 24) : 0xffffffffu;
}
template <int GW>
__device__ __forceinline__ void group_sync() {
    if (GW == 0) __syncthreads(); else __syncwarp(group_mask<GW>());
}

template <int GW>
__device__ __forceinline__ float group_max(float v, float* red, int t, int tpw) {
    const unsigned mask = group_mask<GW>();
    for (int off = (GW == 8 ? 4 : 16); off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(mask, v, off));
    if (GW != 0) return v;
    __syncthreads();
    if ((t & 31) == 0) red[t >> 5] = v;
    __syncthreads();
    float r = red[0];
    for (int i = 1; i < (tpw >> 5); ++i) r = fmaxf(r, red[i]);
    return r;
}

// One group per workflow, workflow slice staged in shared memory.
template <int GW>
__global__ void hx_cpath_staged_kernel(HxForestDev f, const uint32_t* __restrict__ wf_ids, uint32_t count,
                                       int tpw, int wfs_per_block, uint32_t smem_per_wf) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ float red[32];
    const int g = threadIdx.x / tpw, t = threadIdx.x % tpw;
    const uint32_t slot = blockIdx.x * wfs_per_block + g;
    if (slot >= count) return;                // a whole group (warp, or the only group of a block) leaves
    const uint32_t w = wf_ids[slot];
    const uint32_t ns = f.wf_node_start[w], n = f.wf_node_start[w + 1] - ns;
    const uint32_t es = f.wf_edge_start[w], ne = f.wf_edge_start[w + 1] - es;
    const uint32_t ss = f.wf_seg_start[w], nlev = f.wf_seg_start[w + 1] - ss - 1;

    unsigned char* base = smem_raw + (size_t)g * smem_per_wf;
    float* cpS = reinterpret_cast<float*>(base);
    float* costS = cpS + n;                                   // becomes tail once a node is done
    uint32_t* rowS = reinterpret_cast<uint32_t*>(costS + n);  // n + 1 entries, absolute edge offsets
    uint32_t* segS = rowS + n + 1;                            // nlev + 1 entries
    uint16_t* colW = reinterpret_cast<uint16_t*>(segS + nlev + 1);   // copied as 32-bit words from an even edge offset
    const uint32_t eodd = es & 1u;
    uint16_t* colS = colW + eodd;                             // colS[e - es] = successor of edge e

    // the slice goes to shared memory with asynchronous 4-byte copies: all of them are in flight at once,
    // where a load-then-store loop of one warp would pay one memory latency per iteration
    auto cp4 = [](void* dst, const void* src) {
        const unsigned sa = (unsigned)__cvta_generic_to_shared(dst);
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" :: "r"(sa), "l"(src) : "memory");
    };
    for (uint32_t i = t; i < n; i += tpw) cp4(costS + i, f.icost + ns + i);
    for (uint32_t i = t; i <= n; i += tpw) cp4(rowS + i, f.irow + ns + i);
    for (uint32_t i = t; i <= nlev; i += tpw) cp4(segS + i, f.seg_off + ss + i);
    {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(f.icol16 + (es - eodd));
        const uint32_t nw = (ne + eodd + 1) >> 1;             // the last word may reach one entry past the slice (padded array)
        for (uint32_t i = t; i < nw; i += tpw) cp4(reinterpret_cast<uint32_t*>(colW) + i, src + i);
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    group_sync<GW>();

    float hmax = 0.0f;
    for (uint32_t lev = 0; lev < nlev; ++lev) {
        const uint32_t hi = segS[lev + 1];
        for (uint32_t i = segS[lev] + t; i < hi; i += tpw) {
            float tl = 0.0f;
            const uint32_t e1 = rowS[i + 1] - es;
            uint32_t e = rowS[i] - es;
            for (; e + 4 <= e1; e += 4) {                     // four successors in flight (max is exact: any order)
                const uint32_t c0 = colS[e], c1 = colS[e + 1], c2 = colS[e + 2], c3 = colS[e + 3];
                const float v0 = cpS[c0], v1 = cpS[c1], v2 = cpS[c2], v3 = cpS[c3];
                tl = fmaxf(fmaxf(tl, fmaxf(v0, v1)), fmaxf(v2, v3));
            }
            for (; e < e1; ++e) tl = fmaxf(tl, cpS[colS[e]]);
            const float c = __fadd_rn(costS[i], tl);
            cpS[i] = c;
            costS[i] = tl;
            hmax = fmaxf(hmax, c);
        }
        group_sync<GW>();
    }
    for (uint32_t i0 = t; i0 < n; i0 += 4 * tpw) {            // four node numbers in flight per thread
        uint32_t v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = i0 + u * tpw < n ? __ldg(f.perm + ns + i0 + u * tpw) : 0u;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t i = i0 + u * tpw;
            if (i < n) { f.cp[v[u]] = cpS[i]; f.tail[v[u]] = costS[i]; }
        }
    }
    hmax = group_max<GW>(hmax, red, t, tpw);
    if (t == 0) f.H[f.wf_gid ? f.wf_gid[w] : w] = hmax;
}

// One block per workflow, everything in global memory: for workflows too large
// to stage.  cp is written and re-read by the same block; the block barrier
// between levels orders those accesses, and the reads bypass L1.
__global__ void hx_cpath_global_kernel(HxForestDev f, const uint32_t* __restrict__ wf_ids, uint32_t count) {
    __shared__ float red[32];
    const uint32_t w = wf_ids[blockIdx.x];
    const int t = threadIdx.x, tpw = blockDim.x;
    const uint32_t ns = f.wf_node_start[w];
    const uint32_t ss = f.wf_seg_start[w], nlev = f.wf_seg_start[w + 1] - ss - 1;
    float hmax = 0.0f;
    for (uint32_t lev = 0; lev < nlev; ++lev) {
        const uint32_t lo = f.seg_off[ss + lev], hi = f.seg_off[ss + lev + 1];
        for (uint32_t i = lo + t; i < hi; i += tpw) {
            float tl = 0.0f;
            const uint32_t e1 = f.irow[ns + i + 1];
            for (uint32_t e = f.irow[ns + i]; e < e1; ++e)
                tl = fmaxf(tl, __ldcg(&f.cp[f.perm[ns + f.icol32[e]]]));
            const float c = __fadd_rn(f.icost[ns + i], tl);
            const uint32_t v = f.perm[ns + i];
            __stcg(&f.cp[v], c);
            f.tail[v] = tl;
            hmax = fmaxf(hmax, c);
        }
        __syncthreads();
    }
    hmax = group_max<false>(hmax, red, t, tpw);
    if (t == 0) f.H[f.wf_gid ? f.wf_gid[w] : w] = hmax;
}

// Replaces the cost estimates of some nodes (internal numbering) by newer values, e.g. observed
// latencies (Section 5.1, "Define online workflow horizon").
__global__ void hx_cost_update_kernel(float* __restrict__ icost, const uint32_t* __restrict__ idx,
                                      const float* __restrict__ cost, uint32_t n) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) icost[idx[i]] = cost[i];
}

}  // namespace

cudaError_t hx_launch_cost_update(const HxForestDev& f, const uint32_t* idx, const float* cost, uint32_t n,
                                  cudaStream_t stream, long long* launches) {
    if (n == 0) return cudaSuccess;
    hx_cost_update_kernel<<<(n + 255) / 256, 256, 0, stream>>>(const_cast<float*>(f.icost), idx, cost, n);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t hx_launch_cpath(const HxForestDev& f, const HxCpClass* classes, int n_classes,
                            cudaStream_t stream, long long* launches, const HxForkJoin* fj) {
    // the classes touch disjoint workflows: with side streams the second and later classes run
    // beside the first one and join the caller's stream afterwards
    int n_live = 0;
    for (int k = 0; k < n_classes; ++k) n_live += classes[k].count != 0;
    const bool fork = fj && fj->ready && n_live > 1;
    if (fork) {
        cudaError_t e = cudaEventRecord(fj->fork, stream);
        if (e != cudaSuccess) return e;
    }
    int side = 0;
    bool first = true;
    for (int k = 0; k < n_classes; ++k) {
        const HxCpClass& c = classes[k];
        if (c.count == 0) continue;
        cudaStream_t s = stream;
        int my_side = -1;
        if (fork && !first && side < HX_CP_SIDE) {
            my_side = side++;
            s = fj->aux[my_side];
            cudaError_t e = cudaStreamWaitEvent(s, fj->fork, 0);
            if (e != cudaSuccess) return e;
        }
        first = false;
        if (c.smem_per_wf == 0) {
            hx_cpath_global_kernel<<<c.count, 256, 0, s>>>(f, c.wf_ids, c.count);
        } else {
            const int threads = c.threads_per_wf * c.wfs_per_block;
            const size_t smem = c.smem_per_wf * c.wfs_per_block;
            const unsigned grid = (c.count + c.wfs_per_block - 1) / c.wfs_per_block;
            cudaError_t e = cudaSuccess;
            if (c.threads_per_wf == 8) {
                static size_t allowed[64];
                if ((e = hx_opt_in_smem(hx_cpath_staged_kernel<8>, smem, allowed, 40 * 1024)) != cudaSuccess) return e;
                hx_cpath_staged_kernel<8><<<grid, threads, smem, s>>>(
                    f, c.wf_ids, c.count, 8, c.wfs_per_block, (uint32_t)c.smem_per_wf);
            } else if (c.threads_per_wf == 32) {
                static size_t allowed[64];     // static + dynamic shared memory may exceed the 48 KB default
                if ((e = hx_opt_in_smem(hx_cpath_staged_kernel<32>, smem, allowed, 40 * 1024)) != cudaSuccess) return e;
                hx_cpath_staged_kernel<32><<<grid, threads, smem, s>>>(
                    f, c.wf_ids, c.count, 32, c.wfs_per_block, (uint32_t)c.smem_per_wf);
            } else {
                static size_t allowed[64];
                if ((e = hx_opt_in_smem(hx_cpath_staged_kernel<0>, smem, allowed, 40 * 1024)) != cudaSuccess) return e;
                hx_cpath_staged_kernel<0><<<grid, threads, smem, s>>>(
                    f, c.wf_ids, c.count, c.threads_per_wf, 1, (uint32_t)c.smem_per_wf);
            }
        }
        ++*launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        if (my_side >= 0) {
            if ((e = cudaEventRecord(fj->join[my_side], s)) != cudaSuccess) return e;
            if ((e = cudaStreamWaitEvent(stream, fj->join[my_side], 0)) != cudaSuccess) return e;
        }
    }
    return cudaSuccess;
}
