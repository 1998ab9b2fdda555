// Issue-rate micro-kernels for the roofline of the scoring kernel: register-only loops of the instruction kinds
// its candidate loop is made of (fused multiply-add, packed fused multiply-add on two binary32 values,
// three-input minimum, and the loop's own one-to-one mix of the last two), timed on the device.  They measure
// what the FP32 pipes of this GPU sustain at the clock it runs at, which the nominal lanes x clock figure
// only bounds from above.
#include "hx_internal.h"

namespace {

typedef unsigned long long u64;

__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c) {
    u64 d;
    asm volatile("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ float min3(float a, float b, float c) {
    float d;
    asm volatile("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float fma1(float a, float b, float c) {
    float d;
    asm volatile("fma.rn.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

constexpr int kChains = 8;        // independent dependency chains per thread
constexpr int kUnroll = 4;        // rounds over the chains per loop iteration

// MODE 0: fma.rn.f32; 1: fma.rn.f32x2; 2: three-input min.f32; 3: one fma.rn.f32x2 and one min.f32 in turn.
// Every mode issues kChains * kUnroll instructions per iteration (mode 3: half of each kind).
template <int MODE>
__global__ void __launch_bounds__(256) hx_micro_kernel(int iters, float seed, float* sink) {
    float f[kChains]; u64 p[kChains];
#pragma unroll
    for (int k = 0; k < kChains; ++k) {
        f[k] = seed + (float)(threadIdx.x + k);
        const float lo = f[k], hi = f[k] + 0.5f;
        asm("mov.b64 %0, {%1, %2};" : "=l"(p[k]) : "f"(lo), "f"(hi));
    }
    const float a = 0.999f, b = 1e-3f;
    u64 a2, b2;
    asm("mov.b64 %0, {%1, %1};" : "=l"(a2) : "f"(a));
    asm("mov.b64 %0, {%1, %1};" : "=l"(b2) : "f"(b));
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
#pragma unroll
            for (int k = 0; k < kChains; ++k) {
                if (MODE == 0) f[k] = fma1(f[k], a, b);
                if (MODE == 1) p[k] = fma2(p[k], a2, b2);
                if (MODE == 2) f[k] = min3(f[k], f[(k + 1) % kChains], a);
                if (MODE == 3) {
                    if (k & 1) f[k] = min3(f[k], f[k - 1], a);
                    else p[k] = fma2(p[k], a2, b2);
                }
            }
        }
    }
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < kChains; ++k) {
        float lo, hi;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p[k]));
        acc += f[k] + lo + hi;
    }
    if (acc == 12345.678f) *sink = acc;                     // keeps the loop alive; never true in practice
}

template <int MODE>
cudaError_t time_one(int grid, int iters, float* sink, cudaStream_t s, cudaEvent_t e0, cudaEvent_t e1, float* ms) {
    hx_micro_kernel<MODE><<<grid, 256, 0, s>>>(iters / 8, 1.0f, sink);          // warm-up
    cudaError_t e = cudaEventRecord(e0, s);
    if (e != cudaSuccess) return e;
    hx_micro_kernel<MODE><<<grid, 256, 0, s>>>(iters, 1.0f, sink);
    if ((e = cudaEventRecord(e1, s)) != cudaSuccess) return e;
    if ((e = cudaEventSynchronize(e1)) != cudaSuccess) return e;
    return cudaEventElapsedTime(ms, e0, e1);
}

}  // namespace

cudaError_t hx_run_micro(int n_sm, float* sink, cudaStream_t stream, double* lane_instr_per_s, float* ms, long long* launches) {
    const int grid = n_sm * 8, iters = 16384;
    cudaEvent_t e0, e1;
    cudaError_t e = cudaEventCreate(&e0);
    if (e != cudaSuccess) return e;
    if ((e = cudaEventCreate(&e1)) != cudaSuccess) { cudaEventDestroy(e0); return e; }
    if (e == cudaSuccess) e = time_one<0>(grid, iters, sink, stream, e0, e1, ms + 0);
    if (e == cudaSuccess) e = time_one<1>(grid, iters, sink, stream, e0, e1, ms + 1);
    if (e == cudaSuccess) e = time_one<2>(grid, iters, sink, stream, e0, e1, ms + 2);
    if (e == cudaSuccess) e = time_one<3>(grid, iters, sink, stream, e0, e1, ms + 3);
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    if (e != cudaSuccess) return e;
    const double instr = (double)grid * 256.0 * (double)iters * kChains * kUnroll;   // lane-instructions per timed launch
    for (int k = 0; k < 4; ++k) lane_instr_per_s[k] = instr / ((double)ms[k] * 1e-3);
    *launches += 8;
    return cudaGetLastError();
}
