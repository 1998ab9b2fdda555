// Per-call service-time estimates (the Estimator of Section 4.2, "Scheduler internals": prefill time, decode
// time, KV-transfer volume and decode memory demand from a call's input and output length, with a
// roofline-style model): the same binary32 sequence the scoring, greedy and decode kernels use inside,
// written out for callers that need the terms themselves (the event-driven replay).
#include "hx_internal.h"

namespace {

__global__ void hx_estimate_kernel(HxConstTables ct, int G, int M, const hx_call* calls, int n,
                                   float* tpre, float* tdec, float* kvB_out, float* m_out, int* status) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n * G) return;
    const int c = i / G, g = i - c * G;
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(calls) + c);
    const float nt = __uint_as_float(raw.z), o = __uint_as_float(raw.w);
    if (raw.y >= (unsigned)M) {                                   // unknown model: flagged, no estimate
        atomicExch(status, HX_ERR_INVALID_ARG);
        tpre[i] = __int_as_float(0x7f800000); tdec[i] = __int_as_float(0x7f800000);
        if (g == 0) { kvB_out[c] = 0.f; m_out[c] = __fadd_rn(nt, o); }
        return;
    }
    const float phi = ct.phi[raw.y], omega = ct.omega[raw.y], kappa = ct.kappa[raw.y], psi = ct.psi[raw.y];
    const float kvB = __fmul_rn(nt, kappa);
    const float ctx = __fmaf_rn(0.5f, __fsub_rn(o, 1.0f), nt);
    const float step = __fmaf_rn(kappa, ctx, omega);
    const float flops = __fmaf_rn(__fmul_rn(nt, psi), nt, __fmul_rn(nt, phi));     // exactly n * phi when psi = 0
    tpre[i] = fmaxf(__fmul_rn(flops, ct.invF[g]), __fmul_rn(__fadd_rn(omega, kvB), ct.invB[g]));
    tdec[i] = __fmul_rn(__fmul_rn(o, step), ct.invB[g]);
    if (g == 0) { kvB_out[c] = kvB; m_out[c] = __fadd_rn(nt, o); }
}

}  // namespace

cudaError_t hx_launch_estimate(const HxConstTables& ct, int G, int M, const hx_call* calls, int n_calls,
                               float* tpre, float* tdec, float* kvB, float* m, int* status, cudaStream_t stream,
                               long long* launches) {
    const long long work = (long long)n_calls * G;
    hx_estimate_kernel<<<(unsigned)((work + 255) / 256), 256, 0, stream>>>(ct, G, M, calls, n_calls, tpre, tdec, kvB, m, status);
    ++*launches;
    return cudaGetLastError();
}
