// Receiving side of a message and the model step (Algorithm 1, server lines):
//   k_apply_packed  u^_m += C_m(.)  scatter-add of the packed (index, value) entries of every worker
//   k_aggregate     x <- x - gamma * sum_m w_m u^_m, a dense stream over W + 1 arrays
#pragma once
#include "kimad_kernels.cuh"

namespace kimad {

// One CTA row per worker (blockIdx.y); entries are visited with a grid-stride loop because their number
// is only known on the device (offs[L]).  The layer of an entry is found by bisection in offs.
template <bool BF16>
__global__ void __launch_bounds__(kThreads)
k_apply_packed(const uint32_t* __restrict__ idx, const void* __restrict__ val, const uint64_t* __restrict__ offs,
               const LayerDesc* __restrict__ layers, uint32_t L, uint64_t cap, uint64_t stride,
               float* __restrict__ est) {
    const uint32_t w = blockIdx.y;
    const uint64_t* of = offs + (size_t)w * (L + 1);
    const uint64_t total = min(of[L], cap);
    const uint32_t* ix = idx + (size_t)w * cap;
    float* e = est + (size_t)w * stride;
    for (uint64_t p = (uint64_t)blockIdx.x * kThreads + threadIdx.x; p < total; p += (uint64_t)gridDim.x * kThreads) {
        uint32_t lo = 0, hi = L; // invariant: of[lo] <= p < of[hi]
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (of[mid] <= p) lo = mid; else hi = mid;
        }
        const LayerDesc ld = layers[lo];
        const uint32_t i = ix[p];
        if ((uint64_t)i >= ld.n) continue;
        const float v = BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(val)[(size_t)w * cap + p])
                             : reinterpret_cast<const float*>(val)[(size_t)w * cap + p];
        float* dst = e + ld.begin + i;
        *dst = __fadd_rn(*dst, v); // every index occurs once per message: no two threads share an element
    }
}

struct AggWeights { float w[KIMAD_MAX_AGG_WORKERS]; };

template <bool VEC>
__global__ void __launch_bounds__(kThreads)
k_aggregate(float* __restrict__ x, const float* __restrict__ est, uint64_t stride, uint32_t W, uint64_t n,
            AggWeights wt, float gamma) {
    const uint64_t step = (uint64_t)gridDim.x * kThreads;
    if (VEC) {
        const uint64_t nq = n / 4;
        for (uint64_t q = (uint64_t)blockIdx.x * kThreads + threadIdx.x; q < nq; q += step) {
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (uint32_t m = 0; m < W; ++m) {
                const float4 e = __ldcs(reinterpret_cast<const float4*>(est + (size_t)m * stride) + q);
                const float wm = wt.w[m];
                acc.x = __fadd_rn(acc.x, __fmul_rn(wm, e.x)); acc.y = __fadd_rn(acc.y, __fmul_rn(wm, e.y));
                acc.z = __fadd_rn(acc.z, __fmul_rn(wm, e.z)); acc.w = __fadd_rn(acc.w, __fmul_rn(wm, e.w));
            }
            float4 v = reinterpret_cast<float4*>(x)[q];
            v.x = __fsub_rn(v.x, __fmul_rn(gamma, acc.x)); v.y = __fsub_rn(v.y, __fmul_rn(gamma, acc.y));
            v.z = __fsub_rn(v.z, __fmul_rn(gamma, acc.z)); v.w = __fsub_rn(v.w, __fmul_rn(gamma, acc.w));
            reinterpret_cast<float4*>(x)[q] = v;
        }
    }
    const uint64_t tail0 = VEC ? (n / 4) * 4 : 0;
    for (uint64_t i = tail0 + (uint64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += step) {
        float acc = 0.f;
        for (uint32_t m = 0; m < W; ++m) acc = __fadd_rn(acc, __fmul_rn(wt.w[m], est[(size_t)m * stride + i]));
        x[i] = __fsub_rn(x[i], __fmul_rn(gamma, acc));
    }
}

} // namespace kimad
