// Master-side second-moment update of Algorithm 2 for one coordinate of I_{t-1}, shared by the kernels that
// apply it.  Device-side only.
#pragma once
#include <cstdint>
#include "sk_internal.h"

namespace sk {

// v is kept lazily: vstamp[j] is the step at which v[j] was last brought up to date.  A coordinate outside
// I_{t-1} only decays, v <- beta2 v (Algorithm 2's v update with h_t = 0 there), and vhat = max(vhat, v) cannot
// change, so the decays are applied one fp32 multiply per owed step when the coordinate is next touched --
// the same chain of roundings as applying them every step.
__device__ __forceinline__ float decay_owed(float v, float beta2, uint32_t owed) {
    for (uint32_t s = 0; s < owed && v != 0.0f; ++s) v = __fmul_rn(beta2, v);
    return v;
}

// The same decay by square-and-multiply: v * beta2^owed with at most 2 log2(owed) roundings instead of `owed`
// (a few ulp away from the multiply chain; used on the hot path, where `owed` is typically d/k steps and the
// chain would serialise a divergent lane for that long).
__device__ __forceinline__ float decay_owed_fast(float v, float beta2, uint32_t owed) {
    float p = beta2;
    while (owed) {
        if (owed & 1u) v *= p;
        p *= p;
        owed >>= 1;
    }
    return v;
}

// h = gsum / n ; v = beta2 v + (1-beta2) h^2, after the decay owed since `stamp`; `step` is t (1-based)
__device__ __forceinline__ float second_moment_value(const Params& P, float v, uint32_t stamp, uint32_t step, float gsum) {
    const float h = gsum / (float)P.n_all;
    return fmaf(P.beta2, decay_owed_fast(v, P.beta2, step - 1u - stamp), (1.0f - P.beta2) * h * h);
}

// Gradient entries are stored as fp32 or as bf16 (the upper half of an fp32: widening is exact).
// Four consecutive entries of quad index q (q-th group of four in the worker-major array):
__device__ __forceinline__ float4 load_grad4(const void* grads, uint64_t q, uint32_t bf16) {
    if (bf16) {
        const uint2 raw = __ldcs((const uint2*)grads + q);
        return make_float4(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xFFFF0000u),
                           __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xFFFF0000u));
    }
    return __ldcs((const float4*)grads + q);
}
// The same in two halves, for software pipelines: the load leaves bf16 entries unwidened (in .x and .y of the
// result), and the widening happens where the values are consumed, so that nothing depends on the load at issue time.
__device__ __forceinline__ float4 load_grad4_raw(const void* grads, uint64_t q, uint32_t bf16) {
    if (bf16) {
        const uint2 raw = __ldcs((const uint2*)grads + q);
        return make_float4(__uint_as_float(raw.x), __uint_as_float(raw.y), 0.0f, 0.0f);
    }
    return __ldcs((const float4*)grads + q);
}
__device__ __forceinline__ float4 widen_grad4(float4 raw, uint32_t bf16) {
    if (!bf16) return raw;
    const uint32_t lo = __float_as_uint(raw.x), hi = __float_as_uint(raw.y);
    return make_float4(__uint_as_float(lo << 16), __uint_as_float(lo & 0xFFFF0000u),
                       __uint_as_float(hi << 16), __uint_as_float(hi & 0xFFFF0000u));
}
__device__ __forceinline__ float load_grad1(const void* grads, uint64_t q, uint32_t bf16) {
    if (bf16) return __uint_as_float((uint32_t)((const uint16_t*)grads)[q] << 16);
    return ((const float*)grads)[q];
}

}  // namespace sk
