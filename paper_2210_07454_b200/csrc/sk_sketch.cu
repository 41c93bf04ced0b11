// Dense half of the step: second moments on I_{t-1}, momentum + error-feedback accumulate + Count Sketch of
// every worker's vector (Algorithm 2, worker side; Section II-C), and the fixed-order sum of the n sketches.
#include "sk_internal.h"
#include "sk_hash.cuh"

namespace sk {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ void red_add_v4(float* addr, float4 v) {
    // one 16-byte reduction into the L2-resident table; nothing in this kernel reads the tables back
    asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                 :: "l"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w));
}

__global__ void __launch_bounds__(kThreads) k_zero(float4* p, uint64_t n4) {
    const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    for (uint64_t t = blockIdx.x * (uint64_t)kThreads + threadIdx.x; t < n4; t += (uint64_t)gridDim.x * kThreads)
        p[t] = z;
}

__global__ void __launch_bounds__(kThreads) k_fill_u32(uint32_t* p, uint64_t n, uint32_t value) {
    for (uint64_t t = blockIdx.x * (uint64_t)kThreads + threadIdx.x; t < n; t += (uint64_t)gridDim.x * kThreads)
        p[t] = value;
}

// v is kept lazily: vstamp[j] is the step at which v[j] was last brought up to date.  A coordinate outside
// I_{t-1} only decays, v <- beta2 v (Algorithm 2's v update with h_t = 0 there), and vhat = max(vhat, v) cannot
// change, so the decays are applied one fp32 multiply per owed step when the coordinate is next touched --
// the same chain of roundings as applying them every step.
__device__ __forceinline__ float decay_owed(float v, float beta2, uint32_t owed) {
    for (uint32_t s = 0; s < owed && v != 0.0f; ++s) v = __fmul_rn(beta2, v);
    return v;
}

// For j in I_{t-1}: h = mean_w g^(w)_j ; v_j = beta2 v_j + (1-beta2) h^2 ; vhat_j = max(vhat_j, v_j).
__global__ void __launch_bounds__(kThreads)
k_second_moment(const __grid_constant__ Params P, const float* __restrict__ grads, float* v, float* vhat,
                uint32_t* vstamp, const uint32_t* __restrict__ I_prev, uint32_t k_prev, uint32_t t) {
    const uint32_t q = blockIdx.x * kThreads + threadIdx.x;
    if (q >= k_prev) return;
    const uint32_t j = I_prev[q];
    float h = 0.0f;
#pragma unroll 4
    for (uint32_t w = 0; w < P.n; ++w) h += __ldg(grads + (uint64_t)w * P.d + j);
    h = h / (float)P.n;
    float vj = decay_owed(v[j], P.beta2, t - 1u - vstamp[j]);
    vj = fmaf(P.beta2, vj, (1.0f - P.beta2) * h * h);
    v[j] = vj;
    vstamp[j] = t;
    if (vj > vhat[j]) vhat[j] = vj;
}

__global__ void __launch_bounds__(kThreads)
k_v_materialize(const __grid_constant__ Params P, const float* __restrict__ v,
                const uint32_t* __restrict__ vstamp, uint32_t t, float* out) {
    for (uint32_t j = blockIdx.x * kThreads + threadIdx.x; j < P.d; j += gridDim.x * kThreads)
        out[j] = decay_owed(v[j], P.beta2, t - vstamp[j]);
}

// m = beta1 m + (1-beta1) g ; a = m + e (kept in the e buffer) ; S^(w)[row, h_row(j)] += s_row(j) a_j.
// Vector form: one thread owns 4 consecutive coordinates and walks the workers w0..w0+nw-1, so the hashes are
// evaluated once per coordinate quad and reused for every worker (all workers share h and s, or the sketches
// could not be added).  R > 0: rows known at compile time; R == 0: any r <= kMaxRows.
template <int R>
__global__ void __launch_bounds__(kThreads)
k_moment_sketch_v4(const __grid_constant__ Params P, const float4* __restrict__ grads, float4* m, float4* e,
                   float* tables, uint32_t w0, uint32_t nw) {
    const uint32_t r = R > 0 ? (uint32_t)R : P.r;
    const uint32_t d4 = P.d >> 2;
    const float b1 = P.beta1, omb1 = 1.0f - P.beta1;
    const uint64_t tstride = (uint64_t)P.r * P.cs;
    for (uint32_t t = blockIdx.x * kThreads + threadIdx.x; t < d4; t += gridDim.x * kThreads) {
        Quad h[R > 0 ? R : (int)kMaxRows];
#pragma unroll
        for (uint32_t row = 0; row < r; ++row) h[row] = quad_hash(P.row_key[row], P.log2g, P.G, t << 2);
        uint32_t w = w0;
        const uint32_t wend = w0 + nw;
        for (; w + 2 <= wend; w += 2) {          // two workers per trip: six 16-byte loads in flight
            const uint64_t q0 = (uint64_t)w * d4 + t, q1 = q0 + d4;
            const float4 g0 = __ldcs(grads + q0), g1 = __ldcs(grads + q1);
            float4 m0 = __ldcs(m + q0), m1 = __ldcs(m + q1);
            float4 a0 = __ldcs(e + q0), a1 = __ldcs(e + q1);
            m0.x = fmaf(b1, m0.x, omb1 * g0.x); m0.y = fmaf(b1, m0.y, omb1 * g0.y);
            m0.z = fmaf(b1, m0.z, omb1 * g0.z); m0.w = fmaf(b1, m0.w, omb1 * g0.w);
            m1.x = fmaf(b1, m1.x, omb1 * g1.x); m1.y = fmaf(b1, m1.y, omb1 * g1.y);
            m1.z = fmaf(b1, m1.z, omb1 * g1.z); m1.w = fmaf(b1, m1.w, omb1 * g1.w);
            a0.x += m0.x; a0.y += m0.y; a0.z += m0.z; a0.w += m0.w;
            a1.x += m1.x; a1.y += m1.y; a1.z += m1.z; a1.w += m1.w;
            __stcs(m + q0, m0); __stcs(m + q1, m1);
            __stcs(e + q0, a0); __stcs(e + q1, a1);
            float* t0 = tables + (uint64_t)w * tstride;
            float* t1 = t0 + tstride;
#pragma unroll
            for (uint32_t row = 0; row < r; ++row) {
                red_add_v4(t0 + (uint64_t)row * P.cs + h[row].off, quad_scatter(h[row], a0));
                red_add_v4(t1 + (uint64_t)row * P.cs + h[row].off, quad_scatter(h[row], a1));
            }
        }
        if (w < wend) {
            const uint64_t q0 = (uint64_t)w * d4 + t;
            const float4 g0 = __ldcs(grads + q0);
            float4 m0 = __ldcs(m + q0);
            float4 a0 = __ldcs(e + q0);
            m0.x = fmaf(b1, m0.x, omb1 * g0.x); m0.y = fmaf(b1, m0.y, omb1 * g0.y);
            m0.z = fmaf(b1, m0.z, omb1 * g0.z); m0.w = fmaf(b1, m0.w, omb1 * g0.w);
            a0.x += m0.x; a0.y += m0.y; a0.z += m0.z; a0.w += m0.w;
            __stcs(m + q0, m0);
            __stcs(e + q0, a0);
            float* t0 = tables + (uint64_t)w * tstride;
#pragma unroll
            for (uint32_t row = 0; row < r; ++row)
                red_add_v4(t0 + (uint64_t)row * P.cs + h[row].off, quad_scatter(h[row], a0));
        }
    }
}

// Scalar form: any d, any alignment, any group size.  One thread per coordinate.
__global__ void __launch_bounds__(kThreads)
k_moment_sketch_scalar(const __grid_constant__ Params P, const float* __restrict__ grads, float* m, float* e,
                       float* tables, uint32_t w0, uint32_t nw) {
    const float b1 = P.beta1, omb1 = 1.0f - P.beta1;
    const uint64_t tstride = (uint64_t)P.r * P.cs;
    for (uint32_t j = blockIdx.x * kThreads + threadIdx.x; j < P.d; j += gridDim.x * kThreads) {
        for (uint32_t w = w0; w < w0 + nw; ++w) {
            const uint64_t q = (uint64_t)w * P.d + j;
            const float mm = fmaf(b1, m[q], omb1 * grads[q]);
            const float a = mm + e[q];
            m[q] = mm;
            e[q] = a;
            for (uint32_t row = 0; row < P.r; ++row) {
                uint32_t b; float s;
                coord_hash(P.row_key[row], P.log2g, P.G, j, b, s);
                atomicAdd(tables + (uint64_t)w * tstride + (uint64_t)row * P.cs + b, s * a);
            }
        }
    }
}

// S = (S^(0) + S^(1) + ... + S^(n-1)) / n, workers added in index order (Algorithm 2, master side).
__global__ void __launch_bounds__(kThreads)
k_sum_tables(const __grid_constant__ Params P, const float4* __restrict__ tables, float4* sum) {
    const uint32_t q4 = (P.r * P.cs) >> 2;
    const float fn = (float)P.n;
    for (uint32_t t = blockIdx.x * kThreads + threadIdx.x; t < q4; t += gridDim.x * kThreads) {
        float4 acc = __ldcs(tables + t);
        for (uint32_t w = 1; w < P.n; ++w) {
            const float4 x = __ldcs(tables + (uint64_t)w * q4 + t);
            acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
        }
        acc.x = acc.x / fn; acc.y = acc.y / fn; acc.z = acc.z / fn; acc.w = acc.w / fn;
        sum[t] = acc;
    }
}

inline int grid_for(uint64_t items, int sm_count, int per_sm) {
    const uint64_t want = (items + kThreads - 1) / kThreads;
    const uint64_t cap = (uint64_t)sm_count * per_sm;
    return (int)(want < cap ? (want ? want : 1) : cap);
}

}  // namespace

int launch_zero(float* p, uint64_t nfloats, cudaStream_t st) {
    k_zero<<<grid_for(nfloats / 4, 148, 8), kThreads, 0, st>>>((float4*)p, nfloats / 4);
    return 1;
}

int launch_fill_u32(uint32_t* p, uint64_t n, uint32_t value, cudaStream_t st) {
    k_fill_u32<<<grid_for(n, 148, 8), kThreads, 0, st>>>(p, n, value);
    return 1;
}

int launch_second_moment(const Params& P, const float* grads, float* v, float* vhat, uint32_t* vstamp,
                         const uint32_t* I_prev, uint32_t k_prev, uint32_t t, cudaStream_t st) {
    if (k_prev == 0) return 0;
    k_second_moment<<<(k_prev + kThreads - 1) / kThreads, kThreads, 0, st>>>(P, grads, v, vhat, vstamp, I_prev,
                                                                           k_prev, t);
    return 1;
}

int launch_v_materialize(const Params& P, const float* v, const uint32_t* vstamp, uint32_t t, float* out,
                         cudaStream_t st) {
    k_v_materialize<<<grid_for(P.d, 148, 8), kThreads, 0, st>>>(P, v, vstamp, t, out);
    return 1;
}

int launch_moment_sketch(const Params& P, const float* grads, float* m, float* e, float* tables, uint32_t w0,
                         uint32_t nw, bool vec, int sm_count, cudaStream_t st) {
    if (!vec) {
        k_moment_sketch_scalar<<<grid_for(P.d, sm_count, 8), kThreads, 0, st>>>(P, grads, m, e, tables, w0, nw);
        return 1;
    }
    const int grid = grid_for(P.d >> 2, sm_count, 8);
    const float4* g4 = (const float4*)grads;
    float4* m4 = (float4*)m;
    float4* e4 = (float4*)e;
#define SK_CASE(RR) case RR: k_moment_sketch_v4<RR><<<grid, kThreads, 0, st>>>(P, g4, m4, e4, tables, w0, nw); break;
    switch (P.r) {
        SK_CASE(1) SK_CASE(2) SK_CASE(3) SK_CASE(4) SK_CASE(5) SK_CASE(6) SK_CASE(7) SK_CASE(8) SK_CASE(10)
        default: k_moment_sketch_v4<0><<<grid, kThreads, 0, st>>>(P, g4, m4, e4, tables, w0, nw); break;
    }
#undef SK_CASE
    return 1;
}

int launch_sum_tables(const Params& P, const float* tables, float* sum, cudaStream_t st) {
    k_sum_tables<<<grid_for((P.r * P.cs) >> 2, 148, 8), kThreads, 0, st>>>(P, (const float4*)tables, (float4*)sum);
    return 1;
}

}  // namespace sk
