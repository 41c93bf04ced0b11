// Dense half of the step: momentum + error-feedback accumulate + Count Sketch of every worker's vector
// (Algorithm 2, worker side; Section II-C), the gradient sums on I_{t-1} that the master's second-moment update
// needs (the update itself rides on the key pass in sk_select.cu), and the fixed-order sum of the n sketches.
#include "sk_internal.h"
#include "sk_hash.cuh"
#include "sk_moment.cuh"

namespace sk {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ void red_add_v4(float* addr, float4 v) {
    // one 16-byte reduction into the L2-resident table; nothing in this kernel reads the tables back
    asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                 :: "l"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w));
}

// the reduction of one signed quad into row `row` of a table, at the chunk the hash gives (checked in the debug build)
__device__ __forceinline__ void sketch_quad(const Params& P, float* table, uint32_t row, const Quad h, float4 a) {
    SK_GUARD(h.off + 4u <= P.cs, kStatusBucket) red_add_v4(table + (uint64_t)row * P.cs + h.off, quad_scatter(h, a));
}

__global__ void __launch_bounds__(kThreads) k_zero(float4* p, uint64_t n4) {
    chain_acquire();
    const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    for (uint64_t t = blockIdx.x * (uint64_t)kThreads + threadIdx.x; t < n4; t += (uint64_t)gridDim.x * kThreads)
        p[t] = z;
}

__global__ void __launch_bounds__(kThreads) k_fill_u32(uint32_t* p, uint64_t n, uint32_t value) {
    for (uint64_t t = blockIdx.x * (uint64_t)kThreads + threadIdx.x; t < n; t += (uint64_t)gridDim.x * kThreads)
        p[t] = value;
}

__global__ void __launch_bounds__(kThreads)
k_set_bits(const __grid_constant__ Params P, const uint32_t* __restrict__ I, uint32_t count, uint32_t* bitmap) {
    const uint32_t q = blockIdx.x * kThreads + threadIdx.x;
    if (q < count) SK_GUARD(I[q] < P.d, kStatusIndex) atomicOr(&bitmap[I[q] >> 5], 1u << (I[q] & 31u));
}

__global__ void __launch_bounds__(kThreads)
k_v_materialize(const __grid_constant__ Params P, const float* __restrict__ v,
                const uint32_t* __restrict__ vstamp, uint32_t t, float* out) {
    for (uint32_t j = blockIdx.x * kThreads + threadIdx.x; j < P.d; j += gridDim.x * kThreads)
        out[j] = decay_owed(v[j], P.beta2, t - vstamp[j]);
}

// e as Algorithm 2 defines it: the buffer keeps a_t everywhere and the bitmap of I_t marks the zeros
__global__ void __launch_bounds__(kThreads)
k_masked_copy(const float* __restrict__ e, const uint32_t* __restrict__ bitmap, uint32_t d, uint64_t total, float* out) {
    for (uint64_t q = blockIdx.x * (uint64_t)kThreads + threadIdx.x; q < total; q += (uint64_t)gridDim.x * kThreads) {
        const uint32_t j = (uint32_t)(q % d);
        out[q] = ((bitmap[j >> 5] >> (j & 31u)) & 1u) ? 0.0f : e[q];
    }
}

#define SK_MOMENT(mm, aa, gg, mask)                                                     \
    mm.x = fmaf(b1, mm.x, omb1 * gg.x); mm.y = fmaf(b1, mm.y, omb1 * gg.y);             \
    mm.z = fmaf(b1, mm.z, omb1 * gg.z); mm.w = fmaf(b1, mm.w, omb1 * gg.w);             \
    aa.x = fmaf(rho, (mask & 1u) ? 0.0f : aa.x, mm.x); aa.y = fmaf(rho, (mask & 2u) ? 0.0f : aa.y, mm.y); \
    aa.z = fmaf(rho, (mask & 4u) ? 0.0f : aa.z, mm.z); aa.w = fmaf(rho, (mask & 8u) ? 0.0f : aa.w, mm.w);

// Option: S_t = (1/n) sum_w S(a^(w)) = S((1/n) sum_w a^(w)) because the sketch is linear (Section II-C), so one sketch
// of the worker sum replaces the n per-worker sketches and their sum.  `as` is the sum over this launch's workers.
// The exact values of Section III-A's second round are read from asum = sum_w a^(w): each launch adds its workers'
// sum to what the earlier launches of the step left there.
__device__ __forceinline__ void store_worker_sum(const MomentArgs& A, uint32_t t, float4 as, uint32_t w0) {
    if (w0 > 0) {
        const float4 prev = ((const float4*)A.asum)[t];
        as.x += prev.x; as.y += prev.y; as.z += prev.z; as.w += prev.w;
    }
    ((float4*)A.asum)[t] = as;
}

template <int RMAX>
__device__ __forceinline__ void sketch_of_sum(const Params& P, const MomentArgs& A, uint32_t r, const Quad (&h)[RMAX],
                                              float4 as) {
    const float fn = (float)P.n_all;
    as.x = as.x / fn; as.y = as.y / fn; as.z = as.z / fn; as.w = as.w / fn;
#pragma unroll
    for (uint32_t row = 0; row < (uint32_t)RMAX; ++row)
        if (row < r) sketch_quad(P, A.sum_table, row, h[row], as);
}

// m = beta1 m + (1-beta1) g ; a = m + rho e (kept in the e buffer; e counts as 0 on I_{t-1}; rho = alpha_{t-1}/alpha_t,
// and fmaf(1, e, m) is m + e to the bit) ;
// S^(w)[row, h_row(j)] += s_row(j) a_j ; and on I_{t-1} the gradient sum that feeds v and vhat.
// Vector form: one thread owns 4 consecutive coordinates and walks the workers w0..w0+nw-1, so the hashes are
// evaluated once per coordinate quad and reused for every worker (all workers share h and s, or the sketches
// could not be added).  R > 0: rows known at compile time; R == 0: any r <= kMaxRows.
template <int R>
__global__ void __launch_bounds__(kThreads, 3)
k_moment_sketch_v4(const __grid_constant__ Params P, const __grid_constant__ MomentArgs A, uint32_t w0, uint32_t nw) {
    chain_acquire();
    float4* m = (float4*)A.m;
    float4* e = (float4*)A.e;
    const uint32_t r = R > 0 ? (uint32_t)R : P.r;
    const uint32_t d4 = P.d >> 2;
    const float b1 = P.beta1, omb1 = 1.0f - P.beta1, rho = P.rho;
    const uint32_t gb = A.grad_bf16;
    const uint64_t tstride = (uint64_t)P.r * P.cs;
    constexpr int RMAX = R > 0 ? R : (int)kMaxRows;
    const uint32_t trips = (d4 + gridDim.x * kThreads - 1) / (gridDim.x * kThreads);
    for (uint32_t it = 0; it < trips; ++it) {            // uniform trip count: the hash exchange needs whole warps
        const uint32_t t = (it * gridDim.x + blockIdx.x) * kThreads + threadIdx.x;
        Quad h[RMAX];
        quad_hashes<RMAX>(P, r, t < d4 ? t : d4 - 1, h);
        if (t >= d4) continue;
        const uint32_t mask = A.members ? ((__ldg(A.bitmap + (t >> 3)) >> ((t & 7u) * 4u)) & 0xFu) : 0u;
        float4 gs = make_float4(0.f, 0.f, 0.f, 0.f);     // running gradient sum in worker order (used on I_{t-1})
        if (mask && w0 > 0) gs = ((const float4*)A.gsum)[t];
        float4 as = make_float4(0.f, 0.f, 0.f, 0.f);     // sum of a over this launch's workers, in worker order
        uint32_t w = w0;
        const uint32_t wend = w0 + nw;
        for (; w + 2 <= wend; w += 2) {                  // two workers per trip: six 16-byte loads in flight
            const uint64_t q0 = (uint64_t)w * d4 + t, q1 = q0 + d4;
            const float4 g0 = load_grad4(A.grads, q0, gb), g1 = load_grad4(A.grads, q1, gb);
            float4 m0 = __ldcs(m + q0), m1 = __ldcs(m + q1);
            float4 a0 = __ldcs(e + q0), a1 = __ldcs(e + q1);
            SK_CHECK_FINITE4(g0); SK_CHECK_FINITE4(g1);
            SK_MOMENT(m0, a0, g0, mask)
            SK_MOMENT(m1, a1, g1, mask)
            gs.x = (gs.x + g0.x) + g1.x; gs.y = (gs.y + g0.y) + g1.y;
            gs.z = (gs.z + g0.z) + g1.z; gs.w = (gs.w + g0.w) + g1.w;
            as.x = (as.x + a0.x) + a1.x; as.y = (as.y + a0.y) + a1.y;
            as.z = (as.z + a0.z) + a1.z; as.w = (as.w + a0.w) + a1.w;
            __stcs(m + q0, m0); __stcs(m + q1, m1);
            __stcs(e + q0, a0); __stcs(e + q1, a1);
            float* t0 = A.tables + (uint64_t)w * tstride;
            float* t1 = t0 + tstride;
            if (!A.sum_table) {
#pragma unroll
                for (uint32_t row = 0; row < (uint32_t)RMAX; ++row)
                    if (row < r) {
                        sketch_quad(P, t0, row, h[row], a0);
                        sketch_quad(P, t1, row, h[row], a1);
                    }
            }
        }
        if (w < wend) {
            const uint64_t q0 = (uint64_t)w * d4 + t;
            const float4 g0 = load_grad4(A.grads, q0, gb);
            float4 m0 = __ldcs(m + q0);
            float4 a0 = __ldcs(e + q0);
            SK_CHECK_FINITE4(g0);
            SK_MOMENT(m0, a0, g0, mask)
            gs.x += g0.x; gs.y += g0.y; gs.z += g0.z; gs.w += g0.w;
            as.x += a0.x; as.y += a0.y; as.z += a0.z; as.w += a0.w;
            __stcs(m + q0, m0);
            __stcs(e + q0, a0);
            float* t0 = A.tables + (uint64_t)w * tstride;
            if (!A.sum_table) {
#pragma unroll
                for (uint32_t row = 0; row < (uint32_t)RMAX; ++row)
                    if (row < r) sketch_quad(P, t0, row, h[row], a0);
            }
        }
        if (mask) ((float4*)A.gsum)[t] = gs;             // consumed by the key pass (or by the next launch)
        if (A.sum_table) sketch_of_sum<RMAX>(P, A, r, h, as);
        if (A.asum) store_worker_sum(A, t, as, w0);
    }
}

// Parameter averaging (Algorithm 1): every worker keeps its own v and vhat from its own gradient,
//   m = beta1 m + (1-beta1) g ; v = beta2 v + (1-beta2) g^2 ; vhat = max(vhat, v) ; a = m / sqrt(vhat) + e,
// and a is what is sketched.  Reads g, m, v, vhat, e and writes m, v, vhat, a: 36 bytes per worker-coordinate.
__device__ __forceinline__ void pa_moment(float b1, float omb1, float b2, float omb2, float rho, float g, float& m,
                                          float& v, float& vh, float& a, bool masked) {
    m = fmaf(b1, m, omb1 * g);
    v = fmaf(b2, v, omb2 * g * g);
    vh = fmaxf(vh, v);
    a = fmaf(rho, masked ? 0.0f : a, __fdiv_rn(m, __fsqrt_rn(vh)));
}

template <int R>
__global__ void __launch_bounds__(kThreads, 3)
k_moment_sketch_pa_v4(const __grid_constant__ Params P, const __grid_constant__ MomentArgs A, uint32_t w0, uint32_t nw) {
    chain_acquire();
    float4* m = (float4*)A.m;
    float4* e = (float4*)A.e;
    float4* vw = (float4*)A.vw;
    float4* vhw = (float4*)A.vhatw;
    const uint32_t r = R > 0 ? (uint32_t)R : P.r;
    const uint32_t d4 = P.d >> 2;
    const float b1 = P.beta1, omb1 = 1.0f - P.beta1, b2 = P.beta2, omb2 = 1.0f - P.beta2, rho = P.rho;
    const uint32_t gb = A.grad_bf16;
    const uint64_t tstride = (uint64_t)P.r * P.cs;
    constexpr int RMAX = R > 0 ? R : (int)kMaxRows;
    const uint32_t trips = (d4 + gridDim.x * kThreads - 1) / (gridDim.x * kThreads);
    for (uint32_t it = 0; it < trips; ++it) {
        const uint32_t t = (it * gridDim.x + blockIdx.x) * kThreads + threadIdx.x;
        Quad h[RMAX];
        quad_hashes<RMAX>(P, r, t < d4 ? t : d4 - 1, h);
        if (t >= d4) continue;
        const uint32_t mask = A.members ? ((__ldg(A.bitmap + (t >> 3)) >> ((t & 7u) * 4u)) & 0xFu) : 0u;
        float4 as = make_float4(0.f, 0.f, 0.f, 0.f);     // sum of a over this launch's workers, in worker order
        for (uint32_t w = w0; w < w0 + nw; ++w) {
            const uint64_t q0 = (uint64_t)w * d4 + t;
            const float4 g0 = load_grad4(A.grads, q0, gb);
            float4 m0 = __ldcs(m + q0), v0 = __ldcs(vw + q0), h0 = __ldcs(vhw + q0), a0 = __ldcs(e + q0);
            pa_moment(b1, omb1, b2, omb2, rho, g0.x, m0.x, v0.x, h0.x, a0.x, mask & 1u);
            pa_moment(b1, omb1, b2, omb2, rho, g0.y, m0.y, v0.y, h0.y, a0.y, mask & 2u);
            pa_moment(b1, omb1, b2, omb2, rho, g0.z, m0.z, v0.z, h0.z, a0.z, mask & 4u);
            pa_moment(b1, omb1, b2, omb2, rho, g0.w, m0.w, v0.w, h0.w, a0.w, mask & 8u);
            __stcs(m + q0, m0); __stcs(vw + q0, v0); __stcs(vhw + q0, h0); __stcs(e + q0, a0);
            float* t0 = A.tables + (uint64_t)w * tstride;
            if (!A.sum_table) {
#pragma unroll
                for (uint32_t row = 0; row < (uint32_t)RMAX; ++row)
                    if (row < r) sketch_quad(P, t0, row, h[row], a0);
            }
            as.x += a0.x; as.y += a0.y; as.z += a0.z; as.w += a0.w;
        }
        if (A.sum_table) sketch_of_sum<RMAX>(P, A, r, h, as);
        if (A.asum) store_worker_sum(A, t, as, w0);
    }
}

// Scalar form: any d, any alignment, any group size.  One thread per coordinate.
__global__ void __launch_bounds__(kThreads)
k_moment_sketch_scalar(const __grid_constant__ Params P, const __grid_constant__ MomentArgs A, uint32_t w0, uint32_t nw) {
    chain_acquire();
    const float b1 = P.beta1, omb1 = 1.0f - P.beta1, rho = P.rho;
    const uint64_t tstride = (uint64_t)P.r * P.cs;
    for (uint32_t j = blockIdx.x * kThreads + threadIdx.x; j < P.d; j += gridDim.x * kThreads) {
        const bool member = A.members && ((A.bitmap[j >> 5] >> (j & 31u)) & 1u);
        float gs = (member && w0 > 0) ? A.gsum[j] : 0.0f;
        float as = 0.0f;                             // sum of a over this launch's workers
        for (uint32_t w = w0; w < w0 + nw; ++w) {
            const uint64_t q = (uint64_t)w * P.d + j;
            const float g = load_grad1(A.grads, q, A.grad_bf16);
            float mm, a;
            if (A.variant == 1) {
                float vv = A.vw[q], vh = A.vhatw[q];
                mm = A.m[q]; a = A.e[q];
                pa_moment(b1, omb1, P.beta2, 1.0f - P.beta2, rho, g, mm, vv, vh, a, member);
                A.vw[q] = vv; A.vhatw[q] = vh;
            } else {
                mm = fmaf(b1, A.m[q], omb1 * g);
                a = fmaf(rho, member ? 0.0f : A.e[q], mm);
            }
            gs += g;
            as += a;
            A.m[q] = mm;
            A.e[q] = a;
            for (uint32_t row = 0; row < P.r && !A.sum_table; ++row) {
                uint32_t b; float s;
                coord_hash(P, P.row_key[row], j, b, s);
                SK_GUARD(b < P.c, kStatusBucket) atomicAdd(A.tables + (uint64_t)w * tstride + (uint64_t)row * P.cs + b, s * a);
            }
        }
        if (member && A.variant == 0) A.gsum[j] = gs;
        if (A.asum) A.asum[j] = (w0 > 0 ? A.asum[j] : 0.0f) + as;
        if (A.sum_table) {
            const float share = as / (float)P.n_all;
            for (uint32_t row = 0; row < P.r; ++row) {
                uint32_t b; float s;
                coord_hash(P, P.row_key[row], j, b, s);
                SK_GUARD(b < P.c, kStatusBucket) atomicAdd(A.sum_table + (uint64_t)row * P.cs + b, s * share);
            }
        }
    }
}

// S = (S^(0) + S^(1) + ... + S^(n-1)) / n_all, workers added in index order (Algorithm 2, master side); with the
// workers partitioned over processes this is the process's share of the mean.
__global__ void __launch_bounds__(kThreads)
k_sum_tables(const __grid_constant__ Params P, const float4* __restrict__ tables, float4* sum) {
    chain_acquire();
    const uint32_t q4 = (P.r * P.cs) >> 2;
    const float fn = (float)P.n_all;
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

// multiprocessors of the current device (queried once per device), for the grids of the helper kernels
int sm_count_of_device() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

#ifdef SK_DEBUG
namespace {
__global__ void k_debug_violation(const __grid_constant__ Params P, uint32_t bit) {
    SK_GUARD(false, bit) { }
}
}  // namespace
#endif

int launch_debug_violation(const Params& P, uint32_t bit, cudaStream_t st) {
#ifdef SK_DEBUG
    k_debug_violation<<<1, 1, 0, st>>>(P, bit);
    return 1;
#else
    (void)P; (void)bit; (void)st;
    return 0;
#endif
}

int launch_zero(void* p, uint64_t bytes, cudaStream_t st, bool chain) {   // bytes must be a multiple of 16
    launch_kernel(chain, k_zero, grid_for(bytes / 16, sm_count_of_device(), 8), kThreads, 0, st, (float4*)p, bytes / 16);
    return 1;
}

int launch_fill_u32(uint32_t* p, uint64_t n, uint32_t value, cudaStream_t st) {
    k_fill_u32<<<grid_for(n, sm_count_of_device(), 8), kThreads, 0, st>>>(p, n, value);
    return 1;
}

int launch_set_bits(const Params& P, const uint32_t* I, uint32_t count, uint32_t* bitmap, cudaStream_t st) {
    if (count == 0) return 0;
    k_set_bits<<<(count + kThreads - 1) / kThreads, kThreads, 0, st>>>(P, I, count, bitmap);
    return 1;
}

int launch_v_materialize(const Params& P, const float* v, const uint32_t* vstamp, uint32_t t, float* out,
                         cudaStream_t st) {
    k_v_materialize<<<grid_for(P.d, sm_count_of_device(), 8), kThreads, 0, st>>>(P, v, vstamp, t, out);
    return 1;
}

int launch_masked_copy(const Params& P, const float* e, const uint32_t* bitmap, uint32_t workers, float* out,
                       cudaStream_t st) {
    const uint64_t total = (uint64_t)workers * P.d;
    k_masked_copy<<<grid_for(total, sm_count_of_device(), 16), kThreads, 0, st>>>(e, bitmap, P.d, total, out);
    return 1;
}

int launch_moment_sketch(const Params& P, const MomentArgs& A, uint32_t w0, uint32_t nw, bool vec, int sm_count,
                         cudaStream_t st) {
    const bool chain = (P.chain & kChainSketch) != 0;
    if (!vec) {
        launch_kernel(chain, k_moment_sketch_scalar, grid_for(P.d, sm_count, 1), kThreads, 0, st, P, A, w0, nw);
        return 1;
    }
    const int grid = grid_for(P.d >> 2, sm_count, 1);    // the caller passes SMs x CTAs per SM
    if (A.variant == 1) {
#define SK_CASE(RR) case RR: launch_kernel(chain, k_moment_sketch_pa_v4<RR>, grid, kThreads, 0, st, P, A, w0, nw); break;
        switch (P.r) {
            SK_CASE(1) SK_CASE(2) SK_CASE(3) SK_CASE(4) SK_CASE(5) SK_CASE(6) SK_CASE(7) SK_CASE(8) SK_CASE(10)
            default: launch_kernel(chain, k_moment_sketch_pa_v4<0>, grid, kThreads, 0, st, P, A, w0, nw); break;
        }
#undef SK_CASE
        return 1;
    }
#define SK_CASE(RR) case RR: launch_kernel(chain, k_moment_sketch_v4<RR>, grid, kThreads, 0, st, P, A, w0, nw); break;
    switch (P.r) {
        SK_CASE(1) SK_CASE(2) SK_CASE(3) SK_CASE(4) SK_CASE(5) SK_CASE(6) SK_CASE(7) SK_CASE(8) SK_CASE(10)
        default: launch_kernel(chain, k_moment_sketch_v4<0>, grid, kThreads, 0, st, P, A, w0, nw); break;
    }
#undef SK_CASE
    return 1;
}

int launch_sum_tables(const Params& P, const float* tables, float* sum, cudaStream_t st) {
    launch_kernel((P.chain & kChainSum) != 0, k_sum_tables, grid_for((P.r * P.cs) >> 2, sm_count_of_device(), 8), kThreads, 0, st, P,
                  (const float4*)tables, (float4*)sum);
    return 1;
}

}  // namespace sk
