// Sparse half of the step: unsketch every coordinate as the median of its r signed bucket values scaled by
// vhat^{-1/2} (Algorithm 3), select the k largest magnitudes (Algorithm 2, "Top-k"), and apply the update with
// the exact worker means on I_t together with the error-feedback reset.
//
// Selection never stores the d estimates: they are recomputed from the L2-resident aggregate sketch in two
// streaming passes (histogram of the top key bits, then emit-above-threshold + collect-threshold-bin), and
// the small candidate list of the threshold bin is resolved exactly by one thread block.
#include "sk_internal.h"
#include "sk_hash.cuh"

namespace sk {

namespace {

constexpr int kThreads = 256;

// lower median of r values held in registers: ascending compare-exchange sort, element (r-1)/2
template <int R>
__device__ __forceinline__ float median_fixed(float (&q)[R]) {
#pragma unroll
    for (int a = 0; a < R - 1; ++a)
#pragma unroll
        for (int b = 0; b < R - 1 - a; ++b) {
            const float lo = fminf(q[b], q[b + 1]), hi = fmaxf(q[b], q[b + 1]);
            q[b] = lo; q[b + 1] = hi;
        }
    return q[(R - 1) / 2];
}

__device__ __forceinline__ float median_any(float* q, uint32_t r) {
    for (uint32_t a = 1; a < r; ++a) {
        const float key = q[a];
        uint32_t b = a;
        while (b > 0 && q[b - 1] > key) { q[b] = q[b - 1]; --b; }
        q[b] = key;
    }
    return q[(r - 1) / 2];
}

__device__ __forceinline__ float scale_est(float med, float vhat) { return __fdiv_rn(med, __fsqrt_rn(vhat)); }

// estimates of the 4 coordinates 4t..4t+3 (vector form, g >= 4)
template <int R>
__device__ __forceinline__ float4 estimate4(const Params& P, const float* __restrict__ sum, uint32_t t,
                                            float4 vh) {
    const uint32_t r = R > 0 ? (uint32_t)R : P.r;
    float qx[R > 0 ? R : (int)kMaxRows], qy[R > 0 ? R : (int)kMaxRows];
    float qz[R > 0 ? R : (int)kMaxRows], qw[R > 0 ? R : (int)kMaxRows];
#pragma unroll
    for (uint32_t row = 0; row < r; ++row) {
        const Quad h = quad_hash(P.row_key[row], P.log2g, P.G, t << 2);
        float4 cch = __ldg((const float4*)(sum + (uint64_t)row * P.cs + h.off));
        cch = quad_gather(h, cch);
        qx[row] = cch.x; qy[row] = cch.y; qz[row] = cch.z; qw[row] = cch.w;
    }
    float4 est;
    if constexpr (R > 0) {
        est.x = median_fixed(qx); est.y = median_fixed(qy); est.z = median_fixed(qz); est.w = median_fixed(qw);
    } else {
        est.x = median_any(qx, r); est.y = median_any(qy, r); est.z = median_any(qz, r); est.w = median_any(qw, r);
    }
    est.x = scale_est(est.x, vh.x); est.y = scale_est(est.y, vh.y);
    est.z = scale_est(est.z, vh.z); est.w = scale_est(est.w, vh.w);
    return est;
}

// scalar form, any group size / alignment
__device__ __forceinline__ float estimate1(const Params& P, const float* __restrict__ sum, uint32_t j, float vh) {
    float q[kMaxRows];
    for (uint32_t row = 0; row < P.r; ++row) {
        uint32_t b; float s;
        coord_hash(P.row_key[row], P.log2g, P.G, j, b, s);
        q[row] = s * __ldg(sum + (uint64_t)row * P.cs + b);
    }
    return scale_est(median_any(q, P.r), vh);
}

__device__ __forceinline__ uint32_t key_of(float est) { return __float_as_uint(est) & 0x7FFFFFFFu; }

// ---- pass A: histogram of key bits 30..19 ------------------------------------------------------------
template <int R, bool VEC>
__global__ void __launch_bounds__(kThreads)
k_unsketch_hist(const __grid_constant__ Params P, const float* __restrict__ sum, const float* __restrict__ vhat,
                uint32_t* hist) {
    __shared__ uint32_t sh[kHistBins];
    for (uint32_t b = threadIdx.x; b < kHistBins; b += kThreads) sh[b] = 0;
    __syncthreads();
    if (VEC) {
        const uint32_t d4 = P.d >> 2;
        for (uint32_t t = blockIdx.x * kThreads + threadIdx.x; t < d4; t += gridDim.x * kThreads) {
            const float4 est = estimate4<R>(P, sum, t, __ldcs((const float4*)vhat + t));
            atomicAdd(&sh[key_of(est.x) >> kHistShift], 1u);
            atomicAdd(&sh[key_of(est.y) >> kHistShift], 1u);
            atomicAdd(&sh[key_of(est.z) >> kHistShift], 1u);
            atomicAdd(&sh[key_of(est.w) >> kHistShift], 1u);
        }
    } else {
        for (uint32_t j = blockIdx.x * kThreads + threadIdx.x; j < P.d; j += gridDim.x * kThreads)
            atomicAdd(&sh[key_of(estimate1(P, sum, j, vhat[j])) >> kHistShift], 1u);
    }
    __syncthreads();
    for (uint32_t b = threadIdx.x; b < kHistBins; b += kThreads)
        if (sh[b]) atomicAdd(&hist[b], sh[b]);
}

// ---- threshold bin: largest b with count(bins >= b) >= k; clears the histogram for the next step ----------
__global__ void __launch_bounds__(1024) k_pick_bin(uint32_t k, uint32_t* hist, Select* sel) {
    __shared__ uint32_t part[1024];
    constexpr uint32_t per = kHistBins / 1024;
    uint32_t mine[per];
    uint32_t s = 0;
    // thread i owns bins in DESCENDING order: its first bin is kHistBins-1 - i*per
    const uint32_t top = kHistBins - 1 - threadIdx.x * per;
#pragma unroll
    for (uint32_t q = 0; q < per; ++q) { mine[q] = hist[top - q]; hist[top - q] = 0; s += mine[q]; }
    part[threadIdx.x] = s;
    __syncthreads();
    for (uint32_t off = 1; off < 1024; off <<= 1) {       // inclusive scan over threads (descending bins)
        const uint32_t add = threadIdx.x >= off ? part[threadIdx.x - off] : 0;
        __syncthreads();
        part[threadIdx.x] += add;
        __syncthreads();
    }
    uint32_t above = part[threadIdx.x] - s;               // keys in bins above this thread's first bin
#pragma unroll
    for (uint32_t q = 0; q < per; ++q) {
        if (above < k && above + mine[q] >= k) {
            sel->bin = top - q;
            sel->need = k - above;
            sel->cnt_out = 0;
            sel->cnt_cand = 0;
        }
        above += mine[q];
    }
}

// ---- pass B: emit indices above the threshold bin, collect the threshold bin's candidates -----------------
// Block-aggregated appends: one atomic per block-iteration and list.
__device__ __forceinline__ void block_append(uint32_t n_out, uint32_t n_cand, uint32_t* cnt_out, uint32_t* cnt_cand,
                                             uint32_t& base_out, uint32_t& base_cand) {
    __shared__ uint32_t warp_tot[kThreads / 32];
    __shared__ uint32_t block_base[2];
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    uint32_t packed = n_out | (n_cand << 16);              // each <= 4 per thread, <= 1024 per block
    uint32_t incl = packed;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= (uint32_t)off) incl += o;
    }
    if (lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    uint32_t before = 0, total = 0;
#pragma unroll
    for (uint32_t q = 0; q < kThreads / 32; ++q) {
        const uint32_t wtot = warp_tot[q];
        if (q < wid) before += wtot;
        total += wtot;
    }
    if (threadIdx.x == 0) {
        block_base[0] = (total & 0xFFFFu) ? atomicAdd(cnt_out, total & 0xFFFFu) : 0u;
        block_base[1] = (total >> 16) ? atomicAdd(cnt_cand, total >> 16) : 0u;
    }
    __syncthreads();
    const uint32_t excl = before + incl - packed;
    base_out = block_base[0] + (excl & 0xFFFFu);
    base_cand = block_base[1] + (excl >> 16);
    __syncthreads();                                       // shared scratch is reused by the next iteration
}

template <int R, bool VEC>
__global__ void __launch_bounds__(kThreads)
k_unsketch_emit(const __grid_constant__ Params P, const float* __restrict__ sum, const float* __restrict__ vhat,
                Select* sel, uint32_t* I_out, Cand* cand) {
    const uint32_t bin = sel->bin;
    const uint32_t items = VEC ? (P.d >> 2) : P.d;
    const uint32_t trips = (items + gridDim.x * kThreads - 1) / (gridDim.x * kThreads);
    for (uint32_t it = 0; it < trips; ++it) {               // uniform trip count: the block scans need all threads
        const uint32_t t = (it * gridDim.x + blockIdx.x) * kThreads + threadIdx.x;
        uint32_t keys[4], idx0 = VEC ? (t << 2) : t, nk = 0;
        if (t < items) {
            if (VEC) {
                const float4 est = estimate4<R>(P, sum, t, __ldcs((const float4*)vhat + t));
                keys[0] = key_of(est.x); keys[1] = key_of(est.y); keys[2] = key_of(est.z); keys[3] = key_of(est.w);
                nk = 4;
            } else {
                keys[0] = key_of(estimate1(P, sum, t, vhat[t]));
                nk = 1;
            }
        }
        uint32_t n_out = 0, n_cand = 0;
#pragma unroll
        for (uint32_t q = 0; q < 4; ++q)
            if (q < nk) {
                const uint32_t b = keys[q] >> kHistShift;
                n_out += b > bin;
                n_cand += b == bin;
            }
        uint32_t po, pc;
        block_append(n_out, n_cand, &sel->cnt_out, &sel->cnt_cand, po, pc);
#pragma unroll
        for (uint32_t q = 0; q < 4; ++q)
            if (q < nk) {
                const uint32_t b = keys[q] >> kHistShift;
                if (b > bin) I_out[po++] = idx0 + q;
                else if (b == bin) { cand[pc].key = keys[q]; cand[pc].idx = idx0 + q; ++pc; }
            }
    }
}

// ---- refinement: of the candidates in the threshold bin take the `need` largest (key, then smaller index) ----
// Radix select, one block, on the 51-bit composite (key bits 18..0 , ~idx): all composites are distinct, so the
// selection is exact and ties in the key go to the smaller index.
__global__ void __launch_bounds__(1024) k_refine(uint32_t k, Select* sel, const Cand* __restrict__ cand,
                                                 uint32_t* I_out) {
    constexpr uint32_t W = 11, BINS = 1u << W;
    __shared__ uint32_t hist[BINS];
    __shared__ uint32_t s_bin, s_need, s_done, s_pos;
    __shared__ uint32_t s_wtot[32];
    const uint32_t ncand = sel->cnt_cand;
    uint32_t need = sel->need;
    const uint64_t lowmask = (1ull << kHistShift) - 1;
    uint64_t prefix = 0;        // composite >> shift must equal prefix for an element to be still undecided
    int shift = 51;
    bool exact = false;         // true once every element with composite >= threshold is known to be wanted
    while (shift > 0 && !exact) {
        const int w = shift >= (int)W ? (int)W : shift;
        shift -= w;
        for (uint32_t b = threadIdx.x; b < BINS; b += blockDim.x) hist[b] = 0;
        __syncthreads();
        for (uint32_t q = threadIdx.x; q < ncand; q += blockDim.x) {
            const Cand cnd = cand[q];
            const uint64_t comp = ((uint64_t)(cnd.key & lowmask) << 32) | (uint32_t)~cnd.idx;
            if ((comp >> (shift + w)) == prefix) atomicAdd(&hist[(comp >> shift) & ((1u << w) - 1u)], 1u);
        }
        __syncthreads();
        {   // scan the bins from the top: the bin in which the running count first reaches `need`
            const int nb = 1 << w;
            const int b0 = nb - 1 - 2 * (int)threadIdx.x, b1 = b0 - 1;
            const uint32_t c0 = b0 >= 0 ? hist[b0] : 0u, c1 = b1 >= 0 ? hist[b1] : 0u;
            const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
            uint32_t incl = c0 + c1;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= (uint32_t)off) incl += o;
            }
            if (lane == 31) s_wtot[wid] = incl;
            __syncthreads();
            uint32_t above = incl - (c0 + c1);
            for (uint32_t q = 0; q < wid; ++q) above += s_wtot[q];
            if (above < need && above + c0 >= need) { s_bin = (uint32_t)b0; s_need = need - above; s_done = (c0 == need - above); }
            above += c0;
            if (above < need && above + c1 >= need) { s_bin = (uint32_t)b1; s_need = need - above; s_done = (c1 == need - above); }
        }
        __syncthreads();
        prefix = (prefix << w) | s_bin;
        need = s_need;
        exact = s_done != 0;
        __syncthreads();
    }
    const uint64_t threshold = prefix << shift;
    if (threadIdx.x == 0) s_pos = sel->cnt_out;
    __syncthreads();
    for (uint32_t q0 = 0; q0 < ncand; q0 += blockDim.x) {
        const uint32_t q = q0 + threadIdx.x;
        bool take = false;
        uint32_t idx = 0;
        if (q < ncand) {
            const Cand cnd = cand[q];
            idx = cnd.idx;
            const uint64_t comp = ((uint64_t)(cnd.key & lowmask) << 32) | (uint32_t)~cnd.idx;
            take = comp >= threshold;
        }
        if (take) {
            const uint32_t pos = atomicAdd(&s_pos, 1u);
            if (pos < k) I_out[pos] = idx;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        sel->cnt_out = s_pos;
        if (s_pos != k) sel->status |= 1u;
    }
}

// ---- apply on I_t: x_j -= lr * mean_w a^(w)_j / sqrt(vhat_j) ; e^(w)_j = 0 ----------------------------------
__global__ void __launch_bounds__(kThreads)
k_apply(const __grid_constant__ Params P, const uint32_t* __restrict__ I, const float* __restrict__ vhat, float* e,
        float* x) {
    const uint32_t q = blockIdx.x * kThreads + threadIdx.x;
    if (q >= P.k) return;
    const uint32_t j = I[q];
    float abar = 0.0f;
#pragma unroll 4
    for (uint32_t w = 0; w < P.n; ++w) abar += e[(uint64_t)w * P.d + j];
    abar = abar / (float)P.n;
    const float delta = scale_est(abar, vhat[j]);
    x[j] = x[j] - P.lr * delta;
    for (uint32_t w = 0; w < P.n; ++w) e[(uint64_t)w * P.d + j] = 0.0f;
}

__global__ void __launch_bounds__(kThreads)
k_estimates(const __grid_constant__ Params P, const float* __restrict__ sum, const float* __restrict__ vhat,
            float* est) {
    for (uint32_t j = blockIdx.x * kThreads + threadIdx.x; j < P.d; j += gridDim.x * kThreads)
        est[j] = estimate1(P, sum, j, vhat[j]);
}

__global__ void __launch_bounds__(kThreads)
k_hash_export(const __grid_constant__ Params P, uint32_t row, uint64_t i0, uint64_t count, uint32_t* idx,
              int8_t* sgn) {
    for (uint64_t t = blockIdx.x * (uint64_t)kThreads + threadIdx.x; t < count; t += (uint64_t)gridDim.x * kThreads) {
        uint32_t b; float s;
        coord_hash(P.row_key[row], P.log2g, P.G, (uint32_t)(i0 + t), b, s);
        idx[t] = b;
        sgn[t] = s < 0.0f ? (int8_t)-1 : (int8_t)1;
    }
}

inline int grid_for(uint64_t items, int sm_count, int per_sm) {
    const uint64_t want = (items + kThreads - 1) / kThreads;
    const uint64_t cap = (uint64_t)sm_count * per_sm;
    return (int)(want < cap ? (want ? want : 1) : cap);
}

}  // namespace

#define SK_ROWS_SWITCH(KERNEL, ...)                                                                        \
    switch (P.r) {                                                                                         \
        case 1: KERNEL<1, true><<<grid, kThreads, 0, st>>>(__VA_ARGS__); break;                            \
        case 2: KERNEL<2, true><<<grid, kThreads, 0, st>>>(__VA_ARGS__); break;                            \
        case 3: KERNEL<3, true><<<grid, kThreads, 0, st>>>(__VA_ARGS__); break;                            \
        case 4: KERNEL<4, true><<<grid, kThreads, 0, st>>>(__VA_ARGS__); break;                            \
        case 5: KERNEL<5, true><<<grid, kThreads, 0, st>>>(__VA_ARGS__); break;                            \
        case 6: KERNEL<6, true><<<grid, kThreads, 0, st>>>(__VA_ARGS__); break;                            \
        case 7: KERNEL<7, true><<<grid, kThreads, 0, st>>>(__VA_ARGS__); break;                            \
        case 8: KERNEL<8, true><<<grid, kThreads, 0, st>>>(__VA_ARGS__); break;                            \
        case 10: KERNEL<10, true><<<grid, kThreads, 0, st>>>(__VA_ARGS__); break;                          \
        default: KERNEL<0, true><<<grid, kThreads, 0, st>>>(__VA_ARGS__); break;                           \
    }

int launch_unsketch_hist(const Params& P, const float* sum, const float* vhat, uint32_t* hist, bool vec,
                         int sm_count, cudaStream_t st) {
    if (!vec) {
        k_unsketch_hist<0, false><<<grid_for(P.d, sm_count, 4), kThreads, 0, st>>>(P, sum, vhat, hist);
        return 1;
    }
    const int grid = grid_for(P.d >> 2, sm_count, 4);
    SK_ROWS_SWITCH(k_unsketch_hist, P, sum, vhat, hist)
    return 1;
}

int launch_pick_bin(const Params& P, uint32_t* hist, Select* sel, cudaStream_t st) {
    k_pick_bin<<<1, 1024, 0, st>>>(P.k, hist, sel);
    return 1;
}

int launch_unsketch_emit(const Params& P, const float* sum, const float* vhat, Select* sel, uint32_t* I_out,
                         Cand* cand, bool vec, int sm_count, cudaStream_t st) {
    if (!vec) {
        k_unsketch_emit<0, false><<<grid_for(P.d, sm_count, 4), kThreads, 0, st>>>(P, sum, vhat, sel, I_out, cand);
        return 1;
    }
    const int grid = grid_for(P.d >> 2, sm_count, 4);
    SK_ROWS_SWITCH(k_unsketch_emit, P, sum, vhat, sel, I_out, cand)
    return 1;
}

int launch_refine(const Params& P, Select* sel, const Cand* cand, uint32_t* I_out, cudaStream_t st) {
    k_refine<<<1, 1024, 0, st>>>(P.k, sel, cand, I_out);
    return 1;
}

int launch_apply(const Params& P, const uint32_t* I, const float* vhat, float* e, float* x, cudaStream_t st) {
    k_apply<<<(P.k + kThreads - 1) / kThreads, kThreads, 0, st>>>(P, I, vhat, e, x);
    return 1;
}

int launch_estimates(const Params& P, const float* sum, const float* vhat, float* est, cudaStream_t st) {
    k_estimates<<<grid_for(P.d, 148, 8), kThreads, 0, st>>>(P, sum, vhat, est);
    return 1;
}

int launch_hash_export(const Params& P, uint32_t row, uint64_t i0, uint64_t count, uint32_t* idx, int8_t* sgn,
                       cudaStream_t st) {
    k_hash_export<<<grid_for(count, 148, 8), kThreads, 0, st>>>(P, row, i0, count, idx, sgn);
    return 1;
}

}  // namespace sk
