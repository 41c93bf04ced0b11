// Sparse half of the step: unsketch every coordinate as the median of its r signed bucket values scaled by
// vhat^{-1/2} (Algorithm 3), select the k largest magnitudes (Algorithm 2, "Top-k"), and apply the update with
// the exact worker means on I_t together with the error-feedback reset.
//
// Selection: (A) one pass over the coordinates computes every ranking key from the L2-resident aggregate sketch,
// stores it (4 bytes per coordinate) and histograms key bits 30..19; (B) one pass over the stored keys emits the
// indices above the threshold bin, collects the threshold bin's candidates and histograms their next 12 key
// bits; (C) the candidates are split once more and (D) the handful that share the first 24 key bits with the
// threshold are resolved exactly by one block.
// key = bit pattern of |estimate| (monotone for finite non-negative floats); ties go to the smaller index.
#include "sk_internal.h"
#include "sk_hash.cuh"
#include "sk_moment.cuh"

namespace sk {

namespace {

constexpr int kThreads = 256;

// ---- median of r values held in registers (lower median for even r) ----------------------------------------
__device__ __forceinline__ float med3(float x, float y, float z) {
    return fmaxf(fminf(x, y), fminf(fmaxf(x, y), z));
}

template <int R>
__device__ __forceinline__ float median_fixed(float (&q)[R]) {
    if constexpr (R == 1) return q[0];
    else if constexpr (R == 2) return fminf(q[0], q[1]);
    else if constexpr (R == 3) return med3(q[0], q[1], q[2]);
    else if constexpr (R == 5) {
        // the median of five is the median of: the larger of the two pair-minima, the smaller of the two
        // pair-maxima, and the fifth element
        const float f = fmaxf(fminf(q[0], q[1]), fminf(q[2], q[3]));
        const float g = fminf(fmaxf(q[0], q[1]), fmaxf(q[2], q[3]));
        return med3(q[4], f, g);
    } else {
        // bubble passes until position (R-1)/2 is final
#pragma unroll
        for (int a = 0; a < R - (R - 1) / 2; ++a)
#pragma unroll
            for (int b = 0; b < R - 1 - a; ++b) {
                const float lo = fminf(q[b], q[b + 1]), hi = fmaxf(q[b], q[b + 1]);
                q[b] = lo; q[b + 1] = hi;
            }
        return q[(R - 1) / 2];
    }
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

// est = med / sqrt(vhat), both operations correctly rounded (this is the value the selection is defined on)
__device__ __forceinline__ float scale_est(float med, float vhat) { return __fdiv_rn(med, __fsqrt_rn(vhat)); }
__device__ __forceinline__ uint32_t key_of(float est) { return __float_as_uint(est) & 0x7FFFFFFFu; }

// Ranking key of a coordinate: the bit pattern of |med * rsqrt(vhat)|.  The hardware reciprocal square root is
// within 2 ulp, so the key is within a few ulp (< 4e-7 relative) of the correctly rounded estimate -- two orders
// of magnitude inside the tolerance within which the selected set is defined -- and it is a deterministic
// function of (med, vhat), which is all the selection needs.  Denormal vhat takes the exact path.
__device__ __forceinline__ uint32_t key_rank(float med, float vhat) {
    float rs;                                         // one MUFU: vhat is a normal number on this branch
    asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(rs) : "f"(vhat));
    return key_of(vhat > 1e-30f ? med * rs : scale_est(med, vhat));
}

// medians of the 4 coordinates 4t..4t+3 (vector form, g >= 4).  All lanes of the warp call this together.
template <int R>
__device__ __forceinline__ float4 medians4(const Params& P, const float* __restrict__ sum, uint32_t t) {
    constexpr int RMAX = R > 0 ? R : (int)kMaxRows;
    const uint32_t r = R > 0 ? (uint32_t)R : P.r;
    Quad h[RMAX];
    quad_hashes<RMAX>(P, r, t, h);
    float qx[RMAX], qy[RMAX], qz[RMAX], qw[RMAX];
#pragma unroll
    for (uint32_t row = 0; row < (uint32_t)RMAX; ++row)
        if (row < r) {
            float4 cch = make_float4(0.f, 0.f, 0.f, 0.f);
            SK_GUARD(h[row].off + 4u <= P.cs, kStatusBucket) cch = __ldg((const float4*)(sum + (uint64_t)row * P.cs + h[row].off));
            cch = quad_gather(h[row], cch);
            qx[row] = cch.x; qy[row] = cch.y; qz[row] = cch.z; qw[row] = cch.w;
        }
    float4 med;
    if constexpr (R > 0) {
        med.x = median_fixed(qx); med.y = median_fixed(qy); med.z = median_fixed(qz); med.w = median_fixed(qw);
    } else {
        med.x = median_any(qx, r); med.y = median_any(qy, r); med.z = median_any(qz, r); med.w = median_any(qw, r);
    }
    return med;
}

// scalar form, any group size / alignment
__device__ __forceinline__ float median1(const Params& P, const float* __restrict__ sum, uint32_t j) {
    float q[kMaxRows];
    for (uint32_t row = 0; row < P.r; ++row) {
        uint32_t b; float s;
        coord_hash(P, P.row_key[row], j, b, s);
        q[row] = 0.0f;
        SK_GUARD(b < P.c, kStatusBucket) q[row] = s * __ldg(sum + (uint64_t)row * P.cs + b);
    }
    return median_any(q, P.r);
}

// a 16-byte global load that stays where it is written (the compiler would otherwise move it down to its first use)
template <typename T4>
__device__ __forceinline__ T4 ldg128_here(const T4* p) {
    uint32_t a, b, c, d;
    asm volatile("ld.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "l"(p) : "memory");
    T4 out;
    uint32_t* w = reinterpret_cast<uint32_t*>(&out);
    w[0] = a; w[1] = b; w[2] = c; w[3] = d;
    return out;
}

// one count in a shared-memory histogram of kHistBins bins (the bin is checked in the debug build)
__device__ __forceinline__ void hist_add(const Params& P, uint32_t* sh, uint32_t bin) {
    SK_GUARD(bin < kHistBins, kStatusBin) atomicAdd(&sh[bin], 1u);
}

// ---- pass A: ranking keys of all coordinates (stored) + histogram of key bits 30..19 -----------------------------
// The pass streams vhat anyway, so it also carries the master's update of v and vhat on I_{t-1} (Algorithm 2):
// where the membership bitmap is set, v and vhat are brought up to date from the gradient sums the moment kernel
// left in gsum, before vhat is used.  A.members = 0 turns that off (a re-run of the selection must not repeat it).
__device__ __forceinline__ void update_member(const Params& P, const MomentArgs& A, float gsum, float& v, uint32_t& stamp,
                                              float& vh) {
    v = second_moment_value(P, v, stamp, A.step, gsum);
    stamp = A.step;
    vh = fmaxf(vh, v);
}

template <int R, bool VEC>
__global__ void __launch_bounds__(kThreads)
k_unsketch_hist(const __grid_constant__ Params P, const __grid_constant__ MomentArgs A, const float* __restrict__ sum,
                uint32_t* keys, uint32_t* hist) {
    __shared__ uint32_t sh[kHistBins];
    for (uint32_t b = threadIdx.x; b < kHistBins; b += kThreads) sh[b] = 0;
    chain_acquire();                // nothing above touches global memory
    __syncthreads();
    const uint32_t items = VEC ? (P.d >> 2) : P.d;
    const uint32_t trips = (items + gridDim.x * kThreads - 1) / (gridDim.x * kThreads);
    for (uint32_t it = 0; it < trips; ++it) {                // uniform trip count: warps stay whole
        const uint32_t t = (it * gridDim.x + blockIdx.x) * kThreads + threadIdx.x;
        const bool live = t < items;
        const uint32_t tc = live ? t : items - 1;
        if (VEC) {
            const float4 med = medians4<R>(P, sum, tc);
            if (live && A.variant == 1) {                     // parameter averaging: U(S) takes no vhat (Algorithm 1)
                uint4 k4;
                k4.x = key_of(med.x); k4.y = key_of(med.y); k4.z = key_of(med.z); k4.w = key_of(med.w);
                ((uint4*)keys)[t] = k4;
                hist_add(P, sh, k4.x >> kHistShift); hist_add(P, sh, k4.y >> kHistShift);
                hist_add(P, sh, k4.z >> kHistShift); hist_add(P, sh, k4.w >> kHistShift);
            } else if (live) {
                float4 vh = ((const float4*)A.vhat)[t];
                const uint32_t mask = A.members ? ((__ldg(A.bitmap + (t >> 3)) >> ((t & 7u) * 4u)) & 0xFu) : 0u;
                if (mask) {
                    const float4 gs = ((const float4*)A.gsum)[t];
                    float4 vv = ((const float4*)A.v)[t];
                    uint4 vs = ((const uint4*)A.vstamp)[t];
                    if (mask & 1u) update_member(P, A, gs.x, vv.x, vs.x, vh.x);
                    if (mask & 2u) update_member(P, A, gs.y, vv.y, vs.y, vh.y);
                    if (mask & 4u) update_member(P, A, gs.z, vv.z, vs.z, vh.z);
                    if (mask & 8u) update_member(P, A, gs.w, vv.w, vs.w, vh.w);
                    ((float4*)A.v)[t] = vv;
                    ((uint4*)A.vstamp)[t] = vs;
                    ((float4*)A.vhat)[t] = vh;
                    ((float4*)A.gsum)[t] = make_float4(0.f, 0.f, 0.f, 0.f);   // consumed: the sums start from zero next step
                }
                uint4 k4;
                k4.x = key_rank(med.x, vh.x); k4.y = key_rank(med.y, vh.y);
                k4.z = key_rank(med.z, vh.z); k4.w = key_rank(med.w, vh.w);
                ((uint4*)keys)[t] = k4;
                hist_add(P, sh, k4.x >> kHistShift); hist_add(P, sh, k4.y >> kHistShift);
                hist_add(P, sh, k4.z >> kHistShift); hist_add(P, sh, k4.w >> kHistShift);
            }
        } else if (live && A.variant == 1) {
            const uint32_t key = key_of(median1(P, sum, t));
            keys[t] = key;
            hist_add(P, sh, key >> kHistShift);
        } else if (live) {
            float vh = A.vhat[t];
            if (A.members && ((A.bitmap[t >> 5] >> (t & 31u)) & 1u)) {
                float vv = A.v[t];
                uint32_t vs = A.vstamp[t];
                update_member(P, A, A.gsum[t], vv, vs, vh);
                A.gsum[t] = 0.0f;
                A.v[t] = vv; A.vstamp[t] = vs; A.vhat[t] = vh;
            }
            const uint32_t key = key_rank(median1(P, sum, t), vh);
            keys[t] = key;
            hist_add(P, sh, key >> kHistShift);
        }
    }
    __syncthreads();
    for (uint32_t b = threadIdx.x; b < kHistBins; b += kThreads)
        if (sh[b]) atomicAdd(&hist[b], sh[b]);
}

// ---- pass A for the windowed hash family ---------------------------------------------------------------------------
// A unit of 1024 coordinates reads, in every row, only its panel's window of the aggregate sketch.  A block walks a
// run of units in panel-major order (the order the sketch kernel uses), keeps the current panel's windows (r x 32L
// floats) and the unit's r x 32 group hashes in shared memory, and every thread takes one coordinate quad per unit:
// r 16-byte shared-memory reads, sign and xor-permutation undone in registers, median, key, histogram.  Against the
// general kernel this drops the per-quad hash exchange by shuffles and the L2 gathers.
template <int R>
__global__ void __launch_bounds__(kThreads, 5)
k_unsketch_hist_win(const __grid_constant__ Params P, const __grid_constant__ MomentArgs A, const float* __restrict__ sum,
                    uint32_t* keys, uint32_t* hist, uint32_t units_total, uint32_t tbig, uint32_t rem) {
    extern __shared__ __align__(16) uint32_t dyn[];
    constexpr int RMAX = R > 0 ? R : (int)kMaxRows;
    const uint32_t r = R > 0 ? (uint32_t)R : P.r;
    const uint32_t cw = P.win_cw;
    uint32_t* sh = dyn;                                            // [4096] histogram
    uint2* hsh = (uint2*)(sh + kHistBins);                         // [2][r][32]: x = line*32 | perm, y = sign as +-1.0f
    float* win = (float*)(hsh + 2u * r * kGroupsPerUnit);          // [r][cw]: the panel's window of every row
    const uint32_t tid = threadIdx.x;
    chain_release();
    for (uint32_t b = tid; b < kHistBins; b += kThreads) sh[b] = 0;
    const uint32_t s_begin = (uint32_t)((uint64_t)units_total * blockIdx.x / gridDim.x);
    const uint32_t s_end = (uint32_t)((uint64_t)units_total * (blockIdx.x + 1) / gridDim.x);
    const uint32_t d4 = P.d >> 2;
    const uint32_t sg = tid >> 3, o = (tid & 7u) * 4u;             // this thread's group inside the unit, offset inside it
    const uint32_t bm_words = (P.d + 31u) >> 5;

    auto fill_hashes = [&](uint32_t unit, uint32_t buf) {
        for (uint32_t hq = tid; hq < r * kGroupsPerUnit; hq += kThreads) {
            const uint32_t row = hq >> 5, s = hq & 31u;
            const GroupHash gh = group_from_draw(P, stream(P.row_key[row & (kMaxRows - 1u)], (uint64_t)unit * kGroupsPerUnit + s + 1));
            hsh[buf * r * kGroupsPerUnit + hq] = make_uint2(gh.base | gh.perm, 0x3F800000u | (gh.sign << 31));
        }
    };
    auto load_windows = [&](uint32_t panel) {
        for (uint32_t q = tid; q < r * (cw >> 2); q += kThreads) {
            const uint32_t row = q / (cw >> 2), c4 = q - row * (cw >> 2);
            ((float4*)win)[q] = __ldg((const float4*)(sum + (uint64_t)row * P.cs + (uint64_t)panel * cw) + c4);
        }
    };

    // this thread's four membership bits of I_{t-1} in a unit (0 where the pass does not update v and vhat)
    const bool members = A.variant != 1 && A.members;
    auto member_bits = [&](uint32_t unit) -> uint32_t {
        const uint32_t word = unit * kGroupsPerUnit + sg;
        return (members && word < bm_words && unit * kQuadsPerUnit + tid < d4) ? (__ldg(A.bitmap + word) >> o) & 0xFu : 0u;
    };

    UnitWalk walk{P.win_panels, tbig, rem, 0u, 0u};
    uint32_t mask_ahead = 0;
    if (s_begin < s_end) {
        walk.seek(s_begin);
        fill_hashes(walk.unit(), 0u);
    }
    chain_acquire();                // nothing above touches global memory
    if (s_begin < s_end) {
        load_windows(walk.panel);
        mask_ahead = member_bits(walk.unit());
    }
    __syncthreads();
    for (uint32_t s = s_begin; s < s_end; ++s) {
        const uint32_t buf = (s - s_begin) & 1u;
        const uint32_t unit = walk.unit(), panel = walk.panel;
        const bool have_next = s + 1 < s_end;
        walk.next();
        // The membership word was fetched one unit ahead, so the loads of a member's gsum, v and stamp can be issued
        // here, with the load of vhat, and the row work below hides their latency.
        const uint32_t mask = mask_ahead;
        const uint32_t t = unit * kQuadsPerUnit + tid;
        float4 gs = make_float4(0.f, 0.f, 0.f, 0.f), vv = gs;
        uint4 vs = make_uint4(0u, 0u, 0u, 0u);
        float4 vh = make_float4(1.f, 1.f, 1.f, 1.f);
        if (t < d4 && A.variant != 1) vh = ldg128_here<float4>((const float4*)A.vhat + t);
        if (mask) {
            gs = ldg128_here<float4>((const float4*)A.gsum + t);
            vv = ldg128_here<float4>((const float4*)A.v + t);
            vs = ldg128_here<uint4>((const uint4*)A.vstamp + t);
        }
        mask_ahead = have_next ? member_bits(walk.unit()) : 0u;
        if (have_next) fill_hashes(walk.unit(), buf ^ 1u);
        const uint2* hs = hsh + buf * r * kGroupsPerUnit + sg;
        if (t < d4) {
            float qx[RMAX], qy[RMAX], qz[RMAX], qw[RMAX];
#pragma unroll
            for (uint32_t row = 0; row < (uint32_t)RMAX; ++row)
                if (row < r) {
                    const uint2 h = hs[row * kGroupsPerUnit];
                    const uint32_t woff = (h.x ^ o) & ~3u;
                    // coordinate l of the quad sits at element l xor p3 of the chunk: bit 1 of p3 is taken by the
                    // address (which 8-byte half is read first), bit 0 by a swap; h.y is the group's sign (+-1.0f)
                    float2 c01 = make_float2(0.f, 0.f), c23 = c01;
                    SK_GUARD(woff + 4u <= cw, kStatusWindow) {
                        const float* chunk = win + row * cw + woff;
                        c01 = *(const float2*)(chunk + (h.x & 2u));
                        c23 = *(const float2*)(chunk + ((h.x & 2u) ^ 2u));
                    }
                    if (h.x & 1u) { float u = c01.x; c01.x = c01.y; c01.y = u; u = c23.x; c23.x = c23.y; c23.y = u; }
                    const float sg = __uint_as_float(h.y);
                    qx[row] = sg * c01.x; qy[row] = sg * c01.y; qz[row] = sg * c23.x; qw[row] = sg * c23.y;
                }
            float4 med;
            if constexpr (R > 0) {
                med.x = median_fixed(qx); med.y = median_fixed(qy); med.z = median_fixed(qz); med.w = median_fixed(qw);
            } else {
                med.x = median_any(qx, r); med.y = median_any(qy, r); med.z = median_any(qz, r); med.w = median_any(qw, r);
            }
            uint4 k4;
            if (A.variant == 1) {                                  // parameter averaging: U(S) takes no vhat (Algorithm 1)
                k4.x = key_of(med.x); k4.y = key_of(med.y); k4.z = key_of(med.z); k4.w = key_of(med.w);
            } else {
                if (mask) {
                    if (mask & 1u) update_member(P, A, gs.x, vv.x, vs.x, vh.x);
                    if (mask & 2u) update_member(P, A, gs.y, vv.y, vs.y, vh.y);
                    if (mask & 4u) update_member(P, A, gs.z, vv.z, vs.z, vh.z);
                    if (mask & 8u) update_member(P, A, gs.w, vv.w, vs.w, vh.w);
                    ((float4*)A.v)[t] = vv;
                    ((uint4*)A.vstamp)[t] = vs;
                    ((float4*)A.vhat)[t] = vh;
                    ((float4*)A.gsum)[t] = make_float4(0.f, 0.f, 0.f, 0.f);   // consumed: the sums start from zero next step
                }
                k4.x = key_rank(med.x, vh.x); k4.y = key_rank(med.y, vh.y);
                k4.z = key_rank(med.z, vh.z); k4.w = key_rank(med.w, vh.w);
            }
            ((uint4*)keys)[t] = k4;
            hist_add(P, sh, k4.x >> kHistShift); hist_add(P, sh, k4.y >> kHistShift);
            hist_add(P, sh, k4.z >> kHistShift); hist_add(P, sh, k4.w >> kHistShift);
        }
        __syncthreads();            // everyone is done with this unit's hashes (and with the windows, if the panel ends)
        if (have_next && walk.panel != panel) {
            load_windows(walk.panel);
            __syncthreads();
        }
    }
    __syncthreads();
    for (uint32_t b = tid; b < kHistBins; b += kThreads)
        if (sh[b]) atomicAdd(&hist[b], sh[b]);
}

// ---- threshold bin of a 4096-bin histogram: largest b with count(bins >= b) >= need ------------------------
// level 0: need = k, result -> sel->bin/need, counters reset.  level 1: need = sel->need, result -> bin2/need2.
__global__ void __launch_bounds__(1024) k_pick_bin(uint32_t k, uint32_t* hist, Select* sel, int level) {
    __shared__ uint32_t part[1024];
    constexpr uint32_t per = kHistBins / 1024;
    chain_acquire();
    const uint32_t need = level == 0 ? k : sel->need;
    uint32_t mine[per];
    uint32_t s = 0;
    const uint32_t top = kHistBins - 1 - threadIdx.x * per;   // thread i owns `per` bins in descending order
#pragma unroll
    for (uint32_t q = 0; q < per; ++q) { mine[q] = hist[top - q]; hist[top - q] = 0; s += mine[q]; }
    // inclusive scan of the 1024 per-thread counts: inside each warp by shuffles, then over the 32 warp totals
    const uint32_t lane = threadIdx.x & 31u, wid = threadIdx.x >> 5;
    uint32_t incl = s;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= (uint32_t)off) incl += o;
    }
    if (lane == 31u) part[wid] = incl;
    __syncthreads();
    if (wid == 0) {
        uint32_t w = part[lane];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, w, off);
            if (lane >= (uint32_t)off) w += o;
        }
        part[32u + lane] = w;                                 // inclusive totals of warps 0..lane
    }
    __syncthreads();
    uint32_t above = incl - s + (wid ? part[32u + wid - 1u] : 0u);
#pragma unroll
    for (uint32_t q = 0; q < per; ++q) {
        if (above < need && above + mine[q] >= need) {
            if (level == 0) {
                sel->bin = top - q; sel->need = need - above;
                sel->cnt_out = 0; sel->cnt_cand = 0; sel->cnt_cand2 = 0;
            } else {
                sel->bin2 = top - q; sel->need2 = need - above;
            }
        }
        above += mine[q];
    }
}

// Block-aggregated appends to two lists: one atomic per block-iteration and list.
__device__ __forceinline__ void block_append(uint32_t n_a, uint32_t n_b, uint32_t* cnt_a, uint32_t* cnt_b,
                                             uint32_t& base_a, uint32_t& base_b) {
    __shared__ uint32_t warp_tot[kThreads / 32];
    __shared__ uint32_t block_base[2];
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t packed = n_a | (n_b << 16);              // each <= 16 per thread, <= 4096 per block
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
        block_base[0] = (total & 0xFFFFu) ? atomicAdd(cnt_a, total & 0xFFFFu) : 0u;
        block_base[1] = (total >> 16) ? atomicAdd(cnt_b, total >> 16) : 0u;
    }
    __syncthreads();
    const uint32_t excl = before + incl - packed;
    base_a = block_base[0] + (excl & 0xFFFFu);
    base_b = block_base[1] + (excl >> 16);
    __syncthreads();                                        // the shared scratch is reused by the next call
}

// ---- pass B over the stored keys: emit above the threshold bin, collect the threshold bin, histogram its next
// 12 key bits ---------------------------------------------------------------------------------------------------
// Appends go through per-warp staging buffers in shared memory: a warp reserves room in the global list with one
// atomic per kWarpBuf entries and copies them out coalesced, so the pass needs no block-wide barrier per tile.
constexpr uint32_t kWarpBuf = 128;

template <typename T>
__device__ __forceinline__ void warp_flush(const Params& P, T* buf, uint32_t& fill, uint32_t* counter, T* list, uint32_t cap) {
    __syncwarp();
    const uint32_t lane = threadIdx.x & 31u;
    uint32_t base = 0;
    if (lane == 0 && fill) base = atomicAdd(counter, fill);
    base = __shfl_sync(0xFFFFFFFFu, base, 0);
    for (uint32_t q = lane; q < fill; q += 32)
        SK_GUARD(base + q < cap, kStatusListPos) list[base + q] = buf[q];
    __syncwarp();
    fill = 0;
}

// where this lane's `mine` entries of the warp's `total` go: into the staging buffer (flushed first if they do not
// fit), or straight into the list when one tile yields more than a buffer holds
// (a tile that yields more than a buffer holds goes straight into the list: the debug build checks the reserved
// range against the capacity and diverts an overflowing warp into its staging buffer, whose flush is checked too)
template <typename T>
__device__ __forceinline__ T* warp_reserve(const Params& P, T* buf, uint32_t& fill, uint32_t* counter, T* list, uint32_t cap,
                                           uint32_t total, uint32_t excl) {
    if (total == 0) return buf;
    if (fill + total > kWarpBuf) warp_flush(P, buf, fill, counter, list, cap);
    if (total > kWarpBuf) {
        uint32_t base = 0;
        if ((threadIdx.x & 31u) == 0) base = atomicAdd(counter, total);
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        if (in_bounds(base + total <= cap, P.status, kStatusListPos)) return list + base + excl;
        return buf;          // debug build only: the entries of this tile are dropped (two lanes may share a slot)
    }
    T* dst = buf + fill + excl;
    fill += total;
    return dst;
}

template <bool VEC>
__global__ void __launch_bounds__(kThreads)
k_emit(const __grid_constant__ Params P, const uint32_t* __restrict__ keys, const uint32_t* __restrict__ idx_map, Select* sel,
       uint32_t* I_out, Cand* cand, uint32_t* hist2, uint4* clear, uint32_t clear_n4) {
    // clear (may be nullptr): clear_n4 16-byte words that this pass also sets to zero -- the membership bitmap of
    // I_{t-1}, which the key pass was the last to read and the update of x will mark with I_t
    // P.d keys, the P.k largest wanted: I_out holds P.k entries, the candidate list P.d
    const uint32_t d = P.d;
    // idx_map (scalar form only): keys[t] belongs to coordinate idx_map[t] instead of t (second round on a candidate list)
    __shared__ uint32_t sh2[kHistBins];
    __shared__ uint32_t wb_out[kThreads / 32][kWarpBuf];
    __shared__ Cand wb_cand[kThreads / 32][kWarpBuf];
    chain_release();
    for (uint32_t b = threadIdx.x; b < kHistBins; b += kThreads) sh2[b] = 0;
    chain_acquire();                // nothing above touches global memory
    __syncthreads();
    if (clear)
        for (uint32_t t = blockIdx.x * kThreads + threadIdx.x; t < clear_n4; t += gridDim.x * kThreads)
            clear[t] = make_uint4(0u, 0u, 0u, 0u);
    const uint32_t bin = sel->bin;
    const uint32_t thr_lo = bin << kHistShift;                  // first key of the threshold bin
    const uint32_t thr_hi = (bin + 1u) << kHistShift;           // first key above it (2^31 for the last bin: no key)
    const uint32_t lane = threadIdx.x & 31u, wid = threadIdx.x >> 5;
    uint32_t fill_out = 0, fill_cand = 0;                       // the same in every lane of the warp
    constexpr uint32_t U = 4;                                   // key loads in flight per thread
    const uint32_t items = VEC ? (d >> 2) : d;
    const uint32_t tile = U * kThreads;
    const uint32_t trips = (items + gridDim.x * tile - 1) / (gridDim.x * tile);
    for (uint32_t it = 0; it < trips; ++it) {                   // uniform trip count: warps stay whole
        const uint32_t t0 = (it * gridDim.x + blockIdx.x) * tile + threadIdx.x;
        uint32_t kq[U][4], nk[U];
#pragma unroll
        for (uint32_t u = 0; u < U; ++u) {
            const uint32_t t = t0 + u * kThreads;
            nk[u] = 0;
            if (t < items) {
                if (VEC) {
                    const uint4 k4 = __ldcs((const uint4*)keys + t);
                    kq[u][0] = k4.x; kq[u][1] = k4.y; kq[u][2] = k4.z; kq[u][3] = k4.w;
                    nk[u] = 4;
                } else {
                    kq[u][0] = keys[t];
                    nk[u] = 1;
                }
            }
        }
        // counting is branch-free: almost every key is below the threshold bin.  The vector form keeps the outcome
        // of its sixteen comparisons as two bit masks (bit 4u+q), so that the append below visits the hits only.
        uint32_t n_out = 0, n_ge = 0, m_out = 0, m_ge = 0;
#pragma unroll
        for (uint32_t u = 0; u < U; ++u)
            if (nk[u]) {
#pragma unroll
                for (uint32_t q = 0; q < 4; ++q)
                    if (VEC) {
                        m_out |= (uint32_t)(kq[u][q] >= thr_hi) << (4u * u + q);
                        m_ge |= (uint32_t)(kq[u][q] >= thr_lo) << (4u * u + q);
                    } else if (q == 0) {
                        n_out += kq[u][q] >= thr_hi;
                        n_ge += kq[u][q] >= thr_lo;
                    }
            }
        if (VEC) { n_out = (uint32_t)__popc(m_out); n_ge = (uint32_t)__popc(m_ge); }
        const uint32_t n_cand = n_ge - n_out;
        const uint32_t packed = n_out | (n_cand << 16);         // each <= 16 per thread, <= 512 per warp
        uint32_t incl = packed;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= (uint32_t)off) incl += o;
        }
        const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 31);
        if (total == 0) continue;
        const uint32_t excl = incl - packed;
        uint32_t* po = warp_reserve(P, wb_out[wid], fill_out, &sel->cnt_out, I_out, P.k, total & 0xFFFFu, excl & 0xFFFFu);
        Cand* pc = warp_reserve(P, wb_cand[wid], fill_cand, &sel->cnt_cand, cand, P.d, total >> 16, excl >> 16);
        if (packed == 0) continue;                              // this lane has nothing to append
        if (VEC) {
            // one iteration per hit, in the order of the bits (u-major): an index above the bin needs no key, a
            // candidate reads its key back (keys[idx]: the vector form has no index map)
            for (uint32_t m = m_ge; m; m &= m - 1u) {
                const uint32_t b = (uint32_t)__ffs((int)m) - 1u;
                const uint32_t idx = ((t0 + (b >> 2) * kThreads) << 2) + (b & 3u);
                if ((m_out >> b) & 1u) {
                    *po++ = idx;
                } else {
                    const uint32_t key = __ldg(keys + idx);
                    hist_add(P, sh2, (key >> 7) & (kHistBins - 1u));
                    pc->key = key; pc->idx = idx; ++pc;
                }
            }
            continue;
        }
#pragma unroll
        for (uint32_t u = 0; u < U; ++u) {
            if (!nk[u]) continue;
            const uint32_t t = t0 + u * kThreads;
            const uint32_t idx0 = VEC ? (t << 2) : (idx_map ? idx_map[t] : t);
#pragma unroll
            for (uint32_t q = 0; q < 4; ++q)
                if (VEC || q == 0) {
                    const uint32_t key = kq[u][q];
                    if (key >= thr_hi) *po++ = idx0 + q;
                    else if (key >= thr_lo) {
                        hist_add(P, sh2, (key >> 7) & (kHistBins - 1u));
                        pc->key = key; pc->idx = idx0 + q; ++pc;
                    }
                }
        }
    }
    warp_flush(P, wb_out[wid], fill_out, &sel->cnt_out, I_out, P.k);
    warp_flush(P, wb_cand[wid], fill_cand, &sel->cnt_cand, cand, P.d);
    __syncthreads();
    for (uint32_t b = threadIdx.x; b < kHistBins; b += kThreads)
        if (sh2[b]) atomicAdd(&hist2[b], sh2[b]);
}

// ---- pass C over the candidates: first 24 key bits above the threshold -> emit, equal -> second list ----------
__global__ void __launch_bounds__(kThreads)
k_split_candidates(const __grid_constant__ Params P, Select* sel, const Cand* __restrict__ cand, uint32_t* I_out, Cand* cand2) {
    chain_acquire();
    const uint32_t ncand = sel->cnt_cand;
    const uint32_t thr = (sel->bin << kHistBits) | sel->bin2;          // leading 24 bits of the threshold key
    const uint32_t trips = (ncand + gridDim.x * kThreads - 1) / (gridDim.x * kThreads);
    for (uint32_t it = 0; it < trips; ++it) {
        const uint32_t q = (it * gridDim.x + blockIdx.x) * kThreads + threadIdx.x;
        Cand cnd{0u, 0u};
        uint32_t n_out = 0, n_eq = 0;
        if (q < ncand) {
            cnd = cand[q];
            const uint32_t lead = cnd.key >> 7;
            n_out = lead > thr;
            n_eq = lead == thr;
        }
        uint32_t po, pc;
        block_append(n_out, n_eq, &sel->cnt_out, &sel->cnt_cand2, po, pc);
        if (n_out) SK_GUARD(po < P.k, kStatusListPos) I_out[po] = cnd.idx;
        if (n_eq) SK_GUARD(pc < P.d, kStatusListPos) cand2[pc] = cnd;
    }
}

// ---- pass D: of the second list take the `need2` largest by (last 7 key bits, then smaller index) -------------
// Radix select by one block on the 39-bit composite (key & 127, ~idx): all composites are distinct, so the
// selection is exact and equal keys go to the smaller index.
__global__ void __launch_bounds__(1024) k_resolve(const __grid_constant__ Params P, Select* sel,
                                                  const Cand* __restrict__ cand2, uint32_t* I_out) {
    const uint32_t k = P.k;
    constexpr uint32_t W = 11, BINS = 1u << W;
    __shared__ uint32_t hist[BINS];
    __shared__ uint32_t s_bin, s_need, s_done, s_pos;
    __shared__ uint32_t s_wtot[32];
    chain_acquire();
    const uint32_t ncand = sel->cnt_cand2;
    uint32_t need = sel->need2;
    uint64_t prefix = 0;        // composite >> shift must equal prefix for an element to be still undecided
    int shift = 39;
    bool exact = false;         // true once every element with composite >= threshold is known to be wanted
    bool first = true;
    while (shift > 0 && !exact) {
        const int w = first ? 7 : (shift >= (int)W ? (int)W : shift);   // the key bits first, then the index
        first = false;
        shift -= w;
        for (uint32_t b = threadIdx.x; b < BINS; b += blockDim.x) hist[b] = 0;
        __syncthreads();
        for (uint32_t q = threadIdx.x; q < ncand; q += blockDim.x) {
            const Cand cnd = cand2[q];
            const uint64_t comp = ((uint64_t)(cnd.key & 127u) << 32) | (uint32_t)~cnd.idx;
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
        if (q < ncand) {
            const Cand cnd = cand2[q];
            const uint64_t comp = ((uint64_t)(cnd.key & 127u) << 32) | (uint32_t)~cnd.idx;
            if (comp >= threshold) {
                const uint32_t pos = atomicAdd(&s_pos, 1u);
                if (pos < k) I_out[pos] = cnd.idx;      // a surplus is not written; the count below reports it
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        sel->cnt_out = s_pos;
        if (s_pos != k) sel->status |= 1u;
    }
}

// ---- second round (Section III-A): exact value of every candidate, as a ranking key, + first-level histogram ----
// candidates C (P*k coordinates by estimate): key2[q] = bits(| mean_w a^(w)_j / sqrt(vhat_j) |), j = C[q]
// (vhat == nullptr: parameter averaging, the exact value is the plain mean).
__global__ void __launch_bounds__(kThreads)
k_exact_keys(const __grid_constant__ Params P, const uint32_t* __restrict__ C, uint32_t count,
             const float* __restrict__ vhat, const float* __restrict__ e, const float* __restrict__ asum,
             uint32_t* keys2, uint32_t* hist) {
    __shared__ uint32_t sh[kHistBins];
    for (uint32_t b = threadIdx.x; b < kHistBins; b += kThreads) sh[b] = 0;
    chain_acquire();                // nothing above touches global memory
    __syncthreads();
    for (uint32_t q = blockIdx.x * kThreads + threadIdx.x; q < count; q += gridDim.x * kThreads) {
        const uint32_t j = C[q];
        float abar = 0.0f;
        if (!in_bounds(j < P.d, P.status, kStatusIndex)) continue;
        if (asum) abar = asum[j];
        else for (uint32_t w = 0; w < P.n; ++w) abar += e[(uint64_t)w * P.d + j];
        abar = abar / (float)P.n_all;
        const uint32_t key = key_of(vhat ? scale_est(abar, vhat[j]) : abar);
        keys2[q] = key;
        hist_add(P, sh, key >> kHistShift);
    }
    __syncthreads();
    for (uint32_t b = threadIdx.x; b < kHistBins; b += kThreads)
        if (sh[b]) atomicAdd(&hist[b], sh[b]);
}

// ---- apply on I_t: x_j -= lr * mean_w a^(w)_j / sqrt(vhat_j).  The error-feedback reset e^(w)_j = 0 is recorded
// as a bit in the membership bitmap of I_t, which the next step's moment kernel honours. -----------------------
__global__ void __launch_bounds__(kThreads)
k_apply(const __grid_constant__ Params P, const uint32_t* __restrict__ I, const float* __restrict__ vhat,
        const float* __restrict__ e, const float* __restrict__ asum, float* x, uint32_t* bitmap) {
    // asum != nullptr: the sketch kernel left sum_w a^(w) (added in worker order) there, one gather instead of n
    chain_acquire();
    const uint32_t q = blockIdx.x * kThreads + threadIdx.x;
    if (q >= P.k) return;
    const uint32_t j = I[q];
    if (!in_bounds(j < P.d, P.status, kStatusIndex)) return;
    float abar = 0.0f;
    uint32_t w = asum ? P.n : 0;
    if (asum) abar = asum[j];
    for (; w + 8 <= P.n; w += 8) {                           // eight independent gathers in flight, added in order
        float a[8];
#pragma unroll
        for (uint32_t u = 0; u < 8; ++u) a[u] = e[(uint64_t)(w + u) * P.d + j];
#pragma unroll
        for (uint32_t u = 0; u < 8; ++u) abar += a[u];
    }
    for (; w < P.n; ++w) abar += e[(uint64_t)w * P.d + j];
    abar = abar / (float)P.n_all;
    const float delta = vhat ? scale_est(abar, vhat[j]) : abar;
    x[j] = x[j] - P.lr * delta;
    atomicOr(&bitmap[j >> 5], 1u << (j & 31u));
}

__global__ void __launch_bounds__(kThreads)
k_estimates(const __grid_constant__ Params P, const float* __restrict__ sum, const float* __restrict__ vhat,
            float* est) {
    for (uint32_t j = blockIdx.x * kThreads + threadIdx.x; j < P.d; j += gridDim.x * kThreads)
        est[j] = vhat ? scale_est(median1(P, sum, j), vhat[j]) : median1(P, sum, j);
}

__global__ void __launch_bounds__(kThreads)
k_hash_export(const __grid_constant__ Params P, uint32_t row, uint64_t i0, uint64_t count, uint32_t* idx,
              int8_t* sgn) {
    for (uint64_t t = blockIdx.x * (uint64_t)kThreads + threadIdx.x; t < count; t += (uint64_t)gridDim.x * kThreads) {
        uint32_t b; float s;
        coord_hash(P, P.row_key[row], (uint32_t)(i0 + t), b, s);
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

// Persistent grids are sized to what is resident at once (registers and shared memory decide): one block more per
// SM than fits would run as a second, nearly empty wave after the first.
template <typename K>
int resident_per_sm(K kernel, int fallback) {
    int nb = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kernel, kThreads, 0) != cudaSuccess || nb < 1) {
        cudaGetLastError();
        return fallback;
    }
    return nb;
}

#define SK_ROWS_CASE(KERNEL, RR, ...)                                                                      \
    { auto kfn = KERNEL<RR, true>;                                                                         \
      launch_kernel((P.chain & kChainKeys) != 0, kfn, grid_for(items, sm_count, resident_per_sm(kfn, 4)), kThreads, 0, st, __VA_ARGS__); } break;
#define SK_ROWS_SWITCH(KERNEL, ...)                                                                        \
    switch (P.r) {                                                                                         \
        case 1: SK_ROWS_CASE(KERNEL, 1, __VA_ARGS__)                                                       \
        case 2: SK_ROWS_CASE(KERNEL, 2, __VA_ARGS__)                                                       \
        case 3: SK_ROWS_CASE(KERNEL, 3, __VA_ARGS__)                                                       \
        case 4: SK_ROWS_CASE(KERNEL, 4, __VA_ARGS__)                                                       \
        case 5: SK_ROWS_CASE(KERNEL, 5, __VA_ARGS__)                                                       \
        case 6: SK_ROWS_CASE(KERNEL, 6, __VA_ARGS__)                                                       \
        case 7: SK_ROWS_CASE(KERNEL, 7, __VA_ARGS__)                                                       \
        case 8: SK_ROWS_CASE(KERNEL, 8, __VA_ARGS__)                                                       \
        case 10: SK_ROWS_CASE(KERNEL, 10, __VA_ARGS__)                                                     \
        default: SK_ROWS_CASE(KERNEL, 0, __VA_ARGS__)                                                      \
    }

int launch_unsketch_hist(const Params& P, const MomentArgs& A, const float* sum, uint32_t* keys, uint32_t* hist,
                         bool vec, int sm_count, cudaStream_t st) {
    if (!vec) {
        auto kfn = k_unsketch_hist<0, false>;
        launch_kernel((P.chain & kChainKeys) != 0, kfn, grid_for(P.d, sm_count, resident_per_sm(kfn, 4)), kThreads, 0, st, P, A, sum, keys, hist);
        return 1;
    }
    if (P.win_cw != 0 && P.log2g == 5) {           // windowed family: shared-memory windows, panel-major walk
        const uint32_t units_total = (P.d + kUnit - 1) / kUnit;
        const uint32_t tbig = (units_total + P.win_panels - 1) / P.win_panels;
        const uint32_t rem = units_total - (tbig - 1u) * P.win_panels;
        const size_t smem = (size_t)kHistBins * 4 + (size_t)2 * P.r * kGroupsPerUnit * 8 + (size_t)P.r * P.win_cw * 4;
#define SK_WIN_CASE(RR)                                                                                              \
        {                                                                                                            \
            auto kfn = k_unsketch_hist_win<RR>;                                                                      \
            int nb = 0;                                                                                              \
            if ((smem <= 48 * 1024 ||                                                                                \
                 cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess) && \
                cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kfn, kThreads, smem) == cudaSuccess && nb >= 1) { \
                const uint64_t cap = (uint64_t)sm_count * nb;                                                        \
                launch_kernel((P.chain & kChainKeys) != 0, kfn, (int)(units_total < cap ? units_total : cap), kThreads, smem, st,   \
                              P, A, sum, keys, hist, units_total, tbig, rem);                                        \
                return 1;                                                                                            \
            }                                                                                                        \
            cudaGetLastError();                                                                                      \
        } break;
        switch (P.r) {
            case 5: SK_WIN_CASE(5)
            case 7: SK_WIN_CASE(7)
            case 10: SK_WIN_CASE(10)
            default: SK_WIN_CASE(0)
        }
#undef SK_WIN_CASE
    }
    const uint64_t items = P.d >> 2;
    SK_ROWS_SWITCH(k_unsketch_hist, P, A, sum, keys, hist)
    return 1;
}

int launch_pick_bin(const Params& P, uint32_t* hist, Select* sel, int level, cudaStream_t st) {
    launch_kernel((P.chain & kChainPick) != 0, k_pick_bin, 1, 1024, 0, st, P.k, hist, sel, level);
    return 1;
}

int launch_emit(const Params& P, const uint32_t* keys, const uint32_t* idx_map, Select* sel, uint32_t* I_out, Cand* cand,
                uint32_t* hist2, int sm_count, cudaStream_t st, void* clear, uint64_t clear_bytes) {
    uint4* c4 = (uint4*)clear;
    const uint32_t n4 = (uint32_t)(clear_bytes / 16);
    if (P.d % 4 == 0 && !idx_map) {
        auto kfn = k_emit<true>;
        launch_kernel((P.chain & kChainEmit) != 0, kfn, grid_for((P.d >> 2) / 4 + 1, sm_count, resident_per_sm(kfn, 4)), kThreads, 0, st, P,
                      keys, (const uint32_t*)nullptr, sel, I_out, cand, hist2, c4, n4);
    } else {
        auto kfn = k_emit<false>;
        launch_kernel((P.chain & kChainEmit) != 0, kfn, grid_for(P.d, sm_count, resident_per_sm(kfn, 4)), kThreads, 0, st, P, keys, idx_map,
                      sel, I_out, cand, hist2, c4, n4);
    }
    return 1;
}

int launch_exact_keys(const Params& P, const uint32_t* C, uint32_t count, const float* vhat, const float* e,
                      const float* asum, uint32_t* keys2, uint32_t* hist, int sm_count, cudaStream_t st) {
    launch_kernel((P.chain & kChainExact) != 0, k_exact_keys, grid_for(count, sm_count, resident_per_sm(k_exact_keys, 4)), kThreads, 0, st, P, C,
                  count, vhat, e, asum, keys2, hist);
    return 1;
}

int launch_refine(const Params& P, Select* sel, const Cand* cand, Cand* cand2, uint32_t* hist2, uint32_t* I_out,
                  int sm_count, cudaStream_t st) {
    const bool chain = (P.chain & kChainRefine) != 0;
    launch_kernel(chain, k_pick_bin, 1, 1024, 0, st, P.k, hist2, sel, 1);
    launch_kernel(chain, k_split_candidates, sm_count, kThreads, 0, st, P, sel, cand, I_out, cand2);
    launch_kernel(chain, k_resolve, 1, 1024, 0, st, P, sel, cand2, I_out);
    return 3;
}

int launch_apply(const Params& P, const uint32_t* I, const float* vhat, const float* e, const float* asum, float* x,
                 uint32_t* bitmap, cudaStream_t st) {
    launch_kernel((P.chain & kChainApply) != 0, k_apply, (P.k + kThreads - 1) / kThreads, kThreads, 0, st, P, I, vhat, e, asum, x, bitmap);
    return 1;
}

int launch_estimates(const Params& P, const float* sum, const float* vhat, float* est, cudaStream_t st) {
    k_estimates<<<grid_for(P.d, sm_count_of_device(), 8), kThreads, 0, st>>>(P, sum, vhat, est);
    return 1;
}

int launch_hash_export(const Params& P, uint32_t row, uint64_t i0, uint64_t count, uint32_t* idx, int8_t* sgn,
                       cudaStream_t st) {
    k_hash_export<<<grid_for(count, sm_count_of_device(), 8), kThreads, 0, st>>>(P, row, i0, count, idx, sgn);
    return 1;
}

}  // namespace sk
