// Moments + error-feedback accumulate + Count Sketch for the WINDOWED hash family, accumulated on chip by
// ownership: one warp per worker, one thread block per panel slice.
//
// In the windowed family every unit of 1024 coordinates hashes, in every row, into one aligned window of the row
// (the window of the unit's panel).  A block walks a run of units in panel-major order and keeps the current
// panel's window of every (worker, row) table in shared memory.  Warp w of the block streams worker w0 + w: 128-bit
// loads of g, m, e, the moment update, 128-bit stores of m and a_t (Algorithm 2, worker side), and r read-add-write
// accesses of 16 bytes into its own worker's windows (Section II-C).  Because only warp w ever touches worker w's
// windows, no atomics are needed, and only the dense stream and one small flush per panel leave the SM, instead
// of one reduction per (coordinate, row, worker).
//
// Inside a warp the lane <-> coordinate map makes every access conflict-free:
//   * a lane owns 4 consecutive coordinates, so 8 lanes own one hash group of 32, whose values land on the 8
//     distinct 16-byte chunks of ONE 128-byte line of a row: a quarter-warp access covers exactly one line;
//   * the 4 groups of a warp's 128 coordinates could pick the same line of a row, so at sub-step i group q works
//     on row (i + q) mod r: the 4 groups are always in 4 different rows, i.e. in 4 different windows (r >= 4;
//     for fewer rows the groups take turns).
// The group hashes of a unit (r x 32 draws) are evaluated once per block into a double-buffered shared stage.
// sum_w a^(w) (used by the update of x) is formed through a shared stage of the unit's a_t values, in worker
// order; the gradient sums on I_{t-1} (about 1 % of the coordinates) are formed with 16-byte reductions into the
// gsum array, which is zero between steps because the key pass clears what it consumes.
#include "sk_internal.h"
#include "sk_hash.cuh"
#include "sk_moment.cuh"

namespace sk {

namespace {

constexpr uint32_t kChunksPerUnit = kUnit / 128;      // 8 warp-wide chunks of 128 coordinates

__device__ __forceinline__ void red_add_v4(float* addr, float4 v) {
    asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                 :: "l"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w));
}

#define SK_MOMENT(mm, aa, gg, mask)                                                     \
    mm.x = fmaf(b1, mm.x, omb1 * gg.x); mm.y = fmaf(b1, mm.y, omb1 * gg.y);             \
    mm.z = fmaf(b1, mm.z, omb1 * gg.z); mm.w = fmaf(b1, mm.w, omb1 * gg.w);             \
    aa.x = fmaf(rho, (mask & 1u) ? 0.0f : aa.x, mm.x); aa.y = fmaf(rho, (mask & 2u) ? 0.0f : aa.y, mm.y); \
    aa.z = fmaf(rho, (mask & 4u) ? 0.0f : aa.z, mm.z); aa.w = fmaf(rho, (mask & 8u) ? 0.0f : aa.w, mm.w);

struct Chunk { float4 g, m, e; };

// One read-add-write of this lane's four signed values into its worker's window of a row.
// h.x = 32 * line + perm of the lane's group in that row, h.y = the group's sign in that row as the float +1 or -1;
// o = 4 * (lane mod 8) is the offset of the lane's first coordinate inside the group.
// The sign rides on the accumulation (one fused multiply-add per element); the logic pipe, which this kernel loads
// most, is left with the selects of the xor-permutation.
__device__ __forceinline__ void window_add(const Params& P, float* wrow, const uint2 h, uint32_t o, float4 a) {
    const uint32_t off = (h.x ^ o) & ~3u;                          // line of the group, chunk after the xor permutation
    if (!in_bounds(off + 4u <= P.win_cw, P.status, kStatusWindow)) return;
    const float sg = __uint_as_float(h.y);
    // element e of the chunk receives local coordinate e xor p3
    if (h.x & 1u) { float t = a.x; a.x = a.y; a.y = t; t = a.z; a.z = a.w; a.w = t; }
    if (h.x & 2u) { float t = a.x; a.x = a.z; a.z = t; t = a.y; a.y = a.w; a.w = t; }
    float4* dst = (float4*)(wrow + off);
    float4 cur = *dst;
    cur.x = fmaf(sg, a.x, cur.x); cur.y = fmaf(sg, a.y, cur.y); cur.z = fmaf(sg, a.z, cur.z); cur.w = fmaf(sg, a.w, cur.w);
    *dst = cur;
}

// General form: any number of rows, partial last unit, any slice [s_lo, s_hi) of the panel-major unit sequence.
template <int R>
__global__ void __launch_bounds__(256)
k_moment_sketch_own_any(const __grid_constant__ Params P, const __grid_constant__ MomentArgs A, uint32_t w0, uint32_t nw,
                        uint32_t s_lo, uint32_t s_hi, uint32_t tbig, uint32_t rem, uint32_t single) {
    // single != 0xFFFFFFFF: the launch covers exactly that unit (s_lo = 0, s_hi = 1, one block)
    extern __shared__ __align__(16) float smem[];
    const uint32_t r = R > 0 ? (uint32_t)R : P.r;
    const uint32_t cw = P.win_cw;
    float* win = smem;                                             // [nw][r][cw]
    uint2* hsh = (uint2*)(win + (size_t)nw * r * cw);              // [2][r][32]: x = line*32 | perm, y = sign as +-1.0f
    float4* ast = (float4*)(hsh + 2u * r * kGroupsPerUnit);        // [nw][256]: a_t of the unit (only with A.asum)

    const uint32_t tid = threadIdx.x, lane = tid & 31u, wid = tid >> 5;
    const uint32_t nthreads = blockDim.x;
    const uint32_t s_begin = s_lo + (uint32_t)((uint64_t)(s_hi - s_lo) * blockIdx.x / gridDim.x);
    const uint32_t s_end = s_lo + (uint32_t)((uint64_t)(s_hi - s_lo) * (blockIdx.x + 1) / gridDim.x);
    chain_acquire();
    if (s_begin >= s_end) return;                                  // the whole block leaves together

    float4* m = (float4*)A.m;
    float4* e = (float4*)A.e;
    const uint32_t d4 = P.d >> 2;
    const uint32_t bm_words = (P.d + 31u) >> 5;
    const float b1 = P.beta1, omb1 = 1.0f - P.beta1, rho = P.rho;
    const uint32_t gb = A.grad_bf16;
    const uint64_t wbase = (uint64_t)(w0 + wid) * d4;
    const uint64_t tstride = (uint64_t)P.r * P.cs;
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    const uint32_t grp = lane >> 3, o = (lane & 7u) * 4u;          // this lane's group in the chunk, offset inside it
    float* mywin = win + (size_t)wid * r * cw;

    auto fill_hashes = [&](uint32_t unit, uint32_t buf) {
        for (uint32_t hq = tid; hq < r * kGroupsPerUnit; hq += nthreads) {
            const uint32_t row = hq >> 5, s = hq & 31u;
            const GroupHash gh = group_from_draw(P, stream(P.row_key[row & (kMaxRows - 1u)], (uint64_t)unit * kGroupsPerUnit + s + 1));
            hsh[buf * r * kGroupsPerUnit + hq] = make_uint2(gh.base | gh.perm, 0x3F800000u | (gh.sign << 31));
        }
    };
    auto issue = [&](uint32_t unit, uint32_t c, bool have, Chunk& k) {
        const uint32_t t = unit * kQuadsPerUnit + c * 32u + lane;
        if (have && t < d4) {
            k.g = load_grad4(A.grads, wbase + t, gb);
            k.m = __ldcs(m + wbase + t);
            k.e = __ldcs(e + wbase + t);
        } else { k.g = zero4; k.m = zero4; k.e = zero4; }
    };

    UnitWalk walk{P.win_panels, tbig, rem, 0u, 0u};
    walk.seek(s_begin);
    if (single != 0xFFFFFFFFu) { walk.panel = single % P.win_panels; walk.tu = single / P.win_panels; }
    for (uint32_t q = tid; q < nw * r * cw / 4u; q += nthreads) ((float4*)win)[q] = zero4;
    fill_hashes(walk.unit(), 0u);
    Chunk ring[2];
    issue(walk.unit(), 0u, true, ring[0]);
    issue(walk.unit(), 1u, true, ring[1]);
    __syncthreads();

    for (uint32_t s = s_begin; s < s_end; ++s) {
        const uint32_t buf = (s - s_begin) & 1u;
        const uint32_t unit = walk.unit(), panel = walk.panel;
        const bool have_next = s + 1 < s_end;
        walk.next();
        const uint32_t unit_next = have_next ? walk.unit() : 0u;
        if (have_next) fill_hashes(unit_next, buf ^ 1u);
        uint32_t bmw = 0;                                          // lane l: word l of the unit's 32 membership words
        if (A.members && unit * 32u + lane < bm_words) bmw = __ldg(A.bitmap + unit * 32u + lane);
        const uint2* hs = hsh + buf * r * kGroupsPerUnit;

#pragma unroll
        for (uint32_t c = 0; c < kChunksPerUnit; ++c) {
            Chunk k = ring[c & 1u];
            if (c + 2u < kChunksPerUnit) issue(unit, c + 2u, true, ring[c & 1u]);
            else issue(unit_next, c + 2u - kChunksPerUnit, have_next, ring[c & 1u]);
            const uint32_t t = unit * kQuadsPerUnit + c * 32u + lane;
            const bool live = t < d4;
            const uint32_t mask = (__shfl_sync(0xFFFFFFFFu, bmw, c * 4u + grp) >> o) & 0xFu;
            float4 mm = k.m, aa = k.e;
            if (live) SK_CHECK_FINITE4(k.g);
            SK_MOMENT(mm, aa, k.g, mask)
            if (live) { __stcs(m + wbase + t, mm); __stcs(e + wbase + t, aa); }
            if (A.asum) ast[wid * kQuadsPerUnit + c * 32u + lane] = aa;
            const uint32_t sg = c * 4u + grp;                      // this lane's group inside the unit
            if (R >= 4 || (R == 0 && r >= 4)) {
#pragma unroll
                for (uint32_t i = 0; i < (R > 0 ? (uint32_t)R : kMaxRows); ++i) {
                    if (i < r) {
                        uint32_t row = i + grp;
                        if (row >= r) row -= r;
                        window_add(P, mywin + row * cw, hs[row * kGroupsPerUnit + sg], o, aa);
                        __syncwarp();                              // the next sub-step's lanes may read what these wrote
                    }
                }
            } else {
                for (uint32_t row = 0; row < r; ++row)
                    for (uint32_t q = 0; q < 4; ++q) {             // fewer rows than groups: the groups take turns
                        if (grp == q) window_add(P, mywin + row * cw, hs[row * kGroupsPerUnit + sg], o, aa);
                        __syncwarp();
                    }
            }
            // gradient sums on I_{t-1}: every worker's warp adds its quad (gsum is zero between steps)
            if (A.gsum_on && mask) red_add_v4(A.gsum + 4u * (size_t)t, k.g);
        }
        __syncthreads();            // every warp is done with this unit's hashes, windows and a_t stage

        if (A.asum) {               // sum_w a^(w) of the unit, workers added in order
            for (uint32_t q = tid; q < kQuadsPerUnit; q += nthreads) {
                const uint32_t t = unit * kQuadsPerUnit + q;
                if (t < d4) {
                    float4 as = zero4;
                    for (uint32_t w = 0; w < nw; ++w) {
                        const float4 a = ast[w * kQuadsPerUnit + q];
                        as.x += a.x; as.y += a.y; as.z += a.z; as.w += a.w;
                    }
                    if (w0 > 0) {
                        const float4 prev = ((const float4*)A.asum)[t];
                        as.x += prev.x; as.y += prev.y; as.z += prev.z; as.w += prev.w;
                    }
                    ((float4*)A.asum)[t] = as;
                }
            }
        }
        const bool flush = !have_next || walk.panel != panel;
        if (flush) {                // the panel ends here for this block: add its windows to the tables and clear them
            for (uint32_t q = tid; q < nw * r * cw / 4u; q += nthreads) {
                const uint32_t pr = q / (cw / 4u), c4 = q - pr * (cw / 4u);
                const uint32_t w = pr / r, row = pr - w * r;
                const float4 val = ((float4*)win)[q];
                ((float4*)win)[q] = zero4;
                SK_GUARD((uint64_t)panel * cw + 4u * c4 + 4u <= P.cs && w0 + w < P.n, kStatusBucket)
                    red_add_v4(A.tables + (uint64_t)(w0 + w) * tstride + (uint64_t)row * P.cs + (uint64_t)panel * cw + 4u * c4, val);
            }
        }
        if (A.asum || flush) __syncthreads();
    }
}


// ---- shared-memory accesses by 32-bit shared address (asm volatile statements keep their program order) -----------
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ float4 lds128(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, float4 v) {
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" :: "r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w));
}

// Fast form: r >= 4 known at compile time, whole units only (the launcher gives a partial last unit to the general
// form).  Differences that matter for the instruction count: no bounds predicates; the row a lane group works on at
// sub-step i, (i + group) mod r, is folded into per-lane address registers (the hash stage repeats its first three
// rows after the last so that the lane's stage address is affine in i); the chunk loop is unrolled by two only, which
// keeps the loop body inside the instruction cache.
template <int R, bool ASUM, bool BF16>
__global__ void __launch_bounds__(256, 3)      // 3 blocks = 24 warps per SM; 2 and 4 (spills) measured slower
k_moment_sketch_own(const __grid_constant__ Params P, const __grid_constant__ MomentArgs A, uint32_t w0, uint32_t nw,
                    uint32_t s_lo, uint32_t s_hi, uint32_t tbig, uint32_t rem) {
    extern __shared__ __align__(16) float smem[];
    constexpr uint32_t r = (uint32_t)R, HR = (uint32_t)R + 3u;     // rows of the hash stage
    const uint32_t cw = P.win_cw;
    float* win = smem;                                             // [nw][r][cw]
    uint2* hsh = (uint2*)(win + (size_t)nw * r * cw);              // [2][HR][32]: x = line*32 | perm, y = sign as +-1.0f
    float4* ast = (float4*)(hsh + 2u * HR * kGroupsPerUnit);       // [nw][256]: a_t of the unit (ASUM)

    const uint32_t tid = threadIdx.x, lane = tid & 31u, wid = tid >> 5;
    const uint32_t nthreads = blockDim.x;
    const uint32_t s_begin = s_lo + (uint32_t)((uint64_t)(s_hi - s_lo) * blockIdx.x / gridDim.x);
    const uint32_t s_end = s_lo + (uint32_t)((uint64_t)(s_hi - s_lo) * (blockIdx.x + 1) / gridDim.x);
    chain_release();
    if (s_begin >= s_end) { chain_acquire(); return; }             // the whole block leaves together

    const uint32_t d4 = P.d >> 2;
    const float b1 = P.beta1, omb1 = 1.0f - P.beta1, rho = P.rho;
    constexpr uint32_t gb = BF16 ? 1u : 0u;      // compile-time: the widening of bf16 entries costs the fp32 path nothing
    const uint64_t wbase = (uint64_t)(w0 + wid) * d4;
    float4* m4 = (float4*)A.m + wbase;
    float4* e4 = (float4*)A.e + wbase;
    const uint64_t tstride = (uint64_t)P.r * P.cs;
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    const uint32_t grp = lane >> 3, o = (lane & 7u) * 4u;          // this lane's group in the chunk, offset inside it
    const uint32_t members = A.members, gsum_on = A.gsum_on;

    // per-lane shared addresses: the window row of sub-step i, and the stage entry of (row = group + i, group of chunk 0)
    const uint32_t sm_win = (uint32_t)__cvta_generic_to_shared(win);
    uint32_t wrow[R];
#pragma unroll
    for (uint32_t i = 0; i < r; ++i) wrow[i] = sm_win + ((wid * r + (i + grp) % r) * cw) * 4u;
    const uint32_t hs_lane = (uint32_t)__cvta_generic_to_shared(hsh) + (grp * kGroupsPerUnit + grp) * 8u;
    const uint32_t ast_lane = (uint32_t)__cvta_generic_to_shared(ast) + (wid * kQuadsPerUnit + lane) * 16u;

    auto fill_hashes = [&](uint32_t unit, uint32_t buf) {
        for (uint32_t hq = tid; hq < HR * kGroupsPerUnit; hq += nthreads) {
            const uint32_t rowx = hq >> 5, s = hq & 31u;
            const uint32_t row = rowx < r ? rowx : rowx - r;
            const GroupHash gh = group_from_draw(P, stream(P.row_key[row & (kMaxRows - 1u)], (uint64_t)unit * kGroupsPerUnit + s + 1));
            hsh[buf * HR * kGroupsPerUnit + hq] = make_uint2(gh.base | gh.perm, 0x3F800000u | (gh.sign << 31));
        }
    };

    UnitWalk walk{P.win_panels, tbig, rem, 0u, 0u};
    walk.seek(s_begin);
    for (uint32_t q = tid; q < nw * r * cw / 4u; q += nthreads) ((float4*)win)[q] = zero4;
    fill_hashes(walk.unit(), 0u);
    chain_acquire();                // nothing above touches global memory
    // ring of two chunks in flight per lane
    float4 G0, M0, E0, G1, M1, E1;
    {
        const uint32_t t = walk.unit() * kQuadsPerUnit + lane;
        G0 = load_grad4_raw(A.grads, wbase + t, gb); M0 = __ldcs(m4 + t); E0 = __ldcs(e4 + t);
        G1 = load_grad4_raw(A.grads, wbase + t + 32u, gb); M1 = __ldcs(m4 + t + 32u); E1 = __ldcs(e4 + t + 32u);
    }
    __syncthreads();

// one chunk: consume ring slot (G_, M_, E_) holding quad tc, refill it with quad tp, sketch into the windows
#define SK_OWN_CHUNK(G_, M_, E_, c_, tc_, tp_)                                                                      \
    {                                                                                                               \
        const float4 gg = widen_grad4(G_, gb);                                                                      \
        float4 mm = M_, aa = E_;                                                                                    \
        G_ = load_grad4_raw(A.grads, wbase + (tp_), gb); M_ = __ldcs(m4 + (tp_)); E_ = __ldcs(e4 + (tp_));          \
        uint2 h[R];                                                                                                 \
        _Pragma("unroll") for (uint32_t i = 0; i < r; ++i) h[i] = lds64(hs_c + i * (kGroupsPerUnit * 8u));          \
        uint32_t mask = 0;                                                                                          \
        if (members) mask = (__shfl_sync(0xFFFFFFFFu, bmw, (c_) * 4u + grp) >> o) & 0xFu;                           \
        SK_CHECK_FINITE4(gg);                                                                                       \
        SK_MOMENT(mm, aa, gg, mask)                                                                                 \
        __stcs(m4 + (tc_), mm); __stcs(e4 + (tc_), aa);                                                             \
        if (ASUM) sts128(ast_lane + (c_) * 512u, aa);                                                               \
        _Pragma("unroll") for (uint32_t i = 0; i < r; ++i) {                                   \
            const uint32_t woff = (h[i].x ^ o) & ~3u;                                                               \
            const uint32_t addr = wrow[i] + woff * 4u;                                                              \
            const bool inside = in_bounds(woff + 4u <= cw, P.status, kStatusWindow);                                \
            float4 cur = inside ? lds128(addr) : zero4;                                                             \
            float4 sa = aa;                                                                                         \
            const float sg = __uint_as_float(h[i].y);     /* the group's sign in this row, +1 or -1 */              \
            if (h[i].x & 1u) { float t = sa.x; sa.x = sa.y; sa.y = t; t = sa.z; sa.z = sa.w; sa.w = t; }            \
            if (h[i].x & 2u) { float t = sa.x; sa.x = sa.z; sa.z = t; t = sa.y; sa.y = sa.w; sa.w = t; }            \
            cur.x = fmaf(sg, sa.x, cur.x); cur.y = fmaf(sg, sa.y, cur.y);                                           \
            cur.z = fmaf(sg, sa.z, cur.z); cur.w = fmaf(sg, sa.w, cur.w);                                           \
            if (inside) sts128(addr, cur);                                                                          \
            __syncwarp();                        /* the next sub-step's lanes may read what these wrote */          \
        }                                                                                                           \
        /* gradient sums on I_{t-1}: every worker's warp adds its quad (gsum is zero between steps) */            \
        if (gsum_on && mask) red_add_v4(A.gsum + 4u * (size_t)(tc_), gg);                                           \
        hs_c += 32u;                                                                                                \
    }

    for (uint32_t s = s_begin; s < s_end; ++s) {
        const uint32_t buf = (s - s_begin) & 1u;
        const uint32_t unit = walk.unit(), panel = walk.panel;
        const bool have_next = s + 1 < s_end;
        walk.next();
        const uint32_t unit_next = have_next ? walk.unit() : unit;  // past the end: prefetch this unit again, unused
        if (have_next) fill_hashes(unit_next, buf ^ 1u);
        uint32_t bmw = 0;                                           // lane l: word l of the unit's 32 membership words
        if (members) bmw = __ldg(A.bitmap + unit * 32u + lane);
        uint32_t hs_c = hs_lane + buf * (HR * kGroupsPerUnit * 8u);
        uint32_t tc = unit * kQuadsPerUnit + lane;
        const uint32_t tn = unit_next * kQuadsPerUnit + lane;
#pragma unroll 1
        for (uint32_t c = 0; c < kChunksPerUnit - 2u; c += 2u) {
            SK_OWN_CHUNK(G0, M0, E0, c, tc, tc + 64u)
            SK_OWN_CHUNK(G1, M1, E1, c + 1u, tc + 32u, tc + 96u)
            tc += 64u;
        }
        SK_OWN_CHUNK(G0, M0, E0, kChunksPerUnit - 2u, tc, tn)
        SK_OWN_CHUNK(G1, M1, E1, kChunksPerUnit - 1u, tc + 32u, tn + 32u)
        __syncthreads();            // every warp is done with this unit's hashes, windows and a_t stage

        if (ASUM) {                 // sum_w a^(w) of the unit, workers added in order
            for (uint32_t q = tid; q < kQuadsPerUnit; q += nthreads) {
                const uint32_t t = unit * kQuadsPerUnit + q;
                float4 as = zero4;
                for (uint32_t w = 0; w < nw; ++w) {
                    const float4 a = ast[w * kQuadsPerUnit + q];
                    as.x += a.x; as.y += a.y; as.z += a.z; as.w += a.w;
                }
                if (w0 > 0) {
                    const float4 prev = ((const float4*)A.asum)[t];
                    as.x += prev.x; as.y += prev.y; as.z += prev.z; as.w += prev.w;
                }
                ((float4*)A.asum)[t] = as;
            }
        }
        const bool flush = !have_next || walk.panel != panel;
        if (flush) {                // the panel ends here for this block: add its windows to the tables and clear them
            for (uint32_t q = tid; q < nw * r * cw / 4u; q += nthreads) {
                const uint32_t pr = q / (cw / 4u), c4 = q - pr * (cw / 4u);
                const uint32_t w = pr / r, row = pr - w * r;
                const float4 val = ((float4*)win)[q];
                ((float4*)win)[q] = zero4;
                SK_GUARD((uint64_t)panel * cw + 4u * c4 + 4u <= P.cs && w0 + w < P.n, kStatusBucket)
                    red_add_v4(A.tables + (uint64_t)(w0 + w) * tstride + (uint64_t)row * P.cs + (uint64_t)panel * cw + 4u * c4, val);
            }
        }
        if (ASUM || flush) __syncthreads();
    }
#undef SK_OWN_CHUNK
}

// shared memory of one block: windows, two hash stages, and (with the worker sum) the unit's a_t values
inline size_t own_smem(const Params& P, uint32_t nw, uint32_t stage_rows, bool asum) {
    return ((size_t)nw * P.r * P.win_cw) * 4 + (size_t)2 * stage_rows * kGroupsPerUnit * 8 +
           (asum ? (size_t)nw * kQuadsPerUnit * 16 : 0);
}

// grid and shared-memory set-up common to both forms; `units` = length of the unit sequence the launch enumerates
template <typename K, typename... Extra>
int launch_own_kernel(bool chain, K kfn, size_t smem, const Params& P, const MomentArgs& A, uint32_t w0, uint32_t nw,
                      uint32_t units, int sm_count, cudaStream_t st, Extra... extra) {
    if (units == 0) return 0;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        cudaGetLastError();
        return -1;
    }
    const int threads = 32 * (int)nw;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kfn, threads, smem) != cudaSuccess || per_sm < 1) {
        cudaGetLastError();
        return -1;
    }
    // the sequence enumerates the units 0..units-1 in panel-major order
    const uint32_t tbig = (units + P.win_panels - 1) / P.win_panels;
    const uint32_t rem = units - (tbig - 1u) * P.win_panels;
    const uint64_t cap = (uint64_t)sm_count * per_sm;
    const int grid = (int)(units < cap ? units : cap);
    launch_kernel(chain, kfn, grid, threads, smem, st, P, A, w0, nw, 0u, units, tbig, rem, extra...);
    return 1;
}

int launch_own_any(const Params& P, const MomentArgs& A, uint32_t w0, uint32_t nw, uint32_t units, uint32_t single,
                   int sm_count, cudaStream_t st) {
    return launch_own_kernel((P.chain & kChainSketch) != 0, k_moment_sketch_own_any<0>, own_smem(P, nw, P.r, A.asum != nullptr), P, A, w0, nw, units,
                             sm_count, st, single);
}

template <int R>
int launch_own(const Params& P, const MomentArgs& A, uint32_t w0, uint32_t nw, int sm_count, cudaStream_t st) {
    // whole units in the fast form; a partial last unit goes to the general form as a launch of its own
    const uint32_t units_total = (P.d + kUnit - 1) / kUnit, units_full = P.d / kUnit;
    const size_t smem = own_smem(P, nw, R + 3, A.asum != nullptr);
    int l;
    if (A.grad_bf16)
        l = A.asum ? launch_own_kernel((P.chain & kChainSketch) != 0, k_moment_sketch_own<R, true, true>, smem, P, A, w0, nw, units_full, sm_count, st)
                   : launch_own_kernel((P.chain & kChainSketch) != 0, k_moment_sketch_own<R, false, true>, smem, P, A, w0, nw, units_full, sm_count, st);
    else
        l = A.asum ? launch_own_kernel((P.chain & kChainSketch) != 0, k_moment_sketch_own<R, true, false>, smem, P, A, w0, nw, units_full, sm_count, st)
                   : launch_own_kernel((P.chain & kChainSketch) != 0, k_moment_sketch_own<R, false, false>, smem, P, A, w0, nw, units_full, sm_count, st);
    if (l < 0) return l;
    if (units_total > units_full) {
        const int l2 = launch_own_any(P, A, w0, nw, 1u, units_full, sm_count, st);
        if (l2 < 0) return l2;
        l += l2;
    }
    return l;
}

}  // namespace

// Enqueues the ownership kernel for workers w0..w0+nw-1 (nw <= kOwnMaxWorkers).  Returns launches, or -1 if the
// configuration does not fit in shared memory.
int launch_moment_sketch_own(const Params& P, const MomentArgs& A, uint32_t w0, uint32_t nw, int sm_count,
                             cudaStream_t st) {
    if (nw < 1 || nw > kOwnMaxWorkers || P.win_cw == 0 || P.log2g != 5) return -1;
    switch (P.r) {
        case 4: return launch_own<4>(P, A, w0, nw, sm_count, st);
        case 5: return launch_own<5>(P, A, w0, nw, sm_count, st);
        case 6: return launch_own<6>(P, A, w0, nw, sm_count, st);
        case 7: return launch_own<7>(P, A, w0, nw, sm_count, st);
        case 8: return launch_own<8>(P, A, w0, nw, sm_count, st);
        case 10: return launch_own<10>(P, A, w0, nw, sm_count, st);
        default: return launch_own_any(P, A, w0, nw, (P.d + kUnit - 1) / kUnit, 0xFFFFFFFFu, sm_count, st);
    }
}

}  // namespace sk
