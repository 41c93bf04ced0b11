// Moments + error-feedback accumulate + Count Sketch for the WINDOWED hash family, accumulating on chip.
//
// In the windowed family every unit of 1024 coordinates hashes, in every row, into one aligned window of the row
// (the window of the unit's panel).  A thread block therefore takes a panel (or a slice of its units), keeps the
// panel's window of every (worker, row) table in shared memory, adds the units' values there, and writes each
// window out once with 16-byte reductions.  Only the dense stream (read g, m, e; write m, a) and these small
// flushes leave the SM, instead of one reduction per (coordinate, row, worker).
//
// Per unit: phase 1 = the dense update, every thread owning 4 coordinates for all workers of the launch, with
// a_t staged in shared memory; phase 2 = the sketch: each warp owns whole (worker, row) windows, so its
// read-add-write needs no atomics, and the 32 lanes of one access hit 32 different banks because a group is a
// xor-permutation of one 32-float line.
#include "sk_internal.h"
#include "sk_hash.cuh"

namespace sk {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr uint32_t kUnit = 1u << kUnitShift;      // 1024 coordinates
constexpr uint32_t kGroupsPerUnit = kUnit / 32;   // 32

__device__ __forceinline__ void red_add_v4(float* addr, float4 v) {
    asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                 :: "l"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w));
}

#define SK_MOMENT(mm, aa, gg, mask)                                                     \
    mm.x = fmaf(b1, mm.x, omb1 * gg.x); mm.y = fmaf(b1, mm.y, omb1 * gg.y);             \
    mm.z = fmaf(b1, mm.z, omb1 * gg.z); mm.w = fmaf(b1, mm.w, omb1 * gg.w);             \
    aa.x = mm.x + ((mask & 1u) ? 0.0f : aa.x); aa.y = mm.y + ((mask & 2u) ? 0.0f : aa.y); \
    aa.z = mm.z + ((mask & 4u) ? 0.0f : aa.z); aa.w = mm.w + ((mask & 8u) ? 0.0f : aa.w);

// one (worker,row) window update for group s of the unit: lane l adds s(l) * a_l at line*32 + (l xor perm)
__device__ __forceinline__ void window_add(float* win, const float* stage_w, uint2 h, uint32_t s, uint32_t lane) {
    const uint32_t idx = (h.x & ~31u) + ((lane ^ h.x) & 31u);
    const float val = flip(stage_w[s * 32u + lane], (h.y >> lane) & 1u);
    win[idx] += val;
}

__global__ void __launch_bounds__(kThreads)
k_moment_sketch_win(const __grid_constant__ Params P, const __grid_constant__ MomentArgs A, uint32_t w0, uint32_t nw,
                    uint32_t slices, uint32_t units_total) {
    extern __shared__ __align__(16) float smem[];
    const uint32_t r = P.r, cw = P.win_cw;
    float* win = smem;                                   // [nw][r][cw]
    float* stage = win + (size_t)nw * r * cw;            // [nw][1024]
    uint2* hsh = (uint2*)(stage + (size_t)nw * kUnit);   // [r][32]: x = line*32 | perm, y = sign bits
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const float4* __restrict__ grads = (const float4*)A.grads;
    float4* m = (float4*)A.m;
    float4* e = (float4*)A.e;
    const uint32_t d4 = P.d >> 2;
    const float b1 = P.beta1, omb1 = 1.0f - P.beta1;
    const uint64_t tstride = (uint64_t)P.r * P.cs;
    const uint32_t items = P.win_panels * slices;
    const uint32_t win_floats = nw * r * cw;
    const uint32_t pairs = nw * r;

    for (uint32_t item = blockIdx.x; item < items; item += gridDim.x) {
        const uint32_t panel = item % P.win_panels, slice = item / P.win_panels;
        // units of this panel: panel, panel + panels, panel + 2 panels, ...
        const uint32_t T = panel < units_total ? (units_total - panel + P.win_panels - 1) / P.win_panels : 0u;
        const uint32_t t_begin = (uint32_t)((uint64_t)T * slice / slices);
        const uint32_t t_end = (uint32_t)((uint64_t)T * (slice + 1) / slices);
        if (t_begin == t_end) continue;                  // uniform over the block
        for (uint32_t q = tid; q < win_floats / 4; q += kThreads) ((float4*)win)[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        __syncthreads();

        for (uint32_t tu = t_begin; tu < t_end; ++tu) {
            const uint32_t unit = panel + P.win_panels * tu;
            // hashes of the unit's 32 groups in every row
            for (uint32_t hq = tid; hq < r * kGroupsPerUnit; hq += kThreads) {
                const uint32_t row = hq >> 5, s = hq & 31u;
                const GroupHash gh = group_from_draw(P, stream(P.row_key[row], (uint64_t)unit * kGroupsPerUnit + s + 1));
                hsh[hq] = make_uint2(gh.base | gh.perm, gh.signs);
            }
            // phase 1: dense update of this thread's 4 coordinates for every worker of the launch
            const uint32_t t = unit * (kUnit / 4) + tid;
            if (t < d4) {
                const uint32_t mask = A.members ? ((__ldg(A.bitmap + (t >> 3)) >> ((t & 7u) * 4u)) & 0xFu) : 0u;
                float4 gs = make_float4(0.f, 0.f, 0.f, 0.f);
                if (mask && w0 > 0) gs = ((const float4*)A.gsum)[t];
                uint32_t w = 0;
                for (; w + 2 <= nw; w += 2) {
                    const uint64_t q0 = (uint64_t)(w0 + w) * d4 + t, q1 = q0 + d4;
                    const float4 g0 = __ldcs(grads + q0), g1 = __ldcs(grads + q1);
                    float4 m0 = __ldcs(m + q0), m1 = __ldcs(m + q1);
                    float4 a0 = __ldcs(e + q0), a1 = __ldcs(e + q1);
                    SK_MOMENT(m0, a0, g0, mask)
                    SK_MOMENT(m1, a1, g1, mask)
                    gs.x = (gs.x + g0.x) + g1.x; gs.y = (gs.y + g0.y) + g1.y;
                    gs.z = (gs.z + g0.z) + g1.z; gs.w = (gs.w + g0.w) + g1.w;
                    __stcs(m + q0, m0); __stcs(m + q1, m1);
                    __stcs(e + q0, a0); __stcs(e + q1, a1);
                    ((float4*)(stage + (size_t)w * kUnit))[tid] = a0;
                    ((float4*)(stage + (size_t)(w + 1) * kUnit))[tid] = a1;
                }
                if (w < nw) {
                    const uint64_t q0 = (uint64_t)(w0 + w) * d4 + t;
                    const float4 g0 = __ldcs(grads + q0);
                    float4 m0 = __ldcs(m + q0);
                    float4 a0 = __ldcs(e + q0);
                    SK_MOMENT(m0, a0, g0, mask)
                    gs.x += g0.x; gs.y += g0.y; gs.z += g0.z; gs.w += g0.w;
                    __stcs(m + q0, m0);
                    __stcs(e + q0, a0);
                    ((float4*)(stage + (size_t)w * kUnit))[tid] = a0;
                }
                if (mask) ((float4*)A.gsum)[t] = gs;
            } else {
                for (uint32_t w = 0; w < nw; ++w)        // past the end of the vector: contribute zeros
                    ((float4*)(stage + (size_t)w * kUnit))[tid] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            __syncthreads();

            // phase 2: each warp owns whole (worker,row) windows; two independent windows are interleaved
            for (uint32_t pa = warp; pa < pairs; pa += 2 * kWarps) {
                const uint32_t pb = pa + kWarps;
                const uint32_t wa = pa % nw, ra = pa / nw;
                float* win_a = win + (size_t)(wa * r + ra) * cw;
                const float* st_a = stage + (size_t)wa * kUnit;
                const uint2* h_a = hsh + ra * kGroupsPerUnit;
                if (pb < pairs) {
                    const uint32_t wb = pb % nw, rb = pb / nw;
                    float* win_b = win + (size_t)(wb * r + rb) * cw;
                    const float* st_b = stage + (size_t)wb * kUnit;
                    const uint2* h_b = hsh + rb * kGroupsPerUnit;
#pragma unroll 4
                    for (uint32_t s = 0; s < kGroupsPerUnit; ++s) {
                        const uint2 ha = h_a[s], hb = h_b[s];
                        const uint32_t ia = (ha.x & ~31u) + ((lane ^ ha.x) & 31u);
                        const uint32_t ib = (hb.x & ~31u) + ((lane ^ hb.x) & 31u);
                        const float va = flip(st_a[s * 32u + lane], (ha.y >> lane) & 1u);
                        const float vb = flip(st_b[s * 32u + lane], (hb.y >> lane) & 1u);
                        const float xa = win_a[ia], xb = win_b[ib];   // different windows: never the same word
                        win_a[ia] = xa + va;
                        win_b[ib] = xb + vb;
                    }
                } else {
#pragma unroll 4
                    for (uint32_t s = 0; s < kGroupsPerUnit; ++s) window_add(win_a, st_a, h_a[s], s, lane);
                }
            }
            __syncthreads();
        }

        // flush the windows: table[w][row][panel*cw + ...] += window
        for (uint32_t q = tid; q < win_floats / 4; q += kThreads) {
            const float4 v = ((const float4*)win)[q];
            const uint32_t f = q * 4u;
            const uint32_t pr = f / cw, off = f % cw;     // pr = w*r + row
            const uint32_t w = pr / r, row = pr % r;
            red_add_v4(A.tables + (uint64_t)(w0 + w) * tstride + (uint64_t)row * P.cs + (uint64_t)panel * cw + off, v);
        }
        __syncthreads();
    }
}

}  // namespace

size_t window_smem_bytes(const Params& P, uint32_t nw) {
    return ((size_t)nw * P.r * P.win_cw + (size_t)nw * kUnit) * 4 + (size_t)P.r * kGroupsPerUnit * 8;
}

// Enqueues the windowed kernel for workers w0..w0+nw-1 (nw <= kWinMaxWorkers).  Returns launches, or -1 if the
// configuration does not fit in shared memory.
int launch_moment_sketch_win(const Params& P, const MomentArgs& A, uint32_t w0, uint32_t nw, int sm_count,
                             cudaStream_t st) {
    const size_t smem = window_smem_bytes(P, nw);
    static size_t configured = 0;
    if (smem > configured) {
        if (cudaFuncSetAttribute(k_moment_sketch_win, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return -1;
        configured = smem;
    }
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_moment_sketch_win, kThreads, smem) != cudaSuccess || per_sm < 1)
        return -1;
    const uint32_t units_total = (P.d + kUnit - 1) / kUnit;
    const uint32_t per_panel = (units_total + P.win_panels - 1) / P.win_panels;
    // slices: about 6 units per work item, and enough items to balance the resident blocks
    uint32_t slices = per_panel / 6u;
    if (slices < 1) slices = 1;
    const uint64_t items = (uint64_t)P.win_panels * slices;
    const uint64_t cap = (uint64_t)sm_count * per_sm;
    const int grid = (int)(items < cap ? items : cap);
    k_moment_sketch_win<<<grid, kThreads, smem, st>>>(P, A, w0, nw, slices, units_total);
    return 1;
}

}  // namespace sk
