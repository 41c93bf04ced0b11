// Moments + error-feedback accumulate + Count Sketch for the WINDOWED hash family, accumulating on chip.
//
// In the windowed family every unit of 1024 coordinates hashes, in every row, into one aligned window of the row
// (the window of the unit's panel).  A thread block therefore takes a panel (or a slice of its units), keeps the
// panel's window of every (worker, row) table in shared memory, adds the units' values there, and writes each
// window out once with 16-byte reductions.  Only the dense stream (read g, m, e; write m, a) and these small
// flushes leave the SM, instead of one reduction per (coordinate, row, worker).
//
// The block is split by role so that the memory stream and the shared-memory accumulation overlap:
//   producers (8 warps): per unit, the dense update of 4 coordinates per thread for every worker of the launch
//       (loads, moments, stores), a_t staged in shared memory, and the unit's 32 x r group hashes;
//   consumers (one 8-lane sub-warp per (worker,row) window): add the staged values into their window with
//       128-bit read-add-write.  A window has one owner, so no atomics; the 8 lanes of one access touch the 8
//       distinct 16-byte chunks of one 128-byte line, so no bank conflicts.
// The two roles hand the double-buffered stage over with the hardware's named barriers (arrive / sync pairs);
// every thread of the block takes part in every barrier the same number of times.
#include "sk_internal.h"
#include "sk_hash.cuh"
#include "sk_moment.cuh"

namespace sk {

namespace {

constexpr int kProducerThreads = 256;
constexpr uint32_t kUnit = 1u << kUnitShift;      // 1024 coordinates
constexpr uint32_t kGroupsPerUnit = kUnit / 32;   // 32
constexpr int kMaxConsumerWarps = 16;
constexpr uint32_t kMaxRedRows = 4;               // at most this many rows go through L2 reductions in this kernel

__device__ __forceinline__ void red_add_v4(float* addr, float4 v) {
    asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                 :: "l"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w));
}

// named barriers 1..4 (0 is left to __syncthreads): FULL[b] = 1 + b, EMPTY[b] = 3 + b
__device__ __forceinline__ void bar_sync(uint32_t id, uint32_t count) {
    asm volatile("bar.sync %0, %1;" :: "r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_arrive(uint32_t id, uint32_t count) {
    asm volatile("bar.arrive %0, %1;" :: "r"(id), "r"(count) : "memory");
}

#define SK_MOMENT(mm, aa, gg, mask)                                                     \
    mm.x = fmaf(b1, mm.x, omb1 * gg.x); mm.y = fmaf(b1, mm.y, omb1 * gg.y);             \
    mm.z = fmaf(b1, mm.z, omb1 * gg.z); mm.w = fmaf(b1, mm.w, omb1 * gg.w);             \
    aa.x = fmaf(rho, (mask & 1u) ? 0.0f : aa.x, mm.x); aa.y = fmaf(rho, (mask & 2u) ? 0.0f : aa.y, mm.y); \
    aa.z = fmaf(rho, (mask & 4u) ? 0.0f : aa.z, mm.z); aa.w = fmaf(rho, (mask & 8u) ? 0.0f : aa.w, mm.w);

// units of work item `item`: panel, and the half-open range [t_begin, t_end) of the panel's unit list
__device__ __forceinline__ void item_range(const Params& P, uint32_t item, uint32_t slices, uint32_t units_total,
                                           uint32_t& panel, uint32_t& t_begin, uint32_t& t_end) {
    panel = item % P.win_panels;
    const uint32_t slice = item / P.win_panels;
    const uint32_t T = panel < units_total ? (units_total - panel + P.win_panels - 1) / P.win_panels : 0u;
    t_begin = (uint32_t)((uint64_t)T * slice / slices);
    t_end = (uint32_t)((uint64_t)T * (slice + 1) / slices);
}

__global__ void __launch_bounds__(kProducerThreads + 32 * kMaxConsumerWarps)
k_moment_sketch_win(const __grid_constant__ Params P, const __grid_constant__ MomentArgs A, uint32_t w0, uint32_t nw,
                    uint32_t slices, uint32_t units_total, uint32_t r_red) {
    // rows [0, r_red) are sketched by the producers with reductions into the L2-resident tables; rows [r_red, r)
    // by the consumers in shared-memory windows: the two mechanisms load different parts of the SM (the request
    // port towards L2, and instruction issue + shared memory), so splitting the rows lets both stay below the
    // time of the memory stream.
    extern __shared__ __align__(16) float smem[];
    const uint32_t r = P.r, cw = P.win_cw;
    const uint32_t pairs = nw * (r - r_red);
    float* win = smem;                                         // [pairs][cw]
    float* stage = win + (size_t)pairs * cw;                   // [2][nw][1024]
    uint2* hsh = (uint2*)(stage + (size_t)2 * nw * kUnit);     // [2][r][32]: x = line*32 | perm, y = sign bits
    const uint32_t tid = threadIdx.x;
    const uint32_t nthreads = blockDim.x;
    const uint32_t items = P.win_panels * slices;

    if (tid < kProducerThreads) {
        // ------------------------------------------------------------------------------------ producer
        float4* m = (float4*)A.m;
        float4* e = (float4*)A.e;
        const uint32_t d4 = P.d >> 2;
        const float b1 = P.beta1, omb1 = 1.0f - P.beta1, rho = P.rho;
        const uint32_t gb = A.grad_bf16;
        const uint64_t tstride = (uint64_t)P.r * P.cs;
        uint32_t seq = 0;                                      // units produced by this block so far
        for (uint32_t item = blockIdx.x; item < items; item += gridDim.x) {
            uint32_t panel, t_begin, t_end;
            item_range(P, item, slices, units_total, panel, t_begin, t_end);
            for (uint32_t tu = t_begin; tu < t_end; ++tu, ++seq) {
                const uint32_t unit = panel + P.win_panels * tu;
                const uint32_t b = seq & 1u;
                if (seq >= 2) bar_sync(3 + b, nthreads);       // wait until the consumers are done with buffer b
                float* st = stage + (size_t)b * nw * kUnit;
                uint2* hs = hsh + (size_t)b * r * kGroupsPerUnit;
                for (uint32_t hq = r_red * kGroupsPerUnit + tid; hq < r * kGroupsPerUnit; hq += kProducerThreads) {
                    const uint32_t row = hq >> 5, s = hq & 31u;
                    const GroupHash gh = group_from_draw(P, stream(P.row_key[row], (uint64_t)unit * kGroupsPerUnit + s + 1));
                    hs[hq] = make_uint2(gh.base | gh.perm, gh.signs);
                }
                const uint32_t t = unit * (kUnit / 4) + tid;
                Quad hr[kMaxRedRows];                          // this quad's hashes in the rows sketched by reductions
                quad_hashes<kMaxRedRows>(P, r_red, t < d4 ? t : d4 - 1, hr);
                if (t < d4) {
                    const uint32_t mask = A.members ? ((__ldg(A.bitmap + (t >> 3)) >> ((t & 7u) * 4u)) & 0xFu) : 0u;
                    float4 gs = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (mask && w0 > 0) gs = ((const float4*)A.gsum)[t];
                    uint32_t w = 0;
                    for (; w + 2 <= nw; w += 2) {
                        const uint64_t q0 = (uint64_t)(w0 + w) * d4 + t, q1 = q0 + d4;
                        const float4 g0 = load_grad4(A.grads, q0, gb), g1 = load_grad4(A.grads, q1, gb);
                        float4 m0 = __ldcs(m + q0), m1 = __ldcs(m + q1);
                        float4 a0 = __ldcs(e + q0), a1 = __ldcs(e + q1);
                        SK_MOMENT(m0, a0, g0, mask)
                        SK_MOMENT(m1, a1, g1, mask)
                        gs.x = (gs.x + g0.x) + g1.x; gs.y = (gs.y + g0.y) + g1.y;
                        gs.z = (gs.z + g0.z) + g1.z; gs.w = (gs.w + g0.w) + g1.w;
                        __stcs(m + q0, m0); __stcs(m + q1, m1);
                        __stcs(e + q0, a0); __stcs(e + q1, a1);
                        ((float4*)(st + (size_t)w * kUnit))[tid] = a0;
                        ((float4*)(st + (size_t)(w + 1) * kUnit))[tid] = a1;
                        float* t0 = A.tables + (uint64_t)(w0 + w) * tstride;
#pragma unroll
                        for (uint32_t row = 0; row < kMaxRedRows; ++row)
                            if (row < r_red) {
                                red_add_v4(t0 + (uint64_t)row * P.cs + hr[row].off, quad_scatter(hr[row], a0));
                                red_add_v4(t0 + tstride + (uint64_t)row * P.cs + hr[row].off, quad_scatter(hr[row], a1));
                            }
                    }
                    if (w < nw) {
                        const uint64_t q0 = (uint64_t)(w0 + w) * d4 + t;
                        const float4 g0 = load_grad4(A.grads, q0, gb);
                        float4 m0 = __ldcs(m + q0);
                        float4 a0 = __ldcs(e + q0);
                        SK_MOMENT(m0, a0, g0, mask)
                        gs.x += g0.x; gs.y += g0.y; gs.z += g0.z; gs.w += g0.w;
                        __stcs(m + q0, m0);
                        __stcs(e + q0, a0);
                        ((float4*)(st + (size_t)w * kUnit))[tid] = a0;
                        float* t0 = A.tables + (uint64_t)(w0 + w) * tstride;
#pragma unroll
                        for (uint32_t row = 0; row < kMaxRedRows; ++row)
                            if (row < r_red) red_add_v4(t0 + (uint64_t)row * P.cs + hr[row].off, quad_scatter(hr[row], a0));
                    }
                    if (mask) ((float4*)A.gsum)[t] = gs;
                } else {
                    for (uint32_t w = 0; w < nw; ++w)          // past the end of the vector: contribute zeros
                        ((float4*)(st + (size_t)w * kUnit))[tid] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                __threadfence_block();
                __syncwarp();
                bar_arrive(1 + b, nthreads);                   // buffer b is full
            }
        }
    } else {
        // ------------------------------------------------------------------------------------ consumer
        const uint32_t ctid = tid - kProducerThreads;
        const uint32_t sub = ctid >> 3, l8 = ctid & 7u;        // sub-warp index and lane inside it
        const uint32_t nsub = (nthreads - kProducerThreads) >> 3;
        const uint32_t submask = 0xFFu << (8u * ((tid & 31u) >> 3));   // the 8 lanes that share this sub-warp
        const uint64_t tstride = (uint64_t)P.r * P.cs;
        // total units of this block (the same count the producers walk through)
        uint32_t total = 0;
        for (uint32_t item = blockIdx.x; item < items; item += gridDim.x) {
            uint32_t panel, t_begin, t_end;
            item_range(P, item, slices, units_total, panel, t_begin, t_end);
            total += t_end - t_begin;
        }
        uint32_t seq = 0;
        for (uint32_t item = blockIdx.x; item < items; item += gridDim.x) {
            uint32_t panel, t_begin, t_end;
            item_range(P, item, slices, units_total, panel, t_begin, t_end);
            if (t_begin == t_end) continue;
            // a sub-warp owns the windows sub, sub + nsub, ... : clear them
            for (uint32_t pr = sub; pr < pairs; pr += nsub)
                for (uint32_t q = l8; q < cw / 4; q += 8) ((float4*)(win + (size_t)pr * cw))[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            __syncwarp();
            for (uint32_t tu = t_begin; tu < t_end; ++tu, ++seq) {
                const uint32_t b = seq & 1u;
                __syncwarp();
                bar_sync(1 + b, nthreads);                     // wait until buffer b is full
                const float* st = stage + (size_t)b * nw * kUnit;
                const uint2* hs = hsh + (size_t)b * r * kGroupsPerUnit;
                for (uint32_t pr = sub; pr < pairs; pr += nsub) {
                    const uint32_t w = pr % nw, row = r_red + pr / nw;
                    float* wn = win + (size_t)pr * cw;
                    const float4* sw = (const float4*)(st + (size_t)w * kUnit) + l8;
                    const uint2* hr = hs + row * kGroupsPerUnit;
                    uint2 h = hr[0];
                    float4 val = sw[0];
#pragma unroll 4
                    for (uint32_t s = 0; s < kGroupsPerUnit; ++s) {
                        // fetch the next group's hash and values before touching the window (they never alias it)
                        const uint32_t sn = s + 1 < kGroupsPerUnit ? s + 1 : s;
                        const uint2 hn = hr[sn];
                        const float4 vn = sw[sn * 8u];
                        Quad qd;
                        qd.off = (h.x & ~31u) + 4u * ((l8 ^ (h.x >> 2)) & 7u);
                        qd.p3sgn = (h.x & 3u) | (((h.y >> (4u * l8)) & 0xFu) << 2);
                        const float4 add = quad_scatter(qd, val);
                        float4* dst = (float4*)(wn + qd.off);
                        float4 cur = *dst;
                        cur.x += add.x; cur.y += add.y; cur.z += add.z; cur.w += add.w;
                        *dst = cur;
                        __syncwarp(submask);                   // the next group may land on chunks other lanes just wrote
                        h = hn; val = vn;
                    }
                }
                __threadfence_block();
                __syncwarp();
                if (seq + 2 < total) bar_arrive(3 + b, nthreads);   // buffer b may be refilled (if anyone still will)
            }
            __syncwarp();
            // flush this sub-warp's windows: table[w][row][panel*cw + ...] += window
            for (uint32_t pr = sub; pr < pairs; pr += nsub) {
                const uint32_t w = pr % nw, row = r_red + pr / nw;
                float* dstrow = A.tables + (uint64_t)(w0 + w) * tstride + (uint64_t)row * P.cs + (uint64_t)panel * cw;
                for (uint32_t q = l8; q < cw / 4; q += 8) red_add_v4(dstrow + 4u * q, ((const float4*)(win + (size_t)pr * cw))[q]);
            }
            __syncwarp();
        }
    }
}

inline uint32_t consumer_warps(uint32_t pairs) {
    const uint32_t want = (pairs + 3) / 4;
    return want < (uint32_t)kMaxConsumerWarps ? (want ? want : 1u) : (uint32_t)kMaxConsumerWarps;
}

}  // namespace

size_t window_smem_bytes(const Params& P, uint32_t nw, uint32_t r_red) {
    return ((size_t)nw * (P.r - r_red) * P.win_cw + (size_t)2 * nw * kUnit) * 4 + (size_t)2 * P.r * kGroupsPerUnit * 8;
}

// Enqueues the windowed kernel for workers w0..w0+nw-1 (nw <= kWinMaxWorkers).  Returns launches, or -1 if the
// configuration does not fit in shared memory.
int launch_moment_sketch_win(const Params& P, const MomentArgs& A, uint32_t w0, uint32_t nw, uint32_t r_red,
                             int sm_count, cudaStream_t st) {
    if (r_red > kMaxRedRows) r_red = kMaxRedRows;
    if (r_red > P.r) r_red = P.r;
    const size_t smem = window_smem_bytes(P, nw, r_red);
    const int threads = kProducerThreads + 32 * (int)consumer_warps(nw * (P.r - r_red));
    static size_t configured = 0;
    if (smem > configured) {
        if (cudaFuncSetAttribute(k_moment_sketch_win, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return -1;
        configured = smem;
    }
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_moment_sketch_win, threads, smem) != cudaSuccess || per_sm < 1)
        return -1;
    const uint32_t units_total = (P.d + kUnit - 1) / kUnit;
    const uint32_t per_panel = (units_total + P.win_panels - 1) / P.win_panels;
    // slices: about 8 units per work item, so that a flush is small next to the stream it closes
    uint32_t slices = per_panel / 8u;
    if (slices < 1) slices = 1;
    const uint64_t items = (uint64_t)P.win_panels * slices;
    const uint64_t cap = (uint64_t)sm_count * per_sm;
    const int grid = (int)(items < cap ? items : cap);
    k_moment_sketch_win<<<grid, threads, smem, st>>>(P, A, w0, nw, slices, units_total, r_red);
    return 1;
}

}  // namespace sk
