// Kernels for a step whose workers are partitioned over several processes (one GPU each): every process sketches
// its own workers, and the processes exchange (sum) three things per iteration, the quantities Section III-B counts:
// the sketch (r*c floats), the gradient entries h_t on I_{t-1} (k floats) and the exact values of the selected
// candidates (P*k floats).  The exchanged vectors are indexed by POSITION in an index list, so every process must
// hold the list in the same order: ascending.  The selection kernels append in arrival order, so the lists are put
// in order here through a bitmap (set the bits, then enumerate them), which costs a pass over d/32 words instead
// of a sort.
#include "sk_internal.h"

namespace sk {
namespace {

constexpr int kThreads = 256;
constexpr uint32_t kWordsPerThread = kScanWordsPerBlock / kThreads;   // 4 consecutive words per thread

__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t mine, uint32_t& total) {
    __shared__ uint32_t warp_tot[kThreads / 32];
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    uint32_t incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= (uint32_t)off) incl += o;
    }
    if (lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    uint32_t before = 0;
    total = 0;
#pragma unroll
    for (uint32_t q = 0; q < kThreads / 32; ++q) {
        const uint32_t wt = warp_tot[q];
        if (q < wid) before += wt;
        total += wt;
    }
    __syncthreads();
    return before + incl - mine;
}

// counts[b] = number of set bits in the block's 1024 words
__global__ void __launch_bounds__(kThreads)
k_bits_count(const uint32_t* __restrict__ bitmap, uint64_t words, uint32_t* counts) {
    const uint64_t w0 = (uint64_t)blockIdx.x * kScanWordsPerBlock + (uint64_t)threadIdx.x * kWordsPerThread;
    uint32_t c = 0;
#pragma unroll
    for (uint32_t q = 0; q < kWordsPerThread; ++q)
        if (w0 + q < words) c += __popc(bitmap[w0 + q]);
    uint32_t total;
    block_exclusive_scan(c, total);
    if (threadIdx.x == 0) counts[blockIdx.x] = total;
}

// in-place exclusive scan of counts[0..n) by one block; counts[n] <- grand total
__global__ void __launch_bounds__(kThreads)
k_scan_counts(uint32_t* counts, uint32_t n) {
    __shared__ uint32_t carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (uint32_t base = 0; base < n; base += kThreads) {
        const uint32_t q = base + threadIdx.x;
        const uint32_t mine = q < n ? counts[q] : 0u;
        uint32_t total;
        const uint32_t excl = block_exclusive_scan(mine, total);
        const uint32_t carry = carry_s;
        if (q < n) counts[q] = carry + excl;
        __syncthreads();
        if (threadIdx.x == 0) carry_s = carry + total;
        __syncthreads();
    }
    if (threadIdx.x == 0) counts[n] = carry_s;
}

// the set bits of the block's words, written as ascending coordinates from offsets[block]
__global__ void __launch_bounds__(kThreads)
k_bits_emit(const __grid_constant__ Params P, const uint32_t* __restrict__ bitmap, uint64_t words,
            const uint32_t* __restrict__ offsets, uint32_t* out, uint32_t cap) {
    const uint64_t w0 = (uint64_t)blockIdx.x * kScanWordsPerBlock + (uint64_t)threadIdx.x * kWordsPerThread;
    uint32_t w[kWordsPerThread];
    uint32_t c = 0;
#pragma unroll
    for (uint32_t q = 0; q < kWordsPerThread; ++q) {
        w[q] = (w0 + q < words) ? bitmap[w0 + q] : 0u;
        c += __popc(w[q]);
    }
    uint32_t total;
    uint32_t pos = offsets[blockIdx.x] + block_exclusive_scan(c, total);
#pragma unroll
    for (uint32_t q = 0; q < kWordsPerThread; ++q) {
        uint32_t bits = w[q];
        const uint32_t first = (uint32_t)((w0 + q) << 5);
        while (bits) {
            SK_GUARD(pos < cap, kStatusListPos) out[pos] = first + (uint32_t)(__ffs((int)bits) - 1);
            ++pos;
            bits &= bits - 1u;
        }
    }
}

__global__ void __launch_bounds__(kThreads)
k_list_set_bits(const __grid_constant__ Params P, const uint32_t* __restrict__ list, uint32_t count, uint32_t* bitmap) {
    const uint32_t q = blockIdx.x * kThreads + threadIdx.x;
    if (q < count) SK_GUARD(list[q] < P.d, kStatusIndex) atomicOr(&bitmap[list[q] >> 5], 1u << (list[q] & 31u));
}

__global__ void __launch_bounds__(kThreads)
k_gather(const __grid_constant__ Params P, const uint32_t* __restrict__ list, uint32_t count, uint32_t padded,
         const float* __restrict__ src, float* out) {
    const uint32_t q = blockIdx.x * kThreads + threadIdx.x;
    if (q >= padded) return;
    float val = 0.0f;
    if (q < count) SK_GUARD(list[q] < P.d, kStatusIndex) val = src[list[q]];
    out[q] = val;
}

__global__ void __launch_bounds__(kThreads)
k_scatter(const __grid_constant__ Params P, const uint32_t* __restrict__ list, uint32_t count, const float* __restrict__ vals,
          float* dst) {
    const uint32_t q = blockIdx.x * kThreads + threadIdx.x;
    if (q < count) SK_GUARD(list[q] < P.d, kStatusIndex) dst[list[q]] = vals[q];
}

__global__ void __launch_bounds__(kThreads)
k_gather_worker_sum(const __grid_constant__ Params P, const uint32_t* __restrict__ list, uint32_t count,
                    const float* __restrict__ e, float* out) {
    const uint32_t q = blockIdx.x * kThreads + threadIdx.x;
    if (q >= count) return;
    const uint32_t j = list[q];
    float acc = 0.0f;
    SK_GUARD(j < P.d, kStatusIndex)
        for (uint32_t w = 0; w < P.n; ++w) acc += e[(uint64_t)w * P.d + j];
    out[q] = acc;
}

inline uint32_t blocks_for(uint64_t items) { return (uint32_t)((items + kThreads - 1) / kThreads); }

}  // namespace

int launch_list_from_bitmap(const Params& P, const uint32_t* bitmap, uint64_t words, uint32_t* scan, uint32_t* out,
                            uint32_t cap, cudaStream_t st) {
    const uint32_t nblocks = (uint32_t)((words + kScanWordsPerBlock - 1) / kScanWordsPerBlock);
    if (nblocks == 0) return 0;
    k_bits_count<<<nblocks, kThreads, 0, st>>>(bitmap, words, scan);
    k_scan_counts<<<1, kThreads, 0, st>>>(scan, nblocks);
    k_bits_emit<<<nblocks, kThreads, 0, st>>>(P, bitmap, words, scan, out, cap);
    return 3;
}

int launch_sort_list(const Params& P, uint32_t* list, uint32_t count, uint32_t* scratch_bitmap, uint64_t words, uint32_t* scan,
                     cudaStream_t st) {
    if (count == 0) return 0;
    int l = launch_zero(scratch_bitmap, words * 4, st);        // words * 4 is a multiple of 16 (the bitmap's padding)
    k_list_set_bits<<<blocks_for(count), kThreads, 0, st>>>(P, list, count, scratch_bitmap);
    return l + 1 + launch_list_from_bitmap(P, scratch_bitmap, words, scan, list, count, st);
}

int launch_gather(const Params& P, const uint32_t* list, uint32_t count, uint32_t padded, const float* src, float* out,
                  cudaStream_t st) {
    if (padded == 0) return 0;
    k_gather<<<blocks_for(padded), kThreads, 0, st>>>(P, list, count, padded, src, out);
    return 1;
}

int launch_scatter(const Params& P, const uint32_t* list, uint32_t count, const float* vals, float* dst, cudaStream_t st) {
    if (count == 0) return 0;
    k_scatter<<<blocks_for(count), kThreads, 0, st>>>(P, list, count, vals, dst);
    return 1;
}

int launch_gather_worker_sum(const Params& P, const uint32_t* list, uint32_t count, const float* e, float* out,
                             cudaStream_t st) {
    if (count == 0) return 0;
    k_gather_worker_sum<<<blocks_for(count), kThreads, 0, st>>>(P, list, count, e, out);
    return 1;
}

}  // namespace sk
