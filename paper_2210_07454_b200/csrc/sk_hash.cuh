// Bucket and sign hashes of the Count Sketch (Section II-C names {h_j},{s_j}; the family is the library's own
// and is documented with sk_hash in the public header).  Device-side evaluation only.
#pragma once
#include <cstdint>
#include "sk_internal.h"

namespace sk {

constexpr uint64_t kGolden = 0x9E3779B97F4A7C15ULL;
constexpr uint32_t kUnitShift = 10;     // windowed family: units of 1024 coordinates
constexpr uint32_t kUnit = 1u << kUnitShift;
constexpr uint32_t kQuadsPerUnit = kUnit / 4;         // 256
constexpr uint32_t kGroupsPerUnit = kUnit / 32;       // 32

__host__ __device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

// t-th output (t >= 1) of splitmix64 started at state s
__host__ __device__ __forceinline__ uint64_t stream(uint64_t s, uint64_t t) { return mix64(s + t * kGolden); }

__host__ __device__ __forceinline__ uint64_t row_key(uint64_t seed, uint32_t row) {
    return stream(seed, (uint64_t)row + 1);
}

// first bucket of the window that coordinate i's unit owns in every row (0 for the plain family)
__device__ __forceinline__ uint32_t window_base(const Params& P, uint32_t i) {
    return P.win_cw ? ((i >> kUnitShift) % P.win_panels) * P.win_cw : 0u;
}

// What one group of g = 2^log2g consecutive coordinates needs in one row.
struct GroupHash {
    uint32_t base;   // first bucket of the group's aligned block (relative to the window base, if any)
    uint32_t perm;   // xor permutation inside the block, in [0,g)
    uint32_t sign;   // 1  <=>  the group's coordinates carry sign -1 in this row (one sign per row and group)
};

// from one 64-bit draw u: high word -> block by multiply-high range reduction over P.G choices, the leading
// bits of the remainder -> xor permutation, bit 0 of the low word -> the group's sign
__device__ __forceinline__ GroupHash group_from_draw(const Params& P, uint64_t u) {
    const uint32_t hi = (uint32_t)(u >> 32);
    GroupHash h;
    h.base = __umulhi(hi, P.G) << P.log2g;
    h.perm = P.log2g ? ((hi * P.G) >> (32u - P.log2g)) : 0u;
    h.sign = (uint32_t)u & 1u;
    return h;
}

// Scalar form: bucket and sign (+1/-1) of coordinate i in the row with key `key`.
__device__ __forceinline__ void coord_hash(const Params& P, uint64_t key, uint32_t i, uint32_t& bucket, float& sign) {
    const uint32_t q = i >> P.log2g, o = i & ((1u << P.log2g) - 1u);
    const GroupHash h = group_from_draw(P, stream(key, (uint64_t)q + 1));
    bucket = window_base(P, i) + h.base + (o ^ h.perm);
    sign = h.sign ? -1.0f : 1.0f;
}

// Vector form for 4 consecutive coordinates i..i+3 (i % 4 == 0, g >= 4): they land in one aligned 16-byte
// chunk of the row.  `off` is the element offset of that chunk inside the row; local coordinate l goes to
// element (l xor p3) of the chunk; all four carry the group's sign.
struct Quad {
    uint32_t off;
    uint32_t p3sgn;  // bits 0..1: p3 ; bit 2: the sign bit (1 = negative)
};

__device__ __forceinline__ Quad quad_from_draw(const Params& P, uint64_t u, uint32_t i, uint32_t wbase) {
    const uint32_t o = i & ((1u << P.log2g) - 1u);
    const GroupHash h = group_from_draw(P, u);
    Quad r;
    r.off = wbase + h.base + ((o ^ h.perm) & ~3u);
    r.p3sgn = (h.perm & 3u) | (h.sign << 2);
    return r;
}

// Hashes of coordinate quad t (coordinates 4t..4t+3) in rows 0..r-1.  With g = 32 the eight lanes that share a
// group split the rows between them (one 64-bit draw per lane and round) and exchange the draws by shuffle, so
// ALL 32 LANES OF THE WARP MUST CALL THIS TOGETHER (callers clamp t for lanes past the end).
template <int RMAX>
__device__ __forceinline__ void quad_hashes(const Params& P, uint32_t r, uint32_t t, Quad (&h)[RMAX]) {
    const uint32_t i = t << 2;
    const uint32_t wbase = window_base(P, i);
    if (P.log2g == 5) {
        const uint32_t lane = threadIdx.x & 31u, li = lane & 7u, q = t >> 3;
#pragma unroll
        for (uint32_t k = 0; k < (uint32_t)RMAX; k += 8) {
            if (k < r) {
                const uint64_t key = P.row_key[(k + li) & (kMaxRows - 1u)];   // indexed read of the kernel parameter
                const uint64_t u = (k + li < r) ? stream(key, (uint64_t)q + 1) : 0ull;
                const uint32_t hi = (uint32_t)(u >> 32), lo = (uint32_t)u;
#pragma unroll
                for (uint32_t j = 0; j < 8; ++j)
                    if (k + j < (uint32_t)RMAX && k + j < r) {
                        const uint32_t src = (lane & ~7u) + j;
                        const uint32_t ohi = __shfl_sync(0xFFFFFFFFu, hi, src);
                        const uint32_t olo = __shfl_sync(0xFFFFFFFFu, lo, src);
                        // g = 32 written out: block = floor(hi * G / 2^32), permutation = the next 5 bits
                        const uint32_t o = i & 31u, perm = (ohi * P.G) >> 27;
                        h[k + j].off = wbase + (__umulhi(ohi, P.G) << 5) + ((o ^ perm) & ~3u);
                        h[k + j].p3sgn = (perm & 3u) | ((olo & 1u) << 2);
                    }
            }
        }
    } else {
#pragma unroll
        for (uint32_t row = 0; row < (uint32_t)RMAX; ++row)
            if (row < r) h[row] = quad_from_draw(P, stream(P.row_key[row], (uint64_t)(i >> P.log2g) + 1), i, wbase);
    }
}

// The units in panel-major order: panel 0's units, then panel 1's, ...  Panel p owns the units p, p + panels,
// p + 2 panels, ...; the first `rem` panels have `tbig` of them, the others tbig - 1.
struct UnitWalk {
    uint32_t panels, tbig, rem;
    uint32_t panel, tu;
    __device__ __forceinline__ void seek(uint32_t s) {
        const uint32_t head = rem * tbig;
        if (s < head) { panel = s / tbig; tu = s - panel * tbig; }
        else { const uint32_t q = s - head; panel = rem + q / (tbig - 1u); tu = q - (panel - rem) * (tbig - 1u); }
    }
    __device__ __forceinline__ uint32_t unit() const { return panel + panels * tu; }
    __device__ __forceinline__ void next() {
        const uint32_t T = panel < rem ? tbig : tbig - 1u;
        if (++tu >= T) { tu = 0; ++panel; }
    }
};

__device__ __forceinline__ float flip(float a, uint32_t bit) {  // a * (bit ? -1 : +1)
    return __uint_as_float(__float_as_uint(a) ^ (bit << 31));
}

// signed and permuted: out element e = s(l) * a_l with l = e xor p3
__device__ __forceinline__ float4 quad_scatter(const Quad h, float4 a) {
    const uint32_t s = (h.p3sgn << 29) & 0x80000000u;  // the group's sign bit, in the sign position of a float
    a.x = __uint_as_float(__float_as_uint(a.x) ^ s);
    a.y = __uint_as_float(__float_as_uint(a.y) ^ s);
    a.z = __uint_as_float(__float_as_uint(a.z) ^ s);
    a.w = __uint_as_float(__float_as_uint(a.w) ^ s);
    if (h.p3sgn & 1u) { float t = a.x; a.x = a.y; a.y = t; t = a.z; a.z = a.w; a.w = t; }
    if (h.p3sgn & 2u) { float t = a.x; a.x = a.z; a.z = t; t = a.y; a.y = a.w; a.w = t; }
    return a;
}

// inverse: given the chunk's 4 values, return s(l) * chunk[l xor p3] for l = 0..3 (xor is an involution)
__device__ __forceinline__ float4 quad_gather(const Quad h, float4 cch) {
    if (h.p3sgn & 1u) { float t = cch.x; cch.x = cch.y; cch.y = t; t = cch.z; cch.z = cch.w; cch.w = t; }
    if (h.p3sgn & 2u) { float t = cch.x; cch.x = cch.z; cch.z = t; t = cch.y; cch.y = cch.w; cch.w = t; }
    const uint32_t s = (h.p3sgn << 29) & 0x80000000u;  // the group's sign bit, in the sign position of a float
    cch.x = __uint_as_float(__float_as_uint(cch.x) ^ s);
    cch.y = __uint_as_float(__float_as_uint(cch.y) ^ s);
    cch.z = __uint_as_float(__float_as_uint(cch.z) ^ s);
    cch.w = __uint_as_float(__float_as_uint(cch.w) ^ s);
    return cch;
}

}  // namespace sk
