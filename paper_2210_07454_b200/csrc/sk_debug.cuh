// Device-side bounds checks of the debug build (-DSK_DEBUG=1).
//
// Every offset a hash produces, every position a list is appended at, every index taken from a list and every
// histogram bin is compared with the size of what it addresses.  A violation sets a bit in the handle's device
// status word (the one sk_sync reads back and reports) and the access is SKIPPED; nothing traps, so the context
// stays usable and the host sees an error code.  In the normal build the checks compile to nothing.
#pragma once
#include <cstdint>

namespace sk {

enum : uint32_t {
    kStatusCount = 1u,      // the selection emitted a number of indices other than k
    kStatusBucket = 2u,     // a hashed table offset outside its row / table
    kStatusIndex = 4u,      // a coordinate index >= d taken from or written to a list
    kStatusListPos = 8u,    // an append position outside the list's capacity
    kStatusBin = 16u,       // a histogram bin outside the histogram
    kStatusWindow = 32u,    // a shared-memory window offset outside the window
    kStatusNonFinite = 64u, // a gradient entry that is not finite (inputs must be finite; the step goes on regardless)
};

#ifdef SK_DEBUG
__device__ __forceinline__ bool in_bounds(bool ok, uint32_t* status, uint32_t bit) {
    if (!ok && status) atomicOr(status, bit);
    return ok;
}
#else
__device__ __forceinline__ bool in_bounds(bool, uint32_t*, uint32_t) { return true; }
#endif

}  // namespace sk

// debug build: a non-finite entry of a gradient quad is recorded (nothing is skipped: the arithmetic cannot fault)
#ifdef SK_DEBUG
#define SK_CHECK_FINITE4(g)                                                                                   \
    sk::in_bounds(isfinite((g).x) && isfinite((g).y) && isfinite((g).z) && isfinite((g).w), P.status, sk::kStatusNonFinite)
#else
#define SK_CHECK_FINITE4(g) ((void)0)
#endif

// `statement` runs only if `cond` holds; in the debug build a failed `cond` is recorded in P.status
#define SK_GUARD(cond, bit) if (sk::in_bounds((cond), P.status, (bit)))
