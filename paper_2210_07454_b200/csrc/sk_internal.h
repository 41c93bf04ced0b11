// Internal declarations shared by the kernel file and the C-ABI file.  Not installed.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>
#include "sk_debug.cuh"
#include "sk_chain.cuh"

namespace sk {

constexpr uint32_t kMaxRows = 16;
constexpr uint32_t kHistBits = 12;                 // first-level histogram: key bits 30..19
constexpr uint32_t kHistBins = 1u << kHistBits;
constexpr uint32_t kHistShift = 31 - kHistBits;    // 19

// Everything a kernel needs to know about the problem; passed by value as a __grid_constant__.
struct Params {
    uint64_t row_key[kMaxRows];
    uint32_t d, n, r, c;
    uint32_t cs;        // row stride of every table in floats (c rounded up to 32)
    uint32_t log2g, G;  // hash group size 2^log2g; number of blocks a group chooses from (c >> log2g, or the
                        // lines of a window in the windowed family)
    uint32_t win_cw;      // windowed family: buckets per window (32 * lines), 0 = plain family
    uint32_t win_panels;  // windowed family: windows per row = c / win_cw
    uint32_t k;
    float beta1, beta2, lr;
    float rho;          // alpha_{t-1}/alpha_t, the weight of e_{t-1} in the sketched vector (1 for a constant step size)
    uint32_t* status;   // the handle's device status word (bits: sk_debug.cuh); nullptr = none
    uint32_t n_all;     // workers the means are taken over: n, or the total over all processes when the workers are
                        // partitioned (the handle then holds n of them)
    uint32_t chain;     // host side only: the step's kernels are launched chained (sk_chain.cuh)
};

// Device-resident selection state (one per handle).
struct Select {
    uint32_t bin;        // first-level threshold bin
    uint32_t need;       // how many candidates of the threshold bin are still to be taken
    uint32_t cnt_out;    // indices emitted so far
    uint32_t cnt_cand;   // candidates collected
    uint32_t status;     // 0 ok; bit 0: emitted count != k
    uint32_t bin2;       // second-level threshold bin (key bits 18..7) inside `bin`
    uint32_t need2;      // how many of the candidates sharing the threshold's first 24 key bits are to be taken
    uint32_t cnt_cand2;  // candidates sharing the threshold's first 24 key bits
};

struct Cand { uint32_t key, idx; };

// Pointers of the moment + sketch kernel (all device memory).
struct MomentArgs {
    const void* grads;       // n*d gradient entries, fp32 or (grad_bf16 != 0) bf16
    uint32_t grad_bf16;
    float *m, *e, *tables;
    float* sum_table;        // not nullptr: sketch the worker sum of a_t once into this r x cs table (already divided by
                             // n_all) instead of one table per worker -- the sketch is linear (Section II-C)
    float* asum;             // d or nullptr: running sum over the workers of a_t, in worker order (second round of Section III-A)
    float* gsum;             // gradient sums on I_{t-1}, per coordinate.  Zero between steps: the key pass clears what it
                             // consumes, so a kernel may either overwrite a member's quad or add to it
    float *v, *vhat;
    uint32_t* vstamp;        // step at which v[j] was last brought up to date
    const uint32_t* bitmap;  // membership of I_{t-1}: bit j of word j/32
    uint32_t step;           // t (1-based)
    uint32_t members;        // 0 when I_{t-1} is empty
    uint32_t gsum_on;        // the gradient sums on I_{t-1} are wanted (members != 0, Algorithm 2, v not frozen)
    // parameter-averaging variant (Algorithm 1): per-worker second moments, n*d each; variant = 1
    float *vw, *vhatw;
    uint32_t variant;        // 0 = gradient averaging (Algorithm 2), 1 = parameter averaging (Algorithm 1)
};

// Launchers.  Each enqueues on `st` and returns the number of kernels it launched.
int sm_count_of_device();
// debug build only: one thread runs a bounds check with a false condition of the given kind (no access is made)
int launch_debug_violation(const Params& P, uint32_t bit, cudaStream_t st);
int launch_zero(void* p, uint64_t bytes, cudaStream_t st, bool chain = false);
int launch_fill_u32(uint32_t* p, uint64_t n, uint32_t value, cudaStream_t st);
int launch_set_bits(const Params& P, const uint32_t* I, uint32_t count, uint32_t* bitmap, cudaStream_t st);
int launch_moment_sketch(const Params& P, const MomentArgs& A, uint32_t w0, uint32_t nw, bool vec, int sm_count,
                         cudaStream_t st);
// windowed hash family, accumulation by ownership (one warp per worker, block-owned windows): at most kOwnMaxWorkers
// workers per launch; fills A.asum when it is set; -1 if it cannot run
constexpr uint32_t kOwnMaxWorkers = 8;
int launch_moment_sketch_own(const Params& P, const MomentArgs& A, uint32_t w0, uint32_t nw, int sm_count,
                             cudaStream_t st);
int launch_sum_tables(const Params& P, const float* tables, float* sum, cudaStream_t st);
// A.members != 0: also apply the second-moment update on I_{t-1} (bitmap, gsum, v, vstamp, vhat of A)
int launch_unsketch_hist(const Params& P, const MomentArgs& A, const float* sum, uint32_t* keys, uint32_t* hist,
                         bool vec, int sm_count, cudaStream_t st);
int launch_pick_bin(const Params& P, uint32_t* hist, Select* sel, int level, cudaStream_t st);
// selection runs over P.d keys for the P.k largest; idx_map != nullptr: key t belongs to coordinate idx_map[t]
// clear / clear_bytes (a multiple of 16, or nullptr / 0): a buffer the pass also zeroes (the bitmap of I_{t-1})
int launch_emit(const Params& P, const uint32_t* keys, const uint32_t* idx_map, Select* sel, uint32_t* I_out, Cand* cand,
                uint32_t* hist2, int sm_count, cudaStream_t st, void* clear = nullptr, uint64_t clear_bytes = 0);
// second round: exact values of `count` candidate coordinates as ranking keys, with their first-level histogram
// asum != nullptr: sum_w a^(w) per coordinate is read from there instead of gathering e for every worker
int launch_exact_keys(const Params& P, const uint32_t* C, uint32_t count, const float* vhat, const float* e,
                      const float* asum,
                      uint32_t* keys2, uint32_t* hist, int sm_count, cudaStream_t st);
int launch_refine(const Params& P, Select* sel, const Cand* cand, Cand* cand2, uint32_t* hist2, uint32_t* I_out,
                  int sm_count, cudaStream_t st);
// vhat == nullptr: parameter averaging, the update is the plain mean (Algorithm 1)
int launch_apply(const Params& P, const uint32_t* I, const float* vhat, const float* e, const float* asum, float* x,
                 uint32_t* bitmap,
                 cudaStream_t st);
// helpers for state export / import
int launch_estimates(const Params& P, const float* sum, const float* vhat, float* est, cudaStream_t st);
int launch_hash_export(const Params& P, uint32_t row, uint64_t i0, uint64_t count, uint32_t* idx, int8_t* sgn,
                       cudaStream_t st);
int launch_v_materialize(const Params& P, const float* v, const uint32_t* vstamp, uint32_t t, float* out,
                         cudaStream_t st);
int launch_masked_copy(const Params& P, const float* e, const uint32_t* bitmap, uint32_t workers, float* out,
                       cudaStream_t st);
// ---- workers partitioned over processes (sk_shard.cu): canonical (ascending) index lists and the packing of what
// the processes exchange
constexpr uint32_t kScanWordsPerBlock = 1024;      // bitmap words one block of the compaction covers
inline uint64_t scan_entries(uint64_t bitmap_words) { return (bitmap_words + kScanWordsPerBlock - 1) / kScanWordsPerBlock + 1; }
// out <- the set bits of the bitmap as ascending coordinates; scan: scratch of scan_entries(words) uint32
// cap: capacity of `out`; P: for the debug build's checks
int launch_list_from_bitmap(const Params& P, const uint32_t* bitmap, uint64_t words, uint32_t* scan, uint32_t* out,
                            uint32_t cap, cudaStream_t st);
// sorts a list of distinct coordinates in place through a scratch bitmap of `words` words
int launch_sort_list(const Params& P, uint32_t* list, uint32_t count, uint32_t* scratch_bitmap, uint64_t words, uint32_t* scan,
                     cudaStream_t st);
// out[q] = src[list[q]] for q < count, 0 for count <= q < padded
int launch_gather(const Params& P, const uint32_t* list, uint32_t count, uint32_t padded, const float* src, float* out,
                  cudaStream_t st);
// dst[list[q]] = vals[q]
int launch_scatter(const Params& P, const uint32_t* list, uint32_t count, const float* vals, float* dst, cudaStream_t st);
// out[q] = sum over this handle's workers (in order) of e[w][list[q]]
int launch_gather_worker_sum(const Params& P, const uint32_t* list, uint32_t count, const float* e, float* out,
                             cudaStream_t st);

}  // namespace sk
