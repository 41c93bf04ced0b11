// Internal declarations shared by the kernel file and the C-ABI file.  Not installed.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

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
    uint32_t log2g, G;  // hash group size 2^log2g and number of bucket groups c >> log2g
    uint32_t k;
    float beta1, beta2, lr;
};

// Device-resident selection state (one per handle).
struct Select {
    uint32_t bin;        // first-level threshold bin
    uint32_t need;       // how many candidates of the threshold bin are still to be taken
    uint32_t cnt_out;    // indices emitted so far
    uint32_t cnt_cand;   // candidates collected
    uint32_t status;     // 0 ok; bit 0: emitted count != k; bit 1: candidate overflow
    uint32_t pad[3];
};

struct Cand { uint32_t key, idx; };

// Launchers.  Each enqueues on `st` and returns the number of kernels it launched.
int launch_zero(float* p, uint64_t nfloats, cudaStream_t st);
int launch_second_moment(const Params& P, const float* grads, float* v, float* vhat, uint32_t* vstamp,
                         const uint32_t* I_prev, uint32_t k_prev, uint32_t t, cudaStream_t st);
int launch_moment_sketch(const Params& P, const float* grads, float* m, float* e, float* tables,
                         uint32_t w0, uint32_t nw, bool vec, int sm_count, cudaStream_t st);
int launch_sum_tables(const Params& P, const float* tables, float* sum, cudaStream_t st);
int launch_unsketch_hist(const Params& P, const float* sum, const float* vhat, uint32_t* hist, bool vec,
                         int sm_count, cudaStream_t st);
int launch_pick_bin(const Params& P, uint32_t* hist, Select* sel, cudaStream_t st);
int launch_unsketch_emit(const Params& P, const float* sum, const float* vhat, Select* sel, uint32_t* I_out,
                         Cand* cand, bool vec, int sm_count, cudaStream_t st);
int launch_refine(const Params& P, Select* sel, const Cand* cand, uint32_t* I_out, cudaStream_t st);
int launch_apply(const Params& P, const uint32_t* I, const float* vhat, float* e, float* x, cudaStream_t st);
// helpers for state export / import
int launch_estimates(const Params& P, const float* sum, const float* vhat, float* est, cudaStream_t st);
int launch_hash_export(const Params& P, uint32_t row, uint64_t i0, uint64_t count, uint32_t* idx, int8_t* sgn,
                       cudaStream_t st);
int launch_v_materialize(const Params& P, const float* v, const uint32_t* vstamp, uint32_t t, float* out,
                         cudaStream_t st);
int launch_fill_u32(uint32_t* p, uint64_t n, uint32_t value, cudaStream_t st);

}  // namespace sk
