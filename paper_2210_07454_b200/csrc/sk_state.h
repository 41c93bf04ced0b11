// The handle behind the C ABI (private to the library's own translation units).
#pragma once
#include "../../include/sketched_amsgrad.h"
#include "sk_internal.h"

#include <vector>

struct TimeRec { int stage; cudaEvent_t a, b; };

struct sk_state {
    sk::Params P{};
    uint64_t seed = 0, t = 0;
    uint64_t vclock = 0;          // steps that updated v, vhat: the clock of the lazy decay stamps (t minus frozen steps)
    float lr_prev = 0;            // alpha_{t-1}: the step size of the last step taken
    bool sum_sketch = false;      // sketch the worker sum once instead of one table per worker (linearity)
    bool freeze_v = false;        // Algorithm 2 without h_t and without the update of v, vhat
    bool grads_bf16 = false;      // gradients are passed as bf16
    float eps = 0;
    uint32_t k_prev = 0;
    int sm_count = 148;
    size_t l2_bytes = 0;
    int64_t worker_chunk = 0;
    int64_t window_lines = 0;
    bool window_explicit = false; // window_lines was set by the caller (else the default may follow the variant)
    int64_t cand_mult = 1;        // P of Section III-A: candidates of the second round = P * k (1 = no second round)
    uint32_t *Ic = nullptr, *keys2 = nullptr;   // the P*k candidates and their exact-value keys
    int64_t variant = 0;          // 0 = gradient averaging (Algorithm 2), 1 = parameter averaging (Algorithm 1)
    float *vw = nullptr, *vhatw = nullptr;   // per-worker v, vhat of the parameter-averaging variant (n*d each)
    int64_t window_workers = 8;
    int64_t always_asum = 0;      // the sketch kernel leaves sum_w a^(w) for the update of x even without a second round
    int64_t sketch_ctas_per_sm = 64;
    bool timing = false;
    cudaStream_t stream = nullptr;
    // device memory owned by the handle
    float *m = nullptr, *e = nullptr, *v = nullptr, *vhat = nullptr, *tables = nullptr, *sum = nullptr;
    uint32_t *vstamp = nullptr, *I = nullptr, *I_prev = nullptr, *hist = nullptr, *hist2 = nullptr;
    uint32_t *keys = nullptr, *bitmap = nullptr;
    float* gsum = nullptr;
    float* asum = nullptr;        // d, only with a second round: sum over the workers of a_t (worker order), written by the sketch kernel
    uint64_t bitmap_bytes = 0;
    // one iteration in three phases (workers partitioned over processes): 0 idle, 1 after local, 2 after select
    int phase = 0;
    bool step_vec = false;        // this step runs the 128-bit kernels
    bool asum_live = false;       // this step's sketch kernel filled asum
    uint32_t *cbitmap = nullptr, *scan = nullptr;   // scratch of the partitioned step: candidate bitmap, block offsets
    sk::Select* sel = nullptr;
    sk::Cand *cand = nullptr, *cand2 = nullptr;
    float *stage_grads = nullptr, *stage_x = nullptr, *stage_vals = nullptr;
    // host-buffer step: the gradients are copied in pieces on a stream of their own (one event per piece, one for x)
    static constexpr uint32_t kHostPieces = 4;
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t copy_done[kHostPieces + 1] = {};
    // timing
    std::vector<TimeRec> recs;
    std::vector<cudaEvent_t> free_events;
    double ms[SK_NUM_STAGES] = {0};
    uint64_t launches[SK_NUM_STAGES] = {0};
    uint64_t timed_steps = 0;
};
