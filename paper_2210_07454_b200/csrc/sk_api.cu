// C ABI of the library (see include/sketched_amsgrad.h): handle life cycle, the step's launch sequence,
// state export/import and stage timing.  Host code only; the kernels live in sk_sketch.cu / sk_select.cu.
#include "../../include/sketched_amsgrad.h"
#include "sk_internal.h"
#include "sk_hash.cuh"
#include "sk_state.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

namespace {

thread_local std::string g_err;
int64_t g_fail_alloc_countdown = -1;     // >= 0: the (countdown+1)-th device allocation of sk_create fails (test hook)

constexpr uint32_t kDefaultWindowLines = 8;

int fail(int code, const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_err = buf;
    return code;
}

#define SK_CUDA(expr)                                                                              \
    do {                                                                                           \
        cudaError_t err__ = (expr);                                                                \
        if (err__ != cudaSuccess)                                                                  \
            return fail(err__ == cudaErrorMemoryAllocation ? SK_ENOMEM : SK_ECUDA, "%s: %s", #expr, \
                        cudaGetErrorString(err__));                                                \
    } while (0)

}  // namespace

namespace {

void refresh_hash(sk_state* s) {
    for (uint32_t j = 0; j < s->P.r; ++j) s->P.row_key[j] = sk::row_key(s->seed, j);
    s->P.G = s->P.c >> s->P.log2g;
    s->P.win_cw = 0;
    s->P.win_panels = 0;
    if (s->window_lines > 0) {        // windowed family: a group picks one of the window's lines
        s->P.G = (uint32_t)s->window_lines;
        s->P.win_cw = 32u * (uint32_t)s->window_lines;
        s->P.win_panels = s->P.c / s->P.win_cw;
    }
}

uint32_t chunk_of(const sk_state* s) {
    if (s->worker_chunk > 0) return (uint32_t)std::min<int64_t>(s->worker_chunk, s->P.n);
    // keep the tables that are being accumulated concurrently within a fraction of L2
    const double budget = s->l2_bytes ? 0.44 * (double)s->l2_bytes : 56e6;   // measured: more than this and L2 spills
    const double per_worker = (double)s->P.r * s->P.cs * 4.0;
    uint32_t wc = (uint32_t)std::max(1.0, std::floor(budget / per_worker));
    wc = std::min(wc, s->P.n);
    const uint32_t chunks = (s->P.n + wc - 1) / wc;
    return (s->P.n + chunks - 1) / chunks;
}

cudaEvent_t get_event(sk_state* s) {
    if (!s->free_events.empty()) {
        cudaEvent_t e = s->free_events.back();
        s->free_events.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

int flush_timing(sk_state* s) {
    if (s->recs.empty()) return SK_OK;
    SK_CUDA(cudaStreamSynchronize(s->stream));
    for (const TimeRec& r : s->recs) {
        float ms = 0;
        SK_CUDA(cudaEventElapsedTime(&ms, r.a, r.b));
        s->ms[r.stage] += ms;
        s->free_events.push_back(r.a);
        s->free_events.push_back(r.b);
    }
    s->recs.clear();
    return SK_OK;
}

struct StageTimer {   // brackets the launches of one stage with events when timing is on
    sk_state* s; int stage; cudaEvent_t a = nullptr;
    StageTimer(sk_state* s_, int stage_) : s(s_), stage(stage_) {
        if (s->timing) { a = get_event(s); cudaEventRecord(a, s->stream); }
    }
    void done(int launches) {
        s->launches[stage] += (uint64_t)launches;
        if (s->timing) {
            cudaEvent_t b = get_event(s);
            cudaEventRecord(b, s->stream);
            s->recs.push_back({stage, a, b});
        }
    }
};

int check_status(sk_state* s) {
    sk::Select h{};
    SK_CUDA(cudaMemcpyAsync(&h, s->sel, sizeof h, cudaMemcpyDeviceToHost, s->stream));
    SK_CUDA(cudaStreamSynchronize(s->stream));
    if (h.status) {
        // reported once: the word is cleared so that the handle stays usable
        SK_CUDA(cudaMemsetAsync(&s->sel->status, 0, sizeof(uint32_t), s->stream));
        SK_CUDA(cudaStreamSynchronize(s->stream));
        return fail(SK_EDEVICE, "device status word = 0x%x (bit 0: selection emitted %u of %u indices; bits 1-5, debug "
                    "build: table offset, index, list position, histogram bin, window offset out of range; bit 6, debug "
                    "build: a gradient entry was not finite)", h.status,
                    h.cnt_out, s->P.k);
    }
    return SK_OK;
}

sk::MomentArgs moment_args(const sk_state* s, const void* grads) {
    sk::MomentArgs A{};
    A.grads = grads; A.grad_bf16 = s->grads_bf16 ? 1u : 0u; A.m = s->m; A.e = s->e; A.tables = s->tables; A.gsum = s->gsum;
    A.v = s->v; A.vhat = s->vhat; A.vstamp = s->vstamp; A.bitmap = s->bitmap;
    A.step = (uint32_t)(s->vclock + 1); A.members = s->k_prev ? 1u : 0u;
    A.gsum_on = (A.members && !s->freeze_v && s->variant == 0) ? 1u : 0u;
    A.vw = s->vw; A.vhatw = s->vhatw; A.variant = (uint32_t)s->variant;
    return A;
}

// One iteration is three phases.  sk_step runs them back to back.  With the workers partitioned over processes
// (sk_step_local / sk_step_select / sk_step_finish) the caller sums an exchange buffer over the processes between
// the phases: x1 = [this process's share of the mean sketch | its gradient sums on I_{t-1}], x2 = [its sums of a_t at
// the candidates]; both index lists are in ascending order so that position q means the same coordinate everywhere.

// Phase 1 (workers): moments, error-compensated vector, sketches of this handle's workers, their sum.
// [wbeg, wend): the workers this call covers; a step may take the phase in several calls over ascending worker ranges
// (the host-buffer step does, one call per gradient piece that has arrived): the first call opens the phase, the
// one that reaches the last worker closes it.
int phase_local(sk_state* s, const void* grads, float* x1, uint32_t wbeg = 0, uint32_t wend = 0xFFFFFFFFu) {
    // alpha_{t-1}/alpha_t weights e_{t-1} in the sketched vector (the sketch lines of Algorithms 1 and 2)
    s->P.rho = (s->lr_prev == s->P.lr) ? 1.0f : (float)((double)s->lr_prev / (double)s->P.lr);
    const sk::Params& P = s->P;
    const bool vec = s->step_vec;
    const bool sharded = x1 != nullptr;
    cudaStream_t st = s->stream;
    wend = std::min(wend, P.n);
    const bool first = wbeg == 0, last = wend == P.n;
    if (first && s->timing && s->recs.size() > 4096) { int rc = flush_timing(s); if (rc) return rc; }

    sk::MomentArgs A = moment_args(s, grads);
    // the windowed kernel implements Algorithm 2 with one table per worker only
    const bool windowed = vec && P.win_cw != 0 && s->variant == 0 && !s->sum_sketch;
    const uint32_t wc = windowed ? std::min<uint32_t>(std::min<uint32_t>((uint32_t)s->window_workers, sk::kOwnMaxWorkers), P.n)
                                 : chunk_of(s);
    // With a second round the sketch kernel also leaves sum_w a^(w) per coordinate, so that each of the P*k exact
    // values costs one gather instead of n (not the windowed kernel, and not a partitioned step, whose exact values
    // are exchanged: there every local worker's value is gathered).
    A.asum = ((s->cand_mult > 1 || s->always_asum) && !sharded) ? s->asum : nullptr;
    s->asum_live = A.asum != nullptr;
    const uint64_t tfloats = (uint64_t)P.r * P.cs;
    float* sum_out = sharded ? x1 : s->sum;
    if (s->sum_sketch) A.sum_table = sum_out;
    if (s->sum_sketch && first) {    // one sketch of the worker sum, accumulated straight into the aggregate
        StageTimer tm(s, 0);
        tm.done(sk::launch_zero(sum_out, tfloats * 4, st));
    }
    if (sharded && s->k_prev && first) {      // I_{t-1} in ascending order, from its bitmap
        StageTimer tm(s, 0);
        tm.done(sk::launch_list_from_bitmap(P, s->bitmap, s->bitmap_bytes / 4, s->scan, s->I_prev, P.k, st));
    }
    for (uint32_t w0 = wbeg; w0 < wend; w0 += wc) {
        const uint32_t nw = std::min(wc, wend - w0);
        if (!s->sum_sketch) {
            StageTimer tm(s, 0);
            tm.done(sk::launch_zero(s->tables + (uint64_t)w0 * tfloats, (uint64_t)nw * tfloats * 4, st, (P.chain & sk::kChainZero) != 0));
        }
        StageTimer tm(s, 2);     // moments + sketch; also leaves the gradient sums on I_{t-1} in gsum
        if (windowed) {
            const int l = sk::launch_moment_sketch_own(P, A, w0, nw, s->sm_count, st);
            if (l < 0) return fail(SK_ECUDA, "the windowed sketch kernel does not fit in shared memory (window_lines=%lld, r=%u)",
                                   (long long)s->window_lines, P.r);
            tm.done(l);
        } else {
            tm.done(sk::launch_moment_sketch(P, A, w0, nw, vec, s->sm_count * (int)s->sketch_ctas_per_sm, st));
        }
    }
    if (last) {
        StageTimer tm(s, 3);
        int l = s->sum_sketch ? 0 : sk::launch_sum_tables(P, s->tables, sum_out, st);
        if (sharded && s->variant == 0)      // h_t: this process's gradient sums on I_{t-1}, zero-padded to k
            l += sk::launch_gather(P, s->I_prev, s->k_prev, P.k, s->gsum, x1 + tfloats, st);
        tm.done(l);
    }
    SK_CUDA(cudaGetLastError());
    return SK_OK;
}

// Phase 2 (master): second moments on I_{t-1}, unsketch of every coordinate, selection of the candidates.
int phase_select(sk_state* s, const float* x1, float* x2) {
    const sk::Params& P = s->P;
    const bool vec = s->step_vec;
    const bool sharded = x1 != nullptr;
    cudaStream_t st = s->stream;
    sk::MomentArgs A = moment_args(s, nullptr);
    if (s->freeze_v) A.members = 0;             // v, vhat stay as they are (Section III-B's fixed-variance remark)
    sk::Params Q = P;                           // first selection: P*k of d (k without a second round)
    Q.k = (uint32_t)s->cand_mult * P.k;
    {
        StageTimer tm(s, 4);
        int l = 0;
        if (sharded) {                          // the summed exchange buffer: mean sketch, then gradient sums on I_{t-1}
            SK_CUDA(cudaMemcpyAsync(s->sum, x1, (uint64_t)P.r * P.cs * 4, cudaMemcpyDeviceToDevice, st));
            if (s->variant == 0) l += sk::launch_scatter(P, s->I_prev, s->k_prev, x1 + (uint64_t)P.r * P.cs, s->gsum, st);
        }
        // ranking keys; v and vhat on I_{t-1} are brought up to date on the way, from the sums in gsum
        l += sk::launch_unsketch_hist(P, A, s->sum, s->keys, s->hist, vec, s->sm_count, st);
        l += sk::launch_pick_bin(Q, s->hist, s->sel, 0, st);
        tm.done(l);
    }
    uint32_t* list = s->cand_mult > 1 ? s->Ic : s->I;
    {
        StageTimer tm(s, 5);
        // the pass also clears the bitmap of I_{t-1}, which has served its purpose once the key pass is through:
        // the update of x then marks I_t in it
        tm.done(sk::launch_emit(Q, s->keys, nullptr, s->sel, list, s->cand, s->hist2, s->sm_count, st, s->bitmap,
                                s->bitmap_bytes));
    }
    {
        StageTimer tm(s, 6);
        int l = sk::launch_refine(Q, s->sel, s->cand, s->cand2, s->hist2, list, s->sm_count, st);
        if (sharded) {                          // candidates in ascending order, and this process's sums of a_t there
            l += sk::launch_sort_list(P, list, Q.k, s->cbitmap, s->bitmap_bytes / 4, s->scan, st);
            l += sk::launch_gather_worker_sum(P, list, Q.k, s->e, x2, st);
        }
        tm.done(l);
    }
    SK_CUDA(cudaGetLastError());
    return SK_OK;
}

// Phase 3: second round on the exact values (P > 1), then the update of x and of the error-feedback residual.
int phase_finish(sk_state* s, const float* x2, float* x) {
    const sk::Params& P = s->P;
    const bool sharded = x2 != nullptr;
    cudaStream_t st = s->stream;
    const float* asum = s->asum_live ? s->asum : nullptr;
    const float* vhat = s->variant == 1 ? nullptr : s->vhat;
    if (sharded) {                              // the summed exact values, placed at their coordinates
        StageTimer tm(s, 6);
        uint32_t* list = s->cand_mult > 1 ? s->Ic : s->I;
        tm.done(sk::launch_scatter(P, list, (uint32_t)s->cand_mult * P.k, x2, s->asum, st));
        asum = s->asum;
    }
    if (s->cand_mult > 1) {
        // Second round (Section III-A): the P*k largest estimates are candidates, their exact values are fetched,
        // and the k candidates of largest exact magnitude are kept (ties: smaller index).
        StageTimer tm(s, 6);
        const uint32_t pk = (uint32_t)s->cand_mult * P.k;
        int l = sk::launch_exact_keys(P, s->Ic, pk, vhat, s->e, asum, s->keys2, s->hist, s->sm_count, st);
        sk::Params Q2 = P;                      // second selection: k of the P*k candidates, keyed by exact value
        Q2.d = pk;
        l += sk::launch_pick_bin(Q2, s->hist, s->sel, 0, st);
        l += sk::launch_emit(Q2, s->keys2, s->Ic, s->sel, s->I, s->cand, s->hist2, s->sm_count, st);
        l += sk::launch_refine(Q2, s->sel, s->cand, s->cand2, s->hist2, s->I, s->sm_count, st);
        tm.done(l);
    }
    {
        StageTimer tm(s, 7);     // apply marks I_t in the bitmap, which the emit pass of the selection cleared
        tm.done(sk::launch_apply(P, s->I, vhat, s->e, asum, x, s->bitmap, st));
    }
    SK_CUDA(cudaGetLastError());
    std::swap(s->I, s->I_prev);      // I_prev now holds I_t
    s->k_prev = P.k;
    s->lr_prev = P.lr;
    if (!s->freeze_v || s->variant == 1) s->vclock += 1;
    s->t += 1;
    if (s->timing) s->timed_steps += 1;
    return SK_OK;
}

int do_step(sk_state* s, const void* grads, float* x) {
    if (s->phase != 0) return fail(SK_ESTATE, "sk_step: a partitioned step is in progress (finish it with sk_step_finish)");
    s->step_vec = (s->P.d % 4 == 0) && s->P.log2g >= 2 && ((uintptr_t)grads % 16 == 0) && ((uintptr_t)x % 16 == 0);
    int rc = phase_local(s, grads, nullptr);
    if (!rc) rc = phase_select(s, nullptr, nullptr);
    if (!rc) rc = phase_finish(s, nullptr, x);
    return rc;
}

// scratch of the partitioned step, allocated at its first use
int shard_buffers(sk_state* s) {
    if (s->cbitmap) return SK_OK;
    SK_CUDA(cudaMalloc((void**)&s->cbitmap, s->bitmap_bytes));
    SK_CUDA(cudaMalloc((void**)&s->scan, sk::scan_entries(s->bitmap_bytes / 4) * 4));
    if (!s->asum) SK_CUDA(cudaMalloc((void**)&s->asum, ((uint64_t)s->P.d + 3) / 4 * 16));
    return SK_OK;
}

enum Field { F_M, F_E, F_V, F_VHAT, F_TABLES, F_SUM, F_EST, F_I, F_T, F_VW, F_VHATW, F_CAND, F_X, F_KEYS, F_BAD };

Field field_of(const char* name) {
    static const char* names[] = {"m", "e", "v", "vhat", "tables", "sum", "est", "I", "t", "vw", "vhatw", "cand", "x", "keys"};
    for (int q = 0; q < 14; ++q) if (!strcmp(name, names[q])) return (Field)q;
    return F_BAD;
}

}  // namespace

int sk_static_prepare(void);      // sk_static.cu

// lets the library's other translation units report through sk_last_error()
int sk_fail_message(int code, const char* message) { return fail(code, "%s", message); }

extern "C" {

const char* sk_last_error(void) { return g_err.c_str(); }
const char* sk_version(void) { return "sketched-amsgrad-b200 0.1 (sm_100a)"; }

sk_state* sk_create(uint64_t d, uint32_t n, uint32_t r, uint32_t c, uint64_t k, uint64_t seed, float lr,
                    float beta1, float beta2, float eps) {
    if (d < 1 || d >= (1ull << 32)) { fail(SK_EINVAL, "d must be in [1, 2^32)"); return nullptr; }
    if (n < 1 || r < 1 || r > sk::kMaxRows || c < 1) { fail(SK_EINVAL, "need n >= 1, 1 <= r <= 16, c >= 1"); return nullptr; }
    if (k < 1 || k > d) { fail(SK_EINVAL, "k must be in [1, d]"); return nullptr; }
    if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f)) { fail(SK_EINVAL, "beta1, beta2 must be in [0,1)"); return nullptr; }
    if (!(eps > 0.f) || !std::isfinite(eps) || !std::isfinite(lr)) { fail(SK_EINVAL, "eps must be > 0 and lr finite"); return nullptr; }
    if ((uint64_t)r * (((uint64_t)c + 31) / 32 * 32) >= (1ull << 32)) { fail(SK_EINVAL, "r*c too large"); return nullptr; }

    int dev = 0;
    cudaDeviceProp prop{};
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
        fail(SK_ECUDA, "no usable CUDA device: %s", cudaGetErrorString(cudaGetLastError()));
        return nullptr;
    }
    sk_state* s = new sk_state();
    s->sm_count = prop.multiProcessorCount;
    s->l2_bytes = (size_t)prop.l2CacheSize;
    s->seed = seed;
    s->eps = eps;
    sk::Params& P = s->P;
    P.d = (uint32_t)d; P.n = n; P.n_all = n; P.r = r; P.c = c; P.k = (uint32_t)k;
    P.cs = (c + 31u) / 32u * 32u;
    P.beta1 = beta1; P.beta2 = beta2; P.lr = lr; P.rho = 1.0f;
    P.chain = sk::kChainAll;                     // the step's kernels are launched chained (option "chained_launches")
    s->lr_prev = lr;
    uint32_t lg = 5;
    while ((1u << lg) > c) --lg;
    P.log2g = lg;
    // default family: groups of 32 confined to windows of kDefaultWindowLines lines, which lets the sketch accumulate
    // on chip; rows too short for one window keep the plain family
    if (lg == 5 && c >= 32u * kDefaultWindowLines) s->window_lines = kDefaultWindowLines;
    refresh_hash(s);

    const uint64_t nd = (uint64_t)n * d, tf = (uint64_t)r * P.cs;
    bool ok = true;
    auto alloc = [&](void** p, uint64_t bytes) {
        if (!ok) return;
        cudaError_t err = cudaErrorMemoryAllocation;               // what an injected failure looks like
        if (g_fail_alloc_countdown < 0 || g_fail_alloc_countdown-- != 0) err = cudaMalloc(p, bytes ? bytes : 4);
        if (err != cudaSuccess) {
            ok = false;
            *p = nullptr;
            cudaGetLastError();
            fail(SK_ENOMEM, "cudaMalloc of %llu bytes failed: %s", (unsigned long long)bytes, cudaGetErrorString(err));
        }
    };
    alloc((void**)&s->m, nd * 4); alloc((void**)&s->e, nd * 4);
    alloc((void**)&s->v, d * 4); alloc((void**)&s->vhat, d * 4); alloc((void**)&s->vstamp, d * 4);
    alloc((void**)&s->tables, (uint64_t)n * tf * 4); alloc((void**)&s->sum, tf * 4);
    alloc((void**)&s->I, k * 4); alloc((void**)&s->I_prev, k * 4);
    alloc((void**)&s->hist, sk::kHistBins * 4); alloc((void**)&s->sel, sizeof(sk::Select));
    alloc((void**)&s->hist2, sk::kHistBins * 4);
    alloc((void**)&s->cand, d * sizeof(sk::Cand)); alloc((void**)&s->cand2, d * sizeof(sk::Cand));
    const uint64_t d_pad = (d + 3) / 4 * 4;
    s->bitmap_bytes = ((d + 31) / 32 * 4 + 15) / 16 * 16;
    alloc((void**)&s->keys, d_pad * 4); alloc((void**)&s->gsum, d_pad * 4);
    alloc((void**)&s->bitmap, s->bitmap_bytes);
    if (!ok) { sk_destroy(s); return nullptr; }
    P.status = &s->sel->status;
    if (d <= SK_STATIC_MAX_D) sk_static_prepare();   // so that sk_select_static finds its scratch resolved (it may not allocate)
    cudaError_t init = cudaSuccess;
    auto clear = [&](void* p, uint64_t bytes) { if (init == cudaSuccess) init = cudaMemset(p, 0, bytes); };
    clear(s->bitmap, s->bitmap_bytes);                                  // I_0 is empty
    clear(s->m, nd * 4); clear(s->e, nd * 4);                           // m_0 = e_0 = 0
    clear(s->vstamp, d * 4);
    clear(s->gsum, d_pad * 4);
    clear(s->tables, (uint64_t)n * tf * 4); clear(s->sum, tf * 4);
    clear(s->hist, sk::kHistBins * 4); clear(s->hist2, sk::kHistBins * 4);
    clear(s->sel, sizeof(sk::Select));
    if (init != cudaSuccess) {
        fail(SK_ECUDA, "initialisation failed: %s", cudaGetErrorString(init));
        cudaGetLastError();
        sk_destroy(s);
        return nullptr;
    }
    uint32_t eps_bits;
    memcpy(&eps_bits, &eps, 4);
    sk::launch_fill_u32((uint32_t*)s->v, d, eps_bits, nullptr);         // v_0 = vhat_0 = eps
    sk::launch_fill_u32((uint32_t*)s->vhat, d, eps_bits, nullptr);
    if (cudaDeviceSynchronize() != cudaSuccess) {
        fail(SK_ECUDA, "initialisation failed: %s", cudaGetErrorString(cudaGetLastError()));
        sk_destroy(s);
        return nullptr;
    }
    return s;
}

void sk_destroy(sk_state* s) {
    if (!s) return;
    if (s->stream) cudaStreamSynchronize(s->stream); else cudaDeviceSynchronize();
    for (void* p : {(void*)s->m, (void*)s->e, (void*)s->v, (void*)s->vhat, (void*)s->vstamp, (void*)s->tables,
                    (void*)s->sum, (void*)s->I, (void*)s->I_prev, (void*)s->hist, (void*)s->hist2, (void*)s->sel, (void*)s->cand, (void*)s->cand2,
                    (void*)s->keys, (void*)s->gsum, (void*)s->asum, (void*)s->bitmap, (void*)s->vw, (void*)s->vhatw, (void*)s->Ic, (void*)s->keys2, (void*)s->cbitmap, (void*)s->scan,
                    (void*)s->stage_grads, (void*)s->stage_x, (void*)s->stage_vals})
        if (p) cudaFree(p);
    if (s->copy_stream) {
        cudaStreamSynchronize(s->copy_stream);
        cudaStreamDestroy(s->copy_stream);
        for (cudaEvent_t ev : s->copy_done) if (ev) cudaEventDestroy(ev);
    }
    for (const TimeRec& r : s->recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    for (cudaEvent_t e : s->free_events) cudaEventDestroy(e);
    delete s;
}

int sk_step(const void* grads, float* x, sk_state* s) {
    if (!s || !grads || !x) return fail(SK_EINVAL, "sk_step: null argument");
    if (((uintptr_t)grads | (uintptr_t)x) % 4) return fail(SK_EINVAL, "sk_step: pointers must be 4-byte aligned");
    return do_step(s, grads, x);
}

// staging buffers of the host-buffer steps; stage_x doubles as the device-resident parameters (field "x")
static int ensure_stage(sk_state* s) {
    if (s->stage_grads) return SK_OK;
    const uint64_t nd = (uint64_t)s->P.n * s->P.d;
    SK_CUDA(cudaMalloc((void**)&s->stage_grads, nd * 4));
    SK_CUDA(cudaMalloc((void**)&s->stage_x, (uint64_t)s->P.d * 4));
    SK_CUDA(cudaMalloc((void**)&s->stage_vals, (uint64_t)s->P.k * 4));
    SK_CUDA(cudaMemsetAsync(s->stage_x, 0, (uint64_t)s->P.d * 4, s->stream));
    return SK_OK;
}

// The step on host gradients up to (not including) the copy back.  x_host != nullptr: x is sent after the gradients
// (only the last stage reads it); nullptr: the parameters already on the device (field "x") are used.
static int host_step(sk_state* s, const void* grads_host, const float* x_host) {
    if (s->phase != 0) return fail(SK_ESTATE, "a partitioned step is in progress");
    int rc = ensure_stage(s);
    if (rc) return rc;
    if (!s->copy_stream) {
        SK_CUDA(cudaStreamCreateWithFlags(&s->copy_stream, cudaStreamNonBlocking));
        for (cudaEvent_t& ev : s->copy_done) SK_CUDA(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
    }
    // The gradients arrive in up to kHostPieces pieces of whole workers on a copy stream of their own, and the sketch
    // kernel starts on a piece as soon as it is there, so all but the last piece's kernel hides behind the transfer.
    const uint32_t n = s->P.n;
    const uint32_t per = (n + sk_state::kHostPieces - 1) / sk_state::kHostPieces;
    const uint64_t wbytes = (uint64_t)s->P.d * (s->grads_bf16 ? 2 : 4);
    SK_CUDA(cudaEventRecord(s->copy_done[sk_state::kHostPieces], s->stream));        // earlier work on the handle's stream
    SK_CUDA(cudaStreamWaitEvent(s->copy_stream, s->copy_done[sk_state::kHostPieces], 0));
    s->step_vec = (s->P.d % 4 == 0) && s->P.log2g >= 2;                               // the staging buffers are aligned
    uint32_t piece = 0;
    for (uint32_t w = 0; w < n; w += per, ++piece) {
        const uint32_t we = std::min(n, w + per);
        SK_CUDA(cudaMemcpyAsync((char*)s->stage_grads + w * wbytes, (const char*)grads_host + w * wbytes, (we - w) * wbytes,
                                cudaMemcpyHostToDevice, s->copy_stream));
        SK_CUDA(cudaEventRecord(s->copy_done[piece], s->copy_stream));
        SK_CUDA(cudaStreamWaitEvent(s->stream, s->copy_done[piece], 0));
        rc = phase_local(s, s->stage_grads, nullptr, w, we);
        if (rc) return rc;
    }
    if (x_host) {
        SK_CUDA(cudaMemcpyAsync(s->stage_x, x_host, (uint64_t)s->P.d * 4, cudaMemcpyHostToDevice, s->copy_stream));
        SK_CUDA(cudaEventRecord(s->copy_done[sk_state::kHostPieces], s->copy_stream));
    }
    rc = phase_select(s, nullptr, nullptr);
    if (rc) return rc;
    if (x_host) SK_CUDA(cudaStreamWaitEvent(s->stream, s->copy_done[sk_state::kHostPieces], 0));
    return phase_finish(s, nullptr, s->stage_x);
}

int sk_step_host(const void* grads_host, float* x_host, sk_state* s) {
    if (!s || !grads_host || !x_host) return fail(SK_EINVAL, "sk_step_host: null argument");
    int rc = host_step(s, grads_host, x_host);
    if (rc) return rc;
    SK_CUDA(cudaMemcpyAsync(x_host, s->stage_x, (uint64_t)s->P.d * 4, cudaMemcpyDeviceToHost, s->stream));
    SK_CUDA(cudaStreamSynchronize(s->stream));
    return SK_OK;
}

int sk_step_host_sparse(const void* grads_host, uint32_t* idx_host, float* values_host, sk_state* s) {
    if (!s || !grads_host || !idx_host || !values_host) return fail(SK_EINVAL, "sk_step_host_sparse: null argument");
    int rc = host_step(s, grads_host, nullptr);
    if (rc) return rc;
    const uint64_t kb = (uint64_t)s->P.k * 4;
    sk::launch_gather(s->P, s->I_prev, s->P.k, s->P.k, s->stage_x, s->stage_vals, s->stream);   // I_prev holds I_t now
    SK_CUDA(cudaMemcpyAsync(idx_host, s->I_prev, kb, cudaMemcpyDeviceToHost, s->stream));
    SK_CUDA(cudaMemcpyAsync(values_host, s->stage_vals, kb, cudaMemcpyDeviceToHost, s->stream));
    SK_CUDA(cudaStreamSynchronize(s->stream));
    return SK_OK;
}

uint64_t sk_exchange_floats(const sk_state* s, int which) {
    if (!s) return 0;
    if (which == 1) return (uint64_t)s->P.r * s->P.cs + (s->variant == 0 ? s->P.k : 0);
    if (which == 2) return (uint64_t)s->cand_mult * s->P.k;
    return 0;
}

int sk_step_local(const void* grads, float* exchange1, sk_state* s) {
    if (!s || !grads || !exchange1) return fail(SK_EINVAL, "sk_step_local: null argument");
    if (((uintptr_t)grads % 4) || ((uintptr_t)exchange1 % 16))
        return fail(SK_EINVAL, "sk_step_local: grads must be 4-byte and exchange1 16-byte aligned");
    if (s->phase != 0) return fail(SK_ESTATE, "sk_step_local: the previous partitioned step was not finished");
    int rc = shard_buffers(s);
    if (rc) return rc;
    s->step_vec = (s->P.d % 4 == 0) && s->P.log2g >= 2 && ((uintptr_t)grads % 16 == 0);
    rc = phase_local(s, grads, exchange1);
    if (!rc) s->phase = 1;
    return rc;
}

int sk_step_select(const float* exchange1, float* exchange2, sk_state* s) {
    if (!s || !exchange1 || !exchange2) return fail(SK_EINVAL, "sk_step_select: null argument");
    if (((uintptr_t)exchange1 % 16) || ((uintptr_t)exchange2 % 4))
        return fail(SK_EINVAL, "sk_step_select: exchange1 must be 16-byte and exchange2 4-byte aligned");
    if (s->phase != 1) return fail(SK_ESTATE, "sk_step_select: call sk_step_local first");
    int rc = phase_select(s, exchange1, exchange2);
    if (!rc) s->phase = 2;
    return rc;
}

int sk_step_finish(const float* exchange2, float* x, sk_state* s) {
    if (!s || !exchange2 || !x) return fail(SK_EINVAL, "sk_step_finish: null argument");
    if (((uintptr_t)exchange2 | (uintptr_t)x) % 4) return fail(SK_EINVAL, "sk_step_finish: pointers must be 4-byte aligned");
    if (s->phase != 2) return fail(SK_ESTATE, "sk_step_finish: call sk_step_select first");
    s->phase = 0;
    return phase_finish(s, exchange2, x);
}

int sk_set_lr(sk_state* s, float lr) {
    if (!s) return fail(SK_EINVAL, "null handle");
    if (!std::isfinite(lr)) return fail(SK_EINVAL, "the step size must be finite");
    if (lr == 0.0f && lr != s->P.lr) return fail(SK_EINVAL, "a zero step size has no ratio alpha_{t-1}/alpha_t");
    if (s->phase != 0) return fail(SK_ESTATE, "the step size cannot change inside a partitioned step");
    if (s->lr_prev == 0.0f && lr != 0.0f) return fail(SK_EINVAL, "a zero step size has no ratio alpha_{t-1}/alpha_t");
    s->P.lr = lr;
    return SK_OK;
}

int sk_set_stream(sk_state* s, void* stream) {
    if (!s) return fail(SK_EINVAL, "null handle");
    int rc = flush_timing(s);
    if (rc) return rc;
    SK_CUDA(cudaStreamSynchronize(s->stream));
    s->stream = (cudaStream_t)stream;
    return SK_OK;
}

int sk_sync(sk_state* s) {
    if (!s) return fail(SK_EINVAL, "null handle");
    return check_status(s);
}

int sk_test_fail_allocation(int64_t nth) {
    g_fail_alloc_countdown = nth;
    return SK_OK;
}

int sk_debug_check(sk_state* s, uint32_t kind) {
    if (!s) return fail(SK_EINVAL, "null handle");
#ifdef SK_DEBUG
    if (kind < 1 || kind > 6) return fail(SK_EINVAL, "kind must be in 1..6");
    sk::launch_debug_violation(s->P, 1u << kind, s->stream);
    SK_CUDA(cudaGetLastError());
    return SK_OK;
#else
    (void)kind;
    return fail(SK_ESTATE, "this build has no device-side checks (build with -DSK_DEBUG=1)");
#endif
}

int sk_get_stats(sk_state* s, double* out, uint32_t count) {
    if (!s || !out) return fail(SK_EINVAL, "null argument");
    if (count < SK_NUM_STATS) return fail(SK_EINVAL, "sk_get_stats needs room for SK_NUM_STATS values");
    if (s->t == 0) return fail(SK_ESTATE, "no step has been taken yet");
    sk::Select h{};
    SK_CUDA(cudaMemcpyAsync(&h, s->sel, sizeof h, cudaMemcpyDeviceToHost, s->stream));
    SK_CUDA(cudaStreamSynchronize(s->stream));
    const uint32_t lead = ((h.bin << sk::kHistBits) | h.bin2) << 7;      // the threshold key's leading 24 bits
    float tau;
    memcpy(&tau, &lead, 4);
    out[0] = (double)tau;
    out[1] = (double)h.cnt_cand;
    out[2] = (double)h.cnt_cand2;
    out[3] = (double)h.cnt_out;
    out[4] = (double)s->P.r * s->P.c + (double)s->cand_mult * s->P.k + (s->variant == 0 ? 2.0 : 1.0) * s->P.k;
    out[5] = (double)h.status;
    return SK_OK;
}

int sk_set_option(sk_state* s, const char* key, int64_t value) {
    if (!s || !key) return fail(SK_EINVAL, "null argument");
    if (!strcmp(key, "log2g")) {
        if (s->t != 0) return fail(SK_ESTATE, "log2g can only be changed before the first step");
        if (value < 0 || value > 5 || (1u << value) > s->P.c) return fail(SK_EINVAL, "log2g must be in 0..5 with 2^log2g <= c");
        s->P.log2g = (uint32_t)value;
        if (value != 5) s->window_lines = 0;
        refresh_hash(s);
        return SK_OK;
    }
    if (!strcmp(key, "window_lines")) {
        if (s->t != 0) return fail(SK_ESTATE, "window_lines can only be changed before the first step");
        if (value < 0 || value > 64 || (value & (value - 1))) return fail(SK_EINVAL, "window_lines must be 0 or a power of two <= 64");
        if (value > 0 && (s->P.log2g != 5 || 32ull * (uint64_t)value > s->P.c))
            return fail(SK_EINVAL, "window_lines needs a hash group of 32 and 32*window_lines <= c");
        s->window_lines = value;
        s->window_explicit = true;
        refresh_hash(s);
        return SK_OK;
    }
    if (!strcmp(key, "P")) {
        if (s->t != 0) return fail(SK_ESTATE, "P can only be changed before the first step");
        if (value < 1 || (uint64_t)value * s->P.k > s->P.d) return fail(SK_EINVAL, "P must be >= 1 with P*k <= d");
        if (value > 1) {
            if (s->Ic) { cudaFree(s->Ic); cudaFree(s->keys2); s->Ic = s->keys2 = nullptr; }
            const uint64_t pk = (uint64_t)value * s->P.k;
            if (cudaMalloc((void**)&s->Ic, pk * 4) != cudaSuccess || cudaMalloc((void**)&s->keys2, pk * 4) != cudaSuccess ||
                (!s->asum && cudaMalloc((void**)&s->asum, ((uint64_t)s->P.d + 3) / 4 * 16) != cudaSuccess))
                return fail(SK_ENOMEM, "cudaMalloc of the candidate buffers failed: %s", cudaGetErrorString(cudaGetLastError()));
        }
        s->cand_mult = value;
        return SK_OK;
    }
    if (!strcmp(key, "sum_sketch")) {
        if (value != 0 && value != 1) return fail(SK_EINVAL, "sum_sketch must be 0 or 1");
        if (s->phase != 0) return fail(SK_ESTATE, "sum_sketch cannot change inside a partitioned step");
        s->sum_sketch = value != 0;
        return SK_OK;
    }
    if (!strcmp(key, "freeze_v")) {
        if (value != 0 && s->variant == 1) return fail(SK_EINVAL, "freeze_v applies to gradient averaging (Algorithm 2) only");
        if (s->phase != 0) return fail(SK_ESTATE, "freeze_v cannot change inside a partitioned step");
        s->freeze_v = value != 0;
        return SK_OK;
    }
    if (!strcmp(key, "grads_bf16")) {
        if (value != 0 && value != 1) return fail(SK_EINVAL, "grads_bf16 must be 0 or 1");
        s->grads_bf16 = value != 0;
        return SK_OK;
    }
    if (!strcmp(key, "workers_total")) {
        if (s->t != 0) return fail(SK_ESTATE, "workers_total can only be changed before the first step");
        if (value < (int64_t)s->P.n || value >= (1ll << 31)) return fail(SK_EINVAL, "workers_total must be >= n");
        s->P.n_all = (uint32_t)value;
        return SK_OK;
    }
    if (!strcmp(key, "variant")) {
        if (s->t != 0) return fail(SK_ESTATE, "variant can only be changed before the first step");
        if (value != 0 && value != 1) return fail(SK_EINVAL, "variant must be 0 (gradient averaging) or 1 (parameter averaging)");
        if (value == 1 && s->freeze_v) return fail(SK_EINVAL, "freeze_v applies to gradient averaging (Algorithm 2) only");
        if (value == 1 && !s->vw) {                   // v_0^(w) = vhat_0^(w) = eps on every worker (Algorithm 1)
            const uint64_t nd = (uint64_t)s->P.n * s->P.d;
            if (cudaMalloc((void**)&s->vw, nd * 4) != cudaSuccess || cudaMalloc((void**)&s->vhatw, nd * 4) != cudaSuccess)
                return fail(SK_ENOMEM, "cudaMalloc of the per-worker second moments failed: %s",
                            cudaGetErrorString(cudaGetLastError()));
            uint32_t eps_bits;
            memcpy(&eps_bits, &s->eps, 4);
            sk::launch_fill_u32((uint32_t*)s->vw, nd, eps_bits, s->stream);
            sk::launch_fill_u32((uint32_t*)s->vhatw, nd, eps_bits, s->stream);
            SK_CUDA(cudaStreamSynchronize(s->stream));
        }
        s->variant = value;
        // Algorithm 1 runs the reduction kernels, whose reductions spread best over the plain family: it becomes the
        // default there (windows confine a tile's reductions to a few lines of every table)
        if (!s->window_explicit) {
            s->window_lines = (value == 0 && s->P.log2g == 5 && s->P.c >= 32u * kDefaultWindowLines) ? kDefaultWindowLines : 0;
            refresh_hash(s);
        }
        return SK_OK;
    }
    if (!strcmp(key, "window_workers")) {
        if (value < 1 || value > (int64_t)sk::kOwnMaxWorkers) return fail(SK_EINVAL, "window_workers must be in 1..8");
        s->window_workers = value;
        return SK_OK;
    }
    if (!strcmp(key, "worker_sum")) {
        if (value != 0 && value != 1) return fail(SK_EINVAL, "worker_sum must be 0 or 1");
        if (s->phase != 0) return fail(SK_ESTATE, "worker_sum cannot change inside a partitioned step");
        if (value && !s->asum && cudaMalloc((void**)&s->asum, ((uint64_t)s->P.d + 3) / 4 * 16) != cudaSuccess)
            return fail(SK_ENOMEM, "cudaMalloc of the worker-sum buffer failed: %s", cudaGetErrorString(cudaGetLastError()));
        s->always_asum = value;
        return SK_OK;
    }
    if (!strcmp(key, "worker_chunk")) {
        if (value < 0) return fail(SK_EINVAL, "worker_chunk must be >= 0");
        s->worker_chunk = value;
        return SK_OK;
    }
    if (!strcmp(key, "sketch_ctas_per_sm")) {
        if (value < 1 || value > 4096) return fail(SK_EINVAL, "sketch_ctas_per_sm must be in 1..4096");
        s->sketch_ctas_per_sm = value;
        return SK_OK;
    }
    if (!strcmp(key, "chained_launches")) {
        if (value < 0 || value > (int64_t)sk::kChainAll) return fail(SK_EINVAL, "chained_launches must be 0, 1 or a mask below 512");
        s->P.chain = value == 1 ? sk::kChainAll : (uint32_t)value;
        return SK_OK;
    }
    if (!strcmp(key, "timing")) {
        int rc = flush_timing(s);
        if (rc) return rc;
        s->timing = value != 0;
        return SK_OK;
    }
    return fail(SK_EINVAL, "unknown option '%s'", key);
}

int sk_get_option(const sk_state* s, const char* key, int64_t* value) {
    if (!s || !key || !value) return fail(SK_EINVAL, "null argument");
    if (!strcmp(key, "log2g")) *value = s->P.log2g;
    else if (!strcmp(key, "window_lines")) *value = s->window_lines;
    else if (!strcmp(key, "window_workers")) *value = s->window_workers;
    else if (!strcmp(key, "worker_sum")) *value = s->always_asum;
    else if (!strcmp(key, "variant")) *value = s->variant;
    else if (!strcmp(key, "P")) *value = s->cand_mult;
    else if (!strcmp(key, "workers_total")) *value = s->P.n_all;
    else if (!strcmp(key, "freeze_v")) *value = s->freeze_v;
    else if (!strcmp(key, "sum_sketch")) *value = s->sum_sketch;
    else if (!strcmp(key, "grads_bf16")) *value = s->grads_bf16;
    else if (!strcmp(key, "worker_chunk")) *value = chunk_of(s);
    else if (!strcmp(key, "timing")) *value = s->timing;
    else if (!strcmp(key, "chained_launches")) *value = s->P.chain == sk::kChainAll ? 1 : s->P.chain;
    else if (!strcmp(key, "sketch_ctas_per_sm")) *value = s->sketch_ctas_per_sm;
    else if (!strcmp(key, "I_count")) *value = s->k_prev;
    else if (!strcmp(key, "vectorised")) *value = (s->P.d % 4 == 0) && s->P.log2g >= 2;
    else return fail(SK_EINVAL, "unknown option '%s'", key);
    return SK_OK;
}

int sk_hash(const sk_state* s, uint32_t row, uint64_t i0, uint64_t count, uint32_t* idx_out, int8_t* sign_out) {
    if (!s || !idx_out || !sign_out) return fail(SK_EINVAL, "null argument");
    if (row >= s->P.r || i0 + count > (1ull << 32)) return fail(SK_EINVAL, "row or coordinate range out of bounds");
    if (count == 0) return SK_OK;
    sk::launch_hash_export(s->P, row, i0, count, idx_out, sign_out, s->stream);
    SK_CUDA(cudaGetLastError());
    return SK_OK;
}

uint64_t sk_algorithmic_bytes(const sk_state* s) {
    if (!s) return 0;
    const uint64_t n = s->P.n, d = s->P.d, r = s->P.r, c = s->P.c, k = s->P.k;
    const uint64_t g = s->grads_bf16 ? 2 : 0;     // bytes saved per gradient entry when they arrive as bf16
    const uint64_t tables = s->sum_sketch ? 8 * r * c : 8 * n * r * c + 4 * r * c;   // one table instead of n + 1
    // second round: per candidate, its index, the n workers' values (and vhat) in, its exact value out
    const uint64_t second = s->cand_mult > 1 ? (uint64_t)s->cand_mult * k * (4 * n + (s->variant == 1 ? 8 : 12)) : 0;
    if (s->variant == 1)     // Algorithm 1: read g,m,v,vhat,e and write m,v,vhat,e; no master-side second moments
        return (36 - g) * n * d + tables + 8 * n * k + 8 * k + second;
    return (20 - g) * n * d + 4 * d + tables + 12 * n * k + 24 * k + second;
}

int sk_get_timing(sk_state* s, double* ms, uint64_t* launches) {
    if (!s || !ms || !launches) return fail(SK_EINVAL, "null argument");
    int rc = flush_timing(s);
    if (rc) return rc;
    for (int q = 0; q < SK_NUM_STAGES; ++q) {
        ms[q] = s->ms[q]; launches[q] = s->launches[q];
        s->ms[q] = 0; s->launches[q] = 0;
    }
    const int steps = (int)s->timed_steps;
    s->timed_steps = 0;
    return steps;
}

}  // extern "C"

#include "sk_api_state.inc"
