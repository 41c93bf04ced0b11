/*
 * sketched_amsgrad.h -- C ABI of the B200 (sm_100a) library for one compressed optimiser step of
 * SketchedAMSGrad with gradient averaging (Algorithm 2 of the paper), all n workers resident on one GPU.
 *
 * One step, in the paper's notation (w = worker, j = coordinate, constant step size so alpha_{t-1}/alpha_t = 1):
 *   m_t^(w)   = beta1 m_{t-1}^(w) + (1-beta1) g_t^(w)                          (Algorithm 2, worker side)
 *   h_t       = mean_w g_t^(w) on I_{t-1}, 0 elsewhere;  v_t = beta2 v_{t-1} + (1-beta2) h_t^2;
 *   vhat_t    = max(vhat_{t-1}, v_t)                                            (Algorithm 2, master side)
 *   a_t^(w)   = m_t^(w) + e_{t-1}^(w);   S_t^(w) = S(a_t^(w))                   (Count Sketch, Section II-C)
 *   S_t       = (1/n) sum_w S_t^(w)       (workers added in the order 0..n-1)
 *   est_j     = median_row( s_row(j) S_t[row, h_row(j)] ) / sqrt(vhat_t,j)      (Algorithm 3)
 *   I_t       = indices of the k largest |est_j| (ties: smaller index)
 *   x_j      -= lr * mean_w a_t^(w)_j / sqrt(vhat_t,j)   for j in I_t           (exact values, Section III-A)
 *   e_t^(w)   = a_t^(w) off I_t, 0 on I_t                                       (error feedback)
 * v_0 = vhat_0 = eps (an initial value, not a denominator term), m_0 = e_0 = 0, I_0 = empty.
 * Options widen this to the rest of the method: Algorithm 1 ("variant"), the second selection round of
 * Section III-A ("P"), a step-size schedule (sk_set_lr), frozen second moments ("freeze_v"), bf16 gradients
 * ("grads_bf16"), and the workers partitioned over several GPUs (sk_step_local / _select / _finish).
 *
 * Conventions for every entry point:
 *   - "device" pointers are CUDA device memory of the current device; "host" pointers are ordinary memory.
 *   - All arrays are dense fp32 / uint32 in C order.  The caller owns what it passes in; the handle owns all
 *     optimiser state and scratch, allocated in sk_create and released in sk_destroy.
 *   - Functions returning int give 0 on success or a negative SK_E* code; sk_last_error() then holds a
 *     message (thread-local).  Nothing throws, nothing calls exit.  There is no CPU fallback: without a
 *     CUDA device every call that needs one fails with SK_ECUDA.
 *   - A handle is used from one thread at a time; kernels run asynchronously on the handle's stream
 *     (the default stream unless sk_set_stream was called).
 */
#ifndef SKETCHED_AMSGRAD_H
#define SKETCHED_AMSGRAD_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SK_OK        0
#define SK_EINVAL   -1   /* bad argument (null, misaligned, out of range, unknown name) */
#define SK_ECUDA    -2   /* a CUDA runtime call or launch failed; message in sk_last_error() */
#define SK_ENOMEM   -3   /* device allocation failed */
#define SK_ESTATE   -4   /* call not allowed in the handle's current state (e.g. hash option after first step) */
#define SK_EDEVICE  -5   /* a kernel reported an internal inconsistency through the device status word */

typedef struct sk_state sk_state;

/* Algorithm 2's "Input/Set" lines.  d coordinates (1 <= d < 2^32), n workers, r x c sketch (1 <= r <= 16),
 * k kept coordinates (1 <= k <= d), hash seed, step size lr, beta1, beta2 in [0,1), eps > 0.
 * Allocates m,e (n*d), v,vhat (d), n+1 sketch tables and selection scratch (8*d bytes) on the current device
 * and initialises them.  Returns NULL on failure (see sk_last_error()). */
sk_state* sk_create(uint64_t d, uint32_t n, uint32_t r, uint32_t c, uint64_t k, uint64_t seed,
                    float lr, float beta1, float beta2, float eps);

/* One iteration of Algorithm 2 (the whole list above).  grads: device, n*d gradient entries, worker-major
 * (grads[w*d + j]), read only: fp32, or bf16 when the option "grads_bf16" is 1 (the entries are widened exactly;
 * everything else stays fp32).  x: device, d fp32, updated in place.  Both must be 4-byte aligned; the
 * vectorised kernels are used when d % 4 == 0 and both are 16-byte aligned, scalar kernels otherwise.
 * Asynchronous: returns after enqueueing on the handle's stream. */
int sk_step(const void* grads, float* x, sk_state* state);

/* Step size alpha_t of the steps taken from now on (Algorithms 1 and 2 allow a schedule; Theorem 2 uses
 * alpha/sqrt(t)).  Each step weights e_{t-1} by alpha_{t-1}/alpha_t, computed in fp64 from the two fp32 values
 * and rounded to fp32, with alpha_{t-1} the step size of the last step taken (1 when they are equal).  Finite;
 * a zero step size cannot precede or follow a different one.  Not inside a partitioned step. */
int sk_set_lr(sk_state* state, float lr);

/* Same step with HOST buffers: copies grads (n*d) to an internal device staging buffer and x (d) in,
 * runs the step, copies x back, and synchronises the stream.  The gradients are copied in up to four pieces of
 * whole workers on an internal copy stream and the sketch kernel starts on each piece as it arrives, so most of
 * the kernel time hides behind the transfer; with pageable memory the copies simply serialise.  Pinned host
 * memory makes the copies faster but is not required.  The staging buffers, the copy stream and its events are
 * created on first use and released by sk_destroy. */
int sk_step_host(const void* grads_host, float* x_host, sk_state* state);

/* Host-buffer step in the method's own exchange pattern (Section III-B: what the master returns is the sparse update,
 * k values and their positions): the parameters stay on the device (field "x": set it once with sk_set, read it with
 * sk_get; zero until set), the gradients come from the host as for sk_step_host, and what goes back is
 * idx_host[q] = the k coordinates of I_t (in no particular order) and values_host[q] = the new value of x there, so
 * that a host copy of the parameters is brought up to date with x[idx_host[q]] = values_host[q].  Both HOST, k
 * entries.  8*k bytes return instead of 4*d, and x is not sent at all.  Synchronises the stream.
 * sk_step_host overwrites the same device-resident parameters with its x_host. */
int sk_step_host_sparse(const void* grads_host, uint32_t* idx_host, float* values_host, sk_state* state);

/* ---- One iteration with the WORKERS PARTITIONED over several processes (one GPU each) -----------------------------
 * Every process creates a handle for its own n workers (same d, r, c, k, seed, hyper-parameters and options on all
 * of them), sets the option "workers_total" to the number of workers over all processes, and keeps a replica of x.
 * Algorithms 1 and 2 couple the workers only through sums, and those sums are what the processes exchange: per
 * iteration the sketch, the gradient entries on I_{t-1} and the exact values of the candidates, i.e. the
 * |S| + k + P*k floats of Section III-B (the update is applied by every replica, so it is not sent back).  An
 * iteration is three calls with one sum over the processes (an all-reduce, done by the caller) between them:
 *
 *   sk_step_local (grads, exchange1, state)      moments, a_t and sketches of this process's workers
 *   -- caller: exchange1 <- sum over processes of exchange1 --
 *   sk_step_select(exchange1, exchange2, state)  second moments on I_{t-1}, unsketch, selection of the candidates
 *   -- caller: exchange2 <- sum over processes of exchange2 --
 *   sk_step_finish(exchange2, x, state)          second round (P > 1), update of x, new I_t
 *
 * exchange1: device, sk_exchange_floats(state, 1) floats, 16-byte aligned: this process's share of the mean sketch
 *   (r rows of c floats, each row padded to a multiple of 32), then, for Algorithm 2, its gradient sums on I_{t-1}
 *   in ascending index order, zero-padded to k.  exchange2: device, sk_exchange_floats(state, 2) = P*k floats: its
 *   sums of a_t at the candidates in ascending index order.  Both are caller-owned; the library writes them in the
 *   first call of each pair and reads the summed values in the second.  The sum must give every process the same
 *   bits (NCCL's all-reduce does), since every process then takes the same selection from them.
 * grads: this process's n*d gradients, as for sk_step.  All work is enqueued on the handle's stream; nothing
 * synchronises.  Calls out of order return SK_ESTATE.  With one process the result equals sk_step's up to the
 * rounding of the sums. */
uint64_t sk_exchange_floats(const sk_state* state, int which /* 1 or 2 */);
int sk_step_local(const void* grads, float* exchange1, sk_state* state);
int sk_step_select(const float* exchange1, float* exchange2, sk_state* state);
int sk_step_finish(const float* exchange2, float* x, sk_state* state);

/* Releases everything sk_create and later calls allocated.  NULL is accepted. */
void sk_destroy(sk_state* state);

/* stream: a cudaStream_t cast to void* (NULL = default stream).  The handle does not own it. */
int sk_set_stream(sk_state* state, void* stream);
/* Waits for everything enqueued on the handle's stream and reports the device status word: SK_EDEVICE with a
 * message if it is not zero, after which the word is cleared (the handle stays usable).  Bit 0: a selection emitted a
 * number of indices other than k.  Bits 1..5 exist in the debug build (compiled with -DSK_DEBUG=1, see
 * paper_2210_07454_b200/build.py --debug), whose kernels compare every hashed table offset, coordinate index, list
 * position, histogram bin and shared-memory window offset with the size of what it addresses, record a violation
 * here and skip the access; nothing traps.  Bit 6 (debug build): a gradient entry was not finite -- inputs must be
 * finite; the step is taken regardless and its results are then unspecified. */
int sk_sync(sk_state* state);

/* Per-step statistics of the last step's selection (Algorithm 2's Top-k) and the method's exchange volume, for
 * logging: out[0] = the threshold key's leading 24 bits as an fp32 value (a lower bound of the k-th largest
 * |estimate|, within 2^-16 relative), out[1] = coordinates whose key fell into the threshold's 4096-way bin,
 * out[2] = coordinates sharing the threshold's leading 24 key bits (the tie group resolved exactly),
 * out[3] = indices emitted (k unless the status word says otherwise), out[4] = floats one iteration puts on the wire
 * by Section III-B's count, r*c + P*k + 2k (r*c + P*k + k for Algorithm 1), out[5] = the device status word.
 * `out` is a HOST array of at least SK_NUM_STATS doubles.  Synchronises the stream. */
#define SK_NUM_STATS 6
int sk_get_stats(sk_state* state, double* out, uint32_t count);

/* Test hooks (host side; neither touches the GPU's state).
 * sk_test_fail_allocation(nth): the (nth+1)-th device allocation of the following sk_create calls fails as if the
 * device were out of memory (sk_create then returns NULL with a message and frees what it had allocated); nth < 0
 * switches the hook off.  Process-wide; not thread-safe.
 * sk_debug_check(state, kind), kind 1..6: in the debug build a one-thread kernel runs the bounds check of that kind
 * with a false condition (no access is made), so the next sk_sync must report bit `kind`; SK_ESTATE in the normal
 * build, which has no device-side checks.  The paper has no counterpart for either. */
int sk_test_fail_allocation(int64_t nth);
int sk_debug_check(sk_state* state, uint32_t kind);

/* Options (integers):
 *   "log2g"        hash group size g = 2^log2g, 0..5 (Section II-C fixes no hash family; see sk_hash).
 *                  Only before the first step.  Default: the largest value <= 5 with 2^log2g <= c.
 *   "P"            candidate multiplier of the second round (Section III-A): the P*k largest
 *                  estimates become candidates, their exact values are fetched from the workers' vectors, and the
 *                  k candidates of largest exact magnitude form I_t (ties: smaller index).  1 (default) = no second
 *                  round.  P*k <= d.  Only before the first step.  The candidates of the last step are field "cand".
 *   "sum_sketch"   1: the n per-worker sketches and their sum are replaced by ONE sketch of the worker sum,
 *                  S((1/n) sum_w a^(w)), which equals (1/n) sum_w S(a^(w)) because the sketch is linear (Section II-C;
 *                  the two differ only in the rounding of fp32 sums).  The per-worker tables are then not formed
 *                  (sk_get "tables" fails) -- they are what a worker would transmit, so this is for a single GPU
 *                  holding all workers, or for the local share of a partitioned step.  Default 0: n sketches.
 *                  Uses the reduction kernel (not the shared-memory windows).  Any time between steps.
 *   "freeze_v"     1: Algorithm 2 without h_t and without the update of v and vhat, which keep the values they have
 *                  (set them with sk_set "v", "vhat"): the fixed-variance scheme Section III-B reduces the method
 *                  to.  0 (default) resumes the updates.  Gradient averaging only.  Any time between steps.
 *   "grads_bf16"   1: the gradient arguments of sk_step, sk_step_host and sk_step_local hold bf16 entries
 *                  (2 bytes each, same layout).  Default 0.  Any time between steps.
 *   "workers_total" number of workers the means are taken over, >= n; default n.  Set it on every handle of a
 *                  partitioned step (see sk_step_local) to the sum of their n.  Only before the first step.
 *   "variant"      0 (default) = gradient averaging, Algorithm 2; 1 = parameter averaging, Algorithm 1: every worker
 *                  keeps its own v and vhat (fields "vw", "vhatw", n*d each, initial value eps) from its own
 *                  gradient, sketches m/sqrt(vhat) + e, the unsketch takes no vhat and x moves by the plain mean
 *                  of the exact values on I_t.  Only before the first step; allocates 8*n*d bytes.
 *   "window_lines" L > 0 selects the windowed variant of the hash family (needs g = 32, 32*L <= c): units of
 *                  1024 coordinates map into one aligned window of 32*L buckets per row, which lets the sketch
 *                  kernel accumulate in shared memory, one warp per worker.  Default: 8 when g = 32 and c >= 256
 *                  (Algorithm 2), else 0 (plain family; also what "log2g" < 5 and, unless set explicitly,
 *                  "variant" = 1 select).  Only before the first step.
 *   "window_workers" (1..8) workers per launch of the shared-memory sketch kernel (one warp each); default 8.
 *   "worker_sum"   1: the sketch kernel also stores sum_w a^(w) per coordinate (4*d bytes more written, allocated
 *                  when first enabled), and the update of x reads one value per index of I_t instead of n.
 *                  Default 0.  Any time between steps.
 *   "worker_chunk" workers whose tables are accumulated concurrently by the sketch kernel (0 = automatic,
 *                  sized so that the concurrently updated tables stay resident in L2).
 *   "sketch_ctas_per_sm" grid size of the plain sketch kernel in blocks per SM (default 64: one tile per block).
 *   "chained_launches" 1 (default): the kernels of a step are launched with the programmatic-serialization
 *                  attribute: each may become resident while its predecessor in the stream still runs, does its
 *                  shared-memory set-up, and waits for the predecessor's completion before it touches global
 *                  memory.  Results do not depend on it; 0 launches them plainly (values 2..511 chain only some
 *                  kinds of launch: a diagnostic mask, see csrc/sk_chain.cuh).  Any time between steps.
 *   "timing"       1 = record CUDA events around each stage (see sk_get_timing); 0 = off (default). */
int sk_set_option(sk_state* state, const char* key, int64_t value);
/* Also readable: "I_count" (entries "I" currently holds: 0 before the first step, else k unless sk_set installed
 * fewer) and "vectorised" (1 when d % 4 == 0 and g >= 4, so aligned buffers take the 128-bit kernels). */
int sk_get_option(const sk_state* state, const char* key, int64_t* value);

/* The bucket hashes h_row and sign hashes s_row of Section II-C for coordinates i0 .. i0+count-1:
 * idx_out[t] in [0,c), sign_out[t] in {+1,-1}; both DEVICE pointers.  Family (all arithmetic mod 2^64):
 *   stream(s,t) = t-th output of splitmix64 started at s;  K_row = stream(seed, row+1);
 *   q = i div g, o = i mod g, G = c div g;  u = stream(K_row, q+1), hi = u div 2^32, lo = u mod 2^32;
 *   x = hi*G;  h_row(i) = g*(x div 2^32) + (o xor p), p = the leading log2(g) bits of (x mod 2^32);
 *   s_row(i) = +1 if bit 0 of lo is clear, else -1: one sign per (row, group).  The coordinates of a group never
 *   share a bucket, so their relative sign never enters a sum; coordinates of different groups carry independent signs. */
int sk_hash(const sk_state* state, uint32_t row, uint64_t i0, uint64_t count,
            uint32_t* idx_out, int8_t* sign_out);

/* State access for checkpointing and for tests.  `buf` may be a host or a device pointer; `bytes` must equal
 * the field's size.  Fields (fp32 unless noted):
 *   "m","e"   n*d  per-worker momentum and error-feedback residual (after a step, "e" is e_t)
 *   "v","vhat" d   second moments ("v" is brought up to date with the decay it is owed before export)
 *   "tables"  n*r*c  the worker sketches S_t^(w) of the last step;  "sum"  r*c  the aggregate S_t
 *   "est"     d    the estimates of the last step (recomputed on request from "sum" and "vhat"; get only)
 *   "keys"    d uint32  the ranking keys the last step's selection ran on: the bit pattern of |median * rsqrt(vhat)|
 *                  (of |median| for Algorithm 1), as the key pass stored them (get only, after the first step)
 *   "I"       k uint32  I_t of the last step, ascending (get);  set: installs I_{t-1} for the next step
 *   "vw","vhatw" n*d  per-worker second moments (parameter-averaging variant only; "v","vhat" are then unavailable)
 *   "cand"    P*k uint32  candidates of the last step's second round, ascending (get only; empty when P = 1)
 *   "x"       d    the device-resident parameters of the host-buffer steps (see sk_step_host_sparse)
 *   "t"       1 uint64  number of steps taken
 * Both calls synchronise the stream. */
int sk_get(sk_state* state, const char* field, void* buf, uint64_t bytes);
int sk_set(sk_state* state, const char* field, const void* buf, uint64_t bytes);

/* Bytes one step must move by the method's own definition, used as the roofline numerator:
 * 20*n*d (read g,m,e; write m,e) + 4*d (vhat) + 8*n*r*c + 4*r*c (worker tables written and read, aggregate
 * written) + 12*n*k + 24*k (sparse gathers and updates on I_{t-1} and I_t).  Algorithm 1: 36*n*d (g, m, v, vhat, e
 * in; m, v, vhat, e out) and no master-side second moments.  bf16 gradients: 2 bytes less per worker-coordinate.
 * Second round: P*k*(4n + 12) more (candidate index, the n workers' values and vhat in, the exact value out). */
uint64_t sk_algorithmic_bytes(const sk_state* state);

/* Stage timing (option "timing" = 1).  Stages: 0 zero tables, 1 unused (the second moments on I_{t-1} are updated
 * inside stage 4), 2 moments+sketch, 3 sum of sketches, 4 ranking keys + histogram (+ v, vhat on I_{t-1}),
 * 5 emit above the threshold bin, 6 threshold refinement, 7 apply on I_t.
 * Adds up the events of all steps since the last call into ms[0..7] (milliseconds) and launches[0..7]
 * (kernel launches), then clears them.  Synchronises the stream.  Returns the number of steps covered, or <0. */
#define SK_NUM_STAGES 8
int sk_get_timing(sk_state* state, double* ms, uint64_t* launches);

/* The paper has no counterpart for this entry point; it exists for callers that must not allocate.
 * Some callers cannot call cudaMalloc at the moment they need a selection: code running under a framework whose
 * caching allocator owns the device and forbids foreign allocations, code on a latency path that cannot afford
 * cudaMalloc's implicit device-wide synchronisation, or code running after device memory has been filled on
 * purpose.  sk_select_static re-runs the top-k selection of the handle's LAST step (same inputs: the aggregated
 * sketch and vhat the handle holds) and writes the k selected indices, in no particular order, to idx_out
 * (DEVICE pointer, k uint32, caller-owned).  It calls no cudaMalloc, cudaFree or any other allocating routine:
 * all its scratch (histograms, ranking keys, candidate lists; about 5 MB) lives in one file-scope device array
 * inside the library, which every GPU that loads the library holds until the process exits.
 *   - Limit: d <= SK_STATIC_MAX_D; larger handles are rejected with SK_EINVAL and a message naming the limit.
 *     SK_ESTATE if the handle has not taken a step yet, is in the middle of a partitioned step, or runs a second
 *     round (P > 1), whose exact values this entry point does not fetch.
 *   - The device address of the scratch array is resolved once per device, with that device current: by sk_create
 *     (which is allowed to allocate, and so absorbs whatever loading the array's module costs) for every handle
 *     with d <= SK_STATIC_MAX_D, else by the first call of this entry point on the device -- make that first call
 *     before starting any stream capture.  The call launches only kernels the handle's last step has already
 *     launched, so nothing is loaded lazily either: it is allocation-free once a handle exists on the device and
 *     has taken a step.
 *   - What the selection finds wrong (a count other than k; in the debug build any out-of-range position) is
 *     OR-ed into the handle's status word, which sk_sync reports.
 *   - Every call, from every handle and stream, shares the one array, and the array keeps the previous call's
 *     contents; the entry point clears the parts that must start at zero itself.  Two calls that overlap on the
 *     GPU (different streams or threads) race on the array: serialise them.
 *   - Asynchronous on the handle's stream, like sk_step; the handle's own state is read, not modified. */
#define SK_STATIC_MAX_D 262144u
int sk_select_static(sk_state* state, uint32_t* idx_out);

const char* sk_last_error(void);
const char* sk_version(void);

#ifdef __cplusplus
}
#endif
#endif
