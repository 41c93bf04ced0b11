/*
 * CPU oracle for one compressed optimiser step of SketchedAMSGrad (gradient averaging).
 *
 * THIS IS TEST INFRASTRUCTURE, not a product path.  It is a plain, slow, single-purpose restatement of
 * the paper's Algorithm 2 (SketchedAMSGrad, gradient averaging), Algorithm 3 (unsketching with v-hat) and
 * the Count Sketch of Section II-C, used only to check the CUDA library and to be timed beside it.
 * It shares no code with the CUDA path and must never be called from it.
 *
 * Arithmetic: optimiser state (m, e, v, vhat, x) and sketch tables are STORED as fp32, because that is
 * the storage type the method is run in; every update is EVALUATED in fp64 and rounded to fp32 once on
 * store.  Top-k decisions are taken on the fp32-rounded estimates.
 *
 * Readings of the paper taken here (each is also a switch or is stated in the function's comment):
 *   - v_0 = vhat_0 = eps (Algorithm 1's initialisation, applied to Algorithm 2 which prints no value);
 *     eps is an initial value, never a denominator term (Section III-A).
 *   - Algorithm 2's v update is applied to ALL coordinates with h_t zero off I_{t-1}
 *     (v decays there); `v_keep=1` switches to "v unchanged off I_{t-1}" (the remark in Lemma 3's proof).
 *   - Algorithm 3 is read as a per-coordinate scale at query time:
 *     est_i = median_j( s_j(i) S[j,h_j(i)] ) / sqrt(vhat_i).
 *   - Delta_t holds the EXACT worker means at I_t, preconditioned (the second communication round of
 *     Section III-A); e_t^(i) is a_t^(i) with the coordinates of I_t set to zero (Lemma 3's proof).
 *   - Even r: lower median.  Ties in top-k: the smaller index wins.
 *
 * ora_step also implements Algorithm 1 (parameter averaging) when the option "variant_pa" is set: per-worker
 * v and vhat from the worker's own gradient, the sketched vector is m/sqrt(vhat) + e, and the unsketch takes no vhat.
 *
 * Parity pins: see tests/test_oracle_*.py.  Nothing here is "parity unpinned" except the five large
 * benchmark workloads themselves, for which the paper prints no expected values.
 */
#ifndef SK_ORACLE_H
#define SK_ORACLE_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- hash / sign family (Section II-C names {h_j},{s_j} but fixes no family; this is the library's own) */
uint64_t ora_mix64(uint64_t z);
uint64_t ora_stream(uint64_t s0, uint64_t t);          /* t-th output (t>=1) of splitmix64 seeded s0 */
uint64_t ora_row_key(uint64_t seed, uint32_t row);
/* bucket in [0,c) and sign in {+1,-1} of coordinate i in row `row`; group size g = 1<<log2g */
void ora_hash_one(uint64_t seed, uint32_t log2g, uint32_t c, uint32_t row, uint64_t i,
                  uint32_t* bucket, int8_t* sign);
void ora_hash(uint64_t seed, uint32_t log2g, uint32_t c, uint32_t row, uint64_t i0, uint64_t count,
              uint32_t* bucket, int8_t* sign);
/* windowed variant of the family (window_lines > 0; see sk_oracle.c); window_lines = 0 is the plain family */
void ora_hash_one_w(uint64_t seed, uint32_t log2g, uint32_t window_lines, uint32_t c, uint32_t row, uint64_t i,
                    uint32_t* bucket, int8_t* sign);
void ora_hash_w(uint64_t seed, uint32_t log2g, uint32_t window_lines, uint32_t c, uint32_t row, uint64_t i0,
                uint64_t count, uint32_t* bucket, int8_t* sign);

/* ---- Count Sketch primitives with EXPLICIT index / sign arrays (idx[row*d+i], sgn[row*d+i]) */
void ora_sketch(const float* a, uint64_t d, uint32_t r, uint32_t c,
                const uint32_t* idx, const int8_t* sgn, float* table /* r*c, overwritten */);
float ora_median(const float* q, uint32_t r);          /* lower median; q is not modified */
void ora_unsketch(const float* table, uint64_t d, uint32_t r, uint32_t c,
                  const uint32_t* idx, const int8_t* sgn, const float* vhat /* may be NULL */,
                  float* est /* d */);
/* indices of the k largest |est|, ties -> smaller index; output ascending by index */
void ora_topk(const float* est, uint64_t d, uint64_t k, uint32_t* I);

/* ---- full optimiser step */
typedef struct ora_state ora_state;
ora_state* ora_create(uint64_t d, uint32_t n, uint32_t r, uint32_t c, uint64_t k, uint64_t seed,
                      uint32_t log2g, float lr, float beta1, float beta2, float eps);
void ora_destroy(ora_state* s);
/* inject explicit hash arrays (r*d each) instead of the seeded family; pointers must outlive the state */
void ora_set_hash(ora_state* s, const uint32_t* idx, const int8_t* sgn);
/* "P" (candidate multiplier of the second round, Section III-A: top P*k by estimate, then top-k by exact value;
   the candidates of the last step are the uint32 field "cand"), "v_keep", "threads", "window_lines" (windowed hash family), "variant_pa" (1 = Algorithm 1, parameter averaging;
   per-worker v and vhat are then the fields "vw" and "vhatw", n*d each) */
void ora_set_option(ora_state* s, const char* key, int value);
/* "freeze_v" (Algorithm 2 only): h_t is not used and v, vhat keep the values they have (Section III-B: with the
   variance term fixed the method becomes the fixed-preconditioner scheme it is compared with).
   ora_set_lr: the step size alpha_t of the steps taken from now on; each step weights e_{t-1} by
   alpha_{t-1}/alpha_t as Algorithms 1 and 2 print it (alpha_0 := alpha_1). */
void ora_set_lr(ora_state* s, float lr);
int  ora_step(ora_state* s, const float* grads /* n*d worker-major */, float* x /* d, in place */);

/* field access: "m","e" (n*d) "v","vhat","est" (d) "tables" (n*r*c) "sum" (r*c) -> float*;
   "I","I_prev" -> uint32_t* (k entries, ascending; I_prev has ora_count(s,"I_prev") valid entries) */
void*    ora_field(ora_state* s, const char* name);
uint64_t ora_count(ora_state* s, const char* name);

/* communication volume per iteration in floats: r*c + P*k + 2k  (Section III-B) */
double ora_comm_floats(uint64_t r, uint64_t c, uint64_t k, uint64_t P);

#ifdef __cplusplus
}
#endif
#endif
