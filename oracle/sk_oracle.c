/*
 * CPU oracle for SketchedAMSGrad (gradient averaging): see sk_oracle.h for what this is and is not.
 * TEST INFRASTRUCTURE ONLY.  Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC.
 */
#include "sk_oracle.h"
#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------------
 * Hash and sign family.  Section II-C only names bucket hashes h_j:[d]->[c] and sign hashes
 * s_j:[d]->{+1,-1}, j=1..r; the family below is this library's definition.
 *
 *   mix64      : the output function of the splitmix64 generator (Steele, Lea, Flood 2014; Vigna)
 *   stream(s,t): t-th output of splitmix64 started at state s, = mix64(s + t*GOLDEN)
 *   K_j        = stream(seed, j+1)                                   row key
 *   g = 2^b consecutive coordinates form a group: q = i div g, o = i mod g, G = floor(c/g)
 *   u  = stream(K_j, q+1);  hi = u div 2^32, lo = u mod 2^32;  x = hi * G  (a 64-bit product)
 *   B  = x div 2^32                                                  bucket group, in [0,G)
 *   p  = (x mod 2^32) div 2^(32-b)                                   xor-permutation inside the group: the
 *                                                                    leading b bits of the remainder of the
 *                                                                    range reduction (p = 0 when g = 1)
 *   h_j(i) = g*B + (o xor p)
 *   s_j(i) = +1 if bit 0 of lo is 0, else -1:  ONE sign per (row, group)
 *
 * Two coordinates of one group never share a bucket, so their relative sign never enters a bucket's sum; two
 * coordinates of different groups share one with probability 1/(G*g) and carry independent signs, which is all
 * the second-moment argument behind the Count Sketch uses.  With g = 1 this is an ordinary per-coordinate hash
 * and sign.
 * ------------------------------------------------------------------------------------------------ */
static const uint64_t GOLDEN = 0x9E3779B97F4A7C15ULL;

uint64_t ora_mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

uint64_t ora_stream(uint64_t s0, uint64_t t) { return ora_mix64(s0 + t * GOLDEN); }

uint64_t ora_row_key(uint64_t seed, uint32_t row) { return ora_stream(seed, (uint64_t)row + 1); }

/* Windowed variant (window_lines = L > 0, needs g = 32): the coordinates are cut into units of 1024; unit u
 * belongs to panel u mod P, where P = floor(c / (32 L)) is the number of aligned windows of 32 L buckets in a
 * row; every group of the unit lands in its panel's window, on one of the window's L lines:
 *   x = hi * L ;  line = x div 2^32 ;  p = leading 5 bits of (x mod 2^32)
 *   h_j(i) = (u mod P) * 32 L + 32 * line + (o xor p) ;   signs as above.
 * A row is then P independent small Count Sketches (one per panel, each of 32 L buckets); coordinates of
 * different panels never meet, coordinates of one panel and different groups meet with probability 1/(32 L).
 * Because units are dealt to panels round-robin, every panel sees every part of the vector. */
#define ORA_UNIT 1024ULL

void ora_hash_one_w(uint64_t seed, uint32_t log2g, uint32_t window_lines, uint32_t c, uint32_t row, uint64_t i,
                    uint32_t* bucket, int8_t* sign) {
    uint64_t g = 1ULL << log2g;
    uint64_t q = i >> log2g;
    uint64_t o = i & (g - 1);
    uint64_t K = ora_row_key(seed, row);
    uint64_t u = ora_stream(K, q + 1);
    uint64_t hi = u >> 32, lo = u & 0xFFFFFFFFULL;
    uint64_t G = window_lines ? window_lines : c / g;      /* lines to choose from */
    uint64_t x = hi * G;
    uint64_t B = x >> 32;
    uint64_t p = log2g ? ((x & 0xFFFFFFFFULL) >> (32 - log2g)) : 0;
    uint64_t base = 0;
    if (window_lines) {
        uint64_t cw = g * window_lines, P = c / cw;
        base = ((i / ORA_UNIT) % P) * cw;
    }
    *bucket = (uint32_t)(base + g * B + (o ^ p));
    *sign = (lo & 1ULL) ? -1 : 1;
}

void ora_hash_one(uint64_t seed, uint32_t log2g, uint32_t c, uint32_t row, uint64_t i,
                  uint32_t* bucket, int8_t* sign) {
    ora_hash_one_w(seed, log2g, 0, c, row, i, bucket, sign);
}

void ora_hash(uint64_t seed, uint32_t log2g, uint32_t c, uint32_t row, uint64_t i0, uint64_t count,
              uint32_t* bucket, int8_t* sign) {
    for (uint64_t t = 0; t < count; ++t) ora_hash_one(seed, log2g, c, row, i0 + t, &bucket[t], &sign[t]);
}

void ora_hash_w(uint64_t seed, uint32_t log2g, uint32_t window_lines, uint32_t c, uint32_t row, uint64_t i0,
                uint64_t count, uint32_t* bucket, int8_t* sign) {
    for (uint64_t t = 0; t < count; ++t)
        ora_hash_one_w(seed, log2g, window_lines, c, row, i0 + t, &bucket[t], &sign[t]);
}

/* ------------------------------------------------------------------------------------------------
 * Count Sketch, Section II-C:  S[j, h_j(i)] += s_j(i) * f_i  for every coordinate i and row j.
 * Each bucket is accumulated in fp64 over coordinates in increasing i and rounded to fp32 once.
 * ------------------------------------------------------------------------------------------------ */
void ora_sketch(const float* a, uint64_t d, uint32_t r, uint32_t c,
                const uint32_t* idx, const int8_t* sgn, float* table) {
    double* acc = (double*)calloc((size_t)c, sizeof(double));
    for (uint32_t j = 0; j < r; ++j) {
        memset(acc, 0, (size_t)c * sizeof(double));
        for (uint64_t i = 0; i < d; ++i) acc[idx[j * d + i]] += (double)sgn[j * d + i] * (double)a[i];
        for (uint32_t b = 0; b < c; ++b) table[(uint64_t)j * c + b] = (float)acc[b];
    }
    free(acc);
}

/* Median of r values, Section II-C ("the median value of s_j(i) S[j,h_j(i)]").
 * For even r the LOWER median (the ceil(r/2)-th smallest) is returned: a member of the set. */
float ora_median(const float* q, uint32_t r) {
    float tmp[64];
    if (r > 64) r = 64;
    for (uint32_t j = 0; j < r; ++j) tmp[j] = q[j];
    for (uint32_t a = 1; a < r; ++a) {            /* insertion sort, ascending */
        float key = tmp[a];
        uint32_t b = a;
        while (b > 0 && tmp[b - 1] > key) { tmp[b] = tmp[b - 1]; --b; }
        tmp[b] = key;
    }
    return tmp[(r - 1) / 2];
}

/* Unsketch: est_i = median_j( s_j(i) * S[j,h_j(i)] ), and, when vhat is given, divided by sqrt(vhat_i)
 * (Algorithm 3 read as a per-coordinate scale at query time: the estimate of
 *  Delta~_t[i] = vhat_i^{-1/2} * mean_w (m + rho e)[i], the unnumbered equation defining Delta~_t). */
void ora_unsketch(const float* table, uint64_t d, uint32_t r, uint32_t c,
                  const uint32_t* idx, const int8_t* sgn, const float* vhat, float* est) {
    float q[64];
    for (uint64_t i = 0; i < d; ++i) {
        for (uint32_t j = 0; j < r; ++j)
            q[j] = (float)sgn[j * d + i] * table[(uint64_t)j * c + idx[j * d + i]];
        double med = (double)ora_median(q, r);
        est[i] = vhat ? (float)(med / sqrt((double)vhat[i])) : (float)med;
    }
}

/* Top-k (Algorithm 2, "Top-k(U(S_t, vhat_t))"): the k indices of largest |est|; equal magnitudes are
 * ordered by index, smaller first.  Done by a full sort of (magnitude desc, index asc). */
typedef struct { float mag; uint32_t idx; } ora_pair;
static int ora_pair_cmp(const void* pa, const void* pb) {
    const ora_pair* a = (const ora_pair*)pa;
    const ora_pair* b = (const ora_pair*)pb;
    if (a->mag > b->mag) return -1;
    if (a->mag < b->mag) return 1;
    return (a->idx > b->idx) - (a->idx < b->idx);
}
static int ora_u32_cmp(const void* pa, const void* pb) {
    uint32_t a = *(const uint32_t*)pa, b = *(const uint32_t*)pb;
    return (a > b) - (a < b);
}
void ora_topk(const float* est, uint64_t d, uint64_t k, uint32_t* I) {
    ora_pair* p = (ora_pair*)malloc((size_t)d * sizeof(ora_pair));
    for (uint64_t i = 0; i < d; ++i) { p[i].mag = fabsf(est[i]); p[i].idx = (uint32_t)i; }
    qsort(p, (size_t)d, sizeof(ora_pair), ora_pair_cmp);
    for (uint64_t t = 0; t < k; ++t) I[t] = p[t].idx;
    qsort(I, (size_t)k, sizeof(uint32_t), ora_u32_cmp);
    free(p);
}

double ora_comm_floats(uint64_t r, uint64_t c, uint64_t k, uint64_t P) {
    return (double)r * (double)c + (double)P * (double)k + 2.0 * (double)k;
}
