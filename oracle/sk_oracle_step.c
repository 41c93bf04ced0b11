/*
 * CPU oracle, part 2: one full step of SketchedAMSGrad with gradient averaging (Algorithm 2), with the
 * unsketching operator of Algorithm 3.  TEST INFRASTRUCTURE ONLY (see sk_oracle.h).
 */
#include "sk_oracle.h"
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

struct ora_state {
    uint64_t d, k, seed, t, k_prev;
    uint32_t n, r, c, log2g, window_lines;
    float lr, beta1, beta2, eps;
    float lr_prev;           /* alpha_{t-1}: the step size of the last step taken (alpha_0 := alpha_1) */
    int v_keep, threads, variant_pa;
    int freeze_v;            /* Algorithm 2 without h_t and without the update of v, vhat (Section III-B's remark) */
    uint32_t P;              /* candidate multiplier of the second round (Section III-A); 1 = no second round */
    uint32_t* cand;          /* the P*k candidates of the last step, ascending */
    float *vw, *vhatw;       /* parameter-averaging variant: per-worker v and vhat (n*d each) */
    float *m, *e, *v, *vhat, *est, *tables, *sum;
    uint32_t *I, *I_prev;
    uint8_t* mask;
    const uint32_t* h_idx;   /* injected hashes, or NULL: use the seeded family */
    const int8_t* h_sgn;
    uint64_t* row_key;
};

ora_state* ora_create(uint64_t d, uint32_t n, uint32_t r, uint32_t c, uint64_t k, uint64_t seed,
                      uint32_t log2g, float lr, float beta1, float beta2, float eps) {
    if (d == 0 || n == 0 || r == 0 || r > 64 || c == 0 || k == 0 || k > d || log2g > 5) return NULL;
    if ((c >> log2g) == 0 || d >= (1ULL << 32)) return NULL;
    ora_state* s = (ora_state*)calloc(1, sizeof(ora_state));
    s->d = d; s->n = n; s->r = r; s->c = c; s->k = k; s->seed = seed; s->log2g = log2g;
    s->lr = lr; s->lr_prev = lr; s->beta1 = beta1; s->beta2 = beta2; s->eps = eps;
    s->threads = 1;
    s->P = 1;
    s->m = (float*)calloc((size_t)n * d, sizeof(float));        /* m_0 = 0 */
    s->e = (float*)calloc((size_t)n * d, sizeof(float));        /* e_0 = 0 */
    s->v = (float*)malloc((size_t)d * sizeof(float));
    s->vhat = (float*)malloc((size_t)d * sizeof(float));
    for (uint64_t j = 0; j < d; ++j) s->v[j] = s->vhat[j] = eps; /* v_0 = vhat_0 = eps */
    s->est = (float*)calloc((size_t)d, sizeof(float));
    s->tables = (float*)calloc((size_t)n * r * c, sizeof(float));
    s->sum = (float*)calloc((size_t)r * c, sizeof(float));
    s->I = (uint32_t*)calloc((size_t)k, sizeof(uint32_t));
    s->I_prev = (uint32_t*)calloc((size_t)k, sizeof(uint32_t));
    s->k_prev = 0;                                               /* I_0 = empty set */
    s->mask = (uint8_t*)calloc((size_t)d, 1);
    s->row_key = (uint64_t*)malloc((size_t)r * sizeof(uint64_t));
    for (uint32_t j = 0; j < r; ++j) s->row_key[j] = ora_row_key(seed, j);
    return s;
}

void ora_destroy(ora_state* s) {
    if (!s) return;
    free(s->m); free(s->e); free(s->v); free(s->vhat); free(s->est); free(s->tables); free(s->sum);
    free(s->I); free(s->I_prev); free(s->mask); free(s->row_key); free(s->vw); free(s->vhatw); free(s->cand); free(s);
}

void ora_set_hash(ora_state* s, const uint32_t* idx, const int8_t* sgn) { s->h_idx = idx; s->h_sgn = sgn; }

/* alpha_t of the steps taken from now on; the step computes alpha_{t-1}/alpha_t from the last step's value */
void ora_set_lr(ora_state* s, float lr) { s->lr = lr; }

void ora_set_option(ora_state* s, const char* key, int value) {
    if (!strcmp(key, "v_keep")) s->v_keep = value;
    else if (!strcmp(key, "freeze_v")) s->freeze_v = value;
    else if (!strcmp(key, "window_lines")) {
        /* only with g = 32 and at least one whole window in a row; otherwise left unchanged */
        if (value >= 0 && (value == 0 || (s->log2g == 5 && (uint64_t)32 * (uint64_t)value <= s->c)))
            s->window_lines = (uint32_t)value;
    }
    else if (!strcmp(key, "threads")) s->threads = value > 0 ? value : 1;
    else if (!strcmp(key, "P")) {
        if (value >= 1 && (uint64_t)value * s->k <= s->d && s->t == 0) {
            s->P = (uint32_t)value;
            free(s->cand);
            s->cand = (uint32_t*)calloc((size_t)s->P * s->k, sizeof(uint32_t));
        }
    }
    else if (!strcmp(key, "variant_pa")) {
        /* Algorithm 1 (parameter averaging); only before the first step.  v_0^(i) = vhat_0^(i) = eps. */
        if (value && !s->vw && s->t == 0) {
            size_t nd = (size_t)s->n * s->d;
            s->vw = (float*)malloc(nd * sizeof(float));
            s->vhatw = (float*)malloc(nd * sizeof(float));
            for (size_t q = 0; q < nd; ++q) s->vw[q] = s->vhatw[q] = s->eps;
        }
        if (s->t == 0) s->variant_pa = value ? 1 : 0;
    }
}

void* ora_field(ora_state* s, const char* name) {
    if (!strcmp(name, "m")) return s->m;
    if (!strcmp(name, "e")) return s->e;
    if (!strcmp(name, "v")) return s->v;
    if (!strcmp(name, "vhat")) return s->vhat;
    if (!strcmp(name, "est")) return s->est;
    if (!strcmp(name, "tables")) return s->tables;
    if (!strcmp(name, "sum")) return s->sum;
    if (!strcmp(name, "I")) return s->I;
    if (!strcmp(name, "I_prev")) return s->I_prev;
    if (!strcmp(name, "cand")) return s->cand;
    if (!strcmp(name, "vw")) return s->vw;
    if (!strcmp(name, "vhatw")) return s->vhatw;
    return NULL;
}

uint64_t ora_count(ora_state* s, const char* name) {
    if (!strcmp(name, "I_prev")) return s->k_prev;
    if (!strcmp(name, "I")) return s->t ? s->k : 0;
    if (!strcmp(name, "t")) return s->t;
    if (!strcmp(name, "cand")) return (s->t && s->P > 1) ? (uint64_t)s->P * s->k : 0;
    return 0;
}

/* bucket and sign of coordinate i in row j: injected arrays if present, else the seeded family */
static inline void hash_at(const ora_state* s, uint32_t j, uint64_t i, uint32_t* b, int8_t* sg) {
    if (s->h_idx) { *b = s->h_idx[j * s->d + i]; *sg = s->h_sgn[j * s->d + i]; return; }
    uint64_t g = 1ULL << s->log2g, G = s->c / g;
    uint64_t q = i >> s->log2g, o = i & (g - 1);
    uint64_t u = ora_stream(s->row_key[j], q + 1);
    uint64_t base = 0;
    if (s->window_lines) {                 /* windowed family: the unit's panel fixes the window, L lines to choose from */
        uint64_t cw = g * s->window_lines;
        base = ((i / 1024) % (s->c / cw)) * cw;
        G = s->window_lines;
    }
    uint64_t x = (u >> 32) * G;
    uint64_t p = s->log2g ? ((x & 0xFFFFFFFFULL) >> (32 - s->log2g)) : 0;
    *b = (uint32_t)(base + g * (x >> 32) + (o ^ p));
    *sg = (u & 1ULL) ? -1 : 1;             /* one sign per (row, group) */
}

static int ora_step_pa(ora_state* s, const float* grads, float* x);

/* Second round of Section III-A: of the estimates take the P*k largest as candidates, fetch the
 * EXACT values of the compressed vector there -- `exact[j]` is computed by the caller for the candidates only --
 * and keep the k candidates of largest exact magnitude (ties: smaller index).  With P = 1 this is plain Top-k of
 * the estimates.  `scale` is vhat for Algorithm 2 (exact value = mean_w a / sqrt(vhat)) or NULL for Algorithm 1. */
static void select_with_second_round(ora_state* s, const float* scale) {
    const uint64_t d = s->d, k = s->k;
    if (s->P <= 1) { ora_topk(s->est, d, k, s->I); return; }
    const uint64_t pk = (uint64_t)s->P * k;
    ora_topk(s->est, d, pk, s->cand);
    float* exact = (float*)calloc((size_t)d, sizeof(float));       /* zero off the candidate set */
    for (uint64_t t = 0; t < pk; ++t) {
        uint64_t j = s->cand[t];
        double abar = 0.0;
        for (uint32_t w = 0; w < s->n; ++w) abar += (double)s->e[(uint64_t)w * d + j];
        abar /= (double)s->n;
        exact[j] = (float)(scale ? abar / sqrt((double)scale[j]) : abar);
    }
    /* top-k of the exact magnitudes among the candidates: every non-candidate holds 0 and, to keep a zero-valued
       candidate ahead of non-candidates, the selection runs over the candidate list itself */
    float* cval = (float*)malloc((size_t)pk * sizeof(float));
    uint32_t* pos = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
    for (uint64_t t = 0; t < pk; ++t) cval[t] = exact[s->cand[t]];
    ora_topk(cval, pk, k, pos);            /* cand is ascending, so "smaller position" = "smaller index" */
    for (uint64_t t = 0; t < k; ++t) s->I[t] = s->cand[pos[t]];
    free(pos); free(cval); free(exact);
}

int ora_step(ora_state* s, const float* grads, float* x) {
    if (s->variant_pa) return ora_step_pa(s, grads, x);
    const uint64_t d = s->d, k = s->k;
    const uint32_t n = s->n, r = s->r, c = s->c;
    const double b1 = (double)s->beta1, b2 = (double)s->beta2, lr = (double)s->lr;
    const double rho = (double)s->lr_prev / (double)s->lr;   /* alpha_{t-1}/alpha_t (Algorithm 2's sketch line) */
#ifdef _OPENMP
    omp_set_num_threads(s->threads);
#endif

    /* Algorithm 2, worker side: m_t = beta1 m_{t-1} + (1-beta1) g_t */
#pragma omp parallel for schedule(static)
    for (uint64_t q = 0; q < (uint64_t)n * d; ++q)
        s->m[q] = (float)(b1 * (double)s->m[q] + (1.0 - b1) * (double)grads[q]);

    /* h_t = mean_w (g_t^(w)) restricted to I_{t-1} (zero elsewhere);
       v_t = beta2 v_{t-1} + (1-beta2) h_t^2 ; vhat_t = max(vhat_{t-1}, v_t)   (master side) */
    memset(s->mask, 0, (size_t)d);
    for (uint64_t t = 0; t < s->k_prev; ++t) s->mask[s->I_prev[t]] = 1;
    /* freeze_v: h_t is not sent and v, vhat keep their initial values (the fixed-variance scheme the paper
       compares with, Section III-B) */
#pragma omp parallel for schedule(static)
    for (uint64_t j = 0; j < (s->freeze_v ? 0 : d); ++j) {
        double h = 0.0;
        if (s->mask[j]) {
            for (uint32_t w = 0; w < n; ++w) h += (double)grads[(uint64_t)w * d + j];
            h /= (double)n;
        }
        if (s->mask[j] || !s->v_keep) s->v[j] = (float)(b2 * (double)s->v[j] + (1.0 - b2) * h * h);
        if (s->v[j] > s->vhat[j]) s->vhat[j] = s->v[j];
    }

    /* a_t^(w) = m_t^(w) + rho e_{t-1}^(w): the vector each worker sketches; kept in the e buffer */
#pragma omp parallel for schedule(static)
    for (uint64_t q = 0; q < (uint64_t)n * d; ++q)
        s->e[q] = (float)((double)s->m[q] + rho * (double)s->e[q]);

    /* S_t^(w) = S(a_t^(w)): one r x c table per worker, fp64 accumulation in increasing coordinate */
#pragma omp parallel
    {
        double* acc = (double*)malloc((size_t)c * sizeof(double));
#pragma omp for schedule(dynamic, 1)
        for (uint64_t wj = 0; wj < (uint64_t)n * r; ++wj) {
            uint32_t w = (uint32_t)(wj / r), j = (uint32_t)(wj % r);
            const float* a = s->e + (uint64_t)w * d;
            memset(acc, 0, (size_t)c * sizeof(double));
            for (uint64_t i = 0; i < d; ++i) {
                uint32_t b; int8_t sg;
                hash_at(s, j, i, &b, &sg);
                acc[b] += (double)sg * (double)a[i];
            }
            float* row = s->tables + ((uint64_t)w * r + j) * c;
            for (uint32_t b = 0; b < c; ++b) row[b] = (float)acc[b];
        }
        free(acc);
    }

    /* S_t = (1/n) sum_w S_t^(w), workers added in the order 0,1,...,n-1 */
#pragma omp parallel for schedule(static)
    for (uint64_t q = 0; q < (uint64_t)r * c; ++q) {
        double acc = 0.0;
        for (uint32_t w = 0; w < n; ++w) acc += (double)s->tables[(uint64_t)w * r * c + q];
        s->sum[q] = (float)(acc / (double)n);
    }

    /* U(S_t, vhat_t): est_i = median_j( s_j(i) S_t[j,h_j(i)] ) / sqrt(vhat_t,i) */
#pragma omp parallel for schedule(static)
    for (uint64_t i = 0; i < d; ++i) {
        float q[64];
        for (uint32_t j = 0; j < r; ++j) {
            uint32_t b; int8_t sg;
            hash_at(s, j, i, &b, &sg);
            q[j] = (float)sg * s->sum[(uint64_t)j * c + b];
        }
        s->est[i] = (float)((double)ora_median(q, r) / sqrt((double)s->vhat[i]));
    }

    /* I_t = index set of Top-k of the estimates (after the second round on P*k candidates when P > 1) */
    select_with_second_round(s, s->vhat);

    /* Delta_t = (1/n) sum_w Delta_t^(w): exact coordinates of vhat^{-1/2} a_t^(w) on I_t;
       x_{t+1} = x_t - alpha_t Delta_t ;  e_t^(w) = a_t^(w) with the coordinates of I_t removed */
    for (uint64_t t = 0; t < k; ++t) {
        uint64_t j = s->I[t];
        double abar = 0.0;
        for (uint32_t w = 0; w < n; ++w) abar += (double)s->e[(uint64_t)w * d + j];
        abar /= (double)n;
        double delta = abar / sqrt((double)s->vhat[j]);
        x[j] = (float)((double)x[j] - lr * delta);
        for (uint32_t w = 0; w < n; ++w) s->e[(uint64_t)w * d + j] = 0.0f;
    }

    memcpy(s->I_prev, s->I, (size_t)k * sizeof(uint32_t));
    s->k_prev = k;
    s->lr_prev = s->lr;
    s->t += 1;
    return 0;
}

/* ------------------------------------------------------------------------------------------------
 * SketchedAMSGrad with PARAMETER averaging (Algorithm 1).  Every worker runs its own AMSGrad moments:
 *   m = beta1 m + (1-beta1) g ;  v = beta2 v + (1-beta2) g^2 ;  vhat = max(vhat, v)        (per worker)
 *   a = m / sqrt(vhat) + rho e            the vector the worker sketches (kept in the e buffer)
 *   S = (1/n) sum_w S(a^(w)) ;  Delta = Top-k(U(S)) with the plain unsketch (no vhat argument)
 *   Delta takes the exact worker means of a on I_t (Section III-A) ;  x -= alpha Delta
 *   e = a with the coordinates of I_t removed
 * est, sum, tables, I are stored in the same fields as for Algorithm 2.
 * ------------------------------------------------------------------------------------------------ */
static int ora_step_pa(ora_state* s, const float* grads, float* x) {
    const uint64_t d = s->d, k = s->k;
    const uint32_t n = s->n, r = s->r, c = s->c;
    const double b1 = (double)s->beta1, b2 = (double)s->beta2, lr = (double)s->lr;
    const double rho = (double)s->lr_prev / (double)s->lr;   /* alpha_{t-1}/alpha_t (Algorithm 1's sketch line) */
#ifdef _OPENMP
    omp_set_num_threads(s->threads);
#endif
#pragma omp parallel for schedule(static)
    for (uint64_t q = 0; q < (uint64_t)n * d; ++q) {
        const double g = (double)grads[q];
        s->m[q] = (float)(b1 * (double)s->m[q] + (1.0 - b1) * g);
        s->vw[q] = (float)(b2 * (double)s->vw[q] + (1.0 - b2) * g * g);
        if (s->vw[q] > s->vhatw[q]) s->vhatw[q] = s->vw[q];
        s->e[q] = (float)((double)s->m[q] / sqrt((double)s->vhatw[q]) + rho * (double)s->e[q]);
    }
#pragma omp parallel
    {
        double* acc = (double*)malloc((size_t)c * sizeof(double));
#pragma omp for schedule(dynamic, 1)
        for (uint64_t wj = 0; wj < (uint64_t)n * r; ++wj) {
            uint32_t w = (uint32_t)(wj / r), j = (uint32_t)(wj % r);
            const float* a = s->e + (uint64_t)w * d;
            memset(acc, 0, (size_t)c * sizeof(double));
            for (uint64_t i = 0; i < d; ++i) {
                uint32_t b; int8_t sg;
                hash_at(s, j, i, &b, &sg);
                acc[b] += (double)sg * (double)a[i];
            }
            float* row = s->tables + ((uint64_t)w * r + j) * c;
            for (uint32_t b = 0; b < c; ++b) row[b] = (float)acc[b];
        }
        free(acc);
    }
#pragma omp parallel for schedule(static)
    for (uint64_t q = 0; q < (uint64_t)r * c; ++q) {
        double acc = 0.0;
        for (uint32_t w = 0; w < n; ++w) acc += (double)s->tables[(uint64_t)w * r * c + q];
        s->sum[q] = (float)(acc / (double)n);
    }
#pragma omp parallel for schedule(static)
    for (uint64_t i = 0; i < d; ++i) {
        float q[64];
        for (uint32_t j = 0; j < r; ++j) {
            uint32_t b; int8_t sg;
            hash_at(s, j, i, &b, &sg);
            q[j] = (float)sg * s->sum[(uint64_t)j * c + b];
        }
        s->est[i] = ora_median(q, r);
    }
    select_with_second_round(s, NULL);
    for (uint64_t t = 0; t < k; ++t) {
        uint64_t j = s->I[t];
        double abar = 0.0;
        for (uint32_t w = 0; w < n; ++w) abar += (double)s->e[(uint64_t)w * d + j];
        abar /= (double)n;
        x[j] = (float)((double)x[j] - lr * abar);
        for (uint32_t w = 0; w < n; ++w) s->e[(uint64_t)w * d + j] = 0.0f;
    }
    memcpy(s->I_prev, s->I, (size_t)k * sizeof(uint32_t));
    s->k_prev = k;
    s->lr_prev = s->lr;
    s->t += 1;
    return 0;
}
