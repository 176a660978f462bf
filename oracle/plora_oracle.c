/*
 * CPU oracle for the batched heterogeneous-adapter LoRA delta.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what
 * the GPU library must compute.  It shares no code, header, table or helper
 * with the CUDA path and must never be reached from it; only the tests, the
 * smoke check and the benchmark's CPU-baseline leg call it.
 *
 * What it follows (paper sections):
 *   - Section II-A: a LoRA adapter is a pair A in R^{D1 x R}, B in R^{R x D2}
 *     and the adapted layer computes y = x (W + A B); the delta is x A B.
 *   - Section III-A: the adapter computation is Y = X A B.
 *   - Section V-A: strategy E1 computes y from A and B held in GPU memory;
 *     strategy E4 names the two halves, shrink m = x A and expand y = m B.
 *   - Section VI-B: a step serves requests tagged by adapter id; B_i is the
 *     number of requests of adapter i; values are 2 bytes wide.
 * Readings the paper leaves open: a per-adapter fp32 scale s_a multiplies the
 * delta; a token with id -1 has no adapter and keeps its row of y; the delta is
 * added to the caller's y (the base projection output); an id outside
 * [-1, N) is an error.
 *
 * All arithmetic is float64.  Inputs are the raw 16-bit patterns the GPU gets,
 * bf16 or IEEE half (widening either to double is exact).  Nothing is blocked, fused or reordered: the
 * loops are the definition written out.  Pins: tests/test_oracle_*.py.
 */
#include <stdint.h>
#include <stdlib.h>
#include <math.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_INVALID_ARG (-1)
#define ORACLE_ERR_BAD_ADAPTER_ID (-3)

static double bf16_bits_to_double(uint16_t bits)
{
    uint32_t u = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* IEEE half (the paper's FP16, Section VI-B: S = 2 bytes per value): 1 sign, 5 exponent, 10 fraction bits. */
static double fp16_bits_to_double(uint16_t bits)
{
    const int sign = bits >> 15, e = (bits >> 10) & 31, f = bits & 1023;
    double v;
    if (e == 0)
        v = ldexp((double)f, -24);                 /* zero and subnormals: f * 2^-24 */
    else if (e == 31)
        v = f ? NAN : INFINITY;
    else
        v = ldexp(1.0 + (double)f / 1024.0, e - 15);
    return sign ? -v : v;
}

/* Which 16-bit type x, A and B hold: 0 = bf16 (default), 1 = IEEE half.  Set by the caller
 * before a call; the conversion to double is exact for both. */
static int g_input_is_fp16 = 0;
void plora_oracle_set_input_type(int is_fp16) { g_input_is_fp16 = is_fp16 != 0; }
double plora_oracle_input_to_double(uint16_t bits)
{
    return g_input_is_fp16 ? fp16_bits_to_double(bits) : bf16_bits_to_double(bits);
}

static double bf16_to_double(uint16_t bits) { return plora_oracle_input_to_double(bits); }

/* ---------------------------------------------------------------------- */
/* Bucketing: tokens stably sorted by adapter id, plus the segment list.   */
/* Section VI-B: the per-adapter request count B_i is the segment length.  */
/* ---------------------------------------------------------------------- */

typedef struct {
    int32_t key;
    int32_t tok;
} key_tok;

static int cmp_key_tok(const void *pa, const void *pb)
{
    const key_tok *a = (const key_tok *)pa, *b = (const key_tok *)pb;
    if (a->key != b->key)
        return a->key < b->key ? -1 : 1;
    if (a->tok != b->tok)
        return a->tok < b->tok ? -1 : 1;
    return 0;
}

/*
 * ids[T] in [-1, N).  -1 means "no adapter".
 * perm[T]            token indices ordered by (key, token) with key = id, or N for id -1
 * seg_adapter[cap]   ascending distinct ids >= 0 that occur; unused tail = -1
 * seg_start[cap+1]   first position in perm of each segment; entry n_seg and the tail = n_active
 * cap = min(T, N).   n_active = number of tokens with id >= 0.
 */
int plora_oracle_bucket(const int32_t *ids, int32_t T, int32_t N, int32_t *perm, int32_t *seg_adapter,
                        int32_t *seg_start, int32_t *n_seg_out, int32_t *n_active_out)
{
    if (T < 0 || N < 1 || (T > 0 && !ids))
        return ORACLE_ERR_INVALID_ARG;
    for (int32_t t = 0; t < T; ++t)
        if (ids[t] < -1 || ids[t] >= N)
            return ORACLE_ERR_BAD_ADAPTER_ID;

    int32_t cap = T < N ? T : N;
    key_tok *kt = (key_tok *)malloc(sizeof(key_tok) * (size_t)(T > 0 ? T : 1));
    if (!kt)
        return ORACLE_ERR_INVALID_ARG;
    int32_t n_active = 0;
    for (int32_t t = 0; t < T; ++t) {
        kt[t].key = ids[t] == -1 ? N : ids[t];
        kt[t].tok = t;
        if (ids[t] >= 0)
            ++n_active;
    }
    /* the comparator is a total order (token index breaks ties), so the result is unique */
    qsort(kt, (size_t)T, sizeof(key_tok), cmp_key_tok);
    for (int32_t p = 0; p < T; ++p)
        perm[p] = kt[p].tok;

    int32_t n_seg = 0;
    for (int32_t p = 0; p < n_active; ++p) {
        if (p == 0 || kt[p].key != kt[p - 1].key) {
            seg_adapter[n_seg] = kt[p].key;
            seg_start[n_seg] = p;
            ++n_seg;
        }
    }
    for (int32_t k = n_seg; k < cap; ++k)
        seg_adapter[k] = -1;
    for (int32_t k = n_seg; k <= cap; ++k)
        seg_start[k] = n_active;
    *n_seg_out = n_seg;
    *n_active_out = n_active;
    free(kt);
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------- */
/* Shrink (Section V-A, E4): m_t = x_t A[a_t], float64, unrounded.         */
/*   x     bf16 bits [T, d_in] row-major                                   */
/*   A[a]  bf16 bits [d_in, ranks[a]] row-major                            */
/*   m     double [T, ldm]; columns >= rank of the token's adapter, and    */
/*         whole rows of tokens with id -1, are set to 0                   */
/* ---------------------------------------------------------------------- */
int plora_oracle_shrink(const uint16_t *x, const int32_t *ids, int32_t T, int32_t d_in, int32_t N,
                        const int32_t *ranks, const uint16_t *const *A, double *m, int32_t ldm)
{
    if (T < 0 || d_in < 1 || N < 1 || ldm < 1)
        return ORACLE_ERR_INVALID_ARG;
    for (int32_t t = 0; t < T; ++t) {
        if (ids[t] < -1 || ids[t] >= N)
            return ORACLE_ERR_BAD_ADAPTER_ID;
        if (ids[t] >= 0 && ranks[ids[t]] > ldm)
            return ORACLE_ERR_INVALID_ARG;
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t t = 0; t < T; ++t) {
        double *mt = m + (size_t)t * ldm;
        for (int32_t k = 0; k < ldm; ++k)
            mt[k] = 0.0;
        int32_t a = ids[t];
        if (a == -1)
            continue;
        int32_t r = ranks[a];
        const uint16_t *Aa = A[a];
        const uint16_t *xt = x + (size_t)t * d_in;
        for (int32_t k = 0; k < r; ++k) {
            double acc = 0.0;
            for (int32_t i = 0; i < d_in; ++i)
                acc += bf16_to_double(xt[i]) * bf16_to_double(Aa[(size_t)i * r + k]);
            mt[k] = acc;
        }
    }
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------- */
/* Expand (Section V-A, E4): y_t = y_in_t + s_a * (m_t B[a_t]).            */
/*   m     double [T, ldm]                                                 */
/*   B[a]  bf16 bits [ranks[a], d_out] row-major                           */
/*   y_in  fp32 [T, d_out] or NULL (= 0);  y_out double [T, d_out]         */
/* ---------------------------------------------------------------------- */
int plora_oracle_expand(const double *m, int32_t ldm, const int32_t *ids, int32_t T, int32_t d_out, int32_t N,
                        const int32_t *ranks, const float *scales, const uint16_t *const *B,
                        const float *y_in, double *y_out)
{
    if (T < 0 || d_out < 1 || N < 1 || ldm < 1)
        return ORACLE_ERR_INVALID_ARG;
    for (int32_t t = 0; t < T; ++t) {
        if (ids[t] < -1 || ids[t] >= N)
            return ORACLE_ERR_BAD_ADAPTER_ID;
        if (ids[t] >= 0 && ranks[ids[t]] > ldm)
            return ORACLE_ERR_INVALID_ARG;
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t t = 0; t < T; ++t) {
        double *yo = y_out + (size_t)t * d_out;
        const float *yi = y_in ? y_in + (size_t)t * d_out : NULL;
        int32_t a = ids[t];
        if (a == -1) {
            for (int32_t j = 0; j < d_out; ++j)
                yo[j] = yi ? (double)yi[j] : 0.0;
            continue;
        }
        int32_t r = ranks[a];
        double s = (double)scales[a];
        const uint16_t *Ba = B[a];
        const double *mt = m + (size_t)t * ldm;
        for (int32_t j = 0; j < d_out; ++j) {
            double acc = 0.0;
            for (int32_t k = 0; k < r; ++k)
                acc += mt[k] * bf16_to_double(Ba[(size_t)k * d_out + j]);
            yo[j] = (yi ? (double)yi[j] : 0.0) + s * acc;
        }
    }
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------- */
/* The whole delta (Section II-A / V-A E1):                                */
/*   y_out_t = y_in_t + s_a * ((x_t A_a) B_a),  a = ids[t];  id -1: y_in   */
/* ---------------------------------------------------------------------- */
int plora_oracle_lora_delta(const uint16_t *x, const int32_t *ids, int32_t T, int32_t d_in, int32_t d_out,
                            int32_t N, const int32_t *ranks, const float *scales, const uint16_t *const *A,
                            const uint16_t *const *B, const float *y_in, double *y_out)
{
    if (T < 0 || d_in < 1 || d_out < 1 || N < 1)
        return ORACLE_ERR_INVALID_ARG;
    for (int32_t t = 0; t < T; ++t)
        if (ids[t] < -1 || ids[t] >= N)
            return ORACLE_ERR_BAD_ADAPTER_ID;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t t = 0; t < T; ++t) {
        double *yo = y_out + (size_t)t * d_out;
        const float *yi = y_in ? y_in + (size_t)t * d_out : NULL;
        int32_t a = ids[t];
        if (a == -1) {
            for (int32_t j = 0; j < d_out; ++j)
                yo[j] = yi ? (double)yi[j] : 0.0;
            continue;
        }
        int32_t r = ranks[a];
        double s = (double)scales[a];
        const uint16_t *Aa = A[a], *Ba = B[a];
        const uint16_t *xt = x + (size_t)t * d_in;
        double m[1024];
        double *mp = r <= 1024 ? m : (double *)malloc(sizeof(double) * (size_t)r);
        for (int32_t k = 0; k < r; ++k) {
            double acc = 0.0;
            for (int32_t i = 0; i < d_in; ++i)
                acc += bf16_to_double(xt[i]) * bf16_to_double(Aa[(size_t)i * r + k]);
            mp[k] = acc;
        }
        for (int32_t j = 0; j < d_out; ++j) {
            double acc = 0.0;
            for (int32_t k = 0; k < r; ++k)
                acc += mp[k] * bf16_to_double(Ba[(size_t)k * d_out + j]);
            yo[j] = (yi ? (double)yi[j] : 0.0) + s * acc;
        }
        if (mp != m)
            free(mp);
    }
    return ORACLE_OK;
}

/* Number of OpenMP threads a parallel region will use (reported by the benchmark). */
#ifdef _OPENMP
#include <omp.h>
int plora_oracle_threads(void) { return omp_get_max_threads(); }
#else
int plora_oracle_threads(void) { return 1; }
#endif
