/*
 * dq_oracle.c -- plain CPU oracle of the DQ-SGD quantizer hot path.
 * TEST INFRASTRUCTURE ONLY; see dq_oracle.h.  Build with
 *   gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC
 * (-ffp-contract=off -frounding-math: every fp32 operation below rounds on its
 * own, in the order written and in the rounding mode set around it; both are
 * part of the definition of the codes).
 */
#include "dq_oracle.h"

#include <fenv.h>
#include <math.h>
#include <stdlib.h>
#include <string.h>

static int32_t g_threads = 1;

void oracle_set_threads(int32_t n) { g_threads = n < 1 ? 1 : n; }
int32_t oracle_get_threads(void) { return g_threads; }

static int64_t roundup32(int64_t n) { return (n + 31) / 32 * 32; }

/* ------------------------------------------------------------------ layout */

int64_t oracle_padded_elems(const int64_t* seg_elems, int32_t n_seg)
{
    int64_t total = 0;
    for (int32_t i = 0; i < n_seg; ++i) total += roundup32(seg_elems[i]);
    return total;
}

int64_t oracle_num_buckets(const int64_t* seg_elems, int32_t n_seg, int32_t bucket)
{
    int64_t nb = 0;
    for (int32_t i = 0; i < n_seg; ++i) nb += (seg_elems[i] + bucket - 1) / bucket;
    return nb;
}

void oracle_seg_offsets(const int64_t* seg_elems, int32_t n_seg, int64_t* offsets)
{
    int64_t p = 0;
    for (int32_t i = 0; i < n_seg; ++i) {
        offsets[i] = p;
        p += roundup32(seg_elems[i]);
    }
}

void oracle_bucket_table(const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                         int64_t* start, int64_t* len)
{
    int64_t p = 0, k = 0;
    for (int32_t i = 0; i < n_seg; ++i) {
        const int64_t n = seg_elems[i];
        for (int64_t o = 0; o < n; o += bucket) {
            start[k] = p + o;
            len[k] = (n - o < bucket) ? (n - o) : bucket;
            ++k;
        }
        p += roundup32(n);
    }
}

/* the table is small; build it once per call */
typedef struct { int64_t nb; int64_t* start; int64_t* len; } table_t;

static table_t make_table(const int64_t* seg_elems, int32_t n_seg, int32_t bucket)
{
    table_t t;
    t.nb = oracle_num_buckets(seg_elems, n_seg, bucket);
    t.start = (int64_t*)malloc(sizeof(int64_t) * (size_t)(t.nb > 0 ? t.nb : 1));
    t.len = (int64_t*)malloc(sizeof(int64_t) * (size_t)(t.nb > 0 ? t.nb : 1));
    oracle_bucket_table(seg_elems, n_seg, bucket, t.start, t.len);
    return t;
}

static void free_table(table_t* t) { free(t->start); free(t->len); }

/* ------------------------------------------------------------------- norms */

void oracle_bucket_norms(const float* grads, int64_t worker_stride, int32_t M,
                         const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                         float* norms)
{
    table_t tb = make_table(seg_elems, n_seg, bucket);
    const int64_t total = (int64_t)M * tb.nb;
#pragma omp parallel for schedule(static) num_threads(g_threads) if (g_threads > 1)
    for (int64_t w = 0; w < total; ++w) {
        const int64_t m = w / tb.nb, k = w % tb.nb;
        const float* g = grads + m * worker_stride + tb.start[k];
        double ss = 0.0;
        for (int64_t j = 0; j < tb.len[k]; ++j) ss += (double)g[j] * (double)g[j];
        norms[w] = (float)sqrt(ss);
    }
    free_table(&tb);
}

/* The l_infinity member of the family ||g||_p of Eq. 5: the largest magnitude of the
 * bucket (exact in fp32).  p_kind 2 is the l_2 norm above, p_kind 0 stands for p = infinity. */
void oracle_bucket_norms_p(const float* grads, int64_t worker_stride, int32_t M,
                           const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                           int32_t p_kind, float* norms)
{
    if (p_kind == 2) {
        oracle_bucket_norms(grads, worker_stride, M, seg_elems, n_seg, bucket, norms);
        return;
    }
    table_t tb = make_table(seg_elems, n_seg, bucket);
    const int64_t total = (int64_t)M * tb.nb;
#pragma omp parallel for schedule(static) num_threads(g_threads) if (g_threads > 1)
    for (int64_t w = 0; w < total; ++w) {
        const int64_t m = w / tb.nb, k = w % tb.nb;
        const float* g = grads + m * worker_stride + tb.start[k];
        float big = 0.0f;
        for (int64_t j = 0; j < tb.len[k]; ++j) {
            const float a = fabsf(g[j]);
            if (a > big || a != a) big = a;          /* a NaN entry makes the norm NaN */
            if (big != big) break;
        }
        norms[w] = big;
    }
    free_table(&tb);
}

/* ---------------------------------------------------------------- bit rule */

int32_t oracle_choose_bits(const float* norms, int64_t nb, int32_t M,
                           int32_t T, int32_t t, double eps_hat, double alpha,
                           int32_t b_min, int32_t b_max, int32_t fixed_b,
                           int32_t* s_out, double* x_out)
{
    /* G-bar^2 = (1/W) sum_i ||g^(i)||^2 ; with p = 2 the squared norm of a
     * worker's vector is the sum of its squared bucket norms. */
    double sum = 0.0;
    for (int64_t i = 0; i < (int64_t)M * nb; ++i) sum += (double)norms[i] * (double)norms[i];
    const double G2 = sum / (double)M;
    /* Eq. 17: b = log2(x + 1) + 1 with x as below */
    const double x = sqrt((double)T / eps_hat) * pow(alpha, (double)(T - 1 - t) / 2.0) * sqrt(G2);
    if (x_out) *x_out = x;
    int32_t b;
    if (fixed_b != 0) {
        b = fixed_b;
    } else {
        /* smallest integer b in [b_min, b_max] with 2^(b-1) - 1 >= x,
         * i.e. ceil(log2(x + 1)) + 1 without a transcendental */
        b = b_max;
        for (int32_t c = b_min; c <= b_max; ++c) {
            if ((double)((1 << (c - 1)) - 1) >= x) { b = c; break; }
        }
    }
    if (s_out) *s_out = (1 << (b - 1)) - 1;
    return b;
}

/* ------------------------------------------------------------------ Philox */

static void mulhilo(uint32_t a, uint32_t b, uint32_t* hi, uint32_t* lo)
{
    const uint64_t p = (uint64_t)a * (uint64_t)b;
    *hi = (uint32_t)(p >> 32);
    *lo = (uint32_t)p;
}

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0, lo0, hi1, lo1;
        mulhilo(0xD2511F53u, c0, &hi0, &lo0);
        mulhilo(0xCD9E8D57u, c2, &hi1, &lo1);
        const uint32_t n0 = hi1 ^ c1 ^ k0;
        const uint32_t n1 = lo1;
        const uint32_t n2 = hi0 ^ c3 ^ k1;
        const uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;   /* golden-ratio Weyl increments of the key */
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Rounding uniform of padded element j of worker m at a step: Philox block
 * with counter (j >> 3, 0, m, step) and key (seed lo, seed hi); element j owns
 * half (j & 1) (0 = low 16 bits) of word ((j >> 1) & 3).  With k that 16-bit
 * value, v = (2k + 1) / 2^17: a midpoint grid on (0, 1), never 0 and never 1. */
static float uniform16(uint64_t seed, uint32_t step, uint32_t m, int64_t j)
{
    const uint64_t q = (uint64_t)j >> 3;
    const uint32_t ctr[4] = { (uint32_t)q, (uint32_t)(q >> 32), m, step };
    const uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t r[4];
    oracle_philox4x32_10(ctr, key, r);
    const uint32_t word = r[(j >> 1) & 3];
    const uint32_t k = (j & 1) ? (word >> 16) : (word & 0xFFFFu);
    return (float)(2u * k + 1u) * 0x1p-17f;            /* exact in fp32 */
}

/* ---------------------------------------------------------------- quantize */

/* Norms below this are treated as zero: s / norm would overflow fp32. */
#define ORACLE_TINY_NORM 0x1p-100f

void oracle_quantize(const float* grads, int64_t worker_stride, int32_t M,
                     const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                     const float* norms, int32_t b, uint64_t seed, uint32_t step,
                     uint32_t* codes, float* x_out, float* v_out)
{
    table_t tb = make_table(seg_elems, n_seg, bucket);
    const int64_t D32 = oracle_padded_elems(seg_elems, n_seg);
    const int32_t s = (1 << (b - 1)) - 1;
    const float sf = (float)s;

    /* pads: value 0, i.e. code s */
    for (int64_t i = 0; i < (int64_t)M * D32; ++i) codes[i] = (uint32_t)s;
    if (x_out) memset(x_out, 0, sizeof(float) * (size_t)((int64_t)M * D32));
    if (v_out) memset(v_out, 0, sizeof(float) * (size_t)((int64_t)M * D32));

    const int64_t total = (int64_t)M * tb.nb;
#pragma omp parallel for schedule(static) num_threads(g_threads) if (g_threads > 1)
    for (int64_t w = 0; w < total; ++w) {
        const int64_t m = w / tb.nb, k = w % tb.nb;
        const float norm = norms[w];
        /* s / norm and g * inv are both rounded toward zero: then |x| <= s for every
         * element with |g| <= norm (the norm of a bucket dominates its entries), so the
         * code stays in 0 .. 2s without a clamp, and inputs on a level stay exact. */
        float* xs = (float*)malloc(sizeof(float) * (size_t)(tb.len[k] > 0 ? tb.len[k] : 1));
        fesetround(FE_TOWARDZERO);
        {
            const volatile float inv = (norm >= ORACLE_TINY_NORM) ? sf / norm : 0.0f;
            for (int64_t e = 0; e < tb.len[k]; ++e) {
                const volatile float g = grads[m * worker_stride + tb.start[k] + e];
                xs[e] = g * inv;             /* s * g_j / ||g||: signed position on the level grid (Eq. 6) */
            }
        }
        fesetround(FE_TONEAREST);
        for (int64_t e = 0; e < tb.len[k]; ++e) {
            const int64_t j = tb.start[k] + e;
            const float x = xs[e];
            const float v = uniform16(seed, step, (uint32_t)m, j);
            /* Eq. 6 on the signed grid: floor(x + v) is the neighbour of x away
             * from zero with probability p_r = frac(|x|) and the one toward zero
             * otherwise.  x + v is exact in fp64 (x has 24 bits below 2^15, v 17 bits). */
            const double q = floor((double)x + (double)v);
            codes[m * D32 + j] = (uint32_t)((int32_t)q + s);      /* excess-s code, 0 .. 2s */
            if (x_out) x_out[m * D32 + j] = x;
            if (v_out) v_out[m * D32 + j] = v;
        }
        free(xs);
    }
    free_table(&tb);
}

/* ------------------------------------------------------------- pack/unpack */

void oracle_pack(const uint32_t* codes, int64_t n, int32_t b, uint32_t* words)
{
    const int64_t nwords = n / 32 * b;
    memset(words, 0, sizeof(uint32_t) * (size_t)nwords);
    /* element e of the stream owns bits [e*b, e*b + b) of the bit string
     * whose bit i is bit (i % 32) of word (i / 32) */
    for (int64_t e = 0; e < n; ++e) {
        for (int32_t i = 0; i < b; ++i) {
            const int64_t bit = e * b + i;
            if ((codes[e] >> i) & 1u) words[bit >> 5] |= 1u << (bit & 31);
        }
    }
}

void oracle_unpack(const uint32_t* words, int64_t n, int32_t b, uint32_t* codes)
{
    for (int64_t e = 0; e < n; ++e) {
        uint32_t c = 0;
        for (int32_t i = 0; i < b; ++i) {
            const int64_t bit = e * b + i;
            c |= ((words[bit >> 5] >> (bit & 31)) & 1u) << i;
        }
        codes[e] = c;
    }
}

void oracle_quantize_pack(const float* grads, int64_t worker_stride, int32_t M,
                          const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                          const float* norms, int32_t b, uint64_t seed, uint32_t step,
                          uint32_t* packed, int64_t packed_stride)
{
    const int64_t D32 = oracle_padded_elems(seg_elems, n_seg);
    uint32_t* codes = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)((int64_t)M * D32 + 1));
    oracle_quantize(grads, worker_stride, M, seg_elems, n_seg, bucket, norms, b, seed, step,
                    codes, NULL, NULL);
#pragma omp parallel for schedule(static) num_threads(g_threads) if (g_threads > 1)
    for (int32_t m = 0; m < M; ++m)
        oracle_pack(codes + (int64_t)m * D32, D32, b, packed + (int64_t)m * packed_stride);
    free(codes);
}

/* -------------------------------------------------------------- dequantize */

void oracle_dequantize(const uint32_t* codes, const float* norms,
                       const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                       int32_t b, double* values)
{
    table_t tb = make_table(seg_elems, n_seg, bucket);
    const int64_t D32 = oracle_padded_elems(seg_elems, n_seg);
    const int32_t s = (1 << (b - 1)) - 1;
    for (int64_t j = 0; j < D32; ++j) values[j] = 0.0;
    for (int64_t k = 0; k < tb.nb; ++k) {
        for (int64_t e = 0; e < tb.len[k]; ++e) {
            const int64_t j = tb.start[k] + e;
            const double q = (double)codes[j] - (double)s;        /* sgn * level */
            values[j] = (s > 0) ? q * (double)norms[k] / (double)s : 0.0;
        }
    }
    free_table(&tb);
}

void oracle_unpack_dequant_average(const uint32_t* packed, int64_t packed_stride,
                                   const float* norms, int32_t M, int32_t b,
                                   const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                                   float* out)
{
    table_t tb = make_table(seg_elems, n_seg, bucket);
    const int64_t D32 = oracle_padded_elems(seg_elems, n_seg);
    const int32_t s = (1 << (b - 1)) - 1;
    uint32_t* codes = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)((int64_t)M * D32 + 1));
#pragma omp parallel for schedule(static) num_threads(g_threads) if (g_threads > 1)
    for (int32_t m = 0; m < M; ++m)
        oracle_unpack(packed + (int64_t)m * packed_stride, D32, b, codes + (int64_t)m * D32);

    for (int64_t j = 0; j < D32; ++j) out[j] = 0.0f;      /* pads: +0 */
#pragma omp parallel for schedule(static) num_threads(g_threads) if (g_threads > 1)
    for (int64_t k = 0; k < tb.nb; ++k) {
        for (int64_t e = 0; e < tb.len[k]; ++e) {
            const int64_t j = tb.start[k] + e;
            double acc = 0.0;
            for (int32_t m = 0; m < M; ++m) {
                const double q = (double)codes[(int64_t)m * D32 + j] - (double)s;     /* sgn * level */
                if (s > 0) acc += q * (double)norms[(int64_t)m * tb.nb + k] / (double)s;
            }
            out[j] = (float)(acc / (double)M);
        }
    }
    free(codes);
    free_table(&tb);
}

/* Eq. 2 / the parameter-update step of Algorithm 1: x <- x - eta * g_hat, with g_hat the
 * average above, all in fp64 and rounded to fp32 once.  Padding elements keep their value. */
void oracle_unpack_average_update(const uint32_t* packed, int64_t packed_stride,
                                  const float* norms, int32_t M, int32_t b,
                                  const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                                  double eta, float* x)
{
    table_t tb = make_table(seg_elems, n_seg, bucket);
    const int64_t D32 = oracle_padded_elems(seg_elems, n_seg);
    const int32_t s = (1 << (b - 1)) - 1;
    uint32_t* codes = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)((int64_t)M * D32 + 1));
#pragma omp parallel for schedule(static) num_threads(g_threads) if (g_threads > 1)
    for (int32_t m = 0; m < M; ++m)
        oracle_unpack(packed + (int64_t)m * packed_stride, D32, b, codes + (int64_t)m * D32);

#pragma omp parallel for schedule(static) num_threads(g_threads) if (g_threads > 1)
    for (int64_t k = 0; k < tb.nb; ++k) {
        for (int64_t e = 0; e < tb.len[k]; ++e) {
            const int64_t j = tb.start[k] + e;
            double acc = 0.0;
            for (int32_t m = 0; m < M; ++m) {
                const double q = (double)codes[(int64_t)m * D32 + j] - (double)s;     /* sgn * level */
                if (s > 0) acc += q * (double)norms[(int64_t)m * tb.nb + k] / (double)s;
            }
            const double g_hat = acc / (double)M;
            x[j] = (float)((double)x[j] - eta * g_hat);
        }
    }
    free(codes);
    free_table(&tb);
}
