/*
 * dq_oracle.h -- plain CPU oracle of the DQ-SGD quantizer hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a slow, single-pass, obviously-correct
 * restatement of the method (arXiv 2107.14575) used to check the CUDA library
 * and to serve as the timed CPU baseline.  It shares no code with the CUDA
 * path and must never be called from it.  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg may load it.
 *
 * What each function follows:
 *   layout            bucketed layout of a list of tensors (the paper normalises
 *                     by the norm of the whole vector, Eq. 5; one bucket per
 *                     tensor reproduces that, smaller buckets apply the same
 *                     formula per bucket)
 *   bucket_norms      ||g||_2 of Eq. 5, per bucket; bucket_norms_p also the l_infinity
 *                     member of the paper's l_p family (Eq. 5 leaves p open)
 *   choose_bits       Eq. 17 with G-bar of Lemma 1, integer b by ceiling
 *   quantize          Eq. 5 and Eq. 6 (stochastic map zeta), s = 2^(b-1)-1; the b-bit
 *                     code of Sec. IV-A (a sign and b-1 bits of zeta) is stored as
 *                     the single number s + sgn * level in 0 .. 2s
 *   pack / unpack     b-bit codes concatenated LSB-first into 32-bit words
 *   unpack_dequant_average   Algorithm 1, server step "Average", with Eq. 5
 *   unpack_average_update    the same followed by the parameter update of Eq. 2
 *                     (the parameter-update step of Algorithm 1)
 *   philox4x32_10     Salmon, Moraes, Dror, Shaw, "Parallel random numbers:
 *                     as easy as 1, 2, 3" (SC'11), Philox-4x32 with 10 rounds
 *
 * Pinned by tests/test_oracle_*.py.  Unpinned (the paper leaves it undefined):
 * the b = 1 case (s = 0), read here as "code 0, value 0" -- parity unpinned
 * for that case.
 *
 * Layout convention: tensor i with n_i elements starts at padded offset
 * P_i = sum_{j<i} roundup32(n_j); the worker buffer holds D32 = sum roundup32(n_i)
 * floats; buckets of `bucket` elements never cross a tensor, the last bucket
 * of a tensor may be short.  `bucket` is a multiple of 32; a bucket at least as
 * large as every tensor is the paper's own case (one norm per vector).
 */
#ifndef DQ_ORACLE_H
#define DQ_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- layout ---- */
int64_t oracle_padded_elems(const int64_t* seg_elems, int32_t n_seg);
int64_t oracle_num_buckets(const int64_t* seg_elems, int32_t n_seg, int32_t bucket);
void    oracle_seg_offsets(const int64_t* seg_elems, int32_t n_seg, int64_t* offsets /*[n_seg]*/);
/* start (padded flat index) and length (valid elements) of every bucket */
void    oracle_bucket_table(const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                            int64_t* start /*[nb]*/, int64_t* len /*[nb]*/);

/* ---- Eq. 5: per-bucket L2 norm, fp64 accumulation, rounded once to fp32 ---- */
void oracle_bucket_norms(const float* grads, int64_t worker_stride, int32_t M,
                         const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                         float* norms /*[M][nb]*/);

/* ---- Eq. 5 with another member of the l_p family: p_kind = 2 is the call above,
 *      p_kind = 0 stands for p = infinity (largest magnitude of the bucket, exact) ---- */
void oracle_bucket_norms_p(const float* grads, int64_t worker_stride, int32_t M,
                           const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                           int32_t p_kind, float* norms /*[M][nb]*/);

/* ---- Eq. 17: bit rule.  Returns b; writes s and the real-valued x with
 *      b* = log2(x + 1) + 1.  fixed_b != 0 bypasses the rule. ---- */
int32_t oracle_choose_bits(const float* norms, int64_t nb, int32_t M,
                           int32_t T, int32_t t, double eps_hat, double alpha,
                           int32_t b_min, int32_t b_max, int32_t fixed_b,
                           int32_t* s_out, double* x_out);

/* ---- Philox4x32-10 ---- */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);

/* ---- Eq. 5/6: codes s + sgn * level, one uint32 per padded element (s for
 *      padding).  x_out / v_out (optional, may be NULL) receive the signed
 *      position x = RZ(g * RZ(s/norm)) on the level grid and the uniform v drawn
 *      for every element; the code is floor(x + v) + s. ---- */
void oracle_quantize(const float* grads, int64_t worker_stride, int32_t M,
                     const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                     const float* norms, int32_t b, uint64_t seed, uint32_t step,
                     uint32_t* codes /*[M][D32]*/, float* x_out, float* v_out);

/* ---- pack / unpack n codes of b bits (n a multiple of 32) ---- */
void oracle_pack(const uint32_t* codes, int64_t n, int32_t b, uint32_t* words /*[b*n/32]*/);
void oracle_unpack(const uint32_t* words, int64_t n, int32_t b, uint32_t* codes /*[n]*/);

/* quantize then pack every worker; worker m's words start at m*packed_stride */
void oracle_quantize_pack(const float* grads, int64_t worker_stride, int32_t M,
                          const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                          const float* norms, int32_t b, uint64_t seed, uint32_t step,
                          uint32_t* packed, int64_t packed_stride);

/* ---- Eq. 5 inverse for one worker: value = norm * (code - s) / s, in fp64 ---- */
void oracle_dequantize(const uint32_t* codes, const float* norms /*[nb]*/,
                       const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                       int32_t b, double* values /*[D32]*/);

/* ---- Algorithm 1 "Average": unpack, dequantize, mean over M workers ---- */
void oracle_unpack_dequant_average(const uint32_t* packed, int64_t packed_stride,
                                   const float* norms /*[M][nb]*/, int32_t M, int32_t b,
                                   const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                                   float* out /*[D32]*/);

/* ---- Eq. 2: x <- x - eta * average, fp64 arithmetic, one rounding to fp32; pads untouched ---- */
void oracle_unpack_average_update(const uint32_t* packed, int64_t packed_stride,
                                  const float* norms /*[M][nb]*/, int32_t M, int32_t b,
                                  const int64_t* seg_elems, int32_t n_seg, int32_t bucket,
                                  double eta, float* x /*[D32], in and out*/);

/* number of OpenMP threads the loops over workers/buckets may use (default 1) */
void    oracle_set_threads(int32_t n);
int32_t oracle_get_threads(void);

#ifdef __cplusplus
}
#endif
#endif
