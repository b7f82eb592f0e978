/*
 * dq.h -- C ABI of the DQ-SGD gradient quantizer hot path for NVIDIA B200 (sm_100a).
 *
 * Method: "DQ-SGD: Dynamic Quantization in SGD for Communication-Efficient
 * Distributed Learning" (arXiv 2107.14575).  The steps of one iteration of
 * Algorithm 1, all asynchronous on the caller's CUDA stream:
 *
 *   dq_bucket_norms            ||g||_2 of Eq. 5, per bucket          (workers)
 *   dq_choose_bits             bit rule Eq. 17 -> b, s on the device (server)
 *   dq_quantize_pack           Q_b[g] of Eq. 5/6, b-bit codes packed (workers)
 *   dq_unpack_dequant_average  "Average" step of Algorithm 1         (server)
 *
 * and two calls that merge neighbouring steps:
 *
 *   dq_norms_quantize_pack     norms and quantizer in one pass over the gradients
 *                              (b_t is known before step t: Algorithm 1 derives
 *                              b_{t+1} from iteration t)
 *   dq_unpack_average_update   the average followed by x <- x - eta * average (Eq. 2)
 *
 * M workers are M gradient buffers on one GPU: worker m's data is at
 * base + m * stride for every per-worker array.  There is no CPU fallback.
 *
 * Conventions
 *  - "dev" pointers are device pointers owned by the caller.  The library never
 *    allocates or frees device memory and never synchronises the host.
 *  - `stream` is a cudaStream_t passed as void* (NULL = legacy default stream).
 *    Kernels are launched with programmatic stream serialization and start by
 *    waiting for the previous kernel of the stream to complete: the usual
 *    stream order holds for everything they read and write, whatever kernel
 *    (the library's or the caller's) precedes them.  The calls of a round
 *    (norms, bit rule with caller scratch, quantizer, average, update) can be
 *    captured in a CUDA graph.
 *  - Return value: DQ_OK or a negative DQ_ERR_* for errors found on the host
 *    before anything is launched (nothing is written in that case).
 *  - Conditions only the device can see are OR-ed into *dev_status (DQ_STAT_*
 *    bits, a caller-owned int32 the caller zeroes and reads when it wants).
 *    A kernel that raises DQ_STAT_BAD_BITS or DQ_STAT_CAPACITY writes no
 *    output.  No kernel traps or spins without bound: every wait has a time
 *    limit, a decision to leave after one ran out is taken by all threads that
 *    later meet at a barrier (a vote or a barrier reduction, never a thread's own
 *    view), and whoever issued copies waits for them before the CTA ends.
 *  - Data layout ("padded layout"): tensor i of n_i elements starts at element
 *    offset P_i = sum_{j<i} roundup32(n_j) of a worker's fp32 buffer; the
 *    buffer holds D32 = sum_i roundup32(n_i) elements.  Buckets of `bucket`
 *    elements tile each tensor separately; the last bucket of a tensor may be
 *    short.  Elements between a tensor's end and the next multiple of 32 are
 *    padding: ignored on input, the code of 0 in the packed stream, +0 in the
 *    output.
 *  - Codes: s = 2^(b-1) - 1 levels per sign (Sec. IV-A).  A b-bit code holds
 *    s + sgn * level, a number in 0 .. 2s (excess-s; 0 has a single code, s).
 *    THIS IS NOT THE WIRE FORMAT SEC. IV-A DESCRIBES, which spends one bit on the
 *    sign and b-1 bits on the level zeta: the information and the b bits per
 *    element of Eq. 7 are the same, the bit patterns are not, so a peer that
 *    follows the paper's layout literally cannot read these words (and has a
 *    second code, -0, that this format does not).
 *  - Packed stream of one worker: group q (padded elements 32q .. 32q+31) owns
 *    words b*q .. b*q+b-1; element e of the group owns bits [e*b, e*b+b) of
 *    that little-endian bit string.
 */
#ifndef DQ_H
#define DQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- host return codes ---- */
#define DQ_OK          0
#define DQ_ERR_ARG    (-1)  /* NULL pointer, M < 1, bad enum                          */
#define DQ_ERR_ALIGN  (-2)  /* pointer not 16-byte aligned, stride not a multiple of 32
                               elements (fp32) / 4 words (packed)                     */
#define DQ_ERR_RANGE  (-3)  /* size, bucket, rule field or capacity out of range       */
#define DQ_ERR_CUDA   (-4)  /* a CUDA call (launch, copy, descriptor encode) failed    */
#define DQ_ERR_STATE  (-5)  /* multi-tensor layout used before its device table was bound */
#define DQ_ERR_TOO_LARGE (-6) /* more data than an allocation-free entry point's built-in scratch covers */

/* ---- device status bits (OR-ed into *dev_status) ---- */
#define DQ_STAT_NONFINITE   1  /* a bucket norm or G-bar is NaN/Inf                    */
#define DQ_STAT_BAD_BITS    2  /* device b outside 1..16                               */
#define DQ_STAT_CAPACITY    4  /* b * D32/32 words exceed packed_stride_words          */
#define DQ_STAT_WAIT        8  /* a bounded wait on an asynchronous copy ran out       */
#define DQ_STAT_INTERNAL   16  /* a kernel found its shared memory misaligned and left  */

#define DQ_MAX_BITS       16
#define DQ_MAX_BUCKET   4096
#define DQ_MAX_WORKERS  4096

/* ---- members of the quantizer family of Eq. 5 (the norm that scales the entries) ---- */
#define DQ_NORM_L2      2   /* p = 2, the default                                      */
#define DQ_NORM_LINF    0   /* p = infinity: the largest magnitude of the bucket        */
#define DQ_BUCKET_WHOLE_TENSOR 0  /* bucket argument: one norm per tensor, as Eq. 5 is written */
#define DQ_MAX_TENSOR_ELEMS (1 << 30)  /* largest tensor of a whole-tensor layout       */

typedef struct dq_layout dq_layout_t;   /* host object, immutable after create */

/* Parameters of the bit rule, Eq. 17:
 *   b_t = log2( sqrt(T / eps_hat) * alpha^((T-1-t)/2) * G-bar_t + 1 ) + 1
 * eps_hat is the paper's hat-epsilon_Q = 8 W eps_Q / (L d eta^2).  The integer b
 * is the smallest b in [b_min, b_max] whose s = 2^(b-1) - 1 reaches the
 * argument of the logarithm minus one (ceiling of Eq. 17), else b_max.
 * fixed_b in 1..16 bypasses the rule; fixed_b = 0 selects it. */
typedef struct dq_rule {
    int32_t T;        /* total iterations, >= 1                */
    int32_t t;        /* current iteration, 0 <= t < T         */
    double  eps_hat;  /* > 0                                   */
    double  alpha;    /* convergence factor of Theorem 1, > 0  */
    int32_t b_min;    /* 1..16 (2 keeps the quantizer unbiased) */
    int32_t b_max;    /* b_min..16                              */
    int32_t fixed_b;  /* 0 or 1..16                             */
} dq_rule_t;

/* ------------------------------------------------------------------ layout
 * Host-only bookkeeping of the padded layout above (no CUDA call).
 * seg_elems[n_seg] are the tensor sizes (>= 0), bucket a multiple of 32 in
 * 32..DQ_MAX_BUCKET.  The padded total must stay below 2^31 elements.
 * Errors: DQ_ERR_ARG (NULL, n_seg < 1), DQ_ERR_RANGE. */
int     dq_layout_create(const int64_t* seg_elems, int32_t n_seg, int32_t bucket, dq_layout_t** out);
/* The same with the member of the family of Eq. 5 chosen: `norm` is DQ_NORM_L2 or
 * DQ_NORM_LINF (what dq_bucket_norms, dq_tensor_norms and dq_norms_quantize_pack compute
 * for this layout; the quantizer and the average take whatever norms they are given).
 * bucket = DQ_BUCKET_WHOLE_TENSOR gives every non-empty tensor a single bucket, which is
 * Eq. 5 as the paper writes it (the vector is normalised by its own norm); tensors may
 * then have up to DQ_MAX_TENSOR_ELEMS elements, and the norms come from dq_tensor_norms.
 * dq_layout_create(.., bucket, ..) is dq_layout_create_ex(.., bucket, DQ_NORM_L2, ..).
 * Errors: as dq_layout_create; DQ_ERR_ARG for an unknown norm. */
int     dq_layout_create_ex(const int64_t* seg_elems, int32_t n_seg, int32_t bucket, int32_t norm,
                            dq_layout_t** out);
int32_t dq_layout_norm(const dq_layout_t* layout);          /* DQ_NORM_L2 / DQ_NORM_LINF          */
int32_t dq_layout_whole_tensor(const dq_layout_t* layout);  /* 1 for a whole-tensor layout, else 0 */
void    dq_layout_destroy(dq_layout_t* layout);
int32_t dq_layout_num_segments(const dq_layout_t* layout);
int64_t dq_layout_padded_elems(const dq_layout_t* layout);            /* D32                     */
int64_t dq_layout_seg_offset(const dq_layout_t* layout, int32_t i);   /* P_i, -1 if i is invalid */
int64_t dq_layout_num_buckets(const dq_layout_t* layout);             /* nb per worker           */
int64_t dq_layout_packed_words(const dq_layout_t* layout, int32_t b); /* b * D32 / 32            */
/* start (padded element index) and valid length of bucket k; DQ_ERR_RANGE if k is invalid */
int     dq_layout_bucket(const dq_layout_t* layout, int64_t k, int64_t* start, int64_t* len);

/* ---- cutting the path across several GPUs (one worker per GPU, Algorithm 1's send /
 * collect / average with the server's work divided among the GPUs).  The padded buffer is
 * cut into contiguous ranges of whole buckets; GPU r averages range r of every worker's
 * packed stream.  Range [k0, k1) of buckets owns the contiguous words
 * [b * first_elem / 32, b * (first_elem + padded_elems(slice)) / 32) of a packed stream, the
 * norms [k0, k1) and the same element range of the output.
 *   dq_layout_shard_bounds  bounds[0..n_shards]: bounds[j] is the first bucket of shard j,
 *                           bounds[n_shards] = nb; shards carry nearly equal numbers of
 *                           elements (a shard may be empty when there are few buckets)
 *   dq_layout_slice         buckets [k0, k1) as a layout of their own (same bucket size and
 *                           norm; its tensors are the pieces of the parent's tensors inside
 *                           the range; bucket j of the slice is bucket k0 + j of the parent);
 *                           *first_elem (optional) = where the slice starts in the parent's
 *                           padded buffer.  The caller destroys the slice, and binds a device
 *                           table to it like to any layout with several tensors.
 * Errors: DQ_ERR_ARG (NULL, n_shards < 1), DQ_ERR_RANGE (empty or invalid bucket range). */
int     dq_layout_shard_bounds(const dq_layout_t* layout, int32_t n_shards, int64_t* bounds);
int     dq_layout_slice(const dq_layout_t* layout, int64_t k0, int64_t k1, dq_layout_t** out,
                        int64_t* first_elem);

/* Layouts with more than one tensor need a small table on the device.  The
 * caller provides dq_layout_table_bytes() bytes of 16-byte aligned device
 * memory and keeps it alive while the layout is in use; bind copies the table
 * there (cudaMemcpyAsync on `stream`, from memory the layout owns) and
 * remembers the pointer.  Single-tensor layouts need no table (bytes = 0 is
 * reported and bind is a no-op).  Errors: DQ_ERR_ARG, DQ_ERR_ALIGN,
 * DQ_ERR_RANGE (buffer too small), DQ_ERR_CUDA. */
size_t  dq_layout_table_bytes(const dq_layout_t* layout);
int     dq_layout_bind_device_table(dq_layout_t* layout, void* dev_buf, size_t bytes, void* stream);

/* ------------------------------------------------------------- norms, Eq. 5
 * dev_norms[m*nb + k] = sqrt( sum of squares of the valid elements of bucket k
 * of worker m ), the l_2 member of the paper's ||g||_p applied per bucket; for a
 * layout created with DQ_NORM_LINF, the largest magnitude among those elements
 * (exact; a NaN element makes the norm NaN).
 * in : dev_grads  fp32, worker m at dev_grads + m*worker_stride_elems,
 *                 each holding D32 elements in the padded layout
 * out: dev_norms  fp32 [M][nb]
 * Sets DQ_STAT_NONFINITE if a norm is not finite (the norm is still written).
 * Accumulation is fp32 in a fixed order: results are deterministic and within
 * 1e-6 relative of an fp64 evaluation. */
int dq_bucket_norms(const dq_layout_t* layout, const float* dev_grads, int64_t worker_stride_elems,
                    int32_t M, float* dev_norms, int32_t* dev_status, void* stream);

/* ------------------------------------------- one norm per tensor, Eq. 5 as written
 * For layouts created with bucket = DQ_BUCKET_WHOLE_TENSOR: dev_norms[m*nb + k] is the
 * norm (l_2 or l_inf, as the layout says) of the k-th non-empty tensor of worker m, nb the
 * number of non-empty tensors.  Two kernels: partial results of 4096-element pieces into
 * dev_scratch, then one reduction per (worker, tensor) in a fixed order (fp64 for the sums
 * of squares), so results are deterministic and the l_2 norms within 1e-6 relative of an
 * fp64 evaluation; l_inf norms are exact.  dq_bucket_norms and dq_norms_quantize_pack
 * return DQ_ERR_RANGE for such layouts (a tensor's codes need the norm of the whole
 * tensor, so the gradients are read twice); dq_quantize_pack, dq_choose_bits and the
 * average calls work on them as on any other layout.
 * dev_scratch: dq_tensor_norms_scratch_bytes() bytes, 16-byte aligned, used only during
 * the call's kernels.  Sets DQ_STAT_NONFINITE if a norm is not finite. */
size_t dq_tensor_norms_scratch_bytes(const dq_layout_t* layout, int32_t M);
int dq_tensor_norms(const dq_layout_t* layout, const float* dev_grads, int64_t worker_stride_elems,
                    int32_t M, float* dev_norms, void* dev_scratch, size_t scratch_bytes,
                    int32_t* dev_status, void* stream);

/* --------------------------------------------------------- bit rule, Eq. 17
 * G-bar^2 = (1/M) sum_m sum_k dev_norms[m][k]^2 (Lemma 1; for p = 2 the sum of
 * squared bucket norms is the squared norm of the worker's gradient), then the
 * rule above.  Writes dev_b[0] = b and dev_b[1] = s.  The reduction is fp64 in
 * a fixed order.  The later calls read b from dev_b, so no host
 * synchronisation is needed between the calls of a step.
 * dev_scratch: dq_choose_bits_scratch_bytes() bytes of 16-byte aligned device
 * memory, used only during the call's kernels.
 * Sets DQ_STAT_NONFINITE if G-bar is not finite (b = b_max is written). */
size_t dq_choose_bits_scratch_bytes(const dq_layout_t* layout, int32_t M);
int dq_choose_bits(const dq_layout_t* layout, const float* dev_norms, int32_t M, const dq_rule_t* rule,
                   int32_t* dev_b, void* dev_scratch, size_t scratch_bytes,
                   int32_t* dev_status, void* stream);

/* ------------------------------------------- bit rule without any allocation
 * (The paper has no counterpart: this entry point exists for the library's
 * users, not for the method.)
 *
 * Same computation and same result as dq_choose_bits, for callers that have no
 * scratch buffer to give and no way to get one: code that runs after start-up
 * in a process whose device memory was handed out once and for all (a
 * framework's caching allocator owns it, or the job runs against a fixed
 * memory budget), and code on a latency-critical path where cudaMalloc is off
 * limits because it synchronises the device and takes an unpredictable time.
 * The chunk sums of the norm reduction live in a 64 KB array inside the
 * library image instead; every GPU that loads the library holds those 64 KB
 * until the process exits.  The call itself allocates and frees nothing.
 *
 *  - Limit: M * nb <= dq_choose_bits_noalloc_max_norms() (8192 * 8192 = 67,108,864
 *    norms).  Beyond it the call returns DQ_ERR_TOO_LARGE and launches nothing;
 *    use dq_choose_bits with caller scratch for larger problems.
 *  - The first call on each device looks up the array's device address (that
 *    device must be current, as for every call) and keeps it for the life of
 *    the process.  Make that first call before any stream capture begins.  The
 *    address belongs to the device's primary context: after a cudaDeviceReset
 *    (or any other teardown of that context) the library must not be used
 *    again in the same process.  Devices with ordinal 64 and above are not
 *    served (DQ_ERR_CUDA).
 *  - All calls on a device share the one array, and it keeps what the last call
 *    wrote.  Nothing in it needs clearing between calls (each call overwrites
 *    every entry it later reads), but two calls whose kernels overlap on the
 *    GPU -- different streams without an ordering between them -- race on it
 *    and may both produce a wrong b.  Calls on one stream are safe.
 * Arguments, outputs, status bits and the other error codes are those of
 * dq_choose_bits without the scratch pair. */
int64_t dq_choose_bits_noalloc_max_norms(void);
int dq_choose_bits_noalloc(const dq_layout_t* layout, const float* dev_norms, int32_t M, const dq_rule_t* rule,
                           int32_t* dev_b, int32_t* dev_status, void* stream);

/* ----------------------------------------------------- quantizer, Eq. 5 and 6
 * For every valid element j of worker m, with norm the norm of its bucket and
 * s = 2^(b-1) - 1, in fp32 with both operations rounded toward zero (RZ):
 *   inv = norm >= 2^-100 ? RZ(s / norm) : 0
 *   x   = RZ(g_j * inv)                          position on the level grid
 *   code = floor(x + v) + s                      (x + v evaluated exactly)
 * Rounding toward zero keeps |x| <= s for every element with |g_j| <= norm, which
 * holds for the norms dq_bucket_norms computes (a bucket's norm dominates its
 * entries).  The codes of a bucket whose norm is smaller than one of its entries
 * are unspecified (nothing outside the packed stream is touched).
 * v = (2k + 1) / 2^17 in (0, 1) is the element's uniform draw: k is half (j & 1)
 * (0 = low 16 bits) of word ((j >> 1) & 3) of Philox4x32-10 with counter
 * (j >> 3, 0, m, step) and key (seed low word, seed high word); j is the
 * element's index in the padded layout.  floor(x + v) is the neighbour of x
 * away from zero with probability p_r = frac(|x|) and the one toward zero
 * otherwise, which is Eq. 6 (to within 2^-17); values that lie on a level are
 * reproduced for every draw.  b = 1 (s = 0) stores zeros.
 * The codes are packed as described at the top of this file.
 * in : dev_grads, dev_norms [M][nb], dev_b (written by dq_choose_bits)
 * out: dev_packed uint32, worker m at dev_packed + m*packed_stride_words; the
 *      first b*D32/32 words are written, the rest left untouched.
 * Device conditions: DQ_STAT_BAD_BITS, DQ_STAT_CAPACITY (nothing is written),
 * DQ_STAT_WAIT, DQ_STAT_INTERNAL. */
int dq_quantize_pack(const dq_layout_t* layout, const float* dev_grads, int64_t worker_stride_elems,
                     int32_t M, const float* dev_norms, const int32_t* dev_b,
                     uint64_t seed, uint32_t step,
                     uint32_t* dev_packed, int64_t packed_stride_words,
                     int32_t* dev_status, void* stream);

/* The same for workers first_worker .. first_worker + M - 1 of a larger job: worker m of
 * the call draws the uniforms of worker first_worker + m (the third counter word above).
 * With one worker per GPU, GPU r passes M = 1 and first_worker = r, and the words it
 * produces are those of row r of a single call over all workers (Lemma 1's 1/W variance
 * of the average needs the workers' draws to be independent). */
int dq_quantize_pack_worker(const dq_layout_t* layout, const float* dev_grads, int64_t worker_stride_elems,
                            int32_t M, const float* dev_norms, const int32_t* dev_b,
                            uint64_t seed, uint32_t step, uint32_t first_worker,
                            uint32_t* dev_packed, int64_t packed_stride_words,
                            int32_t* dev_status, void* stream);

/* --------------------------- norms and quantizer in one pass, Eq. 5 and 6
 * dq_bucket_norms followed by dq_quantize_pack on the same gradients, with every
 * gradient byte read once: dev_norms receives exactly what dq_bucket_norms
 * writes and dev_packed exactly what dq_quantize_pack writes for those norms.
 * Algorithm 1 sets b_{t+1} from the gradients of iteration t (its bit-update step
 * comes after the averaging of step t), so dev_b is known before this step's
 * gradients are and the two steps need not be separate passes.  A step is then
 *   dq_norms_quantize_pack (b_t) -> dq_unpack_dequant_average -> dq_choose_bits (b_{t+1}).
 * in : dev_grads, dev_b
 * out: dev_norms fp32 [M][nb], dev_packed (as for dq_quantize_pack)
 * Device conditions: those of both calls. */
int dq_norms_quantize_pack(const dq_layout_t* layout, const float* dev_grads, int64_t worker_stride_elems,
                           int32_t M, const int32_t* dev_b, uint64_t seed, uint32_t step,
                           float* dev_norms, uint32_t* dev_packed, int64_t packed_stride_words,
                           int32_t* dev_status, void* stream);

/* dq_norms_quantize_pack for workers first_worker .. first_worker + M - 1 (see
 * dq_quantize_pack_worker). */
int dq_norms_quantize_pack_worker(const dq_layout_t* layout, const float* dev_grads, int64_t worker_stride_elems,
                                  int32_t M, const int32_t* dev_b, uint64_t seed, uint32_t step,
                                  uint32_t first_worker, float* dev_norms, uint32_t* dev_packed,
                                  int64_t packed_stride_words, int32_t* dev_status, void* stream);

/* ----------------------------------- Algorithm 1, server side: "Average"
 * dev_out[j] = (1/M) sum_m (code_m - s) * norm_m / s   (Eq. 5 inverted, then
 * the mean over workers); 0 for padding and when s = 0.  fp32 accumulation in
 * worker order: deterministic, within 1e-6 relative L2 of an fp64 evaluation.
 * in : dev_packed, dev_norms [M][nb], dev_b
 * out: dev_out fp32 [D32]
 * Device conditions: DQ_STAT_BAD_BITS, DQ_STAT_CAPACITY (nothing is written),
 * DQ_STAT_WAIT. */
int dq_unpack_dequant_average(const dq_layout_t* layout, const uint32_t* dev_packed,
                              int64_t packed_stride_words, const float* dev_norms, int32_t M,
                              const int32_t* dev_b, float* dev_out, int32_t* dev_status, void* stream);

/* ------------- Algorithm 1, server side: "Average" and the parameter update
 * x <- x - eta * g_hat, with g_hat the average dq_unpack_dequant_average computes
 * (Eq. 2; the parameter-update step that follows the averaging in Algorithm 1.
 * The prose around Eq. 17 prints the step with a plus sign, the listing and
 * Eq. 2 with a minus sign: descent is meant).  The averaged gradient is formed in registers and
 * never written: per element M*b/8 + 4 bytes are read and 4 written.
 *   dev_params[j] <- fmaf(-lr, g_hat[j], dev_params[j])   (one fp32 rounding)
 * Padding elements of dev_params keep their value (their g_hat is 0), and so does
 * everything when s = 0 (b = 1).
 * in : dev_packed, dev_norms [M][nb], dev_b, lr (finite, else DQ_ERR_RANGE)
 * io : dev_params fp32 [D32], 16-byte aligned, caller-owned, in the padded layout
 * Device conditions: as dq_unpack_dequant_average. */
int dq_unpack_average_update(const dq_layout_t* layout, const uint32_t* dev_packed,
                             int64_t packed_stride_words, const float* dev_norms, int32_t M,
                             const int32_t* dev_b, float lr, float* dev_params,
                             int32_t* dev_status, void* stream);

/* Text for a DQ_ERR_* return value (static storage). */
const char* dq_status_string(int code);

/* Test hook for the bounded waits (no counterpart in the paper).  Every wait of a
 * kernel for one of its own asynchronous copies is bounded by `limit_ns` of the GPU's
 * global timer (default 2e9; 0 restores the default).  With `lose_first_wait` != 0 the
 * first such wait of every warp or CTA that consumes copies is declared lost at once,
 * although its copy is valid and lands a moment later: this exercises what a kernel does
 * after a time-out -- raise DQ_STAT_WAIT, stop producing output, wait (with limit_ns)
 * for every copy it has issued, return -- without anything being lost, faulting or
 * hanging.  Host state of the library, read when a call is made; not for production use
 * (the outputs of a call made under it are incomplete). */
void dq_debug_set_wait_limits(uint64_t limit_ns, int32_t lose_first_wait);

#ifdef __cplusplus
}
#endif

#endif /* DQ_H */
