// dq_choose_bits: the bit rule of Eq. 17 evaluated on the device.
//
//   G-bar^2 = (1/M) sum over workers and buckets of norm^2        (Lemma 1)
//   x       = sqrt(T/eps_hat) * alpha^((T-1-t)/2) * G-bar
//   b       = smallest b in [b_min, b_max] with 2^(b-1) - 1 >= x   (else b_max)
//
// Two small kernels: fixed-size chunks of the norm array are summed in fp64
// (fixed assignment of elements to threads, fixed tree), then one CTA adds
// the chunk sums in a fixed order and applies the rule.  The factor
// sqrt(T/eps_hat) * alpha^((T-1-t)/2) is a host scalar.
#include "dq_common.cuh"

#include <cmath>
#include <mutex>

namespace {

// Both kernels are small on purpose (128 threads, well under 100 registers): in the order of
// Algorithm 1 they run on a second stream beside the average, whose persistent CTAs leave
// about a fifth of an SM's registers free, and CTAs of this size fit into that room.
constexpr int kThreads = 128;       // threads of the second kernel
constexpr int kChunk = 8192;        // norms per CTA of the first kernel
constexpr int kSumThreads = 128;    // threads of the first kernel: 64 norms each, all loads in flight at once

// Sum over the CTA in a fixed order: shuffle tree inside each warp, then the warp sums
// added in warp order by thread 0.  Returns the total in thread 0.
template <int NT>
__device__ __forceinline__ double block_sum(double v, double* sh)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    double total = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < NT / 32; ++w) total += sh[w];
    }
    return total;
}

__global__ void __launch_bounds__(kSumThreads, 8)
norm_square_partials(const float* __restrict__ norms, const int64_t n, double* __restrict__ partial)
{
    __shared__ double sh[kSumThreads / 32];
    grid_dependency_wait();
    constexpr int kPer = kChunk / kSumThreads;     // 64 norms per thread, fetched 32 at a time
    constexpr int kBatch = 32;
    const int64_t base = (int64_t)blockIdx.x * kChunk + threadIdx.x;
    double a0 = 0.0, a1 = 0.0;
#pragma unroll
    for (int h = 0; h < kPer / kBatch; ++h) {
        float x[kBatch];
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            const int64_t j = base + (int64_t)(h * kBatch + i) * kSumThreads;
            x[i] = (j < n) ? __ldg(norms + j) : 0.0f;
        }
#pragma unroll
        for (int i = 0; i < kBatch; i += 2) {
            a0 = fma((double)x[i], (double)x[i], a0);
            a1 = fma((double)x[i + 1], (double)x[i + 1], a1);
        }
    }
    const double s = block_sum<kSumThreads>(a0 + a1, sh);
    if (threadIdx.x == 0) partial[blockIdx.x] = s;       // one entry per CTA of the grid: in bounds by construction
}

__global__ void __launch_bounds__(kThreads)
apply_rule(const double* __restrict__ partial, const int npartial, const int M, const double coef,
           const int b_min, const int b_max, const int fixed_b,
           int32_t* __restrict__ dev_b, int32_t* __restrict__ status)
{
    __shared__ double sh[kThreads / 32];
    grid_dependency_wait();
    double acc = 0.0;
    for (int i = threadIdx.x; i < npartial; i += kThreads) acc += partial[i];
    const double sum = block_sum<kThreads>(acc, sh);
    if (threadIdx.x != 0) return;

    int b;
    if (fixed_b != 0) {
        b = fixed_b;
    } else {
        const double x = coef * sqrt(sum / (double)M);
        b = b_max;
        if (isfinite(x)) {
            for (int c = b_min; c <= b_max; ++c) {
                if ((double)((1 << (c - 1)) - 1) >= x) { b = c; break; }
            }
        } else {
            atomicOr(status, DQ_STAT_NONFINITE);
        }
    }
    dev_b[0] = b;
    dev_b[1] = (1 << (b - 1)) - 1;
}

inline int64_t num_chunks(int64_t n) { return (n + kChunk - 1) / kChunk; }

}  // namespace

extern "C" size_t dq_choose_bits_scratch_bytes(const dq_layout_t* L, int32_t M)
{
    if (!L || M < 1) return 0;
    const int64_t c = num_chunks((int64_t)M * L->nb);
    return (size_t)((c * sizeof(double) + 255) / 256 * 256);
}

namespace {

// Argument checks shared by the two entry points (everything but the scratch memory).
int check_rule_args(const dq_layout_t* L, const float* dev_norms, int32_t M, const dq_rule_t* rule, const int32_t* dev_b,
                    const int32_t* dev_status)
{
    if (!L || !rule) return DQ_ERR_ARG;
    if (M < 1) return DQ_ERR_ARG;
    if (M > DQ_MAX_WORKERS) return DQ_ERR_RANGE;
    if (!dev_norms || !dev_b || !dev_status) return DQ_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(dev_norms) & 3u) || (reinterpret_cast<uintptr_t>(dev_b) & 3u) ||
        (reinterpret_cast<uintptr_t>(dev_status) & 3u))
        return DQ_ERR_ALIGN;
    if (rule->fixed_b < 0 || rule->fixed_b > DQ_MAX_BITS) return DQ_ERR_RANGE;
    if (rule->b_min < 1 || rule->b_max > DQ_MAX_BITS || rule->b_min > rule->b_max) return DQ_ERR_RANGE;
    if (rule->fixed_b == 0 &&
        (rule->T < 1 || rule->t < 0 || rule->t >= rule->T || !(rule->eps_hat > 0.0) || !(rule->alpha > 0.0) ||
         !std::isfinite(rule->eps_hat) || !std::isfinite(rule->alpha)))
        return DQ_ERR_RANGE;
    return DQ_OK;
}

// The two kernels of the rule, with the chunk sums in `partial` (at least num_chunks(M * nb) doubles).
int launch_rule(const dq_layout_t* L, const float* dev_norms, int32_t M, const dq_rule_t* rule, int32_t* dev_b,
                double* partial, int32_t* dev_status, void* stream)
{
    const int64_t n = (int64_t)M * L->nb;
    const int64_t chunks = num_chunks(n);
    double coef = 0.0;
    if (rule->fixed_b == 0)
        coef = std::sqrt((double)rule->T / rule->eps_hat) *
               std::pow(rule->alpha, (double)(rule->T - 1 - rule->t) / 2.0);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (rule->fixed_b == 0) {
        dq_launch(norm_square_partials, dim3((unsigned)chunks), dim3(kSumThreads), 0, st, dev_norms, n, partial);
        if (cudaGetLastError() != cudaSuccess) return DQ_ERR_CUDA;
    }
    dq_launch(apply_rule, dim3(1), dim3(kThreads), 0, st, partial, rule->fixed_b == 0 ? (int)chunks : 0, M, coef,
              rule->b_min, rule->b_max, rule->fixed_b, dev_b, dev_status);
    if (cudaGetLastError() != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

}  // namespace

extern "C" int dq_choose_bits(const dq_layout_t* L, const float* dev_norms, int32_t M, const dq_rule_t* rule,
                              int32_t* dev_b, void* dev_scratch, size_t scratch_bytes,
                              int32_t* dev_status, void* stream)
{
    const int rc = check_rule_args(L, dev_norms, M, rule, dev_b, dev_status);
    if (rc != DQ_OK) return rc;
    if (!dev_scratch) return DQ_ERR_ARG;
    if (!aligned16(dev_scratch)) return DQ_ERR_ALIGN;
    if (scratch_bytes < dq_choose_bits_scratch_bytes(L, M)) return DQ_ERR_RANGE;
    return launch_rule(L, dev_norms, M, rule, dev_b, static_cast<double*>(dev_scratch), dev_status, stream);
}

// ---------------------------------------------------------------------------
// dq_choose_bits_noalloc: the same rule with the chunk sums kept in memory that
// belongs to the library image instead of memory the caller hands in.
//
// The array below is part of the loaded module: every GPU that loads the library
// holds these 64 KB from load until the process exits.  Its name is a device
// symbol; in host code the name is only a stand-in and not an address a kernel
// could use, so the address is asked for once per device with
// cudaGetSymbolAddress while that device is current, and the kernels get that.
namespace {

constexpr int kNoAllocMaxChunks = 8192;                        // 8192 doubles = 64 KB
static __device__ __align__(256) double g_noalloc_partials[kNoAllocMaxChunks];

constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mu;
double* g_noalloc_ptr[kMaxDevices] = {};

// Address of the array on the current device (looked up on the first call per device).
int noalloc_scratch(double** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return DQ_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_noalloc_mu);
    if (!g_noalloc_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_partials) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return DQ_ERR_CUDA;
        }
        g_noalloc_ptr[dev] = static_cast<double*>(p);
    }
    *out = g_noalloc_ptr[dev];
    return DQ_OK;
}

}  // namespace

extern "C" int64_t dq_choose_bits_noalloc_max_norms(void) { return (int64_t)kNoAllocMaxChunks * kChunk; }

extern "C" int dq_choose_bits_noalloc(const dq_layout_t* L, const float* dev_norms, int32_t M, const dq_rule_t* rule,
                                      int32_t* dev_b, int32_t* dev_status, void* stream)
{
    const int rc0 = check_rule_args(L, dev_norms, M, rule, dev_b, dev_status);
    if (rc0 != DQ_OK) return rc0;
    if (num_chunks((int64_t)M * L->nb) > kNoAllocMaxChunks) return DQ_ERR_TOO_LARGE;     // more norms than the built-in array covers

    double* partial = nullptr;
    const int rc = noalloc_scratch(&partial);
    if (rc != DQ_OK) return rc;
    // Nothing in the array has to start at zero: the first kernel writes every entry the
    // second one reads, so whatever an earlier call left behind is overwritten, never used.
    return launch_rule(L, dev_norms, M, rule, dev_b, partial, dev_status, stream);
}
