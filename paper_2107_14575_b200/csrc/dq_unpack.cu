// dq_unpack_dequant_average: the server's "Average" step of Algorithm 1 on
// packed codes: out_j = (1/M) sum_m sgn * level * norm_m / s  (Eq. 5 inverted).
//
// A thread owns one 32-element group and keeps its 32 fp32 sums in registers
// while it walks the M workers; each worker contributes b words per group.
// Decoding a code: one funnel shift brings it to the top of a register, the
// masked magnitude converts to fp32 as level * 2^(32-b) (that power of two is
// folded into the per-worker scale), the sign bit is OR-ed into the float, one
// FMA accumulates.  HBM traffic per output element: M*b/8 bytes read, 4 written.
#include "dq_common.cuh"
#include "dq_device.cuh"

namespace {

constexpr int kThreads = 128;

template <int B>
__device__ __forceinline__ void load_words(const uint32_t* __restrict__ src, uint32_t (&wd)[B])
{
    if (B % 4 == 0) {
#pragma unroll
        for (int i = 0; i < B / 4; ++i) {
            const uint4 t = __ldg(reinterpret_cast<const uint4*>(src) + i);
            wd[4 * i] = t.x; wd[4 * i + 1] = t.y; wd[4 * i + 2] = t.z; wd[4 * i + 3] = t.w;
        }
    } else if (B % 2 == 0) {
#pragma unroll
        for (int i = 0; i < B / 2; ++i) {
            const uint2 t = __ldg(reinterpret_cast<const uint2*>(src) + i);
            wd[2 * i] = t.x; wd[2 * i + 1] = t.y;
        }
    } else {
#pragma unroll
        for (int i = 0; i < B; ++i) wd[i] = __ldg(src + i);
    }
}

template <int B, int E>
__device__ __forceinline__ void accumulate_code(float (&acc)[32], const uint32_t (&wd)[B], const float scale)
{
    constexpr uint32_t kMag = ((1u << (B - 1)) - 1u) << (32 - B);
    const uint32_t x = top_code<B, E>(wd);
    const float mag = __uint2float_rn(x & kMag);                       // level * 2^(32-B), exact
    const float val = __uint_as_float(__float_as_uint(mag) | (x & 0x80000000u));
    acc[E] = fmaf(val, scale, acc[E]);
}

template <int B, int E>
struct AccumulateAll {
    static __device__ __forceinline__ void run(float (&acc)[32], const uint32_t (&wd)[B], const float scale)
    {
        accumulate_code<B, E>(acc, wd, scale);
        AccumulateAll<B, E + 1>::run(acc, wd, scale);
    }
};
template <int B>
struct AccumulateAll<B, 32> {
    static __device__ __forceinline__ void run(float (&)[32], const uint32_t (&)[B], const float) {}
};

template <int B>
__device__ __forceinline__ void average_groups(const LayoutView& v, const uint32_t* __restrict__ packed,
                                               const int64_t packed_stride, const float* __restrict__ norms,
                                               const int M, float* __restrict__ out)
{
    constexpr int s = (1 << (B - 1)) - 1;
    // 1 / (s * M) and the 2^-(32-B) that undoes the position of the magnitude bits
    const float unit = (B == 1) ? 0.0f
                                : __fdiv_rn(1.0f, (float)s * (float)M) * __uint_as_float((uint32_t)(127 - (32 - B)) << 23);
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < v.total_groups; g += nthreads) {
        int bucket, valid;
        group_info(v, (int)g, bucket, valid);
        float acc[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) acc[e] = 0.0f;
        if (B > 1) {
#pragma unroll 2
            for (int m = 0; m < M; ++m) {
                uint32_t wd[B];
                load_words<B>(packed + (int64_t)m * packed_stride + g * B, wd);
                const float scale = __ldg(norms + (int64_t)m * v.nb + bucket) * unit;
                AccumulateAll<B, 0>::run(acc, wd, scale);
            }
        }
        if (valid < 32) {
#pragma unroll
            for (int e = 0; e < 32; ++e)
                if (e >= valid) acc[e] = 0.0f;
        }
        float4* dst = reinterpret_cast<float4*>(out + g * 32);
#pragma unroll
        for (int c = 0; c < 8; ++c) dst[c] = make_float4(acc[4 * c], acc[4 * c + 1], acc[4 * c + 2], acc[4 * c + 3]);
    }
}

__global__ void __launch_bounds__(kThreads)
unpack_average_kernel(const LayoutView v, const uint32_t* __restrict__ packed, const int64_t packed_stride,
                      const float* __restrict__ norms, const int M, const int32_t* __restrict__ dev_b,
                      float* __restrict__ out, int32_t* __restrict__ status)
{
    const int b = __ldg(dev_b);
    if (b < 1 || b > DQ_MAX_BITS) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(status, DQ_STAT_BAD_BITS);
        return;
    }
    if ((int64_t)b * v.total_groups > packed_stride) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(status, DQ_STAT_CAPACITY);
        return;
    }
    switch (b) {
#define DQ_CASE(BB) case BB: average_groups<BB>(v, packed, packed_stride, norms, M, out); break;
        DQ_CASE(1) DQ_CASE(2) DQ_CASE(3) DQ_CASE(4) DQ_CASE(5) DQ_CASE(6) DQ_CASE(7) DQ_CASE(8)
        DQ_CASE(9) DQ_CASE(10) DQ_CASE(11) DQ_CASE(12) DQ_CASE(13) DQ_CASE(14) DQ_CASE(15) DQ_CASE(16)
#undef DQ_CASE
        default: break;
    }
}

}  // namespace

extern "C" int dq_unpack_dequant_average(const dq_layout_t* L, const uint32_t* dev_packed,
                                         int64_t packed_stride_words, const float* dev_norms, int32_t M,
                                         const int32_t* dev_b, float* dev_out, int32_t* dev_status, void* stream)
{
    const int rc = dq_check_common(L, M);
    if (rc != DQ_OK) return rc;
    if (!dev_packed || !dev_norms || !dev_b || !dev_out || !dev_status) return DQ_ERR_ARG;
    if (!aligned16(dev_packed) || !aligned16(dev_out) || (packed_stride_words % 4) != 0 ||
        (reinterpret_cast<uintptr_t>(dev_norms) & 3u) || (reinterpret_cast<uintptr_t>(dev_b) & 3u) ||
        (reinterpret_cast<uintptr_t>(dev_status) & 3u))
        return DQ_ERR_ALIGN;
    if (packed_stride_words < L->padded / 32) return DQ_ERR_RANGE;

    const LayoutView v = make_view(L);
    int64_t blocks = ((int64_t)v.total_groups + kThreads - 1) / kThreads;
    const int64_t cap = (int64_t)dq_sm_count() * 8;
    if (blocks > cap) blocks = cap;
    unpack_average_kernel<<<(unsigned)blocks, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        v, dev_packed, packed_stride_words, dev_norms, M, dev_b, dev_out, dev_status);
    if (cudaGetLastError() != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}
