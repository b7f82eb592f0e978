// dq_quantize_pack: the EWU quantizer of Eq. 5/6 fused with the b-bit packer.
//
// A thread owns one 32-element group: it reads the group's 128 bytes, draws the
// eight Philox blocks that cover it, encodes the 32 codes and assembles the
// group's b words in registers (all shifts are constants once b is known), so
// no code ever leaves the register file before it is packed.  b is read from
// device memory and selects one of sixteen specialisations with a
// grid-uniform switch; nothing on the host depends on b.
// HBM traffic: 4 bytes read and b/8 bytes written per element.
#include "dq_common.cuh"
#include "dq_device.cuh"

namespace {

constexpr int kThreads = 128;

template <int B>
__device__ __forceinline__ void store_words(uint32_t* __restrict__ dst, const uint32_t (&acc)[B])
{
    if (B % 4 == 0) {
#pragma unroll
        for (int i = 0; i < B / 4; ++i)
            reinterpret_cast<uint4*>(dst)[i] = make_uint4(acc[4 * i], acc[4 * i + 1], acc[4 * i + 2], acc[4 * i + 3]);
    } else if (B % 2 == 0) {
#pragma unroll
        for (int i = 0; i < B / 2; ++i)
            reinterpret_cast<uint2*>(dst)[i] = make_uint2(acc[2 * i], acc[2 * i + 1]);
    } else {
#pragma unroll
        for (int i = 0; i < B; ++i) dst[i] = acc[i];
    }
}

// Encodes chunk C (elements 4C..4C+3) of a group and ORs the codes into acc.
template <int B, int C>
__device__ __forceinline__ void encode_chunk(uint32_t (&acc)[B], const float4 x, const float inv, const float sf,
                                             const uint32_t q, const uint32_t m, const uint32_t step,
                                             const PhiloxKeys& keys)
{
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    if (B > 1) philox4x32_10(q, 0u, m, step, keys, w);
    put_code<B, 4 * C + 0>(acc, encode<B>(x.x, inv, sf, w[0]));
    put_code<B, 4 * C + 1>(acc, encode<B>(x.y, inv, sf, w[1]));
    put_code<B, 4 * C + 2>(acc, encode<B>(x.z, inv, sf, w[2]));
    put_code<B, 4 * C + 3>(acc, encode<B>(x.w, inv, sf, w[3]));
}

template <int B>
__device__ __forceinline__ void quantize_groups(const LayoutView& v, const float* __restrict__ grads,
                                                const int64_t worker_stride, const int M,
                                                const float* __restrict__ norms, const PhiloxKeys& keys,
                                                const uint32_t step, uint32_t* __restrict__ packed,
                                                const int64_t packed_stride)
{
    constexpr int s = (1 << (B - 1)) - 1;
    const float sf = (float)s;
    const int64_t total = (int64_t)M * v.total_groups;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += nthreads) {
        const int m = (int)(idx / v.total_groups);
        const int g = (int)(idx - (int64_t)m * v.total_groups);
        int bucket, valid;
        group_info(v, g, bucket, valid);
        const float4* row = reinterpret_cast<const float4*>(grads + (int64_t)m * worker_stride + (int64_t)g * 32);
        float4 x[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) x[c] = __ldg(row + c);
        const float norm = __ldg(norms + (int64_t)m * v.nb + bucket);
        const float inv = (norm >= 0x1p-100f) ? __fdiv_rn(sf, norm) : 0.0f;
        if (valid < 32) {                      // padding after a tensor's end encodes as +0
            float* xe = reinterpret_cast<float*>(x);
#pragma unroll
            for (int e = 0; e < 32; ++e)
                if (e >= valid) xe[e] = 0.0f;
        }
        uint32_t acc[B];
        const uint32_t q0 = (uint32_t)g * 8u;
        encode_chunk<B, 0>(acc, x[0], inv, sf, q0 + 0, m, step, keys);
        encode_chunk<B, 1>(acc, x[1], inv, sf, q0 + 1, m, step, keys);
        encode_chunk<B, 2>(acc, x[2], inv, sf, q0 + 2, m, step, keys);
        encode_chunk<B, 3>(acc, x[3], inv, sf, q0 + 3, m, step, keys);
        encode_chunk<B, 4>(acc, x[4], inv, sf, q0 + 4, m, step, keys);
        encode_chunk<B, 5>(acc, x[5], inv, sf, q0 + 5, m, step, keys);
        encode_chunk<B, 6>(acc, x[6], inv, sf, q0 + 6, m, step, keys);
        encode_chunk<B, 7>(acc, x[7], inv, sf, q0 + 7, m, step, keys);
        store_words<B>(packed + (int64_t)m * packed_stride + (int64_t)g * B, acc);
    }
}

__global__ void __launch_bounds__(kThreads)
quantize_pack_kernel(const LayoutView v, const float* __restrict__ grads, const int64_t worker_stride, const int M,
                     const float* __restrict__ norms, const int32_t* __restrict__ dev_b,
                     const __grid_constant__ PhiloxKeys keys, const uint32_t step,
                     uint32_t* __restrict__ packed, const int64_t packed_stride, int32_t* __restrict__ status)
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
#define DQ_CASE(BB) case BB: quantize_groups<BB>(v, grads, worker_stride, M, norms, keys, step, packed, packed_stride); break;
        DQ_CASE(1) DQ_CASE(2) DQ_CASE(3) DQ_CASE(4) DQ_CASE(5) DQ_CASE(6) DQ_CASE(7) DQ_CASE(8)
        DQ_CASE(9) DQ_CASE(10) DQ_CASE(11) DQ_CASE(12) DQ_CASE(13) DQ_CASE(14) DQ_CASE(15) DQ_CASE(16)
#undef DQ_CASE
        default: break;
    }
}

}  // namespace

extern "C" int dq_quantize_pack(const dq_layout_t* L, const float* dev_grads, int64_t worker_stride_elems,
                                int32_t M, const float* dev_norms, const int32_t* dev_b,
                                uint64_t seed, uint32_t step,
                                uint32_t* dev_packed, int64_t packed_stride_words,
                                int32_t* dev_status, void* stream)
{
    const int rc = dq_check_common(L, M);
    if (rc != DQ_OK) return rc;
    if (!dev_grads || !dev_norms || !dev_b || !dev_packed || !dev_status) return DQ_ERR_ARG;
    if (!aligned16(dev_grads) || !aligned16(dev_packed) || (worker_stride_elems % 32) != 0 ||
        (packed_stride_words % 4) != 0 || (reinterpret_cast<uintptr_t>(dev_norms) & 3u) ||
        (reinterpret_cast<uintptr_t>(dev_b) & 3u) || (reinterpret_cast<uintptr_t>(dev_status) & 3u))
        return DQ_ERR_ALIGN;
    if (M > 1 && worker_stride_elems < L->padded && worker_stride_elems != 0) return DQ_ERR_RANGE;
    if (packed_stride_words < L->padded / 32) return DQ_ERR_RANGE;   // not even b = 1 fits

    const LayoutView v = make_view(L);
    const PhiloxKeys keys = make_philox_keys(seed);
    const int64_t total = (int64_t)M * v.total_groups;
    int64_t blocks = (total + kThreads - 1) / kThreads;
    const int64_t cap = (int64_t)dq_sm_count() * 8;
    if (blocks > cap) blocks = cap;
    quantize_pack_kernel<<<(unsigned)blocks, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        v, dev_grads, worker_stride_elems, M, dev_norms, dev_b, keys, step, dev_packed, packed_stride_words,
        dev_status);
    if (cudaGetLastError() != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}
