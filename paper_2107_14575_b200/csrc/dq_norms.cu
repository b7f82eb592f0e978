// dq_bucket_norms: per-bucket l2 norm of every worker's gradient (the scale
// factor ||g||_p of Eq. 5 with p = 2, applied per bucket).
//
// One team of LANES threads (8, 16 or a full warp, by bucket size) owns a
// bucket: 128-bit coalesced loads, four independent fp32 accumulators per
// lane, a shuffle reduction inside the team.  Teams walk the (worker, bucket)
// list with a grid stride, so neighbouring teams read neighbouring memory.
// HBM-bound: 4 bytes read per element, 4/bucket bytes written.
#include "dq_common.cuh"

namespace {

constexpr int kThreads = 256;

template <int LANES>
__global__ void __launch_bounds__(kThreads)
bucket_norms_kernel(const LayoutView v, const float* __restrict__ grads, const int64_t worker_stride,
                    const int M, float* __restrict__ norms, int32_t* __restrict__ status)
{
    constexpr int kTeams = kThreads / LANES;
    const int lane = threadIdx.x % LANES;
    const int64_t total = (int64_t)M * v.nb;
    const int64_t nteams = (int64_t)gridDim.x * kTeams;
    bool bad = false;

    // The loop bound is the same for every lane of a warp (teams of one warp
    // take consecutive buckets), so the full-mask shuffles below are safe; a
    // team past the end runs with an empty bucket.
    constexpr int kTeamsPerWarp = 32 / LANES;
    int64_t w0 = (int64_t)blockIdx.x * kTeams + (threadIdx.x / 32) * kTeamsPerWarp;
    for (; w0 < total; w0 += nteams) {
        const int64_t w = w0 + (threadIdx.x % 32) / LANES;
        const bool active = w < total;
        const int m = active ? (int)(w / v.nb) : 0;
        const int k = active ? (int)(w - (int64_t)m * v.nb) : 0;
        int64_t start;
        int len;
        bucket_info(v, k, start, len);
        if (!active) len = 0;
        const float* g = grads + (int64_t)m * worker_stride + start;   // 128-byte aligned
        const float4* g4 = reinterpret_cast<const float4*>(g);
        const int n4 = len >> 2;

        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        int i = lane;
#pragma unroll 1
        for (; i + 3 * LANES < n4; i += 4 * LANES) {
            const float4 x0 = __ldg(g4 + i);
            const float4 x1 = __ldg(g4 + i + LANES);
            const float4 x2 = __ldg(g4 + i + 2 * LANES);
            const float4 x3 = __ldg(g4 + i + 3 * LANES);
            a0 = fmaf(x0.x, x0.x, a0); a1 = fmaf(x0.y, x0.y, a1); a2 = fmaf(x0.z, x0.z, a2); a3 = fmaf(x0.w, x0.w, a3);
            a0 = fmaf(x1.x, x1.x, a0); a1 = fmaf(x1.y, x1.y, a1); a2 = fmaf(x1.z, x1.z, a2); a3 = fmaf(x1.w, x1.w, a3);
            a0 = fmaf(x2.x, x2.x, a0); a1 = fmaf(x2.y, x2.y, a1); a2 = fmaf(x2.z, x2.z, a2); a3 = fmaf(x2.w, x2.w, a3);
            a0 = fmaf(x3.x, x3.x, a0); a1 = fmaf(x3.y, x3.y, a1); a2 = fmaf(x3.z, x3.z, a2); a3 = fmaf(x3.w, x3.w, a3);
        }
        for (; i < n4; i += LANES) {
            const float4 x = __ldg(g4 + i);
            a0 = fmaf(x.x, x.x, a0); a1 = fmaf(x.y, x.y, a1); a2 = fmaf(x.z, x.z, a2); a3 = fmaf(x.w, x.w, a3);
        }
        if (lane < (len & 3)) {                       // ragged tail of the tensor's last bucket
            const float x = __ldg(g + n4 * 4 + lane);
            a0 = fmaf(x, x, a0);
        }
        float sum = (a0 + a1) + (a2 + a3);
#pragma unroll
        for (int o = LANES / 2; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o, LANES);
        if (lane == 0 && active) {
            const float nrm = sqrtf(sum);
            norms[w] = nrm;
            bad |= !isfinite(nrm);
        }
    }
    if (bad) atomicOr(status, DQ_STAT_NONFINITE);
}

}  // namespace

extern "C" int dq_bucket_norms(const dq_layout_t* L, const float* dev_grads, int64_t worker_stride_elems,
                               int32_t M, float* dev_norms, int32_t* dev_status, void* stream)
{
    const int rc = dq_check_common(L, M);
    if (rc != DQ_OK) return rc;
    if (!dev_grads || !dev_norms || !dev_status) return DQ_ERR_ARG;
    if (!aligned16(dev_grads) || (worker_stride_elems % 32) != 0 || (reinterpret_cast<uintptr_t>(dev_norms) & 3u) ||
        (reinterpret_cast<uintptr_t>(dev_status) & 3u))
        return DQ_ERR_ALIGN;
    if (M > 1 && worker_stride_elems < L->padded && worker_stride_elems != 0) return DQ_ERR_RANGE;

    const LayoutView v = make_view(L);
    const int64_t total = (int64_t)M * L->nb;
    const int lanes = L->bucket >= 128 ? 32 : (L->bucket >= 64 ? 16 : 8);
    const int teams = kThreads / lanes;
    int64_t blocks = (total + teams - 1) / teams;
    const int64_t cap = (int64_t)dq_sm_count() * 8;     // 8 resident CTAs of 256 threads per SM
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (lanes == 32)
        bucket_norms_kernel<32><<<(unsigned)blocks, kThreads, 0, st>>>(v, dev_grads, worker_stride_elems, M, dev_norms, dev_status);
    else if (lanes == 16)
        bucket_norms_kernel<16><<<(unsigned)blocks, kThreads, 0, st>>>(v, dev_grads, worker_stride_elems, M, dev_norms, dev_status);
    else
        bucket_norms_kernel<8><<<(unsigned)blocks, kThreads, 0, st>>>(v, dev_grads, worker_stride_elems, M, dev_norms, dev_status);
    if (cudaGetLastError() != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}
