// dq_unpack_dequant_average: the server's "Average" step of Algorithm 1 on
// packed codes: out_j = (1/M) sum_m sgn * level * norm_m / s  (Eq. 5 inverted).
//
// Persistent CTAs walk tiles of 128 groups (one group = 32 padded elements = one
// thread, which keeps its 32 fp32 sums in registers).  The M workers' words of
// a tile are fetched in chunks of a few workers by linear bulk copies (TMA) into
// a ring of shared-memory stages, so the copies of the next chunks overlap the
// decoding of the current one.  A code is decoded where it stands in its word
// (mask under the exponent of 2^23, subtract 2^23, OR the sign in: see
// decode_code) and accumulated with one FMA; the power of two its position
// carries is removed once per element after the last worker.  Each thread
// stores its 32 results as eight 16-byte pieces of its own 128-byte line.
// HBM traffic per output element: M*b/8 bytes read, 4 written.
#include "dq_common.cuh"
#include "dq_device.cuh"
#include "dq_tma.cuh"

namespace {

constexpr int kThreads = 128;                 // groups per tile
constexpr int kStages = 2;
constexpr int kStageWords = 4096;             // 16 KB per stage
constexpr int kMaxSmemSegs = 1023;

struct AverageArgs {
    LayoutView v;
    const uint32_t* packed;
    int64_t packed_stride;
    const float* norms;
    const int32_t* dev_b;
    float* out;
    int32_t* status;
    int32_t M;
    uint32_t div_magic;
    int32_t div_shift;
};

__device__ __forceinline__ uint32_t div_gpb(const AverageArgs& a, uint32_t n)
{
    if (a.div_shift >= 0) return n >> a.div_shift;
    return (uint32_t)(((uint64_t)n * a.div_magic) >> 33);     // exact for n < 2^26, divisor <= 128
}

// workers per stage: as many as fit 16 KB with 128 groups of B words each, at most 8
// (their scales sit in registers while the chunk is decoded)
template <int B>
struct ChunkOf {
    static constexpr int fit = kStageWords / (kThreads * B);
    static constexpr int value = fit < 1 ? 1 : (fit > 8 ? 8 : fit);
};

template <int B>
__device__ __forceinline__ void load_words(const uint32_t* __restrict__ src, uint32_t (&wd)[B])
{
    if constexpr (B % 4 == 0) {
#pragma unroll
        for (int i = 0; i < B / 4; ++i) {
            const uint4 t = reinterpret_cast<const uint4*>(src)[i];
            wd[4 * i] = t.x; wd[4 * i + 1] = t.y; wd[4 * i + 2] = t.z; wd[4 * i + 3] = t.w;
        }
    } else if constexpr (B % 2 == 0) {
#pragma unroll
        for (int i = 0; i < B / 2; ++i) {
            const uint2 t = reinterpret_cast<const uint2*>(src)[i];
            wd[2 * i] = t.x; wd[2 * i + 1] = t.y;
        }
    } else {
#pragma unroll
        for (int i = 0; i < B; ++i) wd[i] = src[i];
    }
}

template <int B, int E>
struct AccumulateAll {
    static __device__ __forceinline__ void run(float (&acc)[32], const uint32_t (&wd)[B], const uint32_t (&hi)[B],
                                               const float scale)
    {
        acc[E] = fmaf(decode_code<B, E>(wd, hi), scale, acc[E]);
        AccumulateAll<B, E + 1>::run(acc, wd, hi, scale);
    }
};
template <int B>
struct AccumulateAll<B, 32> {
    static __device__ __forceinline__ void run(float (&)[32], const uint32_t (&)[B], const uint32_t (&)[B], const float) {}
};

template <int B, int W>
struct UpperHalves {
    static __device__ __forceinline__ void run(const uint32_t (&wd)[B], uint32_t (&hi)[B])
    {
        if constexpr (NeedsUpper<B, W>::value) hi[W] = wd[W] >> 16;
        else hi[W] = 0u;
        UpperHalves<B, W + 1>::run(wd, hi);
    }
};
template <int B>
struct UpperHalves<B, B> {
    static __device__ __forceinline__ void run(const uint32_t (&)[B], uint32_t (&)[B]) {}
};

// removes the power of two each element's decoded magnitude carried
template <int B, int E>
struct Normalise {
    static __device__ __forceinline__ void run(float (&acc)[32])
    {
        constexpr int k = CodePos<B, E>::k;
        if constexpr (k != 0) acc[E] *= __uint_as_float((uint32_t)(127 - k) << 23);
        Normalise<B, E + 1>::run(acc);
    }
};
template <int B>
struct Normalise<B, 32> {
    static __device__ __forceinline__ void run(float (&)[32]) {}
};

// Issues the bulk copies of one pipeline unit: workers [m0, m0 + mc) of the tile at row0.
template <int B>
__device__ __forceinline__ void issue_unit(const AverageArgs& a, uint32_t* stage, uint64_t* bar, int row0, int m0, int mc)
{
    int rows = a.v.total_groups - row0;
    rows = rows > kThreads ? kThreads : rows;
    const uint32_t bytes = ((uint32_t)(rows * B * 4) + 15u) & ~15u;   // the stream's stride is a multiple of 16 bytes
    tma::mbar_expect_tx(bar, bytes * (uint32_t)mc);
    for (int j = 0; j < mc; ++j)
        tma::load_bulk(stage + j * (kThreads * B), a.packed + (int64_t)(m0 + j) * a.packed_stride + (int64_t)row0 * B,
                       bytes, bar);
}

template <int B>
__device__ __forceinline__ void average_tiles(const AverageArgs& a, uint32_t* stages, float* scales,
                                              uint64_t* full, const int32_t* tbl)
{
    constexpr int s = (1 << (B - 1)) - 1;
    constexpr int MC = ChunkOf<B>::value;
    const int tid = threadIdx.x;
    const int G = a.v.total_groups;
    const int M = a.M;
    const int total_tiles = (G + kThreads - 1) / kThreads;
    const int nchunk = (M + MC - 1) / MC;
    const int n1 = a.v.n_seg + 1;
    const float unit = (B == 1) ? 0.0f : __fdiv_rn(1.0f, (float)s * (float)M);      // 1 / (s * M)
    float* my_scales = scales + tid;              // column tid of a [kMaxChunk][kThreads] array

    // number of pipeline units this CTA will consume, and the prologue that fills the ring
    const int my_tiles = (total_tiles > (int)blockIdx.x) ? (total_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int my_units = (B == 1) ? 0 : my_tiles * nchunk;
    if (tid == 0) {
        for (int u = 0; u < kStages && u < my_units; ++u) {
            const int tile = blockIdx.x + (u / nchunk) * gridDim.x;
            const int m0 = (u % nchunk) * MC;
            issue_unit<B>(a, stages + u * kStageWords, &full[u], tile * kThreads, m0, (M - m0) < MC ? (M - m0) : MC);
        }
    }

    int seg = 0;
    int u = 0;                                    // pipeline unit counter
    bool timed_out = false;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        const int row0 = tile * kThreads;
        const int g = row0 + tid;
        const bool active = g < G;
        int bucket = 0, valid = 32;
        if (active) {
            int local, n, b0;
            if (a.v.n_seg == 1) {
                local = g; n = a.v.seg0_elems; b0 = 0;
            } else {
                while (g >= tbl[seg + 1]) ++seg;
                local = g - tbl[seg];
                b0 = tbl[n1 + seg];
                n = tbl[2 * n1 + seg];
            }
            bucket = b0 + (int)div_gpb(a, (uint32_t)local);
            const int left = n - local * 32;
            valid = left < 32 ? left : 32;
        }
        float acc[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) acc[e] = 0.0f;

        if constexpr (B > 1) {
            for (int c = 0; c < nchunk; ++c, ++u) {
                const int m0 = c * MC;
                const int mc = (M - m0) < MC ? (M - m0) : MC;
                // this thread's per-worker scales of the chunk, parked in its shared-memory column
                const float* nrm = a.norms + (int64_t)m0 * a.v.nb + bucket;
                for (int j = 0; j < mc; ++j)
                    my_scales[j * kThreads] = active ? __ldg(nrm + (int64_t)j * a.v.nb) * unit : 0.0f;

                const int st = u % kStages;
                if (!tma::mbar_wait(&full[st], (u / kStages) & 1)) { timed_out = true; break; }
                const uint32_t* base = stages + st * kStageWords + tid * B;
#pragma unroll 2
                for (int j = 0; j < mc; ++j) {
                    uint32_t wd[B], hi[B];
                    load_words<B>(base + j * (kThreads * B), wd);
                    UpperHalves<B, 0>::run(wd, hi);
                    AccumulateAll<B, 0>::run(acc, wd, hi, my_scales[j * kThreads]);
                }
                __syncthreads();                  // the stage is free again
                if (tid == 0) {
                    const int nu = u + kStages;
                    if (nu < my_units) {
                        tma::fence_proxy_async();
                        const int ntile = blockIdx.x + (nu / nchunk) * gridDim.x;
                        const int nm0 = (nu % nchunk) * MC;
                        issue_unit<B>(a, stages + st * kStageWords, &full[st], ntile * kThreads, nm0,
                                      (M - nm0) < MC ? (M - nm0) : MC);
                    }
                }
            }
            if (timed_out) break;
            Normalise<B, 0>::run(acc);
        }

        if (valid < 32) {
#pragma unroll
            for (int e = 0; e < 32; ++e)
                if (e >= valid) acc[e] = 0.0f;
        }
        if (active) {
            float4* dst = reinterpret_cast<float4*>(a.out + (int64_t)g * 32);
#pragma unroll
            for (int c = 0; c < 8; ++c)
                dst[c] = make_float4(acc[4 * c], acc[4 * c + 1], acc[4 * c + 2], acc[4 * c + 3]);
        }
    }

    if (timed_out) {
        if (tid == 0) atomicOr(a.status, DQ_STAT_WAIT);
        for (int k = 1; k < kStages; ++k)
            if (u + k < my_units) (void)tma::mbar_wait(&full[(u + k) % kStages], ((u + k) / kStages) & 1);
    }
}

__global__ void __launch_bounds__(kThreads, 5)
unpack_average_kernel(const __grid_constant__ AverageArgs a)
{
    extern __shared__ unsigned char smem_raw[];
    // [stages: kStages * 16 KB][scales: 8 * 128 floats][barriers][table]
    unsigned char* p = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    uint32_t* stages = reinterpret_cast<uint32_t*>(p);
    float* scales = reinterpret_cast<float*>(p + kStages * kStageWords * 4);
    uint64_t* full = reinterpret_cast<uint64_t*>(scales + 8 * kThreads);
    int32_t* tbl_s = reinterpret_cast<int32_t*>(full + kStages);

    const int b = __ldg(a.dev_b);
    if (b < 1 || b > DQ_MAX_BITS) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(a.status, DQ_STAT_BAD_BITS);
        return;
    }
    if ((int64_t)b * a.v.total_groups > a.packed_stride) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(a.status, DQ_STAT_CAPACITY);
        return;
    }
    const int32_t* tbl = a.v.seg_group0;
    if (a.v.n_seg > 1 && a.v.n_seg <= kMaxSmemSegs) {
        for (int i = threadIdx.x; i < 3 * (a.v.n_seg + 1); i += kThreads) tbl_s[i] = __ldg(a.v.seg_group0 + i);
        tbl = tbl_s;
    }
    if (threadIdx.x == 0) {
#pragma unroll
        for (int st = 0; st < kStages; ++st) tma::mbar_init(&full[st], 1);
        tma::fence_barrier_init();
    }
    __syncthreads();

    switch (b) {
#define DQ_CASE(BB) case BB: average_tiles<BB>(a, stages, scales, full, tbl); break;
        DQ_CASE(1) DQ_CASE(2) DQ_CASE(3) DQ_CASE(4) DQ_CASE(5) DQ_CASE(6) DQ_CASE(7) DQ_CASE(8)
        DQ_CASE(9) DQ_CASE(10) DQ_CASE(11) DQ_CASE(12) DQ_CASE(13) DQ_CASE(14) DQ_CASE(15) DQ_CASE(16)
#undef DQ_CASE
        default: break;
    }
}

size_t smem_bytes(int n_seg)
{
    size_t n = 128 + (size_t)kStages * kStageWords * 4 + (size_t)8 * kThreads * 4 + kStages * 8;
    if (n_seg > 1 && n_seg <= kMaxSmemSegs) n += (size_t)3 * (n_seg + 1) * 4;
    return n;
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

    AverageArgs a;
    a.v = make_view(L);
    a.packed = dev_packed;
    a.packed_stride = packed_stride_words;
    a.norms = dev_norms;
    a.dev_b = dev_b;
    a.out = dev_out;
    a.status = dev_status;
    a.M = M;
    const uint32_t gpb = (uint32_t)a.v.groups_per_bucket;
    if ((gpb & (gpb - 1)) == 0) {
        a.div_shift = 0;
        while ((1u << a.div_shift) < gpb) ++a.div_shift;
        a.div_magic = 0;
    } else {
        a.div_shift = -1;
        a.div_magic = (uint32_t)(((uint64_t(1) << 33) + gpb - 1) / gpb);
    }

    const size_t smem = smem_bytes(L->n_seg);
    if (cudaFuncSetAttribute(unpack_average_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return DQ_ERR_CUDA;
    }
    const int64_t tiles = ((int64_t)a.v.total_groups + kThreads - 1) / kThreads;
    int64_t blocks = (int64_t)dq_sm_count() * 5;       // five 37 KB CTAs per SM
    if (blocks > tiles) blocks = tiles;
    unpack_average_kernel<<<(unsigned)blocks, kThreads, smem, static_cast<cudaStream_t>(stream)>>>(a);
    if (cudaGetLastError() != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}
