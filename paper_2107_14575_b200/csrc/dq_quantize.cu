// dq_quantize_pack: the EWU quantizer of Eq. 5/6 fused with the b-bit packer.
//
// Every warp is an independent pipeline over a contiguous range of warp tiles
// (32 groups; one group = 32 consecutive padded elements = one thread).  A warp
// tile's 4 KB of gradients arrive by one TMA tensor copy into the warp's own
// ring of shared-memory stages written with the 128-byte swizzle, so that a
// thread reading its own 128-byte row in 16-byte pieces hits every bank group
// once per quarter warp.  The thread draws the four Philox blocks of its group
// (16 random bits per element), encodes the 32 codes and assembles the group's
// b words in a register shift chain (all shifts are constants once b is
// known).  The warp then transposes its 32*b words through the stage it has just
// consumed and writes them with 16-byte coalesced stores, and one lane refills
// the stage.  Warps never wait for each other: there is no CTA barrier in the
// loop.  b is read from device memory and selects one of sixteen
// specialisations with a grid-uniform switch.
// HBM traffic: 4 bytes read and b/8 bytes written per element.
#include "dq_common.cuh"
#include "dq_device.cuh"
#include "dq_tma.cuh"

namespace {

constexpr int kThreads = 128;
constexpr int kWarps = kThreads / 32;
constexpr int kStages = 2;                  // per warp
constexpr int kTileBytes = 32 * 128;        // 4 KB of fp32 per warp tile
constexpr int kMaxSmemSegs = 1023;          // layouts with more tensors read the table from global memory

// Dynamic shared memory, addressed only through this symbol so that every access
// compiles to a shared-memory instruction:
//   [0, kWarps * kStages * 4 KB)   input tiles, warp-major (each 1024-byte aligned for the swizzle)
//   then the stage barriers and the tensor table
extern __shared__ __align__(1024) unsigned char smem[];
constexpr int kBarOffset = kWarps * kStages * kTileBytes;
constexpr int kTblOffset = kBarOffset + kWarps * kStages * 8;

__device__ __forceinline__ uint64_t* full_bar(int warp, int st)
{
    return reinterpret_cast<uint64_t*>(smem + kBarOffset) + warp * kStages + st;
}
__device__ __forceinline__ unsigned char* stage_ptr(int warp, int st)
{
    return smem + (warp * kStages + st) * kTileBytes;
}

struct QuantizeArgs {
    LayoutView v;
    const float* norms;
    const int32_t* dev_b;
    uint32_t* packed;
    int64_t packed_stride;
    int32_t* status;
    PhiloxKeys keys;
    uint32_t step;
    uint32_t worker0;             // worker m of the call draws the uniforms of worker worker0 + m
    int32_t M;
    int32_t map_has_worker_dim;   // 0 when all workers read the same buffer (stride 0)
    uint32_t div_magic;           // groups_per_bucket: division by multiply-shift, or by shift if a power of two
    int32_t div_shift;            // >= 0: power of two, shift; < 0: use div_magic with a 33-bit shift
    int32_t stream_reads;         // 1: the gradients exceed the L2, read them with the evict-first policy
    uint32_t one_bits;            // 0x3F800040 = bits of 1 + 2^-17, kept out of the compiler's sight (see and_or)
    WaitLimits wait;
};

__device__ __forceinline__ uint32_t div_gpb(const QuantizeArgs& a, uint32_t n)
{
    if (a.div_shift >= 0) return n >> a.div_shift;
    return (uint32_t)(((uint64_t)n * a.div_magic) >> 33);     // exact for n < 2^26, divisor <= 128
}

// A norm load that stays where it is written (a volatile statement keeps its place among the other
// volatile statements, the barrier wait among them): the norm of the warp's next tile is requested
// before this tile's wait and encoding, not after them.
__device__ __forceinline__ float load_norm_early(const float* p)
{
    float x;
    asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(x) : "l"(p));
    return x;
}

template <int B>
__device__ __forceinline__ void quantize_tiles(const QuantizeArgs& a, const CUtensorMap* map, const bool tbl_in_smem)
{
    const int32_t* tbl_s = reinterpret_cast<const int32_t*>(smem + kTblOffset);
    auto tbl = [&](int i) -> int { return tbl_in_smem ? tbl_s[i] : __ldg(a.v.seg_group0 + i); };
    constexpr int s = (1 << (B - 1)) - 1;
    const float sf = (float)s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int G = a.v.total_groups;
    const int tiles_per_worker = (G + 31) / 32;
    const int64_t total_tiles = (int64_t)a.M * tiles_per_worker;
    const int n1 = a.v.n_seg + 1;

    // Warp tiles are numbered worker-major and every warp takes one contiguous range of them,
    // so the walk through the tensor table below advances by at most a few entries per tile.
    // (m, rt) = worker and tile-within-worker of the tile being consumed, (pm, prt) of the
    // next tile to prefetch.
    const int64_t nwarps = (int64_t)gridDim.x * kWarps;
    const int64_t gw = (int64_t)blockIdx.x * kWarps + warp;
    const int64_t tile_begin = gw * total_tiles / nwarps;
    const int64_t tile_end = (gw + 1) * total_tiles / nwarps;
    int m = (int)(tile_begin / tiles_per_worker), rt = (int)(tile_begin - (int64_t)m * tiles_per_worker);
    int pm = m, prt = rt;
    int64_t ptile = tile_begin;
    auto advance = [&](int& mm, int& rr) {
        if (++rr == tiles_per_worker) { rr = 0; ++mm; }
    };
    const uint64_t policy = tma::policy_evict_first();
    auto fetch = [&](int st) {
        tma::mbar_expect_tx(full_bar(warp, st), kTileBytes);
        if (a.stream_reads)
            tma::load_tile_3d_hint(stage_ptr(warp, st), map, full_bar(warp, st), 0, prt * 32, a.map_has_worker_dim ? pm : 0, policy);
        else
            tma::load_tile_3d(stage_ptr(warp, st), map, full_bar(warp, st), 0, prt * 32, a.map_has_worker_dim ? pm : 0);
    };

    // prologue: fill the warp's ring
#pragma unroll
    for (int st = 0; st < kStages; ++st) {
        if (ptile < tile_end && lane == 0) fetch(st);
        ++ptile;
        advance(pm, prt);
    }

    int seg = 0, seg_m = -1;
    // Valid elements and bucket norm of this lane's group in tile (mm, rr); the norm is only requested
    // here.  Groups beyond the layout (the last tile's tail) encode zeros that are never stored.
    auto prepare = [&](int mm, int rr, int& valid_o, float& norm_o) {
        const int g = rr * 32 + lane;
        int bucket = 0;
        valid_o = 32;
        norm_o = 0.0f;
        if (g < G) {
            int local, n, b0;
            if (a.v.n_seg == 1) {
                local = g; n = a.v.seg0_elems; b0 = 0;
            } else {
                if (mm != seg_m) { seg = 0; seg_m = mm; }
                while (g >= tbl(seg + 1)) ++seg;                 // groups only move forward within a worker
                local = g - tbl(seg);
                b0 = tbl(n1 + seg);
                n = tbl(2 * n1 + seg);
            }
            bucket = b0 + (int)div_gpb(a, (uint32_t)local);
            const int left = n - local * 32;
            valid_o = left < 32 ? left : 32;
            norm_o = load_norm_early(a.norms + (int64_t)mm * a.v.nb + bucket);
        }
    };
    int next_valid = 32;
    float next_norm = 0.0f;
    if (tile_begin < tile_end) prepare(m, rt, next_valid, next_norm);
    int it = 0;
    // test hook: the warp's first wait counts as lost, and the warp goes straight to what follows a time-out
    bool timed_out = a.wait.lose_first != 0u && tile_begin < tile_end;
    for (int64_t tile = tile_begin; tile < tile_end && !timed_out; ++tile, ++it, advance(m, rt)) {
        const int st = it % kStages;
        const uint32_t parity = (it / kStages) & 1;
        const int row0 = rt * 32;
        const int g = row0 + lane;
        const int valid = next_valid;
        const float norm = next_norm;
        if (tile + 1 < tile_end) {              // the next tile's norm travels while this tile is encoded
            int m2 = m, rt2 = rt;
            advance(m2, rt2);
            prepare(m2, rt2, next_valid, next_norm);
        }
        const float inv = inv_scale(sf, norm);

        // every lane polls the barrier itself; the verdict is made warp-uniform so that the
        // warp-level synchronisations below are always reached by all lanes or by none
        if (!__all_sync(0xffffffffu, tma::mbar_wait(full_bar(warp, st), parity, a.wait))) {
            timed_out = true;
            break;
        }

        unsigned char* tile_base = stage_ptr(warp, st);
        unsigned char* row = tile_base + lane * 128;
        if (valid < 32) {                       // padding after a tensor's end encodes as 0
            for (int e = valid; e < 32; ++e)
                *reinterpret_cast<float*>(row + ((((e >> 2) ^ (lane & 7)) << 4) | ((e & 3) << 2))) = 0.0f;
        }
        uint32_t acc[B];
        if constexpr (B == 1) {
            acc[0] = 0u;                        // s = 0: every code is 0
        } else if (__all_sync(0xffffffffu, inv == 0.0f)) {
            zero_group_words<B>(acc);           // a tile of zero buckets: every code is s, whatever the draw
        } else {
            uint32_t cur = 0;
            const uint32_t q0 = (uint32_t)g * 4u;
            const uint32_t sw = (uint32_t)(lane & 7);
#define DQ_BLOCK(C)                                                                                             \
            encode_block<B, C>(acc, cur,                                                                        \
                               *reinterpret_cast<const float4*>(row + (((uint32_t)(2 * (C)) ^ sw) << 4)),      \
                               *reinterpret_cast<const float4*>(row + (((uint32_t)(2 * (C) + 1) ^ sw) << 4)),  \
                               inv, q0 + (C), (uint32_t)m + a.worker0, a.step, a.keys, a.one_bits);
            DQ_BLOCK(0) DQ_BLOCK(1) DQ_BLOCK(2) DQ_BLOCK(3)
#undef DQ_BLOCK
        }

        // The warp has read all of its rows: reuse the stage to transpose the 32*B words,
        // then store them 16 bytes per lane.
        __syncwarp();
        uint32_t* out_words = reinterpret_cast<uint32_t*>(tile_base);
        stage_words<B>(out_words + lane * B, acc);
        tma::fence_proxy_async();               // these stores precede the bulk copy that refills the stage
        __syncwarp();
        int ng = G - row0;
        ng = ng > 32 ? 32 : ng;
        const int nwords = ng * B;
        uint32_t* dst = a.packed + (int64_t)m * a.packed_stride + (int64_t)row0 * B;
        const int n4 = nwords >> 2;
        for (int i = lane; i < n4; i += 32)
            DQ_STORE(reinterpret_cast<uint4*>(dst) + i, reinterpret_cast<const uint4*>(out_words)[i], a.packed, (int64_t)a.M * a.packed_stride * 4, a.status);
        if (lane < (nwords & 3)) DQ_STORE(dst + (n4 * 4 + lane), out_words[n4 * 4 + lane], a.packed, (int64_t)a.M * a.packed_stride * 4, a.status);
        __syncwarp();

        // refill the stage
        if (ptile < tile_end && lane == 0) fetch(st);
        ++ptile;
        advance(pm, prt);
    }

    if (timed_out) {
        if (lane == 0) atomicOr(a.status, DQ_STAT_WAIT);
        // every copy the warp has issued and not seen land, the one whose wait ran out included, gets the
        // full limit before the CTA's shared memory is released
        for (int k = 0; k < kStages; ++k) {
            const int j = it + k;
            if (tile_begin + j < tile_end) (void)tma::mbar_wait(full_bar(warp, j % kStages), (j / kStages) & 1, a.wait);
        }
    }
}

__global__ void __launch_bounds__(kThreads, 6)
quantize_pack_kernel(const __grid_constant__ QuantizeArgs a, const __grid_constant__ CUtensorMap map)
{
    grid_dependency_wait();
    const int b = __ldg(a.dev_b);       // issued first, looked at after the set-up below so that the loads overlap
    if (tma::smem_addr(smem) & 1023u) {           // the swizzled tiles need a 1024-byte aligned base
        if (threadIdx.x == 0) atomicOr(a.status, DQ_STAT_INTERNAL);
        return;
    }
    const bool tbl_in_smem = a.v.n_seg > 1 && a.v.n_seg <= kMaxSmemSegs;
    if (tbl_in_smem) {
        int32_t* tbl_s = reinterpret_cast<int32_t*>(smem + kTblOffset);
        for (int i = threadIdx.x; i < 3 * (a.v.n_seg + 1); i += kThreads) tbl_s[i] = __ldg(a.v.seg_group0 + i);
    }
    if (threadIdx.x == 0) {
        tma::prefetch_tensor_map(&map);
        for (int i = 0; i < kWarps * kStages; ++i) tma::mbar_init(full_bar(0, i), 1);
        tma::fence_barrier_init();
    }
    __syncthreads();
    if (b < 1 || b > DQ_MAX_BITS) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(a.status, DQ_STAT_BAD_BITS);
        return;
    }
    if ((int64_t)b * a.v.total_groups > a.packed_stride) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(a.status, DQ_STAT_CAPACITY);
        return;
    }

    switch (b) {
#define DQ_CASE(BB) case BB: quantize_tiles<BB>(a, &map, tbl_in_smem); break;
        DQ_CASE(1) DQ_CASE(2) DQ_CASE(3) DQ_CASE(4) DQ_CASE(5) DQ_CASE(6) DQ_CASE(7) DQ_CASE(8)
        DQ_CASE(9) DQ_CASE(10) DQ_CASE(11) DQ_CASE(12) DQ_CASE(13) DQ_CASE(14) DQ_CASE(15) DQ_CASE(16)
#undef DQ_CASE
        default: break;
    }
}

size_t smem_bytes(int n_seg)
{
    size_t n = (size_t)kTblOffset;
    if (n_seg > 1 && n_seg <= kMaxSmemSegs) n += (size_t)3 * (n_seg + 1) * 4;
    return n;
}

}  // namespace

extern "C" int dq_quantize_pack_worker(const dq_layout_t* L, const float* dev_grads, int64_t worker_stride_elems,
                                       int32_t M, const float* dev_norms, const int32_t* dev_b,
                                       uint64_t seed, uint32_t step, uint32_t first_worker,
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

    QuantizeArgs a;
    a.v = make_view(L);
    a.norms = dev_norms;
    a.dev_b = dev_b;
    a.packed = dev_packed;
    a.packed_stride = packed_stride_words;
    a.status = dev_status;
    a.keys = make_philox_keys(seed);
    a.step = step;
    a.worker0 = first_worker;
    a.M = M;
    a.one_bits = 0x3F800040u;
    a.wait = dq_wait_limits();
    a.stream_reads = ((int64_t)M * L->padded * 4 > (int64_t(64) << 20)) ? 1 : 0;
    const bool worker_dim = (M > 1 && worker_stride_elems != 0);
    a.map_has_worker_dim = worker_dim ? 1 : 0;
    const uint32_t gpb = (uint32_t)a.v.groups_per_bucket;
    if ((gpb & (gpb - 1)) == 0) {
        a.div_shift = 0;
        while ((1u << a.div_shift) < gpb) ++a.div_shift;
        a.div_magic = 0;
    } else {
        a.div_shift = -1;
        a.div_magic = (uint32_t)(((uint64_t(1) << 33) + gpb - 1) / gpb);
    }

    // tensor map over the gradients: [worker][group][32 floats], box = one warp tile of 32 groups
    CUtensorMap map;
    const uint64_t dims[3] = {32, (uint64_t)a.v.total_groups, worker_dim ? (uint64_t)M : 1};
    const uint64_t strides[2] = {128, worker_dim ? (uint64_t)worker_stride_elems * 4 : (uint64_t)L->padded * 4};
    const uint32_t box[3] = {32, 32, 1};                 // one warp tile
    if (!dq_encode_tensor_map(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, dev_grads, dims, strides, box,
                              CU_TENSOR_MAP_SWIZZLE_128B))
        return DQ_ERR_CUDA;

    const size_t smem_need = smem_bytes(L->n_seg);
    // raising the dynamic shared-memory limit is per device and idempotent
    if (cudaFuncSetAttribute(quantize_pack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_need) != cudaSuccess) {
        (void)cudaGetLastError();
        return DQ_ERR_CUDA;
    }
    const int64_t warp_tiles = (int64_t)M * ((a.v.total_groups + 31) / 32);
    int64_t blocks = (int64_t)dq_sm_count() * 6;       // six 33 KB CTAs fit one SM
    if (blocks * kWarps > warp_tiles) blocks = (warp_tiles + kWarps - 1) / kWarps;
    dq_launch(quantize_pack_kernel, dim3((unsigned)blocks), dim3(kThreads), smem_need, static_cast<cudaStream_t>(stream), a, map);
    if (cudaGetLastError() != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

extern "C" int dq_quantize_pack(const dq_layout_t* L, const float* dev_grads, int64_t worker_stride_elems,
                                int32_t M, const float* dev_norms, const int32_t* dev_b,
                                uint64_t seed, uint32_t step,
                                uint32_t* dev_packed, int64_t packed_stride_words,
                                int32_t* dev_status, void* stream)
{
    return dq_quantize_pack_worker(L, dev_grads, worker_stride_elems, M, dev_norms, dev_b, seed, step, 0u, dev_packed,
                                   packed_stride_words, dev_status, stream);
}
