// dq_unpack_dequant_average: the server's "Average" step of Algorithm 1 on
// packed codes: out_j = (1/M) sum_m (code_m - s) * norm_m / s  (Eq. 5 inverted;
// a code holds s + sgn * level).
//
// Persistent CTAs each take a contiguous range of tiles of 128 groups (one
// group = 32 padded elements = one thread, which keeps its 32 fp32 sums in
// registers).  The M workers' words of a tile are fetched in chunks of a few
// workers by linear bulk copies (TMA) into a ring of shared-memory stages, so
// the copies of the next chunks overlap the decoding of the current one.  A
// fifth warp does nothing but issue those copies: a bulk copy holds its issuing
// thread until the copy engine accepts it, about a microsecond per tile when the
// SM's four CTAs queue there at once, and nobody waits for that warp.  A
// code is decoded where it stands in its word (mask under the exponent of 2^23,
// subtract 2^23 + s: see decode_code) and accumulated with one FMA; the power
// of two its position carries is removed once per element after the last
// worker.  The 128 x 32 results of a tile go through a swizzled shared-memory
// tile and leave with one bulk tensor store.
// HBM traffic per output element: M*b/8 bytes read, 4 written.
//
// dq_unpack_average_update is the same kernel with the parameter update of
// Algorithm 1 as its epilogue, x <- x - eta * average: the tile of x is fetched into
// the output tile by a bulk tensor load while the codes are decoded, updated in place
// and stored back; the averaged gradient itself never reaches memory (M*b/8 + 4 bytes
// read and 4 written per element).
#include "dq_common.cuh"
#include "dq_device.cuh"
#include "dq_tma.cuh"

namespace {

constexpr int kThreads = 128;                 // groups per tile = consumer threads (warps 0..3)
constexpr int kBlock = kThreads + 32;         // plus the warp that issues the copies
constexpr int kStages = 2;
constexpr int kStageWords = 4096;             // 16 KB per stage
constexpr int kMaxChunk = 8;                  // workers per stage at most
constexpr int kMaxSmemSegs = 1023;

// Dynamic shared memory, addressed only through this symbol so that every access
// compiles to a shared-memory instruction:
//   [0, 16 KB)                 output tile, 128-byte swizzle (1024-byte aligned)
//   then kStages * 16 KB of input stages, 8 * 128 scales, the stage barriers, the tensor table
extern __shared__ __align__(1024) unsigned char smem[];
constexpr int kOutBytes = kThreads * 128;
constexpr int kStageOffset = kOutBytes;
constexpr int kScaleOffset = kStageOffset + kStages * kStageWords * 4;            // [kMaxChunk][kThreads] floats
// barriers: kStages "stage filled" (copies landed), kStages "stage drained" (one arrival per
// consumer warp), then the one of the x tile
constexpr int kBarOffset = kScaleOffset + kMaxChunk * kThreads * 4;
// one word that says "a wait ran out": written by whoever notices, read by the copy warp (so that it
// stops issuing) and fed into the consumers' barrier reductions
constexpr int kAbortOffset = kBarOffset + (2 * kStages + 1) * 8;
constexpr int kTblOffset = kAbortOffset + 8;

__device__ __forceinline__ uint64_t* full_bar(int st) { return reinterpret_cast<uint64_t*>(smem + kBarOffset) + st; }
__device__ __forceinline__ uint64_t* empty_bar(int st) { return reinterpret_cast<uint64_t*>(smem + kBarOffset) + kStages + st; }
__device__ __forceinline__ uint64_t* x_bar() { return reinterpret_cast<uint64_t*>(smem + kBarOffset) + 2 * kStages; }
__device__ __forceinline__ volatile int* abort_flag() { return reinterpret_cast<volatile int*>(smem + kAbortOffset); }
// barrier among the consumer warps only (the copy warp runs ahead on its own)
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory"); }
// The same barrier with an OR over the consumers' predicates: every consumer gets the same answer,
// so a decision to leave taken from it is taken by all of them or by none.
__device__ __forceinline__ bool consumer_sync_or(const bool pred)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred), "n"(kThreads)
        : "memory");
    return r != 0;
}
// Wait of the copy warp for a drained stage: as mbar_wait, but it also gives up when the
// consumers have said that they are leaving.
__device__ __forceinline__ bool wait_unless_aborted(uint64_t* bar, const uint32_t parity, const WaitLimits& lim)
{
    if (tma::mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = tma::global_timer_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (tma::mbar_try_wait(bar, parity)) return true;
        if (*abort_flag() != 0 || tma::global_timer_ns() - t0 > lim.ns) return false;
    }
}
__device__ __forceinline__ uint32_t* stage_words(int st) { return reinterpret_cast<uint32_t*>(smem + kStageOffset) + st * kStageWords; }

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
    uint32_t magic;               // 0x4B000000, kept out of the compiler's sight (see and_or)
    float neg_lr;                 // -eta of the parameter update (update kernel only)
    WaitLimits wait;
};

__device__ __forceinline__ uint32_t div_gpb(const AverageArgs& a, uint32_t n)
{
    if (a.div_shift >= 0) return n >> a.div_shift;
    return (uint32_t)(((uint64_t)n * a.div_magic) >> 33);     // exact for n < 2^26, divisor <= 128
}

// A norm load that stays where it is written: the compiler may not sink it past the barrier wait and
// the decode that follow (a volatile statement keeps its place among the other volatile statements),
// so the value is on its way while the unit is decoded.
__device__ __forceinline__ float load_norm_early(const float* p)
{
    float x;
    asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(x) : "l"(p));
    return x;
}

// workers per stage: as many as fit 16 KB with 128 groups of B words each, at most kMaxChunk
template <int B>
struct ChunkOf {
    static constexpr int fit = kStageWords / (kThreads * B);
    static constexpr int value = fit < 1 ? 1 : (fit > kMaxChunk ? kMaxChunk : fit);
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

// The 32 sums of a group live in 16 register pairs (elements 2q and 2q + 1), see accumulate_pair.
template <int B, int Q>
struct AccumulateAll {
    static __device__ __forceinline__ void run(uint64_t (&acc2)[16], const uint32_t (&wd)[B], const uint32_t (&hi)[B],
                                               const uint64_t scale2, const uint32_t magic)
    {
        acc2[Q] = accumulate_pair<B, Q>(acc2[Q], wd, hi, scale2, magic);
        AccumulateAll<B, Q + 1>::run(acc2, wd, hi, scale2, magic);
    }
};
template <int B>
struct AccumulateAll<B, 16> {
    static __device__ __forceinline__ void run(uint64_t (&)[16], const uint32_t (&)[B], const uint32_t (&)[B], const uint64_t,
                                               const uint32_t) {}
};

// The upper halves of the words whose codes need them (see decode_code) come straight from shared
// memory as 16-bit loads, two bytes into the word: the load pipe has room, the logic pipe, which a
// shift would use, is the busiest one of this kernel.
template <int B, int W>
struct UpperHalves {
    static __device__ __forceinline__ void run(const uint32_t* __restrict__ src, uint32_t (&hi)[B])
    {
        if constexpr (NeedsUpper<B, W>::value) hi[W] = reinterpret_cast<const uint16_t*>(src)[2 * W + 1];
        else hi[W] = 0u;
        UpperHalves<B, W + 1>::run(src, hi);
    }
};
template <int B>
struct UpperHalves<B, B> {
    static __device__ __forceinline__ void run(const uint32_t* __restrict__, uint32_t (&)[B]) {}
};

// removes the power of two each element's decoded value carried
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
__device__ __forceinline__ void issue_unit(const AverageArgs& a, int st, int row0, int m0, int mc)
{
    int rows = a.v.total_groups - row0;
    rows = rows > kThreads ? kThreads : rows;
    const uint32_t bytes = ((uint32_t)(rows * B * 4) + 15u) & ~15u;   // the stream's stride is a multiple of 16 bytes
    tma::mbar_expect_tx(full_bar(st), bytes * (uint32_t)mc);
    for (int j = 0; j < mc; ++j)
        tma::load_bulk(stage_words(st) + j * (kThreads * B),
                       a.packed + (int64_t)(m0 + j) * a.packed_stride + (int64_t)row0 * B, bytes, full_bar(st));
}

// UPDATE = false: out = average.  UPDATE = true: out holds the parameters x and becomes x - eta * average.
template <int B, bool UPDATE>
__device__ __forceinline__ void average_tiles(const AverageArgs& a, const CUtensorMap* out_map, const bool tbl_in_smem)
{
    constexpr int s = (1 << (B - 1)) - 1;
    constexpr int MC = ChunkOf<B>::value;
    const int32_t* tbl_s = reinterpret_cast<const int32_t*>(smem + kTblOffset);
    auto tbl = [&](int i) -> int { return tbl_in_smem ? tbl_s[i] : __ldg(a.v.seg_group0 + i); };
    const int tid = threadIdx.x;
    const int G = a.v.total_groups;
    const int M = a.M;
    const int total_tiles = (G + kThreads - 1) / kThreads;
    const int nchunk = (M + MC - 1) / MC;
    const int n1 = a.v.n_seg + 1;
    const float unit = (B == 1) ? 0.0f : __fdiv_rn(1.0f, (float)s * (float)M);      // 1 / (s * M)
    // this thread's column of the [kMaxChunk][kThreads] scale buffer (only this thread touches it)
    float* my_scales = reinterpret_cast<float*>(smem + kScaleOffset) + tid;
    const uint32_t magic = a.magic;

    // every CTA takes one contiguous range of tiles; its pipeline units are (tile, chunk) pairs
    const int tile_begin = (int)((int64_t)blockIdx.x * total_tiles / gridDim.x);
    const int tile_end = (int)((int64_t)(blockIdx.x + 1) * total_tiles / gridDim.x);
    const int my_units = (B == 1) ? 0 : (tile_end - tile_begin) * nchunk;
    if (tid >= kThreads) {
        // the copy warp: unit u goes into stage u % kStages as soon as the consumers have drained
        // what was there (unit u - kStages)
        if (tid == kThreads) {
            int issued = 0;
            for (int u = 0; u < my_units; ++u) {
                const int st = u % kStages;
                if (u >= kStages && !wait_unless_aborted(empty_bar(st), (uint32_t)(u / kStages - 1) & 1u, a.wait)) {
                    if (*abort_flag() == 0) {            // nobody drained the stage in time
                        atomicOr(a.status, DQ_STAT_WAIT);
                        *abort_flag() = 1;
                    }
                    break;
                }
                const int tile = tile_begin + u / nchunk;
                const int m0 = (u % nchunk) * MC;
                issue_unit<B>(a, st, tile * kThreads, m0, (M - m0) < MC ? (M - m0) : MC);
                issued = u + 1;
            }
            // Whoever issues copies sees them land: the last copy into each stage is the only one the
            // consumers may not have waited for (when they left early), and the CTA's shared memory
            // must not be released under a copy in flight.
            for (int u = issued > kStages ? issued - kStages : 0; u < issued; ++u)
                if (!tma::mbar_wait(full_bar(u % kStages), (uint32_t)(u / kStages) & 1u, a.wait))
                    atomicOr(a.status, DQ_STAT_WAIT);
        }
        return;
    }

    // Bucket and valid elements of this thread's group in a tile.  The first lookup of a CTA
    // is a binary search, later ones walk on from the previous tile's tensor.
    int seg = 0;
    bool seg_known = false;
    auto lookup = [&](int tile, int& bucket, int& valid) {
        const int g = tile * kThreads + tid;
        bucket = 0;
        valid = 0;                                 // 0: the group lies beyond the layout
        if (g >= G) return;
        int local, n, b0;
        if (a.v.n_seg == 1) {
            local = g; n = a.v.seg0_elems; b0 = 0;
        } else {
            if (!seg_known) {
                int lo = 0, hi = a.v.n_seg;
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (tbl(mid) <= g) lo = mid; else hi = mid;
                }
                seg = lo;
                seg_known = true;
            }
            while (g >= tbl(seg + 1)) ++seg;
            local = g - tbl(seg);
            b0 = tbl(n1 + seg);
            n = tbl(2 * n1 + seg);
        }
        bucket = b0 + (int)div_gpb(a, (uint32_t)local);
        const int left = n - local * 32;
        valid = left < 32 ? left : 32;
    };

    if constexpr (B == 1) {
        // s = 0: every value is 0, and an update by 0 leaves x as it is
        if constexpr (!UPDATE) {
            for (int tile = tile_begin; tile < tile_end; ++tile) {
                if (tid == 0) tma::store_wait_read();
                consumer_sync();
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    *reinterpret_cast<float4*>(smem + tma::swizzle128(tid, c)) = make_float4(0.f, 0.f, 0.f, 0.f);
                tma::fence_proxy_async();
                consumer_sync();
                if (tid == 0) {
                    tma::store_tile_2d(out_map, smem, 0, tile * kThreads);
                    tma::store_commit();
                }
            }
            if (tid == 0) tma::store_wait_read();
        }
        return;
    } else {
        // Software pipeline over the units: while unit u is decoded, the norms of unit u + 1 (one
        // per worker of the chunk, for this thread's bucket) are already on their way in registers.
        // Nothing touches them before the decode is done -- the first use of a loaded value is
        // where the warp would wait for it -- and only then do they become scales
        // (norm * 1/(s M)) in the scale buffer.
        int bucket, valid, nbucket = 0, nvalid = 0;
        lookup(tile_begin, bucket, valid);
        float nxt[MC];
        {
            const int mc0 = M < MC ? M : MC;
            const float* nrm = a.norms + bucket;
#pragma unroll
            for (int j = 0; j < MC; ++j)
                nxt[j] = (j < mc0 && valid > 0 && my_units > 0) ? __ldg(nrm + (int64_t)j * a.v.nb) : 0.0f;
#pragma unroll
            for (int j = 0; j < MC; ++j) my_scales[j * kThreads] = nxt[j] * unit;
        }

        // A warp whose wait for a stage ran out raises the flag, decodes no more and releases no more
        // stages; it walks on to the barrier at the tile's end, where all consumers learn of it together
        // and leave.  (Warps that were still waiting for later stages run into their own limit first.)
        uint64_t acc2[16];
        float acc[32];
        // (test hook: every warp's first wait counts as lost, so the warps start out that way)
        bool timed_out = false, warp_out = a.wait.lose_first != 0u, x_pending = false;
        if (warp_out) *abort_flag() = 1;
        int u = 0;
        int tiles_done = 0;
        for (int tile = tile_begin; tile < tile_end; ++tile) {
#pragma unroll
            for (int q = 0; q < 16; ++q) acc2[q] = 0ull;
            for (int c = 0; c < nchunk; ++c, ++u) {
                const int m0 = c * MC;
                const int mc = (M - m0) < MC ? (M - m0) : MC;

                // next unit: same tile and the next chunk of workers, or the first chunk of the next tile
                const bool last_chunk = (c == nchunk - 1);
                const bool has_next = (u + 1 < my_units);
                int nm0 = m0 + MC;
                if (last_chunk) {
                    nm0 = 0;
                    if (has_next) lookup(tile + 1, nbucket, nvalid);
                } else {
                    nbucket = bucket;
                    nvalid = valid;
                }
                {
                    const int nmc = (M - nm0) < MC ? (M - nm0) : MC;
                    const float* nrm = a.norms + (int64_t)nm0 * a.v.nb + nbucket;
#pragma unroll
                    for (int j = 0; j < MC; ++j)
                        nxt[j] = (has_next && j < nmc && nvalid > 0) ? load_norm_early(nrm + (int64_t)j * a.v.nb) : 0.0f;
                }

                if constexpr (UPDATE) {
                    // the tile of x travels into the output tile while the codes are decoded; the
                    // previous tile's store must have drained it first
                    if (c == 0) {
                        if (tid == 0) {
                            tma::store_wait_read();
                            tma::mbar_expect_tx(x_bar(), kOutBytes);
                            tma::load_tile_2d(smem, out_map, x_bar(), 0, tile * kThreads);
                        }
                        x_pending = true;
                    }
                }
                const int st = u % kStages;
                if (!warp_out &&
                    !__all_sync(0xffffffffu, tma::mbar_wait(full_bar(st), (u / kStages) & 1, a.wait))) {
                    warp_out = true;
                    *abort_flag() = 1;
                }
                if (!warp_out) {
                    const uint32_t* base = stage_words(st) + tid * B;
                    if (mc == MC) {              // a full unit: no loop
#pragma unroll
                        for (int j = 0; j < MC; ++j) {
                            uint32_t wd[B], hi[B];
                            load_words<B>(base + j * (kThreads * B), wd);
                            UpperHalves<B, 0>::run(base + j * (kThreads * B), hi);
                            const uint32_t sc = __float_as_uint(my_scales[j * kThreads]);
                            AccumulateAll<B, 0>::run(acc2, wd, hi, pack_pair(sc, sc), magic);
                        }
                    } else {
#pragma unroll 1
                        for (int j = 0; j < mc; ++j) {
                            uint32_t wd[B], hi[B];
                            load_words<B>(base + j * (kThreads * B), wd);
                            UpperHalves<B, 0>::run(base + j * (kThreads * B), hi);
                            const uint32_t sc = __float_as_uint(my_scales[j * kThreads]);
                            AccumulateAll<B, 0>::run(acc2, wd, hi, pack_pair(sc, sc), magic);
                        }
                    }
                }
#pragma unroll
                for (int j = 0; j < MC; ++j) my_scales[j * kThreads] = nxt[j] * unit;

                // this warp is done with the stage: once all four have said so the copy warp refills it
                // (a warp whose wait ran out says nothing: the stage's copy may still be on its way, and the
                // copy warp, which watches the flag, issues no more)
                __syncwarp();
                if ((tid & 31) == 0 && !warp_out) tma::mbar_arrive(empty_bar(st));
            }
            // the previous tile's bulk store must have drained the output tile before it is rewritten below
            if constexpr (!UPDATE) {
                if (tid == 0) tma::store_wait_read();
            }
            if (consumer_sync_or(warp_out || *abort_flag() != 0)) { timed_out = true; break; }
#pragma unroll
            for (int q = 0; q < 16; ++q) unpack_pair(acc2[q], acc[2 * q], acc[2 * q + 1]);
            Normalise<B, 0>::run(acc);
            if (valid < 32) {
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    if (e >= valid) acc[e] = 0.0f;
            }
            // own row of the swizzled output tile (conflict-free), then one bulk tensor store per tile
            bool x_landed = true;
            if constexpr (UPDATE) {
                x_landed = tma::mbar_wait(x_bar(), (uint32_t)tiles_done & 1u, a.wait);
                if (x_landed) {
                    const float neg_lr = a.neg_lr;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        float4* p = reinterpret_cast<float4*>(smem + tma::swizzle128(tid, c));
                        const float4 x = *p;
                        *p = make_float4(fmaf(neg_lr, acc[4 * c], x.x), fmaf(neg_lr, acc[4 * c + 1], x.y),
                                         fmaf(neg_lr, acc[4 * c + 2], x.z), fmaf(neg_lr, acc[4 * c + 3], x.w));
                    }
                }
            } else {
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    *reinterpret_cast<float4*>(smem + tma::swizzle128(tid, c)) =
                        make_float4(acc[4 * c], acc[4 * c + 1], acc[4 * c + 2], acc[4 * c + 3]);
            }
            tma::fence_proxy_async();
            if constexpr (UPDATE) {
                // nothing is stored from a tile whose parameters did not arrive
                if (consumer_sync_or(!x_landed)) { timed_out = true; break; }
                x_pending = false;
            } else {
                consumer_sync();
            }
            if (tid == 0) {
                tma::store_tile_2d(out_map, smem, 0, tile * kThreads);
                tma::store_commit();
            }
            bucket = nbucket;
            valid = nvalid;
            ++tiles_done;
        }

        if (tid == 0) tma::store_wait_read();         // shared memory must outlive the last store's reads
        if (timed_out) {
            // The copy warp stops issuing and sees its own copies land; the consumers' only copy is the
            // tile of x, which gets the full limit before the shared memory is released.
            *abort_flag() = 1;
            if (tid == 0) atomicOr(a.status, DQ_STAT_WAIT);
            if constexpr (UPDATE) {
                if (x_pending) (void)tma::mbar_wait(x_bar(), (uint32_t)tiles_done & 1u, a.wait);
            }
        }
    }
}

template <bool UPDATE>
__global__ void __launch_bounds__(kBlock, 4)
unpack_average_kernel(const __grid_constant__ AverageArgs a, const __grid_constant__ CUtensorMap out_map)
{
    grid_dependency_wait();
    const int b = __ldg(a.dev_b);       // issued first, looked at after the set-up below so that the loads overlap
    if (tma::smem_addr(smem) & 1023u) {           // the swizzled tile needs a 1024-byte aligned base
        if (threadIdx.x == 0) atomicOr(a.status, DQ_STAT_INTERNAL);
        return;
    }
    const bool tbl_in_smem = a.v.n_seg > 1 && a.v.n_seg <= kMaxSmemSegs;
    if (tbl_in_smem) {
        int32_t* tbl_s = reinterpret_cast<int32_t*>(smem + kTblOffset);
        for (int i = threadIdx.x; i < 3 * (a.v.n_seg + 1); i += kBlock) tbl_s[i] = __ldg(a.v.seg_group0 + i);
    }
    if (threadIdx.x == 0) {
        tma::prefetch_tensor_map(&out_map);
#pragma unroll
        for (int st = 0; st < kStages; ++st) {
            tma::mbar_init(full_bar(st), 1);
            tma::mbar_init(empty_bar(st), kThreads / 32);
        }
        tma::mbar_init(x_bar(), 1);
        tma::fence_barrier_init();
        *abort_flag() = 0;
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
#define DQ_CASE(BB) case BB: average_tiles<BB, UPDATE>(a, &out_map, tbl_in_smem); break;
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

// Checks, tensor map and launch shared by the two entry points; `dev_out` is the averaged
// gradient (update = false) or the parameters, read and written (update = true).
template <bool UPDATE>
int launch_average(const dq_layout_t* L, const uint32_t* dev_packed, int64_t packed_stride_words, const float* dev_norms,
                   int32_t M, const int32_t* dev_b, float lr, float* dev_out, int32_t* dev_status, void* stream)
{
    const int rc = dq_check_common(L, M);
    if (rc != DQ_OK) return rc;
    if (!dev_packed || !dev_norms || !dev_b || !dev_out || !dev_status) return DQ_ERR_ARG;
    if (!aligned16(dev_packed) || !aligned16(dev_out) || (packed_stride_words % 4) != 0 ||
        (reinterpret_cast<uintptr_t>(dev_norms) & 3u) || (reinterpret_cast<uintptr_t>(dev_b) & 3u) ||
        (reinterpret_cast<uintptr_t>(dev_status) & 3u))
        return DQ_ERR_ALIGN;
    if (packed_stride_words < L->padded / 32) return DQ_ERR_RANGE;
    if (UPDATE && !(lr == lr && lr - lr == 0.0f)) return DQ_ERR_RANGE;      // eta must be finite

    AverageArgs a;
    a.v = make_view(L);
    a.packed = dev_packed;
    a.packed_stride = packed_stride_words;
    a.norms = dev_norms;
    a.dev_b = dev_b;
    a.out = dev_out;
    a.status = dev_status;
    a.M = M;
    a.magic = 0x4B000000u;
    a.neg_lr = -lr;
    a.wait = dq_wait_limits();
    const uint32_t gpb = (uint32_t)a.v.groups_per_bucket;
    if ((gpb & (gpb - 1)) == 0) {
        a.div_shift = 0;
        while ((1u << a.div_shift) < gpb) ++a.div_shift;
        a.div_magic = 0;
    } else {
        a.div_shift = -1;
        a.div_magic = (uint32_t)(((uint64_t(1) << 33) + gpb - 1) / gpb);
    }

    // tensor map over the output: [group][32 floats], box = one tile of 128 groups, 128-byte swizzle
    CUtensorMap out_map;
    const uint64_t dims[2] = {32, (uint64_t)a.v.total_groups};
    const uint64_t strides[1] = {128};
    const uint32_t box[2] = {32, (uint32_t)kThreads};
    if (!dq_encode_tensor_map(&out_map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, dev_out, dims, strides, box,
                              CU_TENSOR_MAP_SWIZZLE_128B))
        return DQ_ERR_CUDA;

    const size_t smem_need = smem_bytes(L->n_seg);
    if (cudaFuncSetAttribute(unpack_average_kernel<UPDATE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_need) != cudaSuccess) {
        (void)cudaGetLastError();
        return DQ_ERR_CUDA;
    }
    const int64_t tiles = ((int64_t)a.v.total_groups + kThreads - 1) / kThreads;
    int64_t blocks = (int64_t)dq_sm_count() * 4;       // four 53 KB CTAs per SM
    if (blocks > tiles) blocks = tiles;
    dq_launch(unpack_average_kernel<UPDATE>, dim3((unsigned)blocks), dim3(kBlock), smem_need, static_cast<cudaStream_t>(stream), a,
              out_map);
    if (cudaGetLastError() != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

}  // namespace

extern "C" int dq_unpack_dequant_average(const dq_layout_t* L, const uint32_t* dev_packed,
                                         int64_t packed_stride_words, const float* dev_norms, int32_t M,
                                         const int32_t* dev_b, float* dev_out, int32_t* dev_status, void* stream)
{
    return launch_average<false>(L, dev_packed, packed_stride_words, dev_norms, M, dev_b, 0.0f, dev_out, dev_status,
                                 stream);
}

extern "C" int dq_unpack_average_update(const dq_layout_t* L, const uint32_t* dev_packed,
                                        int64_t packed_stride_words, const float* dev_norms, int32_t M,
                                        const int32_t* dev_b, float lr, float* dev_params, int32_t* dev_status,
                                        void* stream)
{
    return launch_average<true>(L, dev_packed, packed_stride_words, dev_norms, M, dev_b, lr, dev_params, dev_status,
                                stream);
}
