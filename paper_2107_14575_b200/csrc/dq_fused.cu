// dq_norms_quantize_pack: bucket norms (Eq. 5; l_2 or l_inf, as the layout says) and
// quantize+pack (Eq. 5/6) in one pass over the gradients.
//
// Algorithm 1 takes b_{t+1} from the gradients of iteration t, so the bit width of
// a step is known before its gradients are: once a bucket sits in shared
// memory its norm can be taken and its codes emitted at once, and every gradient
// byte is read from HBM a single time.  The norms are written out as well: the
// server needs them for the average and for the next bit width.
//
// Every WARP is a pipeline of its own (two 4 KB stages filled by TMA tensor copies with the
// 128-byte swizzle; no CTA barrier in any loop).  A lane owns one 128-byte row (32 elements)
// of a stage: it squares the row, the lanes of a bucket combine by shuffles exactly as
// dq_bucket_norms does, then the lane encodes its row against that norm and the words leave
// with 16-byte coalesced stores through the consumed stage.
//  * Buckets of up to 1024 elements (gpb = bucket / 32 <= 32): tiles of 32 / gpb buckets, fetched
//    two tiles ahead.
//  * Buckets of 2048 and 4096 elements: a team of 2 or 4 warps takes a bucket, 1024 elements each,
//    and exchanges the partial results through shared memory; every warp fetches one bucket ahead.
// HBM traffic: 4 + b/8 bytes per element.
#include "dq_common.cuh"
#include "dq_device.cuh"
#include "dq_tma.cuh"

namespace {

constexpr int kThreads = 128;
constexpr int kMaxSmemSegs = 1023;

// Dynamic shared memory, addressed only through this symbol so that every access compiles to a
// shared-memory instruction:
//   [0, kWarps * kWStages * 4 KB)   input tiles, warp-major (1024-byte aligned for the swizzle); a
//   consumed tile doubles as the staging area of its warp's output words; then the stage barriers
//   and the tensor table
extern __shared__ __align__(1024) unsigned char smem[];
constexpr int kWarps = kThreads / 32;
constexpr int kWStages = 2;
constexpr int kWTileBytes = 32 * 128;
constexpr int kWBarOffset = kWarps * kWStages * kWTileBytes;
constexpr int kWTblOffset = kWBarOffset + kWarps * kWStages * 8;

// The team kernel adds, between the stage barriers and the tensor table, one barrier and two
// slots of four partial results for each team of warps that share a bucket (room for two teams).
constexpr int kTeamBarOffset = kWTblOffset;
constexpr int kTeamPartOffset = kTeamBarOffset + (kWarps / 2) * 8;
constexpr int kBTblOffset = kTeamPartOffset + (kWarps / 2) * 2 * 4 * 4;

__device__ __forceinline__ uint64_t* wbar(int warp, int st)
{
    return reinterpret_cast<uint64_t*>(smem + kWBarOffset) + warp * kWStages + st;
}
__device__ __forceinline__ unsigned char* wstage(int warp, int st)
{
    return smem + (warp * kWStages + st) * kWTileBytes;
}

struct FusedArgs {
    LayoutView v;
    float* norms;
    const int32_t* dev_b;
    uint32_t* packed;
    int64_t packed_stride;
    int32_t* status;
    PhiloxKeys keys;
    uint32_t step;
    uint32_t worker0;             // worker m of the call draws the uniforms of worker worker0 + m
    int32_t M;
    int32_t map_has_worker_dim;
    int32_t gpb_shift;            // log2(groups per bucket)
    int32_t stream_reads;         // 1: the gradients exceed the L2, read them with the evict-first policy
    uint32_t one_bits;            // 0x3F800040, kept out of the compiler's sight (see and_or)
    WaitLimits wait;
};

// ---- l2 norm of a bucket whose fp32 sum of squares is out of range (see l2_sum_in_range) ----
// One reduction of the row at byte offset `own` of the shared memory (swizzle phase folded in:
// chunk c sits at own ^ (c << 4)) over the `gpb` lanes of the row's bucket, in the order of the
// sum of squares it replaces: four accumulators per row, a pairwise join, the xor butterfly.
template <class R>
__device__ __forceinline__ float reduce_row_team(const R& red, const uint32_t own, const int valid, const int gpb)
{
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    if (valid == 32) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const float4 x = *reinterpret_cast<const float4*>(smem + (own ^ (uint32_t)(c << 4)));
            a0 = red.take(a0, x.x); a1 = red.take(a1, x.y); a2 = red.take(a2, x.z); a3 = red.take(a3, x.w);
        }
    } else {
        for (int e = 0; e < valid; ++e) {
            const float x = *reinterpret_cast<const float*>(smem + (own ^ (uint32_t)((e >> 2) << 4)) + ((e & 3) << 2));
            a0 = red.take(a0, x);
        }
    }
    float v = red.join(red.join(a0, a1), red.join(a2, a3));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float other = __shfl_xor_sync(0xffffffffu, v, o);
        if (o < gpb) v = red.join(v, other);
    }
    return v;
}

// Called by the whole warp when some bucket of its tile is out of range; a lane whose own bucket
// was in range keeps `nrm`.  Out of line: the common case does not pay for its registers.
__device__ __noinline__ float rescaled_team_norm(const uint32_t own, const int valid, const int gpb, const float sum,
                                                 const float nrm)
{
    const float mx = reduce_row_team(MaxMagnitude{}, own, valid, gpb);
    // zero buckets (and those with an infinity or a NaN) are settled by the magnitude alone
    if (!__any_sync(0xffffffffu, !l2_sum_in_range(sum) && magnitude_scalable(mx))) return l2_sum_in_range(sum) ? nrm : mx;
    const int e = scale_exponent(mx);
    const float scaled = reduce_row_team(ScaledSquares{e}, own, valid, gpb);
    return l2_sum_in_range(sum) ? nrm : rescaled_l2(mx, scaled, e);
}

// Called by the whole warp for a regular tile in which some bucket's l2 sum is out of range.  If
// every entry of the tile is +0 or -0, stages the tile's words -- the same B words for every group:
// all codes equal s -- in the stream's 16-byte phase, where the general copy expects them, and
// returns true (in all lanes); otherwise touches nothing and returns false.  Out of line: the common
// case does not pay for its registers.
template <int B>
__device__ __noinline__ bool stage_zero_tile(const uint32_t own, uint32_t* out_words, const int row0)
{
    uint32_t bits = 0u;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const uint4 x = *reinterpret_cast<const uint4*>(smem + (own ^ (uint32_t)(c << 4)));
        bits |= x.x | x.y | x.z | x.w;
    }
    if (!__all_sync(0xffffffffu, (bits << 1) == 0u)) return false;
    // (the vote is behind every lane's reads of its row: the rows may be overwritten now)
    uint32_t z[B];
    if constexpr (B == 1) z[0] = 0u;
    else zero_group_words<B>(z);
    const int lane = threadIdx.x & 31;
    const int off = (int)(((int64_t)row0 * B) & 3);
#pragma unroll
    for (int i = 0; i < B; ++i) out_words[off + lane * B + i] = z[i];
    return true;
}

// ---- buckets that fit one warp: a tile that touches the end of a tensor ---------------
// General route of the per-warp pipelines, kept out of line so that the common case does
// not pay for its registers: buckets may be short, rows of the tile may belong to nobody,
// and every lane looks its bucket up in the tensor table.  Leaves the lane's words in the
// staging area (the consumed stage) and returns the tile's span in groups, plus 256 if a
// norm is not finite.
template <int B, int P>
__device__ __noinline__ int irregular_tile(const FusedArgs& a, unsigned char* base, const int row0, const int m, const int kt)
{
    const int32_t* tbl_s = reinterpret_cast<const int32_t*>(smem + kWTblOffset);
    constexpr int s = (1 << (B - 1)) - 1;
    const float sf = (float)s;
    const int lane = threadIdx.x & 31;
    const int n1 = a.v.n_seg + 1;
    const int gpb = 1 << a.gpb_shift;
    const int bsz = gpb * 32;
    const int R = 32 >> a.gpb_shift;
    const int nb = a.v.nb;
    const int r = lane >> a.gpb_shift;           // bucket of the tile this lane works on
    const int l = lane & (gpb - 1);              // its group inside that bucket
    const int k = kt * R + r;
    int first = 0, len = 0;
    if (k < nb) {
        int local, n, g0;
        if (a.v.n_seg == 1) {
            local = k; n = a.v.seg0_elems; g0 = 0;
        } else {
            int lo = 0, hi = a.v.n_seg;          // last tensor whose first bucket is <= k
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (tbl_s[n1 + mid] <= k) lo = mid; else hi = mid;
            }
            local = k - tbl_s[n1 + lo];
            n = tbl_s[2 * n1 + lo];
            g0 = tbl_s[lo];
        }
        first = g0 + (local << a.gpb_shift);
        const int left = n - local * bsz;
        len = left < bsz ? left : bsz;
    }
    const int row = first - row0 + l;            // this lane's row of the tile
    int valid = len - l * 32;                    // elements of its group that count
    valid = valid < 0 ? 0 : (valid > 32 ? 32 : valid);
    const int span = __reduce_max_sync(0xffffffffu, valid > 0 ? row + 1 : 0);   // groups the tile covers

    // norm of the bucket (same operations, same order as dq_bucket_norms)
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    if (valid > 0) {
        if (valid == 32) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 x = *reinterpret_cast<const float4*>(base + tma::swizzle128(row, c));
                a0 = take<P>(a0, x.x); a1 = take<P>(a1, x.y); a2 = take<P>(a2, x.z); a3 = take<P>(a3, x.w);
            }
        } else {                                 // last group of a tensor: what follows is padding
            for (int e = 0; e < valid; ++e) {
                const float x = *reinterpret_cast<const float*>(base + tma::swizzle128(row, e >> 2) + ((e & 3) << 2));
                a0 = take<P>(a0, x);
            }
        }
    }
    float sum = join<P>(join<P>(a0, a1), join<P>(a2, a3));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float other = __shfl_xor_sync(0xffffffffu, sum, o);
        if (o < gpb) sum = join<P>(sum, other);
    }
    float nrm = finish<P>(sum);
    if constexpr (P == DQ_NORM_L2) {
        if (__any_sync(0xffffffffu, !l2_sum_in_range(sum)))
            nrm = rescaled_team_norm((uint32_t)(base - smem) + (uint32_t)(row * 128 + ((row & 7) << 4)), valid, gpb, sum,
                                     nrm);
    }
    int bad = 0;
    if (l == 0 && k < nb) {
        DQ_STORE(a.norms + ((int64_t)m * nb + k), nrm, a.norms, (int64_t)a.M * a.v.nb * 4, a.status);
        bad = isfinite(nrm) ? 0 : 256;
    }

    // codes of this lane's group against that norm
    uint32_t acc[B];
    if (valid > 0) {
        const float inv = inv_scale(sf, nrm);
        unsigned char* rowp = base + row * 128;
        const uint32_t sw = (uint32_t)(row & 7);
        if (valid < 32) {                        // padding after a tensor's end encodes as 0
            for (int e = valid; e < 32; ++e)
                *reinterpret_cast<float*>(rowp + ((((e >> 2) ^ sw) << 4) | ((e & 3) << 2))) = 0.0f;
        }
        if constexpr (B == 1) {
            acc[0] = 0u;
        } else if (inv == 0.0f) {                // a zero bucket (sparse gradients are full of them): every code is s
            zero_group_words<B>(acc);
        } else {
            uint32_t cur = 0;
            const uint32_t q0 = (uint32_t)(row0 + row) * 4u;
#define DQ_BLOCK(C)                                                                                             \
            encode_block<B, C>(acc, cur,                                                                        \
                               *reinterpret_cast<const float4*>(rowp + (((uint32_t)(2 * (C)) ^ sw) << 4)),     \
                               *reinterpret_cast<const float4*>(rowp + (((uint32_t)(2 * (C) + 1) ^ sw) << 4)), \
                               inv, q0 + (C), (uint32_t)m + a.worker0, a.step, a.keys, a.one_bits);
            DQ_BLOCK(0) DQ_BLOCK(1) DQ_BLOCK(2) DQ_BLOCK(3)
#undef DQ_BLOCK
        }
    }
    __syncwarp();                                // the warp has read all of its rows
    uint32_t* out_words = reinterpret_cast<uint32_t*>(base);
    const int off = (int)(((int64_t)row0 * B) & 3);
    if (valid > 0) {
#pragma unroll
        for (int i = 0; i < B; ++i) out_words[off + row * B + i] = acc[i];
    }
    return span | __reduce_or_sync(0xffffffffu, bad);
}

// ---- buckets that fit one warp: per-warp pipelines ---------------------------------
//
// Most warp tiles are "regular": all of their 32 / gpb buckets are full buckets of one
// tensor, so lane i owns row i, every element counts and the tile spans 32 groups.  Whether
// a tile is regular, and where it starts, depends on the layout alone; the warp works it out
// two tiles ahead from a cached description of the tensor it is in (when it fetches the
// tile) and keeps the answer in a two-deep register queue for the consumer side.  Only
// tiles that touch the end of a tensor take the general route with per-lane table walks.
template <int B, int P>
__device__ __forceinline__ void fused_warp_tiles(const FusedArgs& a, const CUtensorMap* map)
{
    const int32_t* tbl_s = reinterpret_cast<const int32_t*>(smem + kWTblOffset);
    auto tbl = [&](int i) -> int { return tbl_s[i]; };
    constexpr int s = (1 << (B - 1)) - 1;
    const float sf = (float)s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n1 = a.v.n_seg + 1;
    const int gpb = 1 << a.gpb_shift;
    const int bsz_shift = a.gpb_shift + 5;
    const int R = 32 >> a.gpb_shift;                          // buckets per warp tile
    const int nb = a.v.nb;
    const int tiles_per_worker = (nb + R - 1) / R;
    const int64_t total_tiles = (int64_t)a.M * tiles_per_worker;
    const int64_t nwarps = (int64_t)gridDim.x * kWarps;
    const int64_t gw = (int64_t)blockIdx.x * kWarps + warp;
    const int64_t tile_begin = gw * total_tiles / nwarps;
    const int64_t tile_end = (gw + 1) * total_tiles / nwarps;

    auto advance = [&](int& mm, int& rr) {
        if (++rr == tiles_per_worker) { rr = 0; ++mm; }
    };

    // ---- producer side: the tensor the fetches are in (first bucket, first group, first bucket
    //      that is not full) and the description of a tile
    int c_b0 = 0, c_g0 = 0, c_full_end = a.v.n_seg == 1 ? (a.v.seg0_elems >> bsz_shift) : 0;
    // first group of tile kt2 of any worker, bit 31 set if the tile is regular (identical in all lanes)
    auto describe = [&](int kt2) -> uint32_t {
        const int k0 = kt2 * R;
        if (k0 < c_b0 || k0 + R > c_full_end) {
            // not inside the full buckets of the cached tensor: look the tile's tensor up again
            if (a.v.n_seg > 1) {
                int lo = 0, hi = a.v.n_seg;      // last tensor whose first bucket is <= k0
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (tbl(n1 + mid) <= k0) lo = mid; else hi = mid;
                }
                c_b0 = tbl(n1 + lo);
                c_g0 = tbl(lo);
                c_full_end = c_b0 + (tbl(2 * n1 + lo) >> bsz_shift);
            }
        }
        const uint32_t regular = (k0 + R <= c_full_end) ? 0x80000000u : 0u;
        return (uint32_t)(c_g0 + ((k0 - c_b0) << a.gpb_shift)) | regular;
    };

    const int n_tiles = (int)(tile_end - tile_begin);
    int m = (int)(tile_begin / tiles_per_worker), kt = (int)(tile_begin - (int64_t)m * tiles_per_worker);
    int pm = m, pkt = kt;
    // lane 0 fetches: a tile starts at the first group of its first bucket and is always 32 rows
    // (rows past the tile's span belong to later tiles or lie outside the tensor map; nobody reads them)
    auto issue = [&](int st, int row0) {
        tma::mbar_expect_tx(wbar(warp, st), kWTileBytes);
        if (a.stream_reads)
            tma::load_tile_3d_hint(wstage(warp, st), map, wbar(warp, st), 0, row0, a.map_has_worker_dim ? pm : 0,
                                   tma::policy_evict_first());
        else
            tma::load_tile_3d(wstage(warp, st), map, wbar(warp, st), 0, row0, a.map_has_worker_dim ? pm : 0);
    };
    uint32_t d_cur = 0, d_nxt = 0;
#pragma unroll
    for (int st = 0; st < kWStages; ++st) {
        uint32_t d = 0;
        if (st < n_tiles) {
            d = describe(pkt);
            if (lane == 0) issue(st, (int)(d & 0x7fffffffu));
        }
        if (st == 0) d_cur = d; else d_nxt = d;
        advance(pm, pkt);
    }

    const int r = lane >> a.gpb_shift;           // bucket of the tile this lane works on
    const int l = lane & (gpb - 1);              // its group inside that bucket
    // byte offset of lane's row in stage 0 of this warp with the row's swizzle phase folded in:
    // chunk c of the row sits at offset own_row ^ (c << 4)
    const uint32_t own_row0 = (uint32_t)(warp * kWStages * kWTileBytes + lane * 128 + ((lane & 7) << 4));
    int it = 0;
    bool timed_out = false, bad = false;
    // (test hook: with lose_first the warp's first wait counts as lost: no tile is taken and the warp
    // goes straight to what follows a time-out)
    const int n_loop = a.wait.lose_first != 0u ? 0 : n_tiles;
    for (; it < n_loop; ++it, advance(m, kt)) {
        const int st = it % kWStages;
        const int row0 = (int)(d_cur & 0x7fffffffu);
        const bool regular = (d_cur >> 31) != 0;
        unsigned char* base = wstage(warp, st);
        uint32_t* out_words = reinterpret_cast<uint32_t*>(base);
        int span = regular ? 32 : -1;            // groups whose words wait in the staging area; -1: the general route decides

        // every lane polls the barrier itself; the verdict is made warp-uniform so that the
        // warp-level synchronisations below are always reached by all lanes or by none
        if (!__all_sync(0xffffffffu, tma::mbar_wait(wbar(warp, st), (it / kWStages) & 1, a.wait))) {
            timed_out = true;
            break;
        }

        if (regular) {
            // ---- norm of the bucket (same operations, same order as dq_bucket_norms)
            const uint32_t own = own_row0 + (uint32_t)(st * kWTileBytes);
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 x = *reinterpret_cast<const float4*>(smem + (own ^ (uint32_t)(c << 4)));
                a0 = take<P>(a0, x.x); a1 = take<P>(a1, x.y); a2 = take<P>(a2, x.z); a3 = take<P>(a3, x.w);
            }
            float sum = join<P>(join<P>(a0, a1), join<P>(a2, a3));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float other = __shfl_xor_sync(0xffffffffu, sum, o);
                if (o < gpb) sum = join<P>(sum, other);
            }
            const float nrm = finish<P>(sum);
            // Rarely, for the l2 norm, a bucket's sum of squares is out of range (see l2_sum_in_range): all
            // zeros, tiny entries, an overflowed square.  The general route takes such a tile: it reduces
            // the bucket a second time where that is needed and skips the encoding of zero buckets.
            if (P == DQ_NORM_L2 && __any_sync(0xffffffffu, !l2_sum_in_range(sum))) {
                // a tile of nothing but zeros (sparse gradients are full of them) needs no arithmetic at all:
                // its norms are 0 and every code is s; the words are staged for the general copy below
                if (stage_zero_tile<B>(own, out_words, row0)) {
                    if (l == 0)
                        DQ_STORE(a.norms + ((int64_t)m * nb + (kt * R + r)), 0.0f, a.norms, (int64_t)a.M * a.v.nb * 4, a.status);
                } else {
                    span = -1;
                }
                goto general_route;
            }
            if (l == 0) {
                DQ_STORE(a.norms + ((int64_t)m * nb + (kt * R + r)), nrm, a.norms, (int64_t)a.M * a.v.nb * 4, a.status);
                bad |= !isfinite(nrm);
            }
            // ---- codes of this lane's group against that norm
            const float inv = inv_scale(sf, nrm);
            uint32_t acc[B];
            if constexpr (B == 1) {
                acc[0] = 0u;
            } else {
                uint32_t cur = 0;
                const uint32_t q0 = (uint32_t)(row0 + lane) * 4u;
#define DQ_BLOCK(C)                                                                                             \
                encode_block<B, C>(acc, cur,                                                                    \
                                   *reinterpret_cast<const float4*>(smem + (own ^ (uint32_t)((2 * (C)) << 4))), \
                                   *reinterpret_cast<const float4*>(smem + (own ^ (uint32_t)((2 * (C) + 1) << 4))), \
                                   inv, q0 + (C), (uint32_t)m + a.worker0, a.step, a.keys, a.one_bits);
                DQ_BLOCK(0) DQ_BLOCK(1) DQ_BLOCK(2) DQ_BLOCK(3)
#undef DQ_BLOCK
            }
            __syncwarp();                        // the warp has read all of its rows
            if constexpr (B % 4 == 0) {
                // 32 * B words from a 16-byte aligned position: B / 4 quads per lane, no ragged ends
                stage_words<B>(out_words + lane * B, acc);
                tma::fence_proxy_async();        // these stores precede the bulk copy that refills the stage
                __syncwarp();
                uint4* dst = reinterpret_cast<uint4*>(a.packed + (int64_t)m * a.packed_stride + (int64_t)row0 * B);
#pragma unroll
                for (int i = 0; i < B / 4; ++i)
                    DQ_STORE(dst + (lane + 32 * i), reinterpret_cast<const uint4*>(out_words)[lane + 32 * i], a.packed, (int64_t)a.M * a.packed_stride * 4, a.status);
                span = 0;                        // nothing left for the general copy below
            } else {
                // 32 * B words from word `off` of a 16-byte unit: quads 0 (or 1) .. 8B - 1 in full, the
                // 4 - off words before quad 1 and the off words after the last quad one by one
                const int off = (int)(((int64_t)row0 * B) & 3);
#pragma unroll
                for (int i = 0; i < B; ++i) out_words[off + lane * B + i] = acc[i];
                tma::fence_proxy_async();
                __syncwarp();
                uint32_t* aligned_dst = a.packed + (int64_t)m * a.packed_stride + ((int64_t)row0 * B - off);
#pragma unroll
                for (int i = 0; i < (8 * B + 31) / 32; ++i) {
                    const int q = lane + 32 * i;
                    if (q < 8 * B && (q > 0 || off == 0))
                        DQ_STORE(reinterpret_cast<uint4*>(aligned_dst) + q, reinterpret_cast<const uint4*>(out_words)[q], a.packed, (int64_t)a.M * a.packed_stride * 4, a.status);
                }
                if (off != 0 && lane < 4) {
                    const int idx = lane >= off ? lane : 32 * B + lane;
                    DQ_STORE(aligned_dst + idx, out_words[idx], a.packed, (int64_t)a.M * a.packed_stride * 4, a.status);
                }
                span = 0;
            }
        }
    general_route:
        if (span < 0) {
            const int res = irregular_tile<B, P>(a, base, row0, m, kt);
            span = res & 0xff;
            bad |= (res >> 8) != 0;
        }

        // The stage now carries the tile's span * B words.  Word i sits at out_words[off + i] and
        // goes to aligned_dst[off + i], so that the staging area keeps the 16-byte phase of the
        // output stream; whole quads move 16 bytes per lane, the ragged ends word by word.
        if (span > 0) {
            tma::fence_proxy_async();            // the staging stores precede the bulk copy that refills the stage
            __syncwarp();
            const int off = (int)(((int64_t)row0 * B) & 3);
            const int jend = off + span * B;
            uint32_t* aligned_dst = a.packed + (int64_t)m * a.packed_stride + ((int64_t)row0 * B - off);
            const int q0 = off ? 1 : 0, q1 = jend >> 2;          // full quads [q0, q1)
            for (int q = q0 + lane; q < q1; q += 32)
                DQ_STORE(reinterpret_cast<uint4*>(aligned_dst) + q, reinterpret_cast<const uint4*>(out_words)[q], a.packed, (int64_t)a.M * a.packed_stride * 4, a.status);
            if (off && lane >= off && lane < 4 && lane < jend) DQ_STORE(aligned_dst + lane, out_words[lane], a.packed, (int64_t)a.M * a.packed_stride * 4, a.status);   // head
            int ts = q1 * 4;                                                                          // tail
            if (off && ts < 4) ts = 4;
            if (lane < jend - ts) DQ_STORE(aligned_dst + (ts + lane), out_words[ts + lane], a.packed, (int64_t)a.M * a.packed_stride * 4, a.status);
        }
        __syncwarp();

        // refill the stage with the tile two ahead and move the queue
        uint32_t d_new = 0;
        if (it + kWStages < n_tiles) {
            d_new = describe(pkt);
            if (lane == 0) issue(st, (int)(d_new & 0x7fffffffu));
        }
        d_cur = d_nxt;
        d_nxt = d_new;
        advance(pm, pkt);
    }
    if (bad) atomicOr(a.status, DQ_STAT_NONFINITE);
    if (timed_out || n_loop < n_tiles) {
        if (lane == 0) atomicOr(a.status, DQ_STAT_WAIT);
        // every copy the warp has issued and not seen land, the one whose wait ran out included, gets the
        // full limit before the CTA's shared memory is released
        for (int j = it; j < it + kWStages; ++j)
            if (j < n_tiles) (void)tma::mbar_wait(wbar(warp, j % kWStages), (j / kWStages) & 1, a.wait);
    }
}

// Five CTAs per SM (up to 102 registers per thread): at six (80 registers) the widest bit widths
// spill in the tile loop, and the kernel, bound by instruction issue, loses nothing at 20 warps per SM.
constexpr int kWarpKernelCtasPerSm = 5;
// The team kernel likewise: five CTAs per SM measured 2-4 % faster than six and than four.
constexpr int kTeamKernelCtasPerSm = 5;
template <int P>
__global__ void __launch_bounds__(kThreads, kWarpKernelCtasPerSm)
norms_quantize_pack_warp_kernel(const __grid_constant__ FusedArgs a, const __grid_constant__ CUtensorMap map)
{
    grid_dependency_wait();
    const int b = __ldg(a.dev_b);       // issued first, looked at after the set-up below so that the loads overlap
    if (tma::smem_addr(smem) & 1023u) {
        if (threadIdx.x == 0) atomicOr(a.status, DQ_STAT_INTERNAL);
        return;
    }
    if (a.v.n_seg > 1) {
        int32_t* tbl_s = reinterpret_cast<int32_t*>(smem + kWTblOffset);
        for (int i = threadIdx.x; i < 3 * (a.v.n_seg + 1); i += kThreads) tbl_s[i] = __ldg(a.v.seg_group0 + i);
    }
    if (threadIdx.x == 0) {
        tma::prefetch_tensor_map(&map);
        for (int i = 0; i < kWarps * kWStages; ++i) tma::mbar_init(wbar(0, i), 1);
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
#define DQ_CASE(BB) case BB: fused_warp_tiles<BB, P>(a, &map); break;
        DQ_CASE(1) DQ_CASE(2) DQ_CASE(3) DQ_CASE(4) DQ_CASE(5) DQ_CASE(6) DQ_CASE(7) DQ_CASE(8)
        DQ_CASE(9) DQ_CASE(10) DQ_CASE(11) DQ_CASE(12) DQ_CASE(13) DQ_CASE(14) DQ_CASE(15) DQ_CASE(16)
#undef DQ_CASE
        default: break;
    }
}

// ---- buckets of 2048 and 4096 elements: a team of T = 2 or 4 warps takes a bucket, one warp tile each ----
//
// Warp `sub` of the team owns elements [1024 sub, 1024 sub + 1024) of every bucket of the team's range.
// Its two stages alternate between consecutive buckets: while the tile of bucket i is reduced and
// encoded in one stage, the tile of bucket i + 1 is on its way into the other, and as soon as the
// words of bucket i have left, that stage is refilled with the tile of bucket i + 2 -- every warp
// keeps one whole tile in flight for the length of a bucket.  Every lane squares its row, the warp
// combines by the butterflies of dq_bucket_norms, and the T partial results are exchanged through
// shared memory (a barrier of the team's own, waited for with the usual limit; every exchange is
// one phase of it and uses the slots of that phase's parity) and added by every warp in the order
// of dq_bucket_norms.  Short buckets (a tensor's last) and padding take the same route with
// per-lane valid counts; a warp whose share of a bucket is empty fetches nothing and contributes 0.
template <int B, int P, int T>
__device__ __forceinline__ void fused_team_buckets(const FusedArgs& a, const CUtensorMap* map)
{
    const int32_t* tbl_s = reinterpret_cast<const int32_t*>(smem + kBTblOffset);
    constexpr int s = (1 << (B - 1)) - 1;
    const float sf = (float)s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n1 = a.v.n_seg + 1;
    const int nb = a.v.nb;
    constexpr int kBucket = 1024 * T;
    const int sub = warp % T;                     // which 1024 elements of the bucket this warp takes
    const int64_t total = (int64_t)a.M * nb;
    const int64_t nteams = (int64_t)gridDim.x * (kWarps / T);
    const int64_t team = (int64_t)blockIdx.x * (kWarps / T) + warp / T;
    const int64_t begin = team * total / nteams;
    const int n_tiles = (int)((team + 1) * total / nteams - begin);
    if (n_tiles <= 0) return;                     // (the whole team: its warps share `team`)

    struct Pos { int m, k, g0, len; };            // worker, bucket, first group and valid elements of the warp's share
    int seg = 0;                                  // walking hint: buckets only move forward inside a worker
    auto locate = [&](Pos& p) {
        int local, n, gs;
        if (a.v.n_seg == 1) {
            local = p.k; n = a.v.seg0_elems; gs = 0;
        } else {
            while (p.k >= tbl_s[n1 + seg + 1]) ++seg;
            local = p.k - tbl_s[n1 + seg];
            n = tbl_s[2 * n1 + seg];
            gs = tbl_s[seg];
        }
        p.g0 = gs + local * (32 * T) + 32 * sub;
        int left = n - local * kBucket - 1024 * sub;
        left = left < 0 ? 0 : left;
        p.len = left < 1024 ? left : 1024;
    };
    // the bucket after p (located only if the team's range holds it)
    auto successor = [&](const Pos& p, bool exists) -> Pos {
        Pos q;
        q.m = p.m; q.k = p.k + 1; q.g0 = 0; q.len = 0;
        if (q.k == nb) { q.k = 0; ++q.m; seg = 0; }
        if (exists) locate(q);
        return q;
    };
    auto issue = [&](int st, const Pos& p) {
        tma::mbar_expect_tx(wbar(warp, st), kWTileBytes);
        if (a.stream_reads)
            tma::load_tile_3d_hint(wstage(warp, st), map, wbar(warp, st), 0, p.g0, a.map_has_worker_dim ? p.m : 0,
                                   tma::policy_evict_first());
        else
            tma::load_tile_3d(wstage(warp, st), map, wbar(warp, st), 0, p.g0, a.map_has_worker_dim ? p.m : 0);
    };

    Pos cur;
    cur.m = (int)(begin / nb);
    cur.k = (int)(begin - (int64_t)cur.m * nb);
    locate(cur);
    Pos nxt = successor(cur, n_tiles > 1);
    if (lane == 0) {
        if (cur.len > 0) issue(0, cur);
        if (nxt.len > 0) issue(1, nxt);
    }
    bool pend0 = cur.len > 0, pend1 = nxt.len > 0;       // a copy into the stage has not been seen to land
    uint32_t ph0 = 0, ph1 = 0;                            // copies into the stage seen to land
    uint64_t* team_bar = reinterpret_cast<uint64_t*>(smem + kTeamBarOffset) + warp / T;
    float* team_part = reinterpret_cast<float*>(smem + kTeamPartOffset) + (warp / T) * 8;
    bool timed_out = false, bad = false;
    // byte offset of this lane's row inside a stage, swizzle phase folded in: chunk c sits at own ^ (c << 4)
    const uint32_t own = (uint32_t)(lane * 128 + ((lane & 7) << 4));

    // sum of squares (or maximum) of the lane's row of a stage, same operations and order as dq_bucket_norms
    auto row_reduce = [&](const auto& red, const unsigned char* base, int valid) -> float {
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        if (valid == 32) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 x = *reinterpret_cast<const float4*>(base + (own ^ (uint32_t)(c << 4)));
                a0 = red.take(a0, x.x); a1 = red.take(a1, x.y); a2 = red.take(a2, x.z); a3 = red.take(a3, x.w);
            }
        } else {
            for (int e = 0; e < valid; ++e) {
                const float x = *reinterpret_cast<const float*>(base + (own ^ (uint32_t)((e >> 2) << 4)) + ((e & 3) << 2));
                a0 = red.take(a0, x);
            }
        }
        float sum = red.join(red.join(a0, a1), red.join(a2, a3));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum = red.join(sum, __shfl_xor_sync(0xffffffffu, sum, o));
        return sum;
    };
    // One reduction of the bucket: the warp's tile, then the exchange of the team's T partial results.
    // False if the wait for the other warps ran out.
    uint32_t exchanges = 0;
    auto bucket_reduce = [&](const auto& red, const unsigned char* base, int rows, int valid, float& result) -> bool {
        const float part = rows > 0 ? row_reduce(red, base, valid) : 0.0f;
        float* slot = team_part + (exchanges & 1u) * 4;
        __syncwarp();                            // the lanes are done with the slots of two exchanges ago
        if (lane == 0) {
            slot[sub] = part;
            tma::mbar_arrive(team_bar);
        }
        if (!__all_sync(0xffffffffu, tma::mbar_wait(team_bar, exchanges & 1u, a.wait))) return false;
        ++exchanges;
        float r = red.join(0.0f, slot[0]);
#pragma unroll
        for (int i = 1; i < T; ++i) r = red.join(r, slot[i]);
        result = r;
        return true;
    };
    // encodes the lane's row of a stage against `inv`, stages the tile's words in the stage itself and
    // sends them to the packed stream; `row0` is the tile's first group, `span` its number of groups
    auto encode_tile = [&](unsigned char* base, int row0, int valid, int span, float inv, int mm) {
        uint32_t acc[B];
        if (valid > 0) {
            unsigned char* rowp = base + lane * 128;
            const uint32_t sw = (uint32_t)(lane & 7);
            if (valid < 32) {                    // padding after a tensor's end encodes as 0
                for (int e = valid; e < 32; ++e)
                    *reinterpret_cast<float*>(rowp + ((((e >> 2) ^ sw) << 4) | ((e & 3) << 2))) = 0.0f;
            }
            if constexpr (B == 1) {
                acc[0] = 0u;
            } else if (inv == 0.0f) {            // a zero bucket (the whole warp works on one bucket)
                zero_group_words<B>(acc);
            } else {
                uint32_t cur_bits = 0;
                const uint32_t q0 = (uint32_t)(row0 + lane) * 4u;
#define DQ_BLOCK(C)                                                                                             \
                encode_block<B, C>(acc, cur_bits,                                                               \
                                   *reinterpret_cast<const float4*>(rowp + (((uint32_t)(2 * (C)) ^ sw) << 4)), \
                                   *reinterpret_cast<const float4*>(rowp + (((uint32_t)(2 * (C) + 1) ^ sw) << 4)), \
                                   inv, q0 + (C), (uint32_t)mm + a.worker0, a.step, a.keys, a.one_bits);
                DQ_BLOCK(0) DQ_BLOCK(1) DQ_BLOCK(2) DQ_BLOCK(3)
#undef DQ_BLOCK
            }
        }
        __syncwarp();                            // the warp has read all of its rows
        uint32_t* out_words = reinterpret_cast<uint32_t*>(base);
        const int off = (int)(((int64_t)row0 * B) & 3);      // staging keeps the stream's 16-byte phase
        if (valid > 0) {
#pragma unroll
            for (int i = 0; i < B; ++i) out_words[off + lane * B + i] = acc[i];
        }
        tma::fence_proxy_async();                // these stores precede the bulk copy that refills the stage
        __syncwarp();
        const int jend = off + span * B;
        uint32_t* aligned_dst = a.packed + (int64_t)mm * a.packed_stride + ((int64_t)row0 * B - off);
        const int q0 = off ? 1 : 0, q1 = jend >> 2;          // full quads [q0, q1)
        for (int q = q0 + lane; q < q1; q += 32)
            DQ_STORE(reinterpret_cast<uint4*>(aligned_dst) + q, reinterpret_cast<const uint4*>(out_words)[q], a.packed, (int64_t)a.M * a.packed_stride * 4, a.status);
        if (off && lane >= off && lane < 4 && lane < jend) DQ_STORE(aligned_dst + lane, out_words[lane], a.packed, (int64_t)a.M * a.packed_stride * 4, a.status);   // head
        int ts = q1 * 4;                                                                          // tail
        if (off && ts < 4) ts = 4;
        if (lane < jend - ts) DQ_STORE(aligned_dst + (ts + lane), out_words[ts + lane], a.packed, (int64_t)a.M * a.packed_stride * 4, a.status);
        __syncwarp();
    };

    // test hook: the warp's first wait counts as lost, and the warp goes straight to what follows a time-out
    timed_out = a.wait.lose_first != 0u;
    for (int it = 0; it < n_tiles && !timed_out; ++it) {
        const int st = it & 1;
        unsigned char* base = wstage(warp, st);
        const int rows = (cur.len + 31) >> 5;
        if (rows > 0) {
            if (!__all_sync(0xffffffffu, tma::mbar_wait(wbar(warp, st), (st ? ph1 : ph0) & 1u, a.wait))) {
                timed_out = true;
                break;
            }
            if (st) { pend1 = false; ++ph1; } else { pend0 = false; ++ph0; }
        }
        int valid = cur.len - lane * 32;
        valid = valid < 0 ? 0 : (valid > 32 ? 32 : valid);

        float sum;
        if (!bucket_reduce(typename FamilyReduction<P>::type{}, base, rows, valid, sum)) { timed_out = true; break; }
        float nrm = finish<P>(sum);
        if constexpr (P == DQ_NORM_L2) {
            // every lane of every warp of the team holds the same sum: the verdict is uniform
            if (!l2_sum_in_range(sum)) {
                float mx, scaled;
                if (!bucket_reduce(MaxMagnitude{}, base, rows, valid, mx)) { timed_out = true; break; }
                const int e = scale_exponent(mx);
                if (!bucket_reduce(ScaledSquares{e}, base, rows, valid, scaled)) { timed_out = true; break; }
                nrm = rescaled_l2(mx, scaled, e);
            }
        }
        if (lane == 0 && sub == 0) {
            DQ_STORE(a.norms + ((int64_t)cur.m * nb + cur.k), nrm, a.norms, (int64_t)a.M * a.v.nb * 4, a.status);
            bad |= !isfinite(nrm);
        }
        const float inv = inv_scale(sf, nrm);

        if (rows > 0) encode_tile(base, cur.g0, valid, rows, inv, cur.m);
        // the stage is free: the warp's tile of the bucket after next goes there
        const Pos after = successor(nxt, it + 2 < n_tiles);
        if (after.len > 0) {
            if (lane == 0) issue(st, after);
            if (st) pend1 = true; else pend0 = true;
        }
        cur = nxt;
        nxt = after;
    }
    if (bad) atomicOr(a.status, DQ_STAT_NONFINITE);
    if (timed_out) {
        if (lane == 0) atomicOr(a.status, DQ_STAT_WAIT);
        // every copy the warp has issued and not seen land, the one whose wait ran out included, gets the
        // full limit before the CTA's shared memory is released
        if (pend0) (void)tma::mbar_wait(wbar(warp, 0), ph0 & 1u, a.wait);
        if (pend1) (void)tma::mbar_wait(wbar(warp, 1), ph1 & 1u, a.wait);
    }
}

template <int P, int T>
__global__ void __launch_bounds__(kThreads, kTeamKernelCtasPerSm)
norms_quantize_pack_bucket_kernel(const __grid_constant__ FusedArgs a, const __grid_constant__ CUtensorMap map)
{
    grid_dependency_wait();
    const int b = __ldg(a.dev_b);       // issued first, looked at after the set-up below so that the loads overlap
    if (tma::smem_addr(smem) & 1023u) {
        if (threadIdx.x == 0) atomicOr(a.status, DQ_STAT_INTERNAL);
        return;
    }
    if (a.v.n_seg > 1) {
        int32_t* tbl_s = reinterpret_cast<int32_t*>(smem + kBTblOffset);
        for (int i = threadIdx.x; i < 3 * (a.v.n_seg + 1); i += kThreads) tbl_s[i] = __ldg(a.v.seg_group0 + i);
    }
    if (threadIdx.x == 0) {
        tma::prefetch_tensor_map(&map);
        for (int i = 0; i < kWarps * kWStages; ++i) tma::mbar_init(wbar(0, i), 1);
        for (int i = 0; i < kWarps / T; ++i) tma::mbar_init(reinterpret_cast<uint64_t*>(smem + kTeamBarOffset) + i, T);
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
#define DQ_CASE(BB) case BB: fused_team_buckets<BB, P, T>(a, &map); break;
        DQ_CASE(1) DQ_CASE(2) DQ_CASE(3) DQ_CASE(4) DQ_CASE(5) DQ_CASE(6) DQ_CASE(7) DQ_CASE(8)
        DQ_CASE(9) DQ_CASE(10) DQ_CASE(11) DQ_CASE(12) DQ_CASE(13) DQ_CASE(14) DQ_CASE(15) DQ_CASE(16)
#undef DQ_CASE
        default: break;
    }
}

}  // namespace

extern "C" int dq_norms_quantize_pack_worker(const dq_layout_t* L, const float* dev_grads, int64_t worker_stride_elems,
                                             int32_t M, const int32_t* dev_b, uint64_t seed, uint32_t step,
                                             uint32_t first_worker, float* dev_norms, uint32_t* dev_packed,
                                             int64_t packed_stride_words, int32_t* dev_status, void* stream)
{
    const int rc = dq_check_common(L, M);
    if (rc != DQ_OK) return rc;
    if (!dev_grads || !dev_norms || !dev_b || !dev_packed || !dev_status) return DQ_ERR_ARG;
    if (!aligned16(dev_grads) || !aligned16(dev_packed) || (worker_stride_elems % 32) != 0 ||
        (packed_stride_words % 4) != 0 || (reinterpret_cast<uintptr_t>(dev_norms) & 3u) ||
        (reinterpret_cast<uintptr_t>(dev_b) & 3u) || (reinterpret_cast<uintptr_t>(dev_status) & 3u))
        return DQ_ERR_ALIGN;
    if (M > 1 && worker_stride_elems < L->padded && worker_stride_elems != 0) return DQ_ERR_RANGE;
    if (packed_stride_words < L->padded / 32) return DQ_ERR_RANGE;
    if (L->whole_tensor) return DQ_ERR_RANGE;           // one norm per tensor: the codes need a second pass

    const uint32_t gpb = (uint32_t)(L->bucket / 32);
    if ((gpb & (gpb - 1)) != 0 || L->n_seg > kMaxSmemSegs) {
        // bucket sizes that are not 32 * 2^k, or more tensors than the kernel's shared-memory table
        // holds: the two separate passes give the same result
        const int r1 = dq_bucket_norms(L, dev_grads, worker_stride_elems, M, dev_norms, dev_status, stream);
        if (r1 != DQ_OK) return r1;
        return dq_quantize_pack_worker(L, dev_grads, worker_stride_elems, M, dev_norms, dev_b, seed, step, first_worker,
                                       dev_packed, packed_stride_words, dev_status, stream);
    }

    FusedArgs a;
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
    a.gpb_shift = 0;
    while ((1u << a.gpb_shift) < gpb) ++a.gpb_shift;
    a.stream_reads = ((int64_t)M * L->padded * 4 > (int64_t(64) << 20)) ? 1 : 0;
    const bool worker_dim = (M > 1 && worker_stride_elems != 0);
    a.map_has_worker_dim = worker_dim ? 1 : 0;

    const bool per_warp = gpb <= 32;
    // otherwise gpb is 64 or 128: a team of 2 or 4 warps per bucket
    CUtensorMap map;
    const uint64_t dims[3] = {32, (uint64_t)a.v.total_groups, worker_dim ? (uint64_t)M : 1};
    const uint64_t strides[2] = {128, worker_dim ? (uint64_t)worker_stride_elems * 4 : (uint64_t)L->padded * 4};
    const uint32_t box[3] = {32, 32, 1};                 // one warp tile
    if (!dq_encode_tensor_map(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, dev_grads, dims, strides, box,
                              CU_TENSOR_MAP_SWIZZLE_128B))
        return DQ_ERR_CUDA;

    const size_t tbl_bytes = L->n_seg > 1 ? (size_t)3 * (L->n_seg + 1) * 4 : 0;
    if (per_warp) {
        const size_t smem_need = (size_t)kWTblOffset + tbl_bytes;
        const auto kernel = (L->norm == DQ_NORM_LINF) ? norms_quantize_pack_warp_kernel<DQ_NORM_LINF>
                                                      : norms_quantize_pack_warp_kernel<DQ_NORM_L2>;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem_need) != cudaSuccess) {
            (void)cudaGetLastError();
            return DQ_ERR_CUDA;
        }
        const int R = 32 >> a.gpb_shift;
        const int64_t warp_tiles = (int64_t)M * ((L->nb + R - 1) / R);
        int64_t blocks = (int64_t)dq_sm_count() * kWarpKernelCtasPerSm;
        if (blocks * kWarps > warp_tiles) blocks = (warp_tiles + kWarps - 1) / kWarps;
        dq_launch(kernel, dim3((unsigned)blocks), dim3(kThreads), smem_need, static_cast<cudaStream_t>(stream), a, map);
    } else {
        const size_t smem_need = (size_t)kBTblOffset + tbl_bytes;
        const bool linf = (L->norm == DQ_NORM_LINF);
        const auto kernel = gpb == 64 ? (linf ? norms_quantize_pack_bucket_kernel<DQ_NORM_LINF, 2>
                                              : norms_quantize_pack_bucket_kernel<DQ_NORM_L2, 2>)
                                      : (linf ? norms_quantize_pack_bucket_kernel<DQ_NORM_LINF, 4>
                                              : norms_quantize_pack_bucket_kernel<DQ_NORM_L2, 4>);
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem_need) != cudaSuccess) {
            (void)cudaGetLastError();
            return DQ_ERR_CUDA;
        }
        const int64_t warp_tiles = (int64_t)M * L->nb * (gpb / 32);        // no more teams than buckets
        int64_t blocks = (int64_t)dq_sm_count() * kTeamKernelCtasPerSm;
        if (blocks * kWarps > warp_tiles) blocks = (warp_tiles + kWarps - 1) / kWarps;
        dq_launch(kernel, dim3((unsigned)blocks), dim3(kThreads), smem_need, static_cast<cudaStream_t>(stream), a, map);
    }
    if (cudaGetLastError() != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

extern "C" int dq_norms_quantize_pack(const dq_layout_t* L, const float* dev_grads, int64_t worker_stride_elems,
                                      int32_t M, const int32_t* dev_b, uint64_t seed, uint32_t step,
                                      float* dev_norms, uint32_t* dev_packed, int64_t packed_stride_words,
                                      int32_t* dev_status, void* stream)
{
    return dq_norms_quantize_pack_worker(L, dev_grads, worker_stride_elems, M, dev_b, seed, step, 0u, dev_norms,
                                         dev_packed, packed_stride_words, dev_status, stream);
}
