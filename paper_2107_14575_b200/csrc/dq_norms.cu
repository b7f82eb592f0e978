// dq_bucket_norms: per-bucket norm of every worker's gradient (the scale factor
// ||g||_p of Eq. 5 applied per bucket; p = 2, or p = infinity for layouts created
// with DQ_NORM_LINF), and dq_tensor_norms: one norm per tensor.
//
// One team of LANES threads (8, 16 or a full warp, by bucket size) owns a
// bucket: 128-bit coalesced loads, four independent fp32 accumulators per
// lane, a shuffle reduction inside the team.  A warp takes runs of consecutive
// buckets of one worker (blockIdx.y), so the tensor a bucket belongs to is
// searched once per run and then followed; neighbouring warps read neighbouring
// memory.  HBM-bound: 4 bytes read per element, 4/bucket bytes written.
#include "dq_common.cuh"
#include "dq_device.cuh"
#include "dq_tma.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kRun = 8;            // bucket rows a warp handles per run

// l2 norm of a bucket whose fp32 sum of squares is out of range (see l2_sum_in_range), read
// again with plain loads by its team of LANES lanes: largest magnitude first, then the squares of
// the scaled entries.  Called by all lanes of the warp; out of line, it is rarely needed.
template <int LANES>
__device__ __noinline__ float rescaled_norm_global(const float* __restrict__ g, const int len, const int lane)
{
    const MaxMagnitude mag;
    float mx = 0.f;
    for (int i = lane; i < len; i += LANES) mx = mag.take(mx, __ldg(g + i));
#pragma unroll
    for (int o = LANES / 2; o > 0; o >>= 1) mx = mag.join(mx, __shfl_xor_sync(0xffffffffu, mx, o, LANES));
    const int e = scale_exponent(mx);
    const ScaledSquares sq{e};
    float ss = 0.f;
    for (int i = lane; i < len; i += LANES) ss = sq.take(ss, __ldg(g + i));
#pragma unroll
    for (int o = LANES / 2; o > 0; o >>= 1) ss = sq.join(ss, __shfl_xor_sync(0xffffffffu, ss, o, LANES));
    return rescaled_l2(mx, ss, e);
}

template <int LANES, int P>
__global__ void __launch_bounds__(kThreads)
bucket_norms_kernel(const LayoutView v, const float* __restrict__ grads, const int64_t worker_stride,
                    float* __restrict__ norms, int32_t* __restrict__ status)
{
    grid_dependency_wait();
    constexpr int kTeamsPerWarp = 32 / LANES;
    constexpr int kChunk = kRun * kTeamsPerWarp;          // buckets per run
    const int lane = threadIdx.x % LANES;
    const int team = (threadIdx.x % 32) / LANES;
    const int m = blockIdx.y;
    const float* gw = grads + (int64_t)m * worker_stride;
    float* nw = norms + (int64_t)m * v.nb;
    const int warps_total = gridDim.x * (kThreads / 32);
    const int nchunks = (v.nb + kChunk - 1) / kChunk;
    const int bsz = v.groups_per_bucket * 32;
    bool bad = false;

    // Every lane of a warp runs the same number of iterations of both loops, so
    // the full-mask shuffles are safe; a team past the end works on an empty bucket.
    for (int chunk = blockIdx.x * (kThreads / 32) + threadIdx.x / 32; chunk < nchunks; chunk += warps_total) {
        int k = chunk * kChunk + team;
        int seg = 0;
        if (v.n_seg > 1) seg = last_not_above(v.seg_bucket0, v.n_seg, k < v.nb ? k : v.nb - 1);
#pragma unroll 1
        for (int r = 0; r < kRun; ++r, k += kTeamsPerWarp) {
            const bool active = k < v.nb;
            int len = 0;
            int64_t start = 0;
            if (active) {
                int local, n, g0;
                if (v.n_seg == 1) {
                    local = k; n = v.seg0_elems; g0 = 0;
                } else {
                    while (k >= __ldg(v.seg_bucket0 + seg + 1)) ++seg;     // buckets only move forward
                    local = k - __ldg(v.seg_bucket0 + seg);
                    n = __ldg(v.seg_elems + seg);
                    g0 = __ldg(v.seg_group0 + seg);
                }
                start = (int64_t)g0 * 32 + (int64_t)local * bsz;
                const int left = n - local * bsz;
                len = left < bsz ? left : bsz;
            }
            const float* g = gw + start;                                   // 128-byte aligned
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
                a0 = take<P>(a0, x0.x); a1 = take<P>(a1, x0.y); a2 = take<P>(a2, x0.z); a3 = take<P>(a3, x0.w);
                a0 = take<P>(a0, x1.x); a1 = take<P>(a1, x1.y); a2 = take<P>(a2, x1.z); a3 = take<P>(a3, x1.w);
                a0 = take<P>(a0, x2.x); a1 = take<P>(a1, x2.y); a2 = take<P>(a2, x2.z); a3 = take<P>(a3, x2.w);
                a0 = take<P>(a0, x3.x); a1 = take<P>(a1, x3.y); a2 = take<P>(a2, x3.z); a3 = take<P>(a3, x3.w);
            }
            for (; i < n4; i += LANES) {
                const float4 x = __ldg(g4 + i);
                a0 = take<P>(a0, x.x); a1 = take<P>(a1, x.y); a2 = take<P>(a2, x.z); a3 = take<P>(a3, x.w);
            }
            if (lane < (len & 3)) {                       // ragged tail of the tensor's last bucket
                const float x = __ldg(g + n4 * 4 + lane);
                a0 = take<P>(a0, x);
            }
            float sum = join<P>(join<P>(a0, a1), join<P>(a2, a3));
#pragma unroll
            for (int o = LANES / 2; o > 0; o >>= 1) sum = join<P>(sum, __shfl_xor_sync(0xffffffffu, sum, o, LANES));
            float nrm = finish<P>(sum);
            if constexpr (P == DQ_NORM_L2) {
                if (__any_sync(0xffffffffu, active && !l2_sum_in_range(sum))) {
                    const float again = rescaled_norm_global<LANES>(g, len, lane);
                    if (!l2_sum_in_range(sum)) nrm = again;
                }
            }
            if (lane == 0 && active) {
                DQ_STORE(nw + k, nrm, norms, (int64_t)gridDim.y * v.nb * 4, status);
                bad |= !isfinite(nrm);
            }
        }
    }
    if (bad) atomicOr(status, DQ_STAT_NONFINITE);
}

// Full-warp variant for buckets of at least 128 elements.  A warp takes a run of
// eight consecutive buckets: it first works out where each of them lies (so
// that table lookups never sit between a load and its use), then streams the
// eight buckets with independent accumulators, and finally reduces the eight
// per-lane sums together with a butterfly that halves the number of live
// values at each of its first three steps (9 shuffles instead of 40).
template <int P>
__global__ void __launch_bounds__(kThreads)
bucket_norms_warp_kernel(const LayoutView v, const float* __restrict__ grads, const int64_t worker_stride,
                         float* __restrict__ norms, int32_t* __restrict__ status)
{
    extern __shared__ int32_t tbl_s[];
    grid_dependency_wait();
    const int lane = threadIdx.x & 31;
    const int m = blockIdx.y;
    const float4* gw4 = reinterpret_cast<const float4*>(grads + (int64_t)m * worker_stride);
    const float* gw = grads + (int64_t)m * worker_stride;
    float* nw = norms + (int64_t)m * v.nb;
    const int warps_total = gridDim.x * (kThreads / 32);
    const int nchunks = (v.nb + kRun - 1) / kRun;
    const int bsz = v.groups_per_bucket * 32;
    const int n1 = v.n_seg + 1;
    bool bad = false;

    const int32_t* tbl = v.seg_group0;                 // [group0 | bucket0 | elems], n_seg + 1 entries each
    if (v.n_seg > 1 && 3 * n1 * 4 <= 12 * 1024) {
        for (int i = threadIdx.x; i < 3 * n1; i += kThreads) tbl_s[i] = __ldg(v.seg_group0 + i);
        __syncthreads();
        tbl = tbl_s;
    }

    for (int chunk = blockIdx.x * (kThreads / 32) + threadIdx.x / 32; chunk < nchunks; chunk += warps_total) {
        const int k0 = chunk * kRun;
        int first[kRun], len[kRun];                    // first float4 and valid elements of each bucket
        {
            int seg = 0;
            if (v.n_seg > 1) {                         // binary search for the run's first bucket
                int lo = 0, hi = v.n_seg;
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (tbl[n1 + mid] <= k0) lo = mid; else hi = mid;
                }
                seg = lo;
            }
#pragma unroll
            for (int r = 0; r < kRun; ++r) {
                const int k = k0 + r;
                first[r] = 0;
                len[r] = 0;
                if (k < v.nb) {
                    int local, n, g0;
                    if (v.n_seg == 1) {
                        local = k; n = v.seg0_elems; g0 = 0;
                    } else {
                        while (k >= tbl[n1 + seg + 1]) ++seg;
                        local = k - tbl[n1 + seg];
                        n = tbl[2 * n1 + seg];
                        g0 = tbl[seg];
                    }
                    first[r] = (g0 + local * v.groups_per_bucket) * 8;
                    const int left = n - local * bsz;
                    len[r] = left < bsz ? left : bsz;
                }
            }
        }
        float part[kRun];
#pragma unroll
        for (int r = 0; r < kRun; ++r) {
            const float4* g4 = gw4 + first[r];
            const int n4 = len[r] >> 2;
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            for (int i = lane; i < n4; i += 128) {
                const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
                const float4 x0 = __ldg(g4 + i);
                const float4 x1 = (i + 32 < n4) ? __ldg(g4 + i + 32) : z;
                const float4 x2 = (i + 64 < n4) ? __ldg(g4 + i + 64) : z;
                const float4 x3 = (i + 96 < n4) ? __ldg(g4 + i + 96) : z;
                a0 = take<P>(a0, x0.x); a1 = take<P>(a1, x0.y); a2 = take<P>(a2, x0.z); a3 = take<P>(a3, x0.w);
                a0 = take<P>(a0, x1.x); a1 = take<P>(a1, x1.y); a2 = take<P>(a2, x1.z); a3 = take<P>(a3, x1.w);
                a0 = take<P>(a0, x2.x); a1 = take<P>(a1, x2.y); a2 = take<P>(a2, x2.z); a3 = take<P>(a3, x2.w);
                a0 = take<P>(a0, x3.x); a1 = take<P>(a1, x3.y); a2 = take<P>(a2, x3.z); a3 = take<P>(a3, x3.w);
            }
            if (lane < (len[r] & 3)) {                 // ragged tail of a tensor's last bucket
                const float x = __ldg(gw + (int64_t)first[r] * 4 + n4 * 4 + lane);
                a0 = take<P>(a0, x);
            }
            part[r] = join<P>(join<P>(a0, a1), join<P>(a2, a3));
        }
        // butterfly: after the three halving steps lane l holds bucket (l & 7) summed over its octet
        float q[4], h[2], t;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float keep = (lane & 1) ? part[2 * i + 1] : part[2 * i];
            const float give = (lane & 1) ? part[2 * i] : part[2 * i + 1];
            q[i] = join<P>(keep, __shfl_xor_sync(0xffffffffu, give, 1));
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const float keep = (lane & 2) ? q[2 * i + 1] : q[2 * i];
            const float give = (lane & 2) ? q[2 * i] : q[2 * i + 1];
            h[i] = join<P>(keep, __shfl_xor_sync(0xffffffffu, give, 2));
        }
        {
            const float keep = (lane & 4) ? h[1] : h[0];
            const float give = (lane & 4) ? h[0] : h[1];
            t = join<P>(keep, __shfl_xor_sync(0xffffffffu, give, 4));
        }
        t = join<P>(t, __shfl_xor_sync(0xffffffffu, t, 8));
        t = join<P>(t, __shfl_xor_sync(0xffffffffu, t, 16));
        float nrm = finish<P>(t);
        if constexpr (P == DQ_NORM_L2) {
            // lane r holds bucket r of the run: the buckets out of range are taken again one by one
            const unsigned need = __ballot_sync(0xffffffffu, lane < kRun && k0 + lane < v.nb && !l2_sum_in_range(t));
            if (need) {
#pragma unroll
                for (int r = 0; r < kRun; ++r) {
                    if ((need >> r) & 1u) {
                        const float again = rescaled_norm_global<32>(gw + (int64_t)first[r] * 4, len[r], lane);
                        if (lane == r) nrm = again;
                    }
                }
            }
        }
        if (lane < kRun && k0 + lane < v.nb) {
            DQ_STORE(nw + (k0 + lane), nrm, norms, (int64_t)gridDim.y * v.nb * 4, status);
            bad |= !isfinite(nrm);
        }
    }
    if (bad) atomicOr(status, DQ_STAT_NONFINITE);
}

// Bulk-copy variant for bucket sizes that are 32 times a power of two (every size in
// common use).  Persistent CTAs each take a contiguous range of tiles of
// R = 4096 / bucket consecutive buckets of one worker; in the padded layout such
// a run is one contiguous span of at most 128 groups, fetched by a single TMA
// tensor copy into a ring of swizzled shared-memory stages, so the bytes in
// flight are set by the ring and not by how many loads the warps manage to
// issue.  Thread t of a tile owns group (t % gpb) of bucket (t / gpb): it squares
// its 128-byte row, the gpb threads of a bucket combine by shuffles (and through
// shared memory when a bucket spans several warps).
constexpr int kTmaThreads = 128;
constexpr int kTmaStages = 4;
constexpr int kTmaTileBytes = kTmaThreads * 128;
constexpr int kTmaMaxSmemSegs = 1023;

extern __shared__ __align__(1024) unsigned char smem[];
constexpr int kPartOffset = kTmaStages * kTmaTileBytes;          // 4 floats: per-warp partial results
constexpr int kAbortOffset = kPartOffset + 16;                   // set by a thread whose wait ran out
constexpr int kBarOffset = kPartOffset + 32;
constexpr int kTblOffset = kBarOffset + kTmaStages * 8;

__device__ __forceinline__ uint64_t* full_bar(int st) { return reinterpret_cast<uint64_t*>(smem + kBarOffset) + st; }

struct NormsArgs {
    LayoutView v;
    const float* grads;
    float* norms;
    int32_t* status;
    int32_t M;
    int32_t map_has_worker_dim;
    int32_t gpb_shift;           // log2(groups per bucket)
    int32_t stream_reads;        // 1: the gradients exceed the L2, read them with the evict-first policy
    WaitLimits wait;
};

template <int P>
__global__ void __launch_bounds__(kTmaThreads)
bucket_norms_tma_kernel(const __grid_constant__ NormsArgs a, const __grid_constant__ CUtensorMap map)
{
    grid_dependency_wait();
    const int tid = threadIdx.x;
    if (tma::smem_addr(smem) & 1023u) {
        if (tid == 0) atomicOr(a.status, DQ_STAT_INTERNAL);
        return;
    }
    const int n1 = a.v.n_seg + 1;
    const bool tbl_in_smem = a.v.n_seg > 1 && a.v.n_seg <= kTmaMaxSmemSegs;
    int32_t* tbl_s = reinterpret_cast<int32_t*>(smem + kTblOffset);
    if (tbl_in_smem)
        for (int i = tid; i < 3 * n1; i += kTmaThreads) tbl_s[i] = __ldg(a.v.seg_group0 + i);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kAbortOffset);
    if (tid == 0) {
        tma::prefetch_tensor_map(&map);
#pragma unroll
        for (int st = 0; st < kTmaStages; ++st) tma::mbar_init(full_bar(st), 1);
        tma::fence_barrier_init();
        *abort_flag = 0;
    }
    __syncthreads();
    auto tbl = [&](int i) -> int { return tbl_in_smem ? tbl_s[i] : __ldg(a.v.seg_group0 + i); };

    const int gpb = 1 << a.gpb_shift;
    const int R = kTmaThreads >> a.gpb_shift;                   // buckets per tile
    const int nb = a.v.nb;
    const int tiles_per_worker = (nb + R - 1) / R;
    const int total_tiles = a.M * tiles_per_worker;
    const int bsz = gpb * 32;
    // every CTA takes one contiguous range of the worker-major tile list
    const int tile_begin = (int)((int64_t)blockIdx.x * total_tiles / gridDim.x);
    const int tile_end = (int)((int64_t)(blockIdx.x + 1) * total_tiles / gridDim.x);

    // first group and valid elements of bucket k; `seg` is a walking hint (buckets only move forward)
    auto locate = [&](int k, int& seg, int& first_group, int& len) {
        int local, n, g0;
        if (a.v.n_seg == 1) {
            local = k; n = a.v.seg0_elems; g0 = 0;
        } else {
            while (k >= tbl(n1 + seg + 1)) ++seg;
            local = k - tbl(n1 + seg);
            n = tbl(2 * n1 + seg);
            g0 = tbl(seg);
        }
        first_group = g0 + (local << a.gpb_shift);
        const int left = n - local * bsz;
        len = left < bsz ? left : bsz;
    };
    auto advance = [&](int& mm, int& rr) {
        if (++rr == tiles_per_worker) { rr = 0; ++mm; }
    };

    int m = tile_begin / tiles_per_worker, kt = tile_begin - m * tiles_per_worker;
    int pm = m, pkt = kt, ptile = tile_begin, pseg = 0, pseg_m = m;
    const uint64_t policy = tma::policy_evict_first();
    auto issue = [&](int st) {
        if (pm != pseg_m) { pseg = 0; pseg_m = pm; }
        int row0, len0;
        locate(pkt * R, pseg, row0, len0);
        tma::mbar_expect_tx(full_bar(st), kTmaTileBytes);
        if (a.stream_reads)
            tma::load_tile_3d_hint(smem + st * kTmaTileBytes, &map, full_bar(st), 0, row0, a.map_has_worker_dim ? pm : 0, policy);
        else
            tma::load_tile_3d(smem + st * kTmaTileBytes, &map, full_bar(st), 0, row0, a.map_has_worker_dim ? pm : 0);
    };
#pragma unroll
    for (int st = 0; st < kTmaStages; ++st) {
        if (ptile < tile_end && tid == 0) issue(st);
        ++ptile;
        advance(pm, pkt);
    }

    const int r = tid >> a.gpb_shift;            // bucket of the tile this thread works on
    const int l = tid & (gpb - 1);               // its group inside that bucket
    const int lane = tid & 31, warp = tid >> 5;
    float* part = reinterpret_cast<float*>(smem + kPartOffset);
    int seg = 0, seg0 = 0, seg_m = -1;
    int it = 0;
    bool timed_out = false, bad = false;
    for (int tile = tile_begin; tile < tile_end; ++tile, ++it, advance(m, kt)) {
        const int st = it % kTmaStages;
        if (m != seg_m) { seg = 0; seg0 = 0; seg_m = m; }
        const int k0 = kt * R;
        const int k = k0 + r;
        int row0, len0, first = 0, len = 0;
        locate(k0, seg0, row0, len0);
        if (k < nb) locate(k, seg, first, len);
        const int row = first - row0 + l;        // this thread's row of the tile
        int valid = len - l * 32;                // elements of its group that count
        valid = valid < 0 ? 0 : (valid > 32 ? 32 : valid);

        // A thread whose wait runs out says so in shared memory and goes on (what it reads from the
        // stage is then arbitrary, and unused): every thread reaches the barriers below, after which all
        // of them see the flag and leave together.
        bool landed = tma::mbar_wait(full_bar(st), (it / kTmaStages) & 1, a.wait);
        if (it == 0 && a.wait.lose_first != 0u) landed = false;      // test hook: the first wait counts as lost
        if (!landed) *abort_flag = 1;

        // One reduction of the tile: the gpb threads of a bucket combine inside a warp by shuffles and
        // across the warps of a bucket through shared memory; the result counts in the threads with l == 0
        // (in all threads of the bucket when it lies inside one warp).
        const unsigned char* base = smem + st * kTmaTileBytes;
        auto tile_reduce = [&](const auto& red) -> float {
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            if (valid > 0) {
                if (valid == 32) {
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const float4 x = *reinterpret_cast<const float4*>(base + tma::swizzle128(row, c));
                        a0 = red.take(a0, x.x); a1 = red.take(a1, x.y); a2 = red.take(a2, x.z); a3 = red.take(a3, x.w);
                    }
                } else {                             // last group of a tensor: what follows is padding
                    for (int e = 0; e < valid; ++e) {
                        const float x = *reinterpret_cast<const float*>(base + tma::swizzle128(row, e >> 2) + ((e & 3) << 2));
                        a0 = red.take(a0, x);
                    }
                }
            }
            float v = red.join(red.join(a0, a1), red.join(a2, a3));
            const int w = gpb < 32 ? gpb : 32;
            for (int o = w >> 1; o > 0; o >>= 1) v = red.join(v, __shfl_xor_sync(0xffffffffu, v, o));
            if (gpb > 32) {
                if (lane == 0) part[warp] = v;
                __syncthreads();
                if (l == 0) {
                    v = 0.f;
                    for (int i = 0; i < (gpb >> 5); ++i) v = red.join(v, part[(tid >> 5) + i]);
                }
            }
            return v;
        };
        const float sum = tile_reduce(typename FamilyReduction<P>::type{});
        float nrm = finish<P>(sum);
        const bool writes = (l == 0 && k < nb);
        const bool out_of_range = (P == DQ_NORM_L2) && writes && !l2_sum_in_range(sum);
        // after this barrier everyone is done with the stage and with part[]
        if (__syncthreads_or(out_of_range || !landed)) {
            if (*abort_flag) { timed_out = true; break; }
            if constexpr (P == DQ_NORM_L2) {
                // some bucket of the tile needs the rescaled reduction (see l2_sum_in_range): the whole
                // CTA takes it, the buckets that were in range keep their norm
                float mx = tile_reduce(MaxMagnitude{});
                if (gpb > 32) {                  // the bucket's largest magnitude, for all of its threads
                    __syncthreads();
                    if (l == 0) part[warp] = mx;
                    __syncthreads();
                    mx = part[(tid >> a.gpb_shift) << (a.gpb_shift - 5)];
                    __syncthreads();
                }
                const int e = scale_exponent(mx);
                const float scaled = tile_reduce(ScaledSquares{e});
                if (out_of_range) nrm = rescaled_l2(mx, scaled, e);
                __syncthreads();
            }
        }
        if (writes) {
            DQ_STORE(a.norms + ((int64_t)m * nb + k), nrm, a.norms, (int64_t)a.M * a.v.nb * 4, a.status);
            bad |= !isfinite(nrm);
        }
        if (ptile < tile_end && tid == 0) issue(st);
        ++ptile;
        advance(pm, pkt);
    }
    if (bad) atomicOr(a.status, DQ_STAT_NONFINITE);
    if (timed_out) {
        if (tid == 0) atomicOr(a.status, DQ_STAT_WAIT);
        // every copy already issued, the one whose wait ran out included, gets the full limit to land
        // before the CTA's shared memory is released
        for (int j = it; j < it + kTmaStages; ++j)
            if (tile_begin + j < tile_end) (void)tma::mbar_wait(full_bar(j % kTmaStages), (j / kTmaStages) & 1, a.wait);
    }
}

// Second step of dq_tensor_norms: block (tensor, worker) joins the norms of the tensor's pieces in
// a fixed order -- thread t takes pieces t, t + 256, ..., then a tree over the block -- and writes
// the tensor's norm.  l2: the squares of the piece norms are exact in fp64 and cannot leave its
// range; their sum is at least p^2 for every piece norm p, the fp64 square root is monotone and
// gives back p for p^2, and so is the rounding to fp32, which has p among its values: the tensor's
// norm is at least every piece norm, which in turn is at least every entry of the piece.
constexpr int kJoinThreads = 256;

template <int P>
__global__ void __launch_bounds__(kJoinThreads)
tensor_norms_join_kernel(const int32_t n_seg, const int32_t* __restrict__ piece0, const int32_t* __restrict__ bucket0,
                         const int32_t n_pieces, const int32_t nb, const float* __restrict__ partial,
                         float* __restrict__ norms, int32_t* __restrict__ status)
{
    __shared__ double part_d[kJoinThreads / 32];
    __shared__ float part_f[kJoinThreads / 32];
    grid_dependency_wait();
    const int seg = blockIdx.x, m = blockIdx.y;
    int c0 = 0, c1 = n_pieces, k = 0;
    if (n_seg > 1) {
        c0 = __ldg(piece0 + seg);
        c1 = __ldg(piece0 + seg + 1);
        k = __ldg(bucket0 + seg);
    }
    if (c0 >= c1) return;                                    // an empty tensor has no norm
    const float* src = partial + (int64_t)m * n_pieces;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float nrm;
    if constexpr (P == DQ_NORM_L2) {
        double acc = 0.0;
        for (int i = c0 + tid; i < c1; i += kJoinThreads) {
            const double p = (double)__ldg(src + i);
            acc = fma(p, p, acc);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) part_d[warp] = acc;
        __syncthreads();
        if (tid != 0) return;
        double total = 0.0;
        for (int w = 0; w < kJoinThreads / 32; ++w) total += part_d[w];
        nrm = (float)sqrt(total);
    } else {
        float acc = 0.0f;
        for (int i = c0 + tid; i < c1; i += kJoinThreads) acc = max_nan(acc, __ldg(src + i));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc = max_nan(acc, __shfl_xor_sync(0xffffffffu, acc, o));
        if (lane == 0) part_f[warp] = acc;
        __syncthreads();
        if (tid != 0) return;
        float total = 0.0f;
        for (int w = 0; w < kJoinThreads / 32; ++w) total = max_nan(total, part_f[w]);
        nrm = total;
    }
    DQ_STORE(norms + ((int64_t)m * nb + k), nrm, norms, (int64_t)gridDim.y * nb * 4, status);
    if (!isfinite(nrm)) atomicOr(status, DQ_STAT_NONFINITE);
}

// Launch of the bulk-copy kernel over view `v` (groups per bucket a power of two, at most 128).
template <int P>
int launch_tma(const dq_layout_t* L, const LayoutView& v, const float* dev_grads, int64_t worker_stride_elems, int32_t M,
               float* dev_out, int32_t* dev_status, cudaStream_t st)
{
    const uint32_t gpb = (uint32_t)v.groups_per_bucket;
    NormsArgs a;
    a.v = v;
    a.grads = dev_grads;
    a.norms = dev_out;
    a.status = dev_status;
    a.M = M;
    a.gpb_shift = 0;
    while ((1u << a.gpb_shift) < gpb) ++a.gpb_shift;
    a.stream_reads = ((int64_t)M * L->padded * 4 > (int64_t(64) << 20)) ? 1 : 0;
    a.wait = dq_wait_limits();
    const bool worker_dim = (M > 1 && worker_stride_elems != 0);
    a.map_has_worker_dim = worker_dim ? 1 : 0;
    CUtensorMap map;
    const uint64_t dims[3] = {32, (uint64_t)v.total_groups, worker_dim ? (uint64_t)M : 1};
    const uint64_t strides[2] = {128, worker_dim ? (uint64_t)worker_stride_elems * 4 : (uint64_t)L->padded * 4};
    const uint32_t box[3] = {32, (uint32_t)kTmaThreads, 1};
    if (!dq_encode_tensor_map(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, dev_grads, dims, strides, box,
                              CU_TENSOR_MAP_SWIZZLE_128B))
        return DQ_ERR_CUDA;
    size_t smem_need = (size_t)kTblOffset;
    if (L->n_seg > 1 && L->n_seg <= kTmaMaxSmemSegs) smem_need += (size_t)3 * (L->n_seg + 1) * 4;
    if (cudaFuncSetAttribute(bucket_norms_tma_kernel<P>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_need) != cudaSuccess) {
        (void)cudaGetLastError();
        return DQ_ERR_CUDA;
    }
    const int R = kTmaThreads >> a.gpb_shift;
    const int64_t tiles = (int64_t)M * ((v.nb + R - 1) / R);
    int64_t blocks = (int64_t)dq_sm_count() * 3;    // three 65 KB CTAs per SM
    if (blocks > tiles) blocks = tiles;
    dq_launch(bucket_norms_tma_kernel<P>, dim3((unsigned)blocks), dim3(kTmaThreads), smem_need, st, a, map);
    if (cudaGetLastError() != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

// other bucket sizes: plain-load kernels
template <int P>
int launch_plain(const dq_layout_t* L, const LayoutView& v, const float* dev_grads, int64_t worker_stride_elems, int32_t M,
                 float* dev_norms, int32_t* dev_status, cudaStream_t st)
{
    const int lanes = L->bucket >= 128 ? 32 : (L->bucket >= 64 ? 16 : 8);
    const int64_t chunk = (int64_t)kRun * (32 / lanes);
    const int64_t nchunks = (L->nb + chunk - 1) / chunk;
    int64_t bx = (nchunks + kThreads / 32 - 1) / (kThreads / 32);
    // about 8 resident CTAs of 256 threads per SM over all workers
    int64_t cap = ((int64_t)dq_sm_count() * 8 + M - 1) / M;
    if (cap < 1) cap = 1;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    const dim3 grid((unsigned)bx, (unsigned)M);
    if (lanes == 32) {
        const size_t smem = (L->n_seg > 1 && (size_t)3 * (L->n_seg + 1) * 4 <= 12 * 1024) ? (size_t)3 * (L->n_seg + 1) * 4 : 0;
        dq_launch(bucket_norms_warp_kernel<P>, grid, dim3(kThreads), smem, st, v, dev_grads, worker_stride_elems, dev_norms, dev_status);
    }
    else if (lanes == 16)
        dq_launch(bucket_norms_kernel<16, P>, grid, dim3(kThreads), 0, st, v, dev_grads, worker_stride_elems, dev_norms, dev_status);
    else
        dq_launch(bucket_norms_kernel<8, P>, grid, dim3(kThreads), 0, st, v, dev_grads, worker_stride_elems, dev_norms, dev_status);
    if (cudaGetLastError() != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

int check_norm_args(const dq_layout_t* L, const float* dev_grads, int64_t worker_stride_elems, int32_t M,
                    const float* dev_norms, const int32_t* dev_status)
{
    const int rc = dq_check_common(L, M);
    if (rc != DQ_OK) return rc;
    if (!dev_grads || !dev_norms || !dev_status) return DQ_ERR_ARG;
    if (!aligned16(dev_grads) || (worker_stride_elems % 32) != 0 || (reinterpret_cast<uintptr_t>(dev_norms) & 3u) ||
        (reinterpret_cast<uintptr_t>(dev_status) & 3u))
        return DQ_ERR_ALIGN;
    if (M > 1 && worker_stride_elems < L->padded && worker_stride_elems != 0) return DQ_ERR_RANGE;
    return DQ_OK;
}

}  // namespace

extern "C" int dq_bucket_norms(const dq_layout_t* L, const float* dev_grads, int64_t worker_stride_elems,
                               int32_t M, float* dev_norms, int32_t* dev_status, void* stream)
{
    const int rc = check_norm_args(L, dev_grads, worker_stride_elems, M, dev_norms, dev_status);
    if (rc != DQ_OK) return rc;
    if (L->whole_tensor) return DQ_ERR_RANGE;           // one norm per tensor comes from dq_tensor_norms

    const LayoutView v = make_view(L);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint32_t gpb = (uint32_t)v.groups_per_bucket;
    const bool linf = (L->norm == DQ_NORM_LINF);
    if ((gpb & (gpb - 1)) == 0) {
        // bucket = 32 * 2^k: bulk-copy kernel
        return linf ? launch_tma<DQ_NORM_LINF>(L, v, dev_grads, worker_stride_elems, M, dev_norms, dev_status, st)
                    : launch_tma<DQ_NORM_L2>(L, v, dev_grads, worker_stride_elems, M, dev_norms, dev_status, st);
    }
    return linf ? launch_plain<DQ_NORM_LINF>(L, v, dev_grads, worker_stride_elems, M, dev_norms, dev_status, st)
                : launch_plain<DQ_NORM_L2>(L, v, dev_grads, worker_stride_elems, M, dev_norms, dev_status, st);
}

extern "C" size_t dq_tensor_norms_scratch_bytes(const dq_layout_t* L, int32_t M)
{
    if (!L || !L->whole_tensor || M < 1) return 0;
    return (size_t)M * (size_t)L->n_pieces * sizeof(float);
}

extern "C" int dq_tensor_norms(const dq_layout_t* L, const float* dev_grads, int64_t worker_stride_elems, int32_t M,
                               float* dev_norms, void* dev_scratch, size_t scratch_bytes, int32_t* dev_status,
                               void* stream)
{
    const int rc = check_norm_args(L, dev_grads, worker_stride_elems, M, dev_norms, dev_status);
    if (rc != DQ_OK) return rc;
    if (!L->whole_tensor) return DQ_ERR_RANGE;          // bucketed layouts: dq_bucket_norms
    if (!dev_scratch) return DQ_ERR_ARG;
    if (!aligned16(dev_scratch)) return DQ_ERR_ALIGN;
    if (scratch_bytes < dq_tensor_norms_scratch_bytes(L, M)) return DQ_ERR_RANGE;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* partial = static_cast<float*>(dev_scratch);
    const LayoutView pv = make_piece_view(L);
    const bool linf = (L->norm == DQ_NORM_LINF);
    const int r1 = linf ? launch_tma<DQ_NORM_LINF>(L, pv, dev_grads, worker_stride_elems, M, partial, dev_status, st)
                        : launch_tma<DQ_NORM_L2>(L, pv, dev_grads, worker_stride_elems, M, partial, dev_status, st);
    if (r1 != DQ_OK) return r1;
    const int32_t n1 = L->n_seg + 1;
    const int32_t* piece0 = L->n_seg > 1 ? L->dev_table + 4 * n1 : nullptr;
    const int32_t* bucket0 = L->n_seg > 1 ? L->dev_table + n1 : nullptr;
    const dim3 grid((unsigned)L->n_seg, (unsigned)M);
    if (linf)
        dq_launch(tensor_norms_join_kernel<DQ_NORM_LINF>, grid, dim3(kJoinThreads), 0, st, L->n_seg, piece0, bucket0,
                  (int32_t)L->n_pieces, (int32_t)L->nb, partial, dev_norms, dev_status);
    else
        dq_launch(tensor_norms_join_kernel<DQ_NORM_L2>, grid, dim3(kJoinThreads), 0, st, L->n_seg, piece0, bucket0,
                  (int32_t)L->n_pieces, (int32_t)L->nb, partial, dev_norms, dev_status);
    if (cudaGetLastError() != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}
