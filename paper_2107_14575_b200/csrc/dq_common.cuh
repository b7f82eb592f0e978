// Shared declarations of the CUDA library: the host layout object, the layout
// view kernels receive, and small device helpers.  Nothing here is used by the
// CPU checker.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>
#include <vector>

#include "dq.h"

// ---------------------------------------------------------------- host layout

struct dq_layout {
    int32_t n_seg = 0;
    int32_t bucket = 0;
    int64_t padded = 0;                 // D32
    int64_t nb = 0;                     // buckets per worker
    std::vector<int64_t> seg_elems;     // n_i
    std::vector<int64_t> seg_offset;    // P_i (elements)
    // device table image: three int32 arrays of n_seg + 1 entries each
    //   [0]            first 32-element group of tensor i (last entry: D32/32)
    //   [n_seg+1]      first bucket of tensor i           (last entry: nb)
    //   [2(n_seg+1)]   valid elements of tensor i         (last entry: 0)
    // A whole-tensor layout appends a second image of the same shape whose middle array counts
    // 4096-element pieces instead of buckets (the pieces dq_tensor_norms reduces first).
    std::vector<int32_t> table;
    const int32_t* dev_table = nullptr; // caller-owned copy, set by bind
    int32_t norm = DQ_NORM_L2;          // member of the l_p family the norm calls compute
    bool whole_tensor = false;          // one bucket per non-empty tensor
    int64_t n_pieces = 0;               // whole-tensor layouts: 4096-element pieces per worker
};

// What a kernel needs to map 32-element groups and buckets to tensors.
struct LayoutView {
    int32_t n_seg;
    int32_t groups_per_bucket;   // bucket / 32
    int32_t total_groups;        // D32 / 32
    int32_t nb;                  // buckets per worker
    int32_t seg0_elems;          // valid elements when n_seg == 1
    const int32_t* seg_group0;   // [n_seg + 1]   (NULL when n_seg == 1)
    const int32_t* seg_bucket0;  // [n_seg + 1]
    const int32_t* seg_elems;    // [n_seg + 1]
};

inline LayoutView make_view(const dq_layout* L)
{
    LayoutView v;
    v.n_seg = L->n_seg;
    v.groups_per_bucket = L->bucket / 32;
    v.total_groups = (int32_t)(L->padded / 32);
    v.nb = (int32_t)L->nb;
    v.seg0_elems = (int32_t)L->seg_elems[0];
    v.seg_group0 = L->dev_table;
    v.seg_bucket0 = L->dev_table ? L->dev_table + (L->n_seg + 1) : nullptr;
    v.seg_elems = L->dev_table ? L->dev_table + 2 * (L->n_seg + 1) : nullptr;
    return v;
}

// The same tensors cut into 4096-element pieces (whole-tensor layouts only): the view the
// first kernel of dq_tensor_norms works on.
inline LayoutView make_piece_view(const dq_layout* L)
{
    LayoutView v;
    const int32_t n1 = L->n_seg + 1;
    v.n_seg = L->n_seg;
    v.groups_per_bucket = 128;
    v.total_groups = (int32_t)(L->padded / 32);
    v.nb = (int32_t)L->n_pieces;
    v.seg0_elems = (int32_t)L->seg_elems[0];
    v.seg_group0 = L->dev_table ? L->dev_table + 3 * n1 : nullptr;
    v.seg_bucket0 = L->dev_table ? L->dev_table + 4 * n1 : nullptr;
    v.seg_elems = L->dev_table ? L->dev_table + 5 * n1 : nullptr;
    return v;
}

// Host-side argument checks shared by the entry points.
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int dq_check_common(const dq_layout* L, int32_t M);   // DQ_OK / DQ_ERR_*
int dq_sm_count();                                    // SMs of the current device (cached per device)

#ifdef __CUDACC__

// Every kernel of the library is launched with programmatic stream serialization and begins
// with grid_dependency_wait(): the grid may be set up while the previous kernel of the stream
// is still draining (which hides the launch latency between the calls of a step), and the wait
// returns once that kernel has completed and its writes are visible, so nothing is read or
// written early.  No kernel signals its dependents ahead of its own end.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline void dq_launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    (void)cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);   // the caller reads cudaGetLastError()
}

// Every store of a kernel to global memory goes through DQ_STORE(pointer, value, base, extent in
// bytes, status word).  In the normal build that is the plain store and nothing else is evaluated.
// Built with -DDQ_CHECKED (build.py --checked -> libdq_checked.so) every store first checks that it
// lies inside [base, base + extent) and, if it does not, raises DQ_STAT_INTERNAL instead of storing:
// the stand-in for a memory checker where none can be run.
#ifdef DQ_CHECKED
template <class T>
__device__ __forceinline__ void dq_checked_store(T* p, const T& v, const void* base, const int64_t extent_bytes, int32_t* status)
{
    const int64_t off = reinterpret_cast<const char*>(p) - reinterpret_cast<const char*>(base);
    if (off < 0 || off + (int64_t)sizeof(T) > extent_bytes) atomicOr(status, DQ_STAT_INTERNAL);
    else *p = v;
}
#define DQ_STORE(p, v, base, extent_bytes, status) dq_checked_store((p), (v), (base), (int64_t)(extent_bytes), (status))
#else
#define DQ_STORE(p, v, base, extent_bytes, status) (*(p) = (v))
#endif

// Index of the last entry of starts[0..n] (n + 1 entries, non-decreasing) that is <= x.
// Tensors of zero size repeat a start; the last repeat is the non-empty one.
__device__ __forceinline__ int last_not_above(const int32_t* __restrict__ starts, int n, int x)
{
    int lo = 0, hi = n;            // invariant: starts[lo] <= x < starts[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(starts + mid) <= x) lo = mid; else hi = mid;
    }
    return lo;
}

// Bucket and number of valid elements of group g (32 padded elements).
__device__ __forceinline__ void group_info(const LayoutView& v, int g, int& bucket, int& valid)
{
    int local, n, b0;
    if (v.n_seg == 1) {
        local = g; n = v.seg0_elems; b0 = 0;
    } else {
        const int i = last_not_above(v.seg_group0, v.n_seg, g);
        local = g - __ldg(v.seg_group0 + i);
        n = __ldg(v.seg_elems + i);
        b0 = __ldg(v.seg_bucket0 + i);
    }
    bucket = b0 + local / v.groups_per_bucket;
    const int left = n - local * 32;
    valid = left < 32 ? left : 32;
}

// First padded element and valid length of bucket k.
__device__ __forceinline__ void bucket_info(const LayoutView& v, int k, int64_t& start, int& len)
{
    int local, n, g0;
    if (v.n_seg == 1) {
        local = k; n = v.seg0_elems; g0 = 0;
    } else {
        const int i = last_not_above(v.seg_bucket0, v.n_seg, k);
        local = k - __ldg(v.seg_bucket0 + i);
        n = __ldg(v.seg_elems + i);
        g0 = __ldg(v.seg_group0 + i);
    }
    const int bsz = v.groups_per_bucket * 32;
    start = (int64_t)g0 * 32 + (int64_t)local * bsz;
    const int left = n - local * bsz;
    len = left < bsz ? left : bsz;
}

#endif  // __CUDACC__
