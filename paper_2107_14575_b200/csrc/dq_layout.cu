// Host layout object of the padded, bucketed gradient layout, and helpers
// shared by the entry points.
#include "dq_common.cuh"

#include <mutex>
#include <new>

static inline int64_t up32(int64_t n) { return (n + 31) / 32 * 32; }

extern "C" int dq_layout_create_ex(const int64_t* seg_elems, int32_t n_seg, int32_t bucket, int32_t norm,
                                   dq_layout_t** out)
{
    if (!seg_elems || !out || n_seg < 1) return DQ_ERR_ARG;
    if (norm != DQ_NORM_L2 && norm != DQ_NORM_LINF) return DQ_ERR_ARG;
    const bool whole = (bucket == DQ_BUCKET_WHOLE_TENSOR);
    if (!whole && (bucket < 32 || bucket > DQ_MAX_BUCKET || bucket % 32 != 0)) return DQ_ERR_RANGE;
    int64_t padded = 0, largest = 0;
    for (int32_t i = 0; i < n_seg; ++i) {
        if (seg_elems[i] < 0 || seg_elems[i] >= (int64_t(1) << 31)) return DQ_ERR_RANGE;
        if (whole && seg_elems[i] > DQ_MAX_TENSOR_ELEMS) return DQ_ERR_RANGE;
        padded += up32(seg_elems[i]);
        if (seg_elems[i] > largest) largest = seg_elems[i];
        if (padded >= (int64_t(1) << 31)) return DQ_ERR_RANGE;
    }
    if (padded == 0) return DQ_ERR_RANGE;
    if (whole) {
        // a bucket of 32 * 2^k elements that holds the largest tensor: every tensor is one bucket,
        // and the kernels that map groups to buckets divide by a power of two
        int64_t bk = 32;
        while (bk < largest) bk *= 2;
        bucket = (int32_t)bk;
    }
    dq_layout* L = new (std::nothrow) dq_layout;
    if (!L) return DQ_ERR_ARG;
    L->n_seg = n_seg;
    L->bucket = bucket;
    L->padded = padded;
    L->norm = norm;
    L->whole_tensor = whole;
    L->seg_elems.assign(seg_elems, seg_elems + n_seg);
    L->seg_offset.resize(n_seg);
    const int32_t n1 = n_seg + 1;
    L->table.assign(size_t(whole ? 6 : 3) * n1, 0);
    constexpr int64_t kPiece = 4096;
    int64_t p = 0, k = 0, c = 0;
    for (int32_t i = 0; i < n_seg; ++i) {
        L->seg_offset[i] = p;
        L->table[i] = (int32_t)(p / 32);
        L->table[n1 + i] = (int32_t)k;
        L->table[2 * n1 + i] = (int32_t)seg_elems[i];
        if (whole) {
            L->table[3 * n1 + i] = (int32_t)(p / 32);
            L->table[4 * n1 + i] = (int32_t)c;
            L->table[5 * n1 + i] = (int32_t)seg_elems[i];
            c += (seg_elems[i] + kPiece - 1) / kPiece;
        }
        p += up32(seg_elems[i]);
        k += (seg_elems[i] + bucket - 1) / bucket;
    }
    L->table[n_seg] = (int32_t)(p / 32);
    L->table[n1 + n_seg] = (int32_t)k;
    L->table[2 * n1 + n_seg] = 0;
    if (whole) {
        L->table[3 * n1 + n_seg] = (int32_t)(p / 32);
        L->table[4 * n1 + n_seg] = (int32_t)c;
        L->table[5 * n1 + n_seg] = 0;
    }
    L->nb = k;
    L->n_pieces = c;
    *out = L;
    return DQ_OK;
}

extern "C" int dq_layout_create(const int64_t* seg_elems, int32_t n_seg, int32_t bucket, dq_layout_t** out)
{
    if (bucket == DQ_BUCKET_WHOLE_TENSOR) return DQ_ERR_RANGE;      // only through dq_layout_create_ex
    return dq_layout_create_ex(seg_elems, n_seg, bucket, DQ_NORM_L2, out);
}

extern "C" int32_t dq_layout_norm(const dq_layout_t* L) { return L ? L->norm : DQ_NORM_L2; }
extern "C" int32_t dq_layout_whole_tensor(const dq_layout_t* L) { return (L && L->whole_tensor) ? 1 : 0; }

extern "C" void dq_layout_destroy(dq_layout_t* layout) { delete layout; }

extern "C" int32_t dq_layout_num_segments(const dq_layout_t* L) { return L ? L->n_seg : 0; }
extern "C" int64_t dq_layout_padded_elems(const dq_layout_t* L) { return L ? L->padded : 0; }
extern "C" int64_t dq_layout_num_buckets(const dq_layout_t* L) { return L ? L->nb : 0; }

extern "C" int64_t dq_layout_seg_offset(const dq_layout_t* L, int32_t i)
{
    if (!L || i < 0 || i >= L->n_seg) return -1;
    return L->seg_offset[i];
}

extern "C" int64_t dq_layout_packed_words(const dq_layout_t* L, int32_t b)
{
    if (!L || b < 1 || b > DQ_MAX_BITS) return 0;
    return L->padded / 32 * b;
}

extern "C" int dq_layout_bucket(const dq_layout_t* L, int64_t k, int64_t* start, int64_t* len)
{
    if (!L || !start || !len) return DQ_ERR_ARG;
    if (k < 0 || k >= L->nb) return DQ_ERR_RANGE;
    const int32_t n1 = L->n_seg + 1;
    // last tensor whose first bucket is <= k
    int32_t lo = 0, hi = L->n_seg;
    while (hi - lo > 1) {
        const int32_t mid = (lo + hi) / 2;
        if (L->table[n1 + mid] <= k) lo = mid; else hi = mid;
    }
    const int64_t local = k - L->table[n1 + lo];
    *start = L->seg_offset[lo] + local * L->bucket;
    const int64_t left = L->seg_elems[lo] - local * L->bucket;
    *len = left < L->bucket ? left : L->bucket;
    return DQ_OK;
}

// Balanced contiguous ranges of whole buckets: bound j is the first bucket whose start lies at or
// beyond j / n_shards of the padded buffer (so shards carry nearly equal numbers of elements).
extern "C" int dq_layout_shard_bounds(const dq_layout_t* L, int32_t n_shards, int64_t* bounds)
{
    if (!L || !bounds || n_shards < 1) return DQ_ERR_ARG;
    bounds[0] = 0;
    for (int32_t j = 1; j < n_shards; ++j) {
        const int64_t target = L->padded * j / n_shards;
        int64_t lo = bounds[j - 1], hi = L->nb;          // first bucket in [lo, nb] that starts at or after target
        while (lo < hi) {
            const int64_t mid = lo + (hi - lo) / 2;
            int64_t start = 0, len = 0;
            dq_layout_bucket(L, mid, &start, &len);
            if (start >= target) hi = mid; else lo = mid + 1;
        }
        bounds[j] = lo;
    }
    bounds[n_shards] = L->nb;
    return DQ_OK;
}

// Buckets [k0, k1) as a layout of their own.  Its tensors are the pieces of the parent's tensors
// that the range covers: every piece but a tensor's last is a whole number of buckets (a multiple
// of 32 elements), so the pieces sit in the slice's padded buffer exactly as they sit in the
// parent's, first_elem elements further on.
extern "C" int dq_layout_slice(const dq_layout_t* L, int64_t k0, int64_t k1, dq_layout_t** out, int64_t* first_elem)
{
    if (!L || !out) return DQ_ERR_ARG;
    if (k0 < 0 || k1 > L->nb || k0 >= k1) return DQ_ERR_RANGE;
    const int32_t n1 = L->n_seg + 1;
    std::vector<int64_t> pieces;
    int64_t first = -1;
    for (int32_t i = 0; i < L->n_seg; ++i) {
        const int64_t b0 = L->table[n1 + i], b1 = L->table[n1 + i + 1];      // this tensor's buckets
        const int64_t lo = (k0 > b0 ? k0 : b0), hi = (k1 < b1 ? k1 : b1);
        if (lo >= hi) continue;
        const int64_t e0 = (lo - b0) * L->bucket;
        int64_t e1 = (hi - b0) * L->bucket;
        if (e1 > L->seg_elems[i]) e1 = L->seg_elems[i];
        if (first < 0) first = L->seg_offset[i] + e0;
        pieces.push_back(e1 - e0);
    }
    if (pieces.empty()) return DQ_ERR_RANGE;
    const int rc = dq_layout_create_ex(pieces.data(), (int32_t)pieces.size(),
                                       L->whole_tensor ? DQ_BUCKET_WHOLE_TENSOR : L->bucket, L->norm, out);
    if (rc != DQ_OK) return rc;
    if (first_elem) *first_elem = first;
    return DQ_OK;
}

extern "C" size_t dq_layout_table_bytes(const dq_layout_t* L)
{
    if (!L || L->n_seg == 1) return 0;
    return L->table.size() * sizeof(int32_t);
}

extern "C" int dq_layout_bind_device_table(dq_layout_t* L, void* dev_buf, size_t bytes, void* stream)
{
    if (!L) return DQ_ERR_ARG;
    if (L->n_seg == 1) return DQ_OK;
    if (!dev_buf) return DQ_ERR_ARG;
    if (!aligned16(dev_buf)) return DQ_ERR_ALIGN;
    const size_t need = L->table.size() * sizeof(int32_t);
    if (bytes < need) return DQ_ERR_RANGE;
    if (cudaMemcpyAsync(dev_buf, L->table.data(), need, cudaMemcpyHostToDevice,
                        static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return DQ_ERR_CUDA;
    }
    L->dev_table = static_cast<const int32_t*>(dev_buf);
    return DQ_OK;
}

int dq_check_common(const dq_layout* L, int32_t M)
{
    if (!L) return DQ_ERR_ARG;
    if (M < 1) return DQ_ERR_ARG;
    if (M > DQ_MAX_WORKERS) return DQ_ERR_RANGE;
    if (L->n_seg > 1 && !L->dev_table) return DQ_ERR_STATE;
    return DQ_OK;
}

int dq_sm_count()
{
    static std::mutex mu;
    static int cached_dev = -1, cached_sms = 0;
    std::lock_guard<std::mutex> lock(mu);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return 148; }
    if (dev != cached_dev) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
            (void)cudaGetLastError();
            sms = 148;
        }
        cached_dev = dev;
        cached_sms = sms;
    }
    return cached_sms;
}

extern "C" const char* dq_status_string(int code)
{
    switch (code) {
        case DQ_OK:        return "ok";
        case DQ_ERR_ARG:   return "invalid argument (NULL pointer, M < 1)";
        case DQ_ERR_ALIGN: return "misaligned pointer or stride";
        case DQ_ERR_RANGE: return "value out of range";
        case DQ_ERR_CUDA:  return "CUDA call failed";
        case DQ_ERR_STATE: return "layout has several tensors but no device table is bound";
        case DQ_ERR_TOO_LARGE: return "problem larger than the built-in scratch of an allocation-free entry point";
        default:           return "unknown status";
    }
}
