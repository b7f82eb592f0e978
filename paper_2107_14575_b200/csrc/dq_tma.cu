// Host side of the TMA plumbing: tensor-map encoding through the driver entry
// point, looked up once at run time.
#include "dq_tma.cuh"

#include <mutex>

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static std::once_flag once;
    static EncodeTiledFn fn = nullptr;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            (void)cudaGetLastError();
    });
    return fn;
}

}  // namespace

bool dq_encode_tensor_map(CUtensorMap* map, CUtensorMapDataType type, uint32_t rank, const void* base,
                          const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box,
                          CUtensorMapSwizzle swizzle)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t d[5], s[4];
    cuuint32_t b[5], e[5];
    for (uint32_t i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; e[i] = 1; }
    for (uint32_t i = 0; i + 1 < rank; ++i) s[i] = strides_bytes[i];
    const CUresult rc = fn(map, type, rank, const_cast<void*>(base), d, s, b, e, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS;
}

// ---- wait limits (see WaitLimits) ----
namespace {
constexpr unsigned long long kDefaultWaitNs = 2000000000ull;
std::mutex g_limits_mu;
WaitLimits g_limits = {kDefaultWaitNs, 0u, 0u};
}  // namespace

WaitLimits dq_wait_limits()
{
    std::lock_guard<std::mutex> lock(g_limits_mu);
    return g_limits;
}

extern "C" void dq_debug_set_wait_limits(uint64_t limit_ns, int32_t lose_first_wait)
{
    std::lock_guard<std::mutex> lock(g_limits_mu);
    g_limits.ns = limit_ns ? limit_ns : kDefaultWaitNs;
    g_limits.lose_first = lose_first_wait ? 1u : 0u;
}
