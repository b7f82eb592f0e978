// Device-side arithmetic of the quantizer: the Philox4x32-10 block function,
// the per-element encoder of Eq. 5/6 and the register bit packer.  All of it
// is written for a thread that owns one 32-element group, so that every shift
// and word index is a compile-time constant once B (bits per code) is known.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

// Round keys of Philox4x32-10: key + r * (0x9E3779B9, 0xBB67AE85).  They are the
// same for the whole grid, so the host computes them and they travel as kernel
// arguments (constant bank), which keeps them out of the register file.
struct PhiloxKeys {
    uint32_t k0[10];
    uint32_t k1[10];
};

inline PhiloxKeys make_philox_keys(uint64_t seed)
{
    PhiloxKeys k;
    uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        k.k0[r] = a;
        k.k1[r] = b;
        a += 0x9E3779B9u;
        b += 0xBB67AE85u;
    }
    return k;
}

#ifdef __CUDACC__

// One Philox4x32-10 block (Salmon et al., SC'11): ten rounds of two 32x32->64
// multiplies and a three-way xor with the counter words and the round key.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              const PhiloxKeys& K, uint32_t (&out)[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ K.k0[r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ K.k1[r];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Eq. 5/6 for one element: r = min(|g| * inv, s); l = floor(r); p_r = r - l;
// level = l + [u < p_r]; code = sign << (B-1) | level.  Every fp32 operation
// rounds on its own (no fused multiply-add), in this order.
// floor: r + 2^23 rounded toward -inf leaves floor(r) in the low mantissa bits
// (0 <= r <= 32767), one full-rate add instead of a conversion.
template <int B>
__device__ __forceinline__ uint32_t encode(const float g, const float inv, const float sf, const uint32_t w)
{
    const uint32_t gb = __float_as_uint(g);
    if constexpr (B == 1) return gb >> 31;
    const float r = fminf(__fmul_rn(fabsf(g), inv), sf);
    const float t = __fadd_rd(r, 8388608.0f);
    const float pr = __fsub_rn(r, __fsub_rn(t, 8388608.0f));          // exact
    const float u = __fmul_rn(__uint2float_rn(w >> 8), 0x1p-24f);     // exact, [0, 1)
    const uint32_t lv = __float_as_uint(t) + (u < pr ? 1u : 0u);
    constexpr uint32_t kLow = (1u << (B - 1)) - 1u;
    constexpr uint32_t kSign = 1u << (B - 1);
    return (lv & kLow) | ((gb >> (32 - B)) & kSign);
}

// OR code number E of a group into the group's B-word little-endian bit string.
template <int B, int E>
__device__ __forceinline__ void put_code(uint32_t (&acc)[B], const uint32_t code)
{
    constexpr int bit = E * B;
    constexpr int w = bit >> 5;
    constexpr int sh = bit & 31;
    if constexpr (sh == 0) acc[w] = code;            // first code of a word
    else acc[w] |= code << sh;
    if constexpr (sh + B > 32) acc[w + 1] = code >> (32 - sh);   // straddles into a fresh word
}

// Code number E of a group, moved to the top of a register: sign at bit 31, the
// level right below it, whatever follows in the stream in the low 32-B bits.
template <int B, int E>
__device__ __forceinline__ uint32_t top_code(const uint32_t (&wd)[B])
{
    constexpr int bit = E * B;
    constexpr int w = bit >> 5;
    constexpr int sh = bit & 31;
    constexpr int end = sh + B;                      // one past the code's last bit, in word w
    if constexpr (end == 32) return wd[w];
    else if constexpr (end < 32) return wd[w] << (32 - end);
    else return __funnelshift_l(wd[w], wd[w + 1], 64 - end);   // straddles words w, w+1
}

#endif  // __CUDACC__
