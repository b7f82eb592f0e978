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
// level = l + [u <= p_r] with u = 1 - v, v = (2k + 1) / 2^24, k the top 23 bits of
// the element's Philox word; code = sign << (B-1) | level.
// Every fp32 operation rounds on its own (no fused multiply-add).
//  * v: the bits 0x3F800000 | k are the float 1 + k / 2^23; subtracting
//    1 - 2^-24 from it is exact and leaves (2k + 1) / 2^24.
//  * level = floor(r + v): u <= p_r  <=>  p_r + v >= 1.  An add rounded toward
//    -inf never crosses an integer downwards, so floor(fl(r + v)) is the floor
//    of the exact sum; adding 2^23, again toward -inf, leaves that integer in
//    the low mantissa bits (0 <= r + v < 32768).  No conversion instruction.
template <int B>
__device__ __forceinline__ uint32_t encode(const float g, const float inv, const float sf, const uint32_t w)
{
    const uint32_t gb = __float_as_uint(g);
    if constexpr (B == 1) return gb >> 31;
    const float r = fminf(__fmul_rn(fabsf(g), inv), sf);
    const float x = __uint_as_float(__funnelshift_r(w, 0x7Fu, 9));      // 1 + k 2^-23
    const float v = __fsub_rn(x, 0.99999994f);                          // (2k + 1) 2^-24, exact
    const float t = __fadd_rd(__fadd_rd(r, v), 8388608.0f);
    constexpr uint32_t kLow = (1u << (B - 1)) - 1u;
    return (__float_as_uint(t) & kLow) | ((gb >> (32 - B)) & ~kLow);    // bits >= B are zero
}

// Appends code number E of a group to the group's little-endian bit string.
// `cur` is a shift register: a funnel shift pushes the B code bits in at the
// top, so after 32 bits the first code sits at bit 0 and the word is complete.
// A code that straddles two words finishes the current word with its low bits
// and seeds the next one with itself at the top; the surplus low bits fall off
// as that word fills up.
template <int B, int E>
__device__ __forceinline__ void push_code(uint32_t (&acc)[B], uint32_t& cur, const uint32_t code)
{
    constexpr int bit = E * B;
    constexpr int w = bit >> 5;
    constexpr int sh = bit & 31;
    constexpr int end = sh + B;
    if constexpr (end < 32) {
        if constexpr (sh == 0) cur = code << (32 - B);
        else cur = __funnelshift_r(cur, code, B);
    } else if constexpr (end == 32) {
        if constexpr (sh == 0) acc[w] = code;                    // B == 32 never happens; kept for completeness
        else acc[w] = __funnelshift_r(cur, code, B);
    } else {
        acc[w] = __funnelshift_r(cur, code, 32 - sh);
        cur = code << (32 - B);
    }
}

// Decoding for the average.  The level bits of a code are masked out of the
// word where they stand and OR-ed under the exponent of 2^23: the float
// 2^23 + level * 2^k minus 2^23 is level * 2^k exactly, one logic operation and
// one add with no shift and no int-to-float conversion.  The sign bit is shifted
// to bit 31 and OR-ed into that float.  k depends only on the code's position
// E, so the caller removes 2^k once after all workers have been accumulated
// (decoded_shift).  Codes whose level bits reach above bit 22 of their word are
// decoded from the word's upper half (shifted down by 16 once per word) or,
// when they straddle two words, from a funnel shift.
template <int B, int E>
struct CodePos {
    static constexpr int bit = E * B;
    static constexpr int w = bit >> 5;
    static constexpr int sh = bit & 31;
    static constexpr int end = sh + B;            // one past the sign bit, counted in word w
    static constexpr bool straddles = end > 32;
    static constexpr bool in_place = !straddles && (end - 1) <= 23;
    static constexpr bool in_upper = !straddles && !in_place && sh >= 16;
    // power of two the decoded magnitude carries
    static constexpr int k = in_place ? sh : (in_upper ? sh - 16 : 0);
};

template <int B, int E>
__device__ __forceinline__ float decode_code(const uint32_t (&wd)[B], const uint32_t (&hi)[B])
{
    using P = CodePos<B, E>;
    constexpr uint32_t kLevel = (1u << (B - 1)) - 1u;
    constexpr uint32_t kMagic = 0x4B000000u;     // 2^23
    uint32_t m, t;
    if constexpr (P::in_place) {
        m = (wd[P::w] & (kLevel << P::k)) | kMagic;
        t = (P::end == 32) ? wd[P::w] : (wd[P::w] << (32 - P::end));
    } else if constexpr (P::in_upper) {
        m = (hi[P::w] & (kLevel << P::k)) | kMagic;
        t = (P::end == 32) ? wd[P::w] : (wd[P::w] << (32 - P::end));
    } else if constexpr (!P::straddles) {
        m = ((wd[P::w] >> P::sh) & kLevel) | kMagic;
        t = (P::end == 32) ? wd[P::w] : (wd[P::w] << (32 - P::end));
    } else {
        m = (__funnelshift_r(wd[P::w], wd[P::w + 1], P::sh) & kLevel) | kMagic;
        t = wd[P::w + 1] << (64 - P::end);
    }
    const float d = __uint_as_float(m) - 8388608.0f;                  // level * 2^k, exact
    return __uint_as_float(__float_as_uint(d) | (t & 0x80000000u));
}

// does any code of word W need the word's upper half?
template <int B, int W, int E = 0>
struct NeedsUpper {
    static constexpr bool value =
        ((CodePos<B, E>::w == W) && CodePos<B, E>::in_upper) || NeedsUpper<B, W, E + 1>::value;
};
template <int B, int W>
struct NeedsUpper<B, W, 32> {
    static constexpr bool value = false;
};

#endif  // __CUDACC__
