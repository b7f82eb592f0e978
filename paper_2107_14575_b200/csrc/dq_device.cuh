// Device-side arithmetic of the quantizer: the Philox4x32-10 block function,
// the per-element encoder of Eq. 5/6, the register bit packer and the in-place
// decoder of the average.  All of it is written for a thread that owns one
// 32-element group, so that every shift and word index is a compile-time
// constant once B (bits per code) is known.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "dq.h"

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

// The three places where the members of the l_p family differ.  P = DQ_NORM_L2: sum of
// squares, square root at the end.  P = DQ_NORM_LINF: running maximum of the magnitudes
// (max.NaN, so that a NaN entry is not skipped and reaches the status word), nothing at the end.
__device__ __forceinline__ float max_nan(const float a, const float b)
{
    float d;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}
template <int P>
__device__ __forceinline__ float take(const float acc, const float x)
{
    if constexpr (P == DQ_NORM_L2) return fmaf(x, x, acc);
    else return max_nan(acc, fabsf(x));
}
template <int P>
__device__ __forceinline__ float join(const float a, const float b)
{
    if constexpr (P == DQ_NORM_L2) return a + b;
    else return max_nan(a, b);
}
template <int P>
__device__ __forceinline__ float finish(const float a)
{
    if constexpr (P == DQ_NORM_L2) return sqrtf(a);
    else return a;
}

// ---- l2 norms of buckets whose squares leave the fp32 range ---------------------------------
// The sum of squares S of a bucket, accumulated with fused multiply-adds, is taken as it is when
// 2^-100 <= S < inf: no square overflowed, every term that fell into the subnormal range (or
// vanished) is below 2^-126 and so below 2^-26 of S, and sqrt(S) >= 2^-50 dominates each of
// those entries while sqrt(fl(g^2)) = |g| for the others.  Outside that range (a bucket of tiny
// entries, an overflowed square, a NaN) the bucket is reduced again: first its largest magnitude
// (exact), then the squares of the entries scaled by the power of two that brings that magnitude
// into [1, 2), in the same order as before, and the square root is scaled back.  The functors
// below are the three reductions; the kernels supply the loads and the joins between threads.
__device__ __forceinline__ bool l2_sum_in_range(const float sum)
{
    return sum >= 0x1p-100f && sum <= 3.402823466e38f;       // false for a NaN as well
}
struct SumSquares {
    __device__ __forceinline__ float take(const float acc, const float x) const { return fmaf(x, x, acc); }
    __device__ __forceinline__ float join(const float a, const float b) const { return a + b; }
};
struct MaxMagnitude {
    __device__ __forceinline__ float take(const float acc, const float x) const { return max_nan(acc, fabsf(x)); }
    __device__ __forceinline__ float join(const float a, const float b) const { return max_nan(a, b); }
};
struct ScaledSquares {
    int e;                          // the entries are multiplied by 2^-e first (exact, or negligible when it underflows)
    __device__ __forceinline__ float take(const float acc, const float x) const
    {
        const float y = scalbnf(x, -e);
        return fmaf(y, y, acc);
    }
    __device__ __forceinline__ float join(const float a, const float b) const { return a + b; }
};
// the reduction a member of the family starts with
template <int P> struct FamilyReduction { using type = SumSquares; };
template <> struct FamilyReduction<DQ_NORM_LINF> { using type = MaxMagnitude; };
// Exponent to scale by, from the bucket's largest magnitude (0 when there is nothing to scale:
// an all-zero bucket, an infinity or a NaN, for which rescaled_l2 returns the magnitude itself).
__device__ __forceinline__ bool magnitude_scalable(const float mx) { return mx > 0.0f && mx <= 3.402823466e38f; }
__device__ __forceinline__ int scale_exponent(const float mx) { return magnitude_scalable(mx) ? ilogbf(mx) : 0; }
// The norm from the largest magnitude and the scaled sum of squares.  An overflow of the
// result (entries near the top of the fp32 range) gives infinity, as the fp64 definition
// rounded to fp32 does.
__device__ __forceinline__ float rescaled_l2(const float mx, const float scaled_sum, const int e)
{
    if (!magnitude_scalable(mx)) return mx;                  // 0, infinity or NaN
    return scalbnf(sqrtf(scaled_sum), e);
}

// (a & mask) | c as one three-input logic operation.  `c` must come from a register the
// compiler cannot fold (callers pass the exponent pattern of 2^23 from a kernel
// argument), otherwise two immediates would cost two instructions.
__device__ __forceinline__ uint32_t and_or(const uint32_t a, const uint32_t mask, const uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(mask), "r"(c));
    return d;
}

// Two fp32 values in one 64-bit register pair, for the packed two-lane forms of sm_100
// (add.f32x2, mul.f32x2, fma.f32x2).
__device__ __forceinline__ uint64_t pack_pair(const uint32_t lo, const uint32_t hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack_pair(const uint64_t v, float& lo, float& hi)
{
    uint32_t a, b;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
    lo = __uint_as_float(a);
    hi = __uint_as_float(b);
}
__device__ __forceinline__ uint64_t add_pair(const uint64_t a, const uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t fma_pair(const uint64_t a, const uint64_t b, const uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
// Eq. 5/6 for one element.  With x = RZ(g * inv), inv = RZ(s / norm), the element's
// position on the level grid and v = (2k + 1) / 2^17 its uniform draw (k a 16-bit
// half of a Philox word), the code is floor(x + v) + s: for either sign the
// neighbour of x away from zero is taken with probability frac(|x|), Eq. 6.
//  * Both roundings are toward zero, so |x| <= s whenever |g| <= norm (a bucket's
//    norm dominates its entries): no clamp, no absolute value, no sign handling.
//  * HALF selects the low (0) or high (1) 16 bits of w.  The bits
//    0x3F800040 | k << 7 are the float 1 + v (the constant comes in a register the
//    compiler cannot fold, see and_or).
//  * An add rounded toward -inf never crosses an integer downwards, so
//    floor(fl(x + (1 + v))) is the floor of the exact sum; adding 2^23 + s - 1,
//    again toward -inf, leaves floor(x + v) + s in the low mantissa bits.  No
//    conversion instruction.
// The result carries the code in its low B bits and the exponent bits of 2^23
// above them; the packer drops everything above bit B-1.
template <int B, int HALF>
__device__ __forceinline__ uint32_t encode(const float g, const float inv, const uint32_t w, const uint32_t one_bits)
{
    constexpr int s = (1 << (B - 1)) - 1;
    const float x = __fmul_rz(g, inv);
    // k << 7 in place: the high half comes down by a multiply-high (w * 2^23 >> 32 = w >> 9),
    // which runs on the multiplier and leaves the logic pipe to the generator
    const uint32_t kbits = HALF ? __umulhi(w, 0x00800000u) : (w << 7);
    const float one_plus_v = __uint_as_float(and_or(kbits, 0x007FFF80u, one_bits));   // one_bits = 0x3F800040
    const float t = __fadd_rd(__fadd_rd(x, one_plus_v), 8388608.0f + (float)(s - 1));
    return __float_as_uint(t);
}

// inv = RZ(s / norm), the scale of Eq. 5 rounded toward zero (0 for norm < 2^-100, where the
// quotient could overflow, and for a NaN norm).  Written out instead of calling the library's
// division so that it stays inline: reciprocal estimate r (relative error <= 2^-23), q = s * r,
// one Newton step q <- q + (s - q * norm) * r, which brings q to within 2^-44 of the quotient
// before its rounding, i.e. to one of the two floats that enclose s / norm; the sign of the
// exactly rounded residual s - q * norm then tells which, and the upper one steps down an ulp.
// Norms above 2^125, whose reciprocal estimate would be flushed to zero, take the library route.
__device__ __forceinline__ float inv_scale(const float sf, const float norm)
{
    if (!(norm >= 0x1p-100f)) return 0.0f;
    if (norm > 0x1p125f) return __fdiv_rz(sf, norm);
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(norm));
    float q = __fmul_rn(sf, r);
    q = __fmaf_rn(__fmaf_rn(-q, norm, sf), r, q);
    const float e = __fmaf_rn(-q, norm, sf);
    return __uint_as_float(__float_as_uint(q) - (e < 0.0f ? 1u : 0u));
}

// Appends code number E of a group to the group's little-endian bit string.
// `cur` is a shift register: a funnel shift pushes the B code bits in at the
// top, so after 32 bits the first code sits at bit 0 and the word is complete.
// A code that straddles two words finishes the current word with its low bits
// and seeds the next one with itself at the top; the surplus low bits fall off
// as that word fills up.  Bits of `code` above B-1 never reach a word.
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
        acc[w] = __funnelshift_r(cur, code, B);
    } else {
        acc[w] = __funnelshift_r(cur, code, 32 - sh);
        cur = code << (32 - B);
    }
}

// The B words of a group whose 32 codes all equal s: what a zero scale gives (x = 0 and
// floor(0 + v) = 0 for every draw v in (0, 1)), so such a group needs neither uniforms nor
// arithmetic.  Everything here folds to constants.
template <int B, int E>
struct PushSame {
    static __device__ __forceinline__ void run(uint32_t (&acc)[B], uint32_t& cur, const uint32_t code)
    {
        push_code<B, E>(acc, cur, code);
        PushSame<B, E + 1>::run(acc, cur, code);
    }
};
template <int B>
struct PushSame<B, 32> {
    static __device__ __forceinline__ void run(uint32_t (&)[B], uint32_t&, const uint32_t) {}
};
template <int B>
__device__ __forceinline__ void zero_group_words(uint32_t (&acc)[B])
{
    uint32_t cur = 0;
    PushSame<B, 0>::run(acc, cur, (1u << (B - 1)) - 1u);
}

// Stores the B words of one group into the warp's staging area (stride B words
// between lanes; the widest access the alignment allows keeps bank conflicts low).
template <int B>
__device__ __forceinline__ void stage_words(uint32_t* __restrict__ dst, const uint32_t (&acc)[B])
{
    if constexpr (B % 4 == 0) {
#pragma unroll
        for (int i = 0; i < B / 4; ++i)
            reinterpret_cast<uint4*>(dst)[i] = make_uint4(acc[4 * i], acc[4 * i + 1], acc[4 * i + 2], acc[4 * i + 3]);
    } else if constexpr (B % 2 == 0) {
#pragma unroll
        for (int i = 0; i < B / 2; ++i)
            reinterpret_cast<uint2*>(dst)[i] = make_uint2(acc[2 * i], acc[2 * i + 1]);
    } else {
#pragma unroll
        for (int i = 0; i < B; ++i) dst[i] = acc[i];
    }
}

// Encodes elements 8C .. 8C+7 of a group (one Philox block) and appends the codes.
template <int B, int C>
__device__ __forceinline__ void encode_block(uint32_t (&acc)[B], uint32_t& cur, const float4 lo, const float4 hi,
                                             const float inv, const uint32_t q, const uint32_t m,
                                             const uint32_t step, const PhiloxKeys& keys, const uint32_t ob)
{
    uint32_t w[4];
    philox4x32_10(q, 0u, m, step, keys, w);
    push_code<B, 8 * C + 0>(acc, cur, encode<B, 0>(lo.x, inv, w[0], ob));
    push_code<B, 8 * C + 1>(acc, cur, encode<B, 1>(lo.y, inv, w[0], ob));
    push_code<B, 8 * C + 2>(acc, cur, encode<B, 0>(lo.z, inv, w[1], ob));
    push_code<B, 8 * C + 3>(acc, cur, encode<B, 1>(lo.w, inv, w[1], ob));
    push_code<B, 8 * C + 4>(acc, cur, encode<B, 0>(hi.x, inv, w[2], ob));
    push_code<B, 8 * C + 5>(acc, cur, encode<B, 1>(hi.y, inv, w[2], ob));
    push_code<B, 8 * C + 6>(acc, cur, encode<B, 0>(hi.z, inv, w[3], ob));
    push_code<B, 8 * C + 7>(acc, cur, encode<B, 1>(hi.w, inv, w[3], ob));
}

// Decoding for the average.  A code holds s + sgn * level.  Its B bits are
// masked out of the word where they stand and OR-ed under the exponent of 2^23:
// that float is 2^23 + code * 2^k, and subtracting 2^23 + s * 2^k leaves
// sgn * level * 2^k exactly -- one logic operation and one add, no shift, no
// int-to-float conversion, no sign handling.  k depends only on the code's
// position E, so the caller removes 2^k once after all workers have been
// accumulated.  Codes that reach above bit 22 of their word are decoded from the
// word's upper half (shifted down by 16 once per word) or, when they straddle
// two words, from a funnel shift.
template <int B, int E>
struct CodePos {
    static constexpr int bit = E * B;
    static constexpr int w = bit >> 5;
    static constexpr int sh = bit & 31;
    static constexpr int end = sh + B;            // one past the code's last bit, counted in word w
    static constexpr bool straddles = end > 32;
    static constexpr bool in_place = !straddles && end <= 23;
    static constexpr bool in_upper = !straddles && !in_place && sh >= 16;
    // power of two the decoded value carries
    static constexpr int k = in_place ? sh : (in_upper ? sh - 16 : 0);
};

template <int B, int E>
__device__ __forceinline__ float decode_code(const uint32_t (&wd)[B], const uint32_t (&hi)[B], const uint32_t magic)
{
    using P = CodePos<B, E>;
    constexpr uint32_t kCode = (1u << B) - 1u;
    constexpr int s = (1 << (B - 1)) - 1;
    uint32_t m;                                  // magic = 0x4B000000, the bits of 2^23
    if constexpr (P::in_place) {
        m = and_or(wd[P::w], kCode << P::k, magic);
    } else if constexpr (P::in_upper) {
        m = and_or(hi[P::w], kCode << P::k, magic);
    } else if constexpr (!P::straddles) {
        m = and_or(wd[P::w] >> P::sh, kCode, magic);
    } else {
        m = and_or(__funnelshift_r(wd[P::w], wd[P::w + 1], P::sh), kCode, magic);
    }
    return __uint_as_float(m) - (8388608.0f + (float)(s << P::k));      // sgn * level * 2^k, exact
}

// The same decoding for two neighbouring codes at once with the packed two-lane fp32 forms of
// sm_100 (add.f32x2, fma.f32x2 on 64-bit register pairs): one packed subtract and one packed FMA
// replace two of each, which halves the operand traffic of the accumulation (the scalar form
// keeps 32 accumulators, a scale and an immediate in flight per code).  Results are bit for bit
// those of decode_code: the same exact subtract, the same single rounding in the FMA.
// bits of the float 2^23 + code * 2^k for code E of a group (the part of decode_code before the subtract)
template <int B, int E>
__device__ __forceinline__ uint32_t code_bits(const uint32_t (&wd)[B], const uint32_t (&hi)[B], const uint32_t magic)
{
    using P = CodePos<B, E>;
    constexpr uint32_t kCode = (1u << B) - 1u;
    if constexpr (P::in_place) return and_or(wd[P::w], kCode << P::k, magic);
    else if constexpr (P::in_upper) return and_or(hi[P::w], kCode << P::k, magic);
    else if constexpr (!P::straddles) return and_or(wd[P::w] >> P::sh, kCode, magic);
    else return and_or(__funnelshift_r(wd[P::w], wd[P::w + 1], P::sh), kCode, magic);
}
// bits of the float -(2^23 + s * 2^k): 2^23 + n has the mantissa n for every integer n < 2^23
template <int B, int E>
struct NegOffsetBits {
    static constexpr uint32_t value = 0xCB000000u + (uint32_t)(((1 << (B - 1)) - 1) << CodePos<B, E>::k);
};
// (sgn * level * 2^k0, sgn * level * 2^k1) of codes 2Q and 2Q + 1 times (scale, scale), added to acc2
template <int B, int Q>
__device__ __forceinline__ uint64_t accumulate_pair(const uint64_t acc2, const uint32_t (&wd)[B], const uint32_t (&hi)[B],
                                                    const uint64_t scale2, const uint32_t magic)
{
    constexpr uint64_t kOff = (uint64_t)NegOffsetBits<B, 2 * Q>::value | ((uint64_t)NegOffsetBits<B, 2 * Q + 1>::value << 32);
    const uint64_t m = pack_pair(code_bits<B, 2 * Q>(wd, hi, magic), code_bits<B, 2 * Q + 1>(wd, hi, magic));
    return fma_pair(add_pair(m, kOff), scale2, acc2);
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
