// Device-side building blocks of the MVUE prune: the counter-based random words,
// the 1:2 and 2:4 block estimators and small packing helpers.
//
// Every floating-point step that decides a mask or a kept value is written with
// the explicit round-to-nearest intrinsics (__fadd_rn, __fmul_rn, ...) so that the
// compiler can neither fuse a multiply with an add nor reorder a sum: the result
// is a pure function of the inputs and the seed, bit for bit.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

namespace mvue {

// ---------------------------------------------------------------------------
// Philox4x32 with ten rounds (Salmon et al., SC'11).  The ten round keys depend
// on the seed only, so the host expands them once and passes them by value; in
// the kernel they sit in the constant bank and cost no instruction.
// ---------------------------------------------------------------------------
struct RoundKeys {
    uint32_t k0[10];
    uint32_t k1[10];
};

__host__ inline RoundKeys make_round_keys(uint64_t seed) {
    RoundKeys rk;
    uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        rk.k0[r] = a;
        rk.k1[r] = b;
        a += 0x9E3779B9u;
        b += 0xBB67AE85u;
    }
    return rk;
}

// Words of generator call number `call` (counter = (lo, hi, 0, 0)).
__device__ __forceinline__ uint4 philox4x32_10(uint64_t call, const RoundKeys& rk) {
    uint32_t c0 = (uint32_t)call, c1 = (uint32_t)(call >> 32), c2 = 0u, c3 = 0u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ rk.k0[r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ rk.k1[r];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    return make_uint4(c0, c1, c2, c3);
}

// eps in [0,1): top 24 bits of the word, exact in binary32.
__device__ __forceinline__ float uniform24(uint32_t word) {
    return __fmul_rn(__uint2float_rn(word >> 8), 5.9604644775390625e-08f);
}

// ---------------------------------------------------------------------------
// MVUE 1:2 (Sec. 4.1): keep a_1 iff eps (|a_1|+|a_2|) < |a_1|; the survivor
// becomes sign(a_i)(|a_1|+|a_2|).  b1, b2 are the binary32 bit patterns.
// Returns the kept index; *kept_bits receives the new value's bit pattern.
// A zero is never preferred to a non-zero; an all-zero block keeps index 0, +0.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t mvue_1of2(uint32_t b1, uint32_t b2, uint32_t word,
                                              uint32_t* kept_bits) {
    const float m1 = __uint_as_float(b1 & 0x7FFFFFFFu);
    const float m2 = __uint_as_float(b2 & 0x7FFFFFFFu);
    const float S = __fadd_rn(m1, m2);
    const float t = __fmul_rn(uniform24(word), S);
    const uint32_t idx = (m2 != 0.0f && !(t < m1)) ? 1u : 0u;
    const uint32_t sign = (idx ? b2 : b1) & 0x80000000u;
    const uint32_t sbits = __float_as_uint(S);
    *kept_bits = sbits ? (sbits | sign) : 0u;
    return idx;
}

// ---------------------------------------------------------------------------
// MVUE 2:4 (marginals: Sec. 4.2; joint law: App. A.2).
//
// Sorted magnitudes s1 <= s2 <= s3 <= s4 (ties by position).  All three cases of
// the appendix are evaluated as one cumulative table over the pairs 13, 14, 23,
// 24 (else 34) with numerators w and common denominator D:
//   case 3 (s4 >= s1+s2+s3): w = (0, s1, 0, s2),                         D = s1+s2+s3
//   case 1 (s4 <= 2 s1 + s3): w = (2s1+s3-s4, 2s1-s3+s4, 2s2+s3-s4, 2s2-s3+s4), D = 2 sum
//   case 2 (otherwise):       w = (0, 2s1, s1+s2+s3-s4, s2-s1+s4-s3),    D = sum
// and the pair is the first whose cumulative numerator exceeds eps * D.
// Kept values: case 3 -> dominant unchanged, the other sign * (s1+s2+s3);
// cases 1, 2 -> both sign * sum / 2.
//
// Key: a 64-bit (or, when the low two magnitude bits are known to be zero, a
// 32-bit) integer whose order is (magnitude, position).
// ---------------------------------------------------------------------------
template <typename KeyT>
__device__ __forceinline__ void cswap(KeyT& a, KeyT& b) {
    const KeyT lo = a < b ? a : b;
    const KeyT hi = a < b ? b : a;
    a = lo;
    b = hi;
}

template <bool kLowBitsFree>
struct SortKey;

template <>
struct SortKey<true> {   // magnitudes widened from bf16: the low 16 bits are zero
    using T = uint32_t;
    static __device__ __forceinline__ T make(uint32_t mag_bits, uint32_t pos) { return mag_bits | pos; }
    static __device__ __forceinline__ float mag(T k) { return __uint_as_float(k & ~3u); }
    static __device__ __forceinline__ uint32_t pos(T k) { return k & 3u; }
};

template <>
struct SortKey<false> {  // arbitrary binary32 magnitudes
    using T = uint64_t;
    static __device__ __forceinline__ T make(uint32_t mag_bits, uint32_t pos) {
        return ((uint64_t)mag_bits << 2) | pos;
    }
    static __device__ __forceinline__ float mag(T k) { return __uint_as_float((uint32_t)(k >> 2)); }
    static __device__ __forceinline__ uint32_t pos(T k) { return (uint32_t)k & 3u; }
};

// b0..b3: binary32 bit patterns of the block.  Outputs: nibble idx0 | idx1 << 2
// (idx0 < idx1) and the two new values' bit patterns in that order.
template <bool kLowBitsFree>
__device__ __forceinline__ void mvue_2of4(uint32_t b0, uint32_t b1, uint32_t b2, uint32_t b3,
                                          uint32_t word, uint32_t* nibble, uint32_t* v0_bits,
                                          uint32_t* v1_bits) {
    using SK = SortKey<kLowBitsFree>;
    typename SK::T k1 = SK::make(b0 & 0x7FFFFFFFu, 0u);
    typename SK::T k2 = SK::make(b1 & 0x7FFFFFFFu, 1u);
    typename SK::T k3 = SK::make(b2 & 0x7FFFFFFFu, 2u);
    typename SK::T k4 = SK::make(b3 & 0x7FFFFFFFu, 3u);
    cswap(k1, k2); cswap(k3, k4); cswap(k1, k3); cswap(k2, k4); cswap(k2, k3);

    const float s1 = SK::mag(k1), s2 = SK::mag(k2), s3 = SK::mag(k3), s4 = SK::mag(k4);
    const float S12 = __fadd_rn(s1, s2);
    const float S3 = __fadd_rn(S12, s3);
    const float S = __fadd_rn(S3, s4);

    const float two_s1 = __fadd_rn(s1, s1);
    const float two_s2 = __fadd_rn(s2, s2);
    const bool capped = s4 >= S3;                               // case 3
    const bool tight = s4 <= __fadd_rn(two_s1, s3);             // case 1 (when not capped)

    // case 1 numerators
    const float a13 = fmaxf(0.0f, __fsub_rn(__fadd_rn(two_s1, s3), s4));
    const float a14 = fmaxf(0.0f, __fadd_rn(__fsub_rn(two_s1, s3), s4));
    const float a23 = fmaxf(0.0f, __fsub_rn(__fadd_rn(two_s2, s3), s4));
    const float a24 = fmaxf(0.0f, __fadd_rn(__fsub_rn(two_s2, s3), s4));
    // case 2 numerators
    const float c23 = fmaxf(0.0f, __fsub_rn(S3, s4));
    const float c24 = fmaxf(0.0f, __fadd_rn(__fsub_rn(s2, s1), __fsub_rn(s4, s3)));

    const float w13 = (tight && !capped) ? a13 : 0.0f;
    const float w14 = capped ? s1 : (tight ? a14 : two_s1);
    const float w23 = capped ? 0.0f : (tight ? a23 : c23);
    const float w24 = capped ? s2 : (tight ? a24 : c24);
    const float D = capped ? S3 : (tight ? __fadd_rn(S, S) : S);

    const float t = __fmul_rn(uniform24(word), D);
    const float c1 = w13;
    const float c2 = __fadd_rn(c1, w14);
    const float c3 = __fadd_rn(c2, w23);
    const float c4 = __fadd_rn(c3, w24);
    // index of the first cumulative numerator above t: 0..3 -> pairs 13,14,23,24; 4 -> pair 34
    const uint32_t pair = (uint32_t)!(t < c1) + (uint32_t)!(t < c2) + (uint32_t)!(t < c3) + (uint32_t)!(t < c4);

    const uint32_t ka = pair >> 1;                              // rank of the smaller survivor: 0,0,1,1,2
    const bool b_is_top = (pair & 1u) | (pair >> 2);            // larger survivor is rank 3 (else rank 2)
    const typename SK::T key_a = ka == 0 ? k1 : (ka == 1 ? k2 : k3);
    const typename SK::T key_b = b_is_top ? k4 : k3;
    uint32_t ia = SK::pos(key_a), ib = SK::pos(key_b);

    const float half = __fmul_rn(0.5f, S);
    uint32_t va = __float_as_uint(capped ? S3 : half);
    uint32_t vb = __float_as_uint(capped ? s4 : half);
    // signs of the original elements at positions ia, ib
    const uint32_t sa = ia == 0 ? b0 : (ia == 1 ? b1 : (ia == 2 ? b2 : b3));
    const uint32_t sb = ib == 0 ? b0 : (ib == 1 ? b1 : (ib == 2 ? b2 : b3));
    va |= sa & 0x80000000u;
    vb |= sb & 0x80000000u;

    if (S3 == 0.0f) {            // at most one non-zero: a zero fills the lowest free position with +0
        ia = (ib == 0u) ? 1u : 0u;
        va = 0u;
    }
    if (s4 == 0.0f) {            // all zero
        ia = 0u; ib = 1u; va = 0u; vb = 0u;
    }
    const bool a_first = ia < ib;
    *nibble = a_first ? (ia | (ib << 2)) : (ib | (ia << 2));
    *v0_bits = a_first ? va : vb;
    *v1_bits = a_first ? vb : va;
}

// Two binary32 values -> one 32-bit word of two bf16 (round to nearest even), lo first.
__device__ __forceinline__ uint32_t pack_bf16x2(uint32_t lo_bits, uint32_t hi_bits) {
    __nv_bfloat162 p = __floats2bfloat162_rn(__uint_as_float(lo_bits), __uint_as_float(hi_bits));
    return *reinterpret_cast<uint32_t*>(&p);
}

}  // namespace mvue
