// Device-side building blocks of the MVUE prune: the counter-based random words,
// the 1:2 and 2:4 block estimators and small packing helpers.
//
// Every floating-point step that decides a mask or a kept value is written with
// the explicit round-to-nearest intrinsics (__fadd_rn, __fmul_rn, __fmaf_rn with an
// exact power-of-two product) so that the compiler can neither fuse nor reorder:
// the result is a pure function of the inputs and the seed, bit for bit.
//
// The prune is bound by the integer/logic pipe, not by memory, unless the
// selection is written tightly; the bf16 paths below therefore keep compares,
// selects and bit operations to a minimum and push what they can onto the
// floating-point and multiply pipes.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

namespace mvue {

// First statement of every kernel launched with launch_dependent(): returns once the grids this launch depends on have
// completed and their stores are visible (at once when the kernel was launched the ordinary way).
__device__ __forceinline__ void grid_dependency_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

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

// Words of generator call number `call` (counter = (lo, hi, stream, 0); the selection draws use stream 0, the
// rounding bits of the survivors stream 1).
__device__ __forceinline__ uint4 philox4x32_10(uint64_t call, const RoundKeys& rk, uint32_t stream = 0u) {
    uint32_t c0 = (uint32_t)call, c1 = (uint32_t)(call >> 32), c2 = stream, c3 = 0u;
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

// The top 24 bits of a word as a float (exact): eps * 2^24.
__device__ __forceinline__ float top24(uint32_t word) {
    return __uint2float_rn(__umulhi(word, 1u << 24));   // high product = word >> 8, on the multiply pipe
}

// Two binary32 values -> one word of two bf16 (round to nearest even), lo first.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&p);
}

// Two binary32 survivors -> one word of two bf16 (lo first): to nearest even, or (kSR) stochastically -- the low 16 bits
// of a survivor are the probability, over 2^16, of its upper bf16 neighbour, and adding the slot's 16 random bits
// (rnd = bits of the low slot | bits of the high slot << 16) carries into the upper half exactly that often:
// stored = (bits + r) >> 16, whose expectation over r is the survivor itself.
template <bool kSR>
__device__ __forceinline__ uint32_t pack_out(float lo, float hi, uint32_t rnd) {
    if (!kSR) return pack_bf16x2(lo, hi);
    return __byte_perm(__float_as_uint(lo) + (rnd & 0xFFFFu), __float_as_uint(hi) + (rnd >> 16), 0x7632u);
}

// ===========================================================================
// MVUE 1:2 (Sec. 4.1): keep a_1 iff eps (|a_1|+|a_2|) < |a_1| (or a_2 = 0); the
// survivor becomes sign(a_i)(|a_1|+|a_2|).
// ===========================================================================
// f0, f1: the pair as binary32.  Returns true when a_1 (f0) is kept; *kept
// receives the new value.
__device__ __forceinline__ bool mvue_1of2(float f0, float f1, uint32_t word, float* kept) {
    const float m0 = fabsf(f0), m1 = fabsf(f1);
    const float S = __fadd_rn(m0, m1);
    const float t = __fmul_rn(top24(word), __fmul_rn(S, 5.9604644775390625e-08f));
    const bool keep0 = (t < m0) || (m1 == 0.0f);
    const uint32_t src = __float_as_uint(keep0 ? f0 : f1);
    *kept = __uint_as_float(__float_as_uint(S) | (src & 0x80000000u));
    return keep0;
}

// Two adjacent bf16 pairs (one group of four): x0 = a0 | a1 << 16, x1 = a2 | a3 << 16.
// Outputs the group's two survivors as bf16 (pair 0 in the low half) and its nibble
// (pair 0 -> position 0/1, pair 1 -> position 2/3).
template <bool kSR = false>
__device__ __forceinline__ void mvue_1of2x2_bf16(uint32_t x0, uint32_t x1, uint32_t word0,
                                                 uint32_t word1, uint32_t* out, uint32_t* nibble, uint32_t rnd = 0u) {
    const float a0 = __uint_as_float(x0 << 16), a1 = __uint_as_float(x0 & 0xFFFF0000u);
    const float b0 = __uint_as_float(x1 << 16), b1 = __uint_as_float(x1 & 0xFFFF0000u);
    const float SA = __fadd_rn(fabsf(a0), fabsf(a1));
    const float SB = __fadd_rn(fabsf(b0), fabsf(b1));
    const float tA = __fmul_rn(top24(word0), __fmul_rn(SA, 5.9604644775390625e-08f));
    const float tB = __fmul_rn(top24(word1), __fmul_rn(SB, 5.9604644775390625e-08f));
    const bool keepA = (tA < fabsf(a0)) || (fabsf(a1) == 0.0f);
    const bool keepB = (tB < fabsf(b0)) || (fabsf(b1) == 0.0f);
    // byte 1 <- high byte of the survivor of pair 0, byte 3 <- high byte of the survivor of pair 1
    const uint32_t sel = (keepA ? 0x0010u : 0x0030u) | (keepB ? 0x5000u : 0x7000u);
    const uint32_t signs = __byte_perm(x0, x1, sel) & 0x80008000u;
    *out = pack_out<kSR>(SA, SB, rnd) | signs;
    *nibble = (keepA ? 0u : 1u) | (keepB ? 8u : 12u);
}

// The same for a group whose four elements are the half kHigh of four row words (K runs down the rows).
template <bool kHigh>
__device__ __forceinline__ void mvue_1of2x2_bf16_rows(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3,
                                                      uint32_t word0, uint32_t word1, uint32_t* out,
                                                      uint32_t* nibble) {
    auto widen = [](uint32_t w) { return __uint_as_float(kHigh ? (w & 0xFFFF0000u) : (w << 16)); };
    const float a0 = widen(w0), a1 = widen(w1), b0 = widen(w2), b1 = widen(w3);
    const float SA = __fadd_rn(fabsf(a0), fabsf(a1));
    const float SB = __fadd_rn(fabsf(b0), fabsf(b1));
    const float tA = __fmul_rn(top24(word0), __fmul_rn(SA, 5.9604644775390625e-08f));
    const float tB = __fmul_rn(top24(word1), __fmul_rn(SB, 5.9604644775390625e-08f));
    const bool keepA = (tA < fabsf(a0)) || (fabsf(a1) == 0.0f);
    const bool keepB = (tB < fabsf(b0)) || (fabsf(b1) == 0.0f);
    const uint32_t srcA = keepA ? w0 : w1, srcB = keepB ? w2 : w3;
    // byte 1 <- high byte of pair 0's survivor, byte 3 <- high byte of pair 1's survivor
    const uint32_t signs = __byte_perm(srcA, srcB, kHigh ? 0x7030u : 0x5010u) & 0x80008000u;
    *out = pack_bf16x2(SA, SB) | signs;
    *nibble = (keepA ? 0u : 1u) | (keepB ? 8u : 12u);
}

// ===========================================================================
// MVUE 2:4 (marginals: Sec. 4.2; joint law over pairs: App. A.2).
//
// With the magnitudes sorted, s1 <= s2 <= s3 <= s4 (ties by position), d = s4-s3,
// the cumulative numerators of the appendix's pair table in the order 13, 14, 23,
// 24 are, for all three of its cases and over the common denominator D,
//     C13 = 2 s1 - d,  C14 = 4 s1,  C23 = 4 s1 + (2 s2 - d) + min(2 s1 - d, 0),
//     C24 = 4 (s1 + s2),  D = 2 (2 S3 + min(s4 - S3, 0)),  S3 = s1 + s2 + s3,
// and the pair is the first with eps D < C (else 34).  When s4 >= S3 the larger
// survivor is always the dominant element.  Survivors become sign(a) D/4, the
// dominant element of the capped case keeps max(s4, D/4) = s4.
// ===========================================================================
template <typename KeyT>
struct Pick24 {
    KeyT key_a, key_b;   // sort keys of the smaller / larger survivor
    float va, vb;        // their new magnitudes
};

// k1..k4: sort keys ascending; KEY_MAG(k) its magnitude, KEY_POS(k) its position.
template <typename KeyT, typename MagF>
__device__ __forceinline__ Pick24<KeyT> pick_2of4(KeyT k1, KeyT k2, KeyT k3, KeyT k4, uint32_t word,
                                                  MagF mag) {
    const float s1 = mag(k1), s2 = mag(k2), s3 = mag(k3), s4 = mag(k4);
    const float S12 = __fadd_rn(s1, s2);
    const float S3 = __fadd_rn(S12, s3);
    const float d = __fsub_rn(s4, s3);
    const float x = __fmaf_rn(2.0f, s1, -d);            // 2 s1 is exact: one rounding, as (s1+s1)-d
    const float y = __fmaf_rn(2.0f, s2, -d);
    const float C14 = __fmul_rn(4.0f, s1);
    // min(v, 0) = (v - |v|) / 2 exactly: keeps the minimum off the compare/select pipe
    const float C23 = __fmaf_rn(0.5f, __fsub_rn(x, fabsf(x)), __fadd_rn(C14, y));
    const float C24 = __fmul_rn(4.0f, S12);
    const float e = __fsub_rn(s4, S3);                  // >= 0: the dominant element is capped at p = 1
    const float Dh = __fmaf_rn(0.5f, __fsub_rn(e, fabsf(e)), __fadd_rn(S3, S3));
    const float t = __fmul_rn(top24(word), __fmul_rn(Dh, 1.1920928955078125e-07f));

    const bool p1 = t < x;
    const bool p12 = p1 || (t < C14);
    const bool p3 = t < C23;
    const bool p34 = p3 || (t < C24);
    const bool capped = e >= 0.0f;
    const KeyT key_a = p12 ? k1 : (p34 ? k2 : k3);
    const bool b_is_third = !capped && (p1 || (!p12 && p3));
    const KeyT key_b = b_is_third ? k3 : k4;

    Pick24<KeyT> r;
    r.key_a = key_a;
    r.key_b = key_b;
    r.va = __fmul_rn(0.5f, Dh);
    r.vb = fmaxf(s4, r.va);
    return r;
}

// ---- bf16 source: x01 = a0 | a1 << 16, x23 = a2 | a3 << 16 ------------------
// The sort key of an element is one byte permute of its source word:
//   bits 31..16  the bf16 itself (widened to binary32 it is the element),
//   bits 15..14  its position in the block, bits 13..8 zero,
//   bits  7..0   a copy of the bf16's high byte (bit 7 = its sign).
// The first comparator layer takes absolute values, which strips bit 31 for free;
// as positive floats the keys then order by (magnitude, position), and the
// survivors' keys still carry position and sign, so nothing is looked up again.
// Outputs: `out` = the two survivors as bf16 (lower position in the low half),
// `nibble` = idx0 | idx1 << 2.
// The four elements are the halves (kH* = false: low, true: high) of the words w0..w3: adjacent pairs of two
// words when K is contiguous (w0 = w1, w2 = w3), or the same half of four row words when K runs down the rows.
template <bool kH0, bool kH1, bool kH2, bool kH3, bool kSR = false>
__device__ __forceinline__ void mvue_2of4_bf16(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3, uint32_t word,
                                               uint32_t* out, uint32_t* nibble, uint32_t rnd = 0u) {
    const float f0 = __uint_as_float(__byte_perm(w0, 0x00u, kH0 ? 0x3243 : 0x1041));
    const float f1 = __uint_as_float(__byte_perm(w1, 0x40u, kH1 ? 0x3243 : 0x1041));
    const float f2 = __uint_as_float(__byte_perm(w2, 0x80u, kH2 ? 0x3243 : 0x1041));
    const float f3 = __uint_as_float(__byte_perm(w3, 0xC0u, kH3 ? 0x3243 : 0x1041));
    const float lo01 = fminf(fabsf(f0), fabsf(f1)), hi01 = fmaxf(fabsf(f0), fabsf(f1));
    const float lo23 = fminf(fabsf(f2), fabsf(f3)), hi23 = fmaxf(fabsf(f2), fabsf(f3));
    const float k1 = fminf(lo01, lo23), mid_a = fmaxf(lo01, lo23);
    const float mid_b = fminf(hi01, hi23), k4 = fmaxf(hi01, hi23);
    const float k2 = fminf(mid_a, mid_b), k3 = fmaxf(mid_a, mid_b);

    const Pick24<float> r = pick_2of4(
        k1, k2, k3, k4, word,
        [](float k) { return __uint_as_float(__float_as_uint(k) & 0xFFFF0000u); });

    const uint32_t ua = __float_as_uint(r.key_a), ub = __float_as_uint(r.key_b);
    const uint32_t signs = __byte_perm(ua, ub, 0x4000) & 0x80008000u;   // byte 1 <- a's sign byte, byte 3 <- b's
    const uint32_t pa = ua << 16, pb = ub << 16;                        // position in the top two bits
    const bool swap = pa > pb;
    // (the rounding bits belong to the slots: when a ends up in the high slot it takes the high slot's bits)
    const uint32_t ab = pack_out<kSR>(r.va, r.vb, kSR ? __byte_perm(rnd, 0u, swap ? 0x1032u : 0x3210u) : 0u) | signs;   // a low, b high
    *out = __byte_perm(ab, 0u, swap ? 0x1032u : 0x3210u);
    // (p >> 30) and (p >> 28) as high products: bits 29..28 of p are zero, so p >> 28 = position << 2
    const uint32_t nib_ab = __umulhi(pa, 4u) + __umulhi(pb, 16u);
    const uint32_t nib_ba = __umulhi(pb, 4u) + __umulhi(pa, 16u);
    *nibble = swap ? nib_ba : nib_ab;
}

// ---- binary32 source ---------------------------------------------------------
// 64-bit keys (magnitude bits << 2 | position); b0..b3 are the raw bit patterns.
template <bool kSR = false>
__device__ __forceinline__ void mvue_2of4_f32(uint32_t b0, uint32_t b1, uint32_t b2, uint32_t b3,
                                              uint32_t word, uint32_t* out, uint32_t* nibble, uint32_t rnd = 0u) {
    auto make = [](uint32_t b, uint32_t p) { return ((uint64_t)(b & 0x7FFFFFFFu) << 2) | p; };
    auto cswap = [](uint64_t& a, uint64_t& b) {
        const uint64_t lo = a < b ? a : b, hi = a < b ? b : a;
        a = lo; b = hi;
    };
    uint64_t k1 = make(b0, 0u), k2 = make(b1, 1u), k3 = make(b2, 2u), k4 = make(b3, 3u);
    cswap(k1, k2); cswap(k3, k4); cswap(k1, k3); cswap(k2, k4); cswap(k2, k3);
    const Pick24<uint64_t> r = pick_2of4(
        k1, k2, k3, k4, word,
        [](uint64_t k) { return __uint_as_float((uint32_t)(k >> 2)); });
    const uint32_t ia = (uint32_t)r.key_a & 3u, ib = (uint32_t)r.key_b & 3u;
    const uint32_t sa = (ia == 0 ? b0 : (ia == 1 ? b1 : (ia == 2 ? b2 : b3))) & 0x80000000u;
    const uint32_t sb = (ib == 0 ? b0 : (ib == 1 ? b1 : (ib == 2 ? b2 : b3))) & 0x80000000u;
    const float va = __uint_as_float(__float_as_uint(r.va) | sa);
    const float vb = __uint_as_float(__float_as_uint(r.vb) | sb);
    const bool swap = ia > ib;
    *out = pack_out<kSR>(swap ? vb : va, swap ? va : vb, rnd);
    *nibble = swap ? (ib | (ia << 2)) : (ia | (ib << 2));
}

// ===========================================================================
// MVUE 2:4, second joint law: systematic sampling (marginals: Sec. 4.2).
//
// Sec. 4.2's block variance depends on the marginals p_i alone, and App. A.2 is one
// joint law with the optimal ones.  This law has the same marginals and kept values
// (so the same mean and the same minimal variance) and needs no sort: in the block's
// own order, element k gets the weight e_k = min(|a_k|, R_k), R_k = sum of the other
// three magnitudes (an element heavier than the rest together is clipped to their
// sum), owns [c_k, c_k + e_k) of [0, D), D = sum e_k, H = D/2; the owners of t and
// t + H survive, t = eps H.  e_k / H is exactly the optimal p_k in both cases of
// Sec. 4.2, and a survivor becomes sign(a_k) max(|a_k|, H) = a_k / p_k.
//   R_k carries + 2^-149 so that a lone non-zero owns a non-empty interval;
//   t2 = (2^23 + n)(D 2^-24), n = top 23 bits of the word; t = t2 - H is exact;
//   i = #{c_1, c_2 <= t},  j = max(i + 1, #{c_1, c_2, c_3 <= t2}).
// Counting is done on "less than": li = #{t < c_1, t < c_2} = 2 - i and
// lj = min(#{t2 < c_k}, li) = 3 - j; x < c is the sign bit of x - c (the difference
// of two finite floats is never rounded across zero).
// ===========================================================================
struct Pick24Sys {
    uint32_t li, lj;     // i = 2 - li, j = 3 - lj
    float H;
};

// kAll3: also count t2 < c_1 (implied by the other two, see below; kept where it schedules better).
template <bool kAll3>
__device__ __forceinline__ Pick24Sys pick_2of4_sys(float m0, float m1, float m2, float m3, uint32_t word) {
    const float tiny = __uint_as_float(1u);                                   // 2^-149
    const float q01 = __fadd_rn(__fadd_rn(m0, m1), tiny), q23 = __fadd_rn(__fadd_rn(m2, m3), tiny);
    const float R0 = __fadd_rn(m1, q23), R1 = __fadd_rn(m0, q23);
    const float R2 = __fadd_rn(q01, m3), R3 = __fadd_rn(q01, m2);
    const float c1 = fminf(m0, R0), e1 = fminf(m1, R1), e2 = fminf(m2, R2), e3 = fminf(m3, R3);
    const float c2 = __fadd_rn(c1, e1), c3 = __fadd_rn(c2, e2), D = __fadd_rn(c3, e3);
    const float Hs = __fmul_rn(D, 5.9604644775390625e-08f);                   // D 2^-24
    Pick24Sys r;
    r.H = __fmul_rn(0.5f, D);
    // 2^23 + n as a float: its bit pattern is 0x4B000000 + n
    const float n2 = __uint_as_float(__umulhi(word, 1u << 23) + 0x4B000000u);
    const float t2 = __fmul_rn(n2, Hs), t = __fsub_rn(t2, r.H);
    auto below = [](float x, float c) { return __umulhi(__float_as_uint(__fsub_rn(x, c)), 2u); };   // x < c ? 1 : 0
    r.li = below(t, c1) + below(t, c2);
    // t2 < c_1 implies t2 < c_2 and t2 < c_3, and then min(3, li) = min(2, li): the c_1 term is never needed
    r.lj = min((kAll3 ? below(t2, c1) : 0u) + below(t2, c2) + below(t2, c3), r.li);
    return r;
}

// bf16 source: x01 = a0 | a1 << 16, x23 = a2 | a3 << 16.  The two survivors are gathered by one byte
// permute (selector bytes 2i, 2i+1, 2j, 2j+1); bf16 rounding is monotone, so the rounded max(|a|, H)
// is the larger of the element's own bits and the rounded H, taken on both halves at once as
// signed 16-bit integers (with equal sign bits the larger magnitude is the larger integer).
template <bool kSR = false>
__device__ __forceinline__ void mvue_2of4_sys_bf16(uint32_t x01, uint32_t x23, uint32_t word, uint32_t* out,
                                                   uint32_t* nibble, uint32_t rnd = 0u) {
    const Pick24Sys r = pick_2of4_sys<false>(fabsf(__uint_as_float(x01 << 16)), fabsf(__uint_as_float(x01 & 0xFFFF0000u)),
                                             fabsf(__uint_as_float(x23 << 16)), fabsf(__uint_as_float(x23 & 0xFFFF0000u)),
                                             word);
    const uint32_t sel = 0x7654u - 0x22u * r.li - 0x2200u * r.lj;
    const uint32_t raw = __byte_perm(x01, x23, sel);
    // (a survivor below H takes H rounded for its own slot; one at or above H is a bf16 number no smaller than either
    // neighbour of H, so the maximum still picks it)
    const uint32_t hs = pack_out<kSR>(r.H, r.H, rnd) | (raw & 0x80008000u);
    *out = __vmaxs2(raw, hs);
    *nibble = 14u - r.li - 4u * r.lj;                                         // i | j << 2
}

// Two blocks at a time on packed binary32 pairs: add.rn.f32x2 / sub.rn.f32x2 round each half exactly as the scalar
// instruction does, so the result is that of mvue_2of4_sys_bf16 on each block, bit for bit, in about three quarters of
// the issue slots (the kernel is bound by instruction issue, not by the arithmetic pipes).  Every multiplication
// stays scalar: a packed multiply that feeds a packed add or subtract gets contracted into a fused multiply-add --
// one rounding instead of two -- which moves a threshold by one unit in the last place on a few draws in 2^23.
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t sub_f32x2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// Blocks A = (xa01, xa23; word wa) and B = (xb01, xb23; word wb), each as in mvue_2of4_sys_bf16.
template <bool kSR = false>
__device__ __forceinline__ void mvue_2of4_sys_bf16_x2(uint32_t xa01, uint32_t xa23, uint32_t xb01, uint32_t xb23,
                                                      uint32_t wa, uint32_t wb, uint32_t* out_a, uint32_t* out_b,
                                                      uint32_t* nibble_a, uint32_t* nibble_b, uint32_t rnd_a = 0u,
                                                      uint32_t rnd_b = 0u) {
    // magnitudes: both sign bits of a word cleared at once, then widened
    const uint32_t ya01 = xa01 & 0x7FFF7FFFu, ya23 = xa23 & 0x7FFF7FFFu, yb01 = xb01 & 0x7FFF7FFFu, yb23 = xb23 & 0x7FFF7FFFu;
    const float a0 = __uint_as_float(ya01 << 16), a1 = __uint_as_float(ya01 & 0xFFFF0000u);
    const float a2 = __uint_as_float(ya23 << 16), a3 = __uint_as_float(ya23 & 0xFFFF0000u);
    const float b0 = __uint_as_float(yb01 << 16), b1 = __uint_as_float(yb01 & 0xFFFF0000u);
    const float b2 = __uint_as_float(yb23 << 16), b3 = __uint_as_float(yb23 & 0xFFFF0000u);
    const uint64_t m0 = pack_f32x2(a0, b0), m1 = pack_f32x2(a1, b1), m2 = pack_f32x2(a2, b2), m3 = pack_f32x2(a3, b3);
    const float tiny1 = __uint_as_float(1u);                                  // 2^-149
    const uint64_t tiny = pack_f32x2(tiny1, tiny1);
    const uint64_t q01 = add_f32x2(add_f32x2(m0, m1), tiny), q23 = add_f32x2(add_f32x2(m2, m3), tiny);
    const uint64_t R0 = add_f32x2(m1, q23), R1 = add_f32x2(m0, q23), R2 = add_f32x2(q01, m3), R3 = add_f32x2(q01, m2);
    float r0a, r0b, r1a, r1b, r2a, r2b, r3a, r3b;
    unpack_f32x2(R0, r0a, r0b); unpack_f32x2(R1, r1a, r1b); unpack_f32x2(R2, r2a, r2b); unpack_f32x2(R3, r3a, r3b);
    const uint64_t c1 = pack_f32x2(fminf(a0, r0a), fminf(b0, r0b)), e1 = pack_f32x2(fminf(a1, r1a), fminf(b1, r1b));
    const uint64_t e2 = pack_f32x2(fminf(a2, r2a), fminf(b2, r2b)), e3 = pack_f32x2(fminf(a3, r3a), fminf(b3, r3b));
    const uint64_t c2 = add_f32x2(c1, e1), c3 = add_f32x2(c2, e2), D = add_f32x2(c3, e3);
    float Da, Db;
    unpack_f32x2(D, Da, Db);
    const float Ha = __fmul_rn(0.5f, Da), Hb = __fmul_rn(0.5f, Db);
    const float t2a = __fmul_rn(__uint_as_float(__umulhi(wa, 1u << 23) + 0x4B000000u), __fmul_rn(Da, 5.9604644775390625e-08f));
    const float t2b = __fmul_rn(__uint_as_float(__umulhi(wb, 1u << 23) + 0x4B000000u), __fmul_rn(Db, 5.9604644775390625e-08f));
    const uint64_t t2 = pack_f32x2(t2a, t2b), t = sub_f32x2(t2, pack_f32x2(Ha, Hb));
    float d1a, d1b, d2a, d2b, d3a, d3b, d4a, d4b;                             // x < c is the sign bit of x - c
    unpack_f32x2(sub_f32x2(t, c1), d1a, d1b); unpack_f32x2(sub_f32x2(t, c2), d2a, d2b);
    unpack_f32x2(sub_f32x2(t2, c2), d3a, d3b); unpack_f32x2(sub_f32x2(t2, c3), d4a, d4b);
    auto sign = [](float x) { return __umulhi(__float_as_uint(x), 2u); };
    {
        const uint32_t li = sign(d1a) + sign(d2a), lj = min(sign(d3a) + sign(d4a), li);
        const uint32_t raw = __byte_perm(xa01, xa23, 0x7654u - 0x22u * li - 0x2200u * lj);
        *out_a = __vmaxs2(raw, pack_out<kSR>(Ha, Ha, rnd_a) | (raw & 0x80008000u));
        *nibble_a = 14u - li - 4u * lj;
    }
    {
        const uint32_t li = sign(d1b) + sign(d2b), lj = min(sign(d3b) + sign(d4b), li);
        const uint32_t raw = __byte_perm(xb01, xb23, 0x7654u - 0x22u * li - 0x2200u * lj);
        *out_b = __vmaxs2(raw, pack_out<kSR>(Hb, Hb, rnd_b) | (raw & 0x80008000u));
        *nibble_b = 14u - li - 4u * lj;
    }
}

// ---- App. A.2 pair table, bf16 source with K contiguous, gathered output ------------------------------------------
// The same law and the same bits as mvue_2of4_bf16 (x01 = a0 | a1 << 16, x23 = a2 | a3 << 16), with the output stage
// of the systematic law:
//   sort key = the bf16 in the upper half, the position in the two lowest bits (the sign comes back with the gather);
//   every survivor's new magnitude is max(|a|, D/4): D/4 for a survivor with p < 1 (then D/4 >= |a|, also after the
//   roundings of pick_2of4: the sums only add non-negative terms, and in the uncapped case D/2 = fl(2 S3 - (S3 - a_4))
//   cannot round below 2 a_4), |a| itself for the capped dominant element;
//   so the two survivors are gathered in position order by one byte permute and raised to bf16(D/4) with one signed
//   16-bit maximum per half.
template <bool kSR = false>
__device__ __forceinline__ void mvue_2of4_bf16_gather(uint32_t x01, uint32_t x23, uint32_t word, uint32_t* out,
                                                      uint32_t* nibble, uint32_t rnd = 0u) {
    const float f0 = __uint_as_float(__byte_perm(x01, 0u, 0x1054)), f1 = __uint_as_float(__byte_perm(x01, 1u, 0x3254));
    const float f2 = __uint_as_float(__byte_perm(x23, 2u, 0x1054)), f3 = __uint_as_float(__byte_perm(x23, 3u, 0x3254));
    const float lo01 = fminf(fabsf(f0), fabsf(f1)), hi01 = fmaxf(fabsf(f0), fabsf(f1));
    const float lo23 = fminf(fabsf(f2), fabsf(f3)), hi23 = fmaxf(fabsf(f2), fabsf(f3));
    const float k1 = fminf(lo01, lo23), mid_a = fmaxf(lo01, lo23);
    const float mid_b = fminf(hi01, hi23), k4 = fmaxf(hi01, hi23);
    const float k2 = fminf(mid_a, mid_b), k3 = fmaxf(mid_a, mid_b);
    const Pick24<float> r = pick_2of4(
        k1, k2, k3, k4, word,
        [](float k) { return __uint_as_float(__float_as_uint(k) & 0xFFFF0000u); });
    const uint32_t pa = __float_as_uint(r.key_a) & 3u, pb = __float_as_uint(r.key_b) & 3u;
    const uint32_t i = min(pa, pb), j = max(pa, pb);
    const uint32_t raw = __byte_perm(x01, x23, 0x1010u + 0x22u * i + 0x2200u * j);
    *out = __vmaxs2(raw, pack_out<kSR>(r.va, r.va, rnd) | (raw & 0x80008000u));
    *nibble = i + 4u * j;
}

// binary32 source: b0..b3 are the raw bit patterns.
template <bool kSR = false>
__device__ __forceinline__ void mvue_2of4_sys_f32(uint32_t b0, uint32_t b1, uint32_t b2, uint32_t b3,
                                                  uint32_t word, uint32_t* out, uint32_t* nibble, uint32_t rnd = 0u) {
    const Pick24Sys r = pick_2of4_sys<true>(fabsf(__uint_as_float(b0)), fabsf(__uint_as_float(b1)),
                                            fabsf(__uint_as_float(b2)), fabsf(__uint_as_float(b3)), word);
    const uint32_t bi = r.li == 2u ? b0 : (r.li == 1u ? b1 : b2);            // i = 2 - li in {0, 1, 2}
    const uint32_t bj = r.lj == 2u ? b1 : (r.lj == 1u ? b2 : b3);            // j = 3 - lj in {1, 2, 3}
    const float vi = __uint_as_float(__float_as_uint(fmaxf(fabsf(__uint_as_float(bi)), r.H)) | (bi & 0x80000000u));
    const float vj = __uint_as_float(__float_as_uint(fmaxf(fabsf(__uint_as_float(bj)), r.H)) | (bj & 0x80000000u));
    *out = pack_out<kSR>(vi, vj, rnd);
    *nibble = 14u - r.li - 4u * r.lj;
}

// ===========================================================================
// Approximately optimal 2:4 (Sec. 4.4, "approx-MVUE"): two sequential draws without
// replacement, each proportional to magnitude; a survivor is divided by its exact
// inclusion probability p_k = (m_k / s)(1 + T_k), T_k = sum_{l != k} m_l / R_l, R_l = sum of
// the magnitudes other than l (the equation of Sec. 4.4), i.e. becomes sign(a_k) s / (1 + T_k).
// Block order, no sort; two random words per block.
//   first draw:  c_1 = m_0, c_2 = c_1 + m_1, c_3 = c_2 + m_2, s = c_3 + m_3,
//                t_1 = n_1 (s 2^-24), i = #{c_k <= t_1};
//   second draw among the others in position order, d_1, d_2 their running sums,
//                t_2 = n_2 (R_i 2^-24), j = the #{d_k <= t_2}-th of them;
//   sums of three run in position order, (x + y) + z; the six divisions are IEEE.
//   R_i = 0 (at most one non-zero): both survivors keep their own values.
// Unlike the two exact laws this one cannot avoid division, so on this hardware it is the
// most expensive of the three estimators, not the cheapest.
// ===========================================================================
__device__ __forceinline__ float sel4(uint32_t k, float x0, float x1, float x2, float x3) {
    return k < 2u ? (k == 0u ? x0 : x1) : (k == 2u ? x2 : x3);
}

// b0..b3: the block as binary32 bit patterns.  out = the two survivors as bf16 (lower position in the
// low half), nibble = idx0 | idx1 << 2.
template <bool kSR = false>
__device__ __forceinline__ void mvue_2of4_approx_f32(uint32_t b0, uint32_t b1, uint32_t b2, uint32_t b3,
                                                     uint32_t word1, uint32_t word2, uint32_t* out,
                                                     uint32_t* nibble, uint32_t rnd = 0u) {
    const float m0 = fabsf(__uint_as_float(b0)), m1 = fabsf(__uint_as_float(b1));
    const float m2 = fabsf(__uint_as_float(b2)), m3 = fabsf(__uint_as_float(b3));
    const float q01 = __fadd_rn(m0, m1), q12 = __fadd_rn(m1, m2), q02 = __fadd_rn(m0, m2);
    const float R3 = __fadd_rn(q01, m2), R2 = __fadd_rn(q01, m3), R1 = __fadd_rn(q02, m3), R0 = __fadd_rn(q12, m3);
    const float s = __fadd_rn(R3, m3);
    const float t1 = __fmul_rn(top24(word1), __fmul_rn(s, 5.9604644775390625e-08f));
    const uint32_t i = (m0 <= t1 ? 1u : 0u) + (q01 <= t1 ? 1u : 0u) + (R3 <= t1 ? 1u : 0u);
    const float Ri = sel4(i, R0, R1, R2, R3);
    const float d1 = i == 0u ? m1 : m0;
    const float d2 = sel4(i, q12, q02, q01, q01);
    const float t2 = __fmul_rn(top24(word2), __fmul_rn(Ri, 5.9604644775390625e-08f));
    const uint32_t jj = (d1 <= t2 ? 1u : 0u) + (d2 <= t2 ? 1u : 0u);
    const uint32_t j = jj + (jj >= i ? 1u : 0u);
    // The IEEE division leaves its short path when an operand is zero, and zeros are everywhere in a
    // ReLU-sparse gradient: divide stand-ins instead (0 / R is 0 whatever R; a quotient by R = 0 is only
    // ever read when R_i = 0, where the survivors keep their own values), so that the warp stays together.
    auto quot = [](float num, float den) {
        const float q = __fdiv_rn(num == 0.0f ? 1.0f : num, den == 0.0f ? 1.0f : den);
        return num == 0.0f ? 0.0f : q;
    };
    const float vv0 = quot(m0, R0), vv1 = quot(m1, R1), vv2 = quot(m2, R2), vv3 = quot(m3, R3);
    const float u01 = __fadd_rn(vv0, vv1), u12 = __fadd_rn(vv1, vv2), u02 = __fadd_rn(vv0, vv2);
    const uint32_t lo = min(i, j), hi = max(i, j);
    // T_k = (sum of two) + (the last of the others)
    const float Tlo = __fadd_rn(sel4(lo, u12, u02, u01, u01), lo == 3u ? vv2 : vv3);
    const float Thi = __fadd_rn(sel4(hi, u12, u02, u01, u01), hi == 3u ? vv2 : vv3);
    const bool own = Ri == 0.0f;
    const float s_div = own ? 1.0f : s;                      // s may be 0 only when own
    const float scaled_lo = __fdiv_rn(s_div, __fadd_rn(1.0f, Tlo)), scaled_hi = __fdiv_rn(s_div, __fadd_rn(1.0f, Thi));
    const float mag_lo = own ? sel4(lo, m0, m1, m2, m3) : scaled_lo;
    const float mag_hi = own ? sel4(hi, m0, m1, m2, m3) : scaled_hi;
    const uint32_t blo = lo < 2u ? (lo == 0u ? b0 : b1) : (lo == 2u ? b2 : b3);
    const uint32_t bhi = hi < 2u ? (hi == 0u ? b0 : b1) : (hi == 2u ? b2 : b3);
    const float vlo = __uint_as_float(__float_as_uint(mag_lo) | (blo & 0x80000000u));
    const float vhi = __uint_as_float(__float_as_uint(mag_hi) | (bhi & 0x80000000u));
    *out = pack_out<kSR>(vlo, vhi, rnd);
    *nibble = lo | (hi << 2);
}

// bf16 source: x01 = a0 | a1 << 16, x23 = a2 | a3 << 16 (widened exactly).
template <bool kSR = false>
__device__ __forceinline__ void mvue_2of4_approx_bf16(uint32_t x01, uint32_t x23, uint32_t word1, uint32_t word2,
                                                      uint32_t* out, uint32_t* nibble, uint32_t rnd = 0u) {
    mvue_2of4_approx_f32<kSR>(x01 << 16, x01 & 0xFFFF0000u, x23 << 16, x23 & 0xFFFF0000u, word1, word2, out, nibble, rnd);
}

// ===========================================================================
// MVUE 1:4 (appendix "Additional sparsity results"; Sec. 4.1's argument with one survivor of four): element i of the block
// survives with probability |a_i| / S, S the sum of the four magnitudes, and becomes sign(a_i) S.
//   c_1 = m_0, c_2 = c_1 + m_1, c_3 = c_2 + m_2, S = c_3 + m_3;  t = n (S 2^-24);  i = #{c_k <= t}.
// The survivor is stored in the 2:4 container beside a +0: positions (i, 3), or (2, 3) when i = 3.
// ===========================================================================
template <bool kSR = false>
__device__ __forceinline__ void mvue_1of4_f32(uint32_t b0, uint32_t b1, uint32_t b2, uint32_t b3, uint32_t word,
                                              uint32_t* out, uint32_t* nibble, uint32_t rnd = 0u) {
    const float m0 = fabsf(__uint_as_float(b0)), m1 = fabsf(__uint_as_float(b1));
    const float m2 = fabsf(__uint_as_float(b2)), m3 = fabsf(__uint_as_float(b3));
    const float c2 = __fadd_rn(m0, m1), c3 = __fadd_rn(c2, m2), S = __fadd_rn(c3, m3);
    const float t = __fmul_rn(top24(word), __fmul_rn(S, 5.9604644775390625e-08f));
    const uint32_t i = (m0 <= t ? 1u : 0u) + (c2 <= t ? 1u : 0u) + (c3 <= t ? 1u : 0u);
    const uint32_t bi = i < 2u ? (i == 0u ? b0 : b1) : (i == 2u ? b2 : b3);
    const float v = __uint_as_float(__float_as_uint(S) | (bi & 0x80000000u));
    if (kSR) {                                               // the survivor takes the rounding bits of the slot it lands in
        *out = pack_out<true>(i < 3u ? v : 0.0f, i < 3u ? 0.0f : v, rnd);
    } else {
        const uint32_t h = pack_bf16x2(v, 0.0f);             // survivor in the low half, +0 in the high half
        *out = i < 3u ? h : h << 16;
    }
    *nibble = i < 3u ? (i | 12u) : 14u;
}

// ===========================================================================
// Approx-4:8 (appendix "Additional sparsity results": Sec. 4.4's procedure with four survivors of eight).  Four
// sequential draws, each proportional to magnitude among the elements still there; a survivor is divided by its exact
// inclusion probability p_i = sum over the sets R (|R| <= 3, i not in R) of u(R) m_i, with
//   rest(Q) = the magnitudes outside Q added left to right,  inv(Q) = 1 / rest(Q) (0 if rest is 0),
//   u({}) = inv({}),  w(R) = sum_{k in R} u(R \ k) m_k,  u(R) = w(R) inv(R),
// sets visited by size, then by increasing bit mask, sums first term first.  A block with at most four non-zeros keeps
// them all with their own values.  No tensor core reads this pattern: prune only.
// b[8]: the block as binary32 bit patterns; words: the block's own generator call.  Returns the mask (bit k = element k
// survives); out[0..1] = the four survivors as bf16, ascending position.
// ===========================================================================
__host__ __device__ constexpr int popcount8_c(unsigned x) {
    return (int)((x & 1u) + ((x >> 1) & 1u) + ((x >> 2) & 1u) + ((x >> 3) & 1u) + ((x >> 4) & 1u) + ((x >> 5) & 1u) +
                 ((x >> 6) & 1u) + ((x >> 7) & 1u));
}

__device__ __forceinline__ uint32_t approx_4of8(const uint32_t (&b)[8], uint4 words, uint32_t (&out)[2]) {
    float m[8];
    int nnz = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        m[k] = fabsf(__uint_as_float(b[k]));
        nnz += m[k] != 0.0f ? 1 : 0;
    }
    auto rest_of = [&](unsigned Q) {                       // left to right over the elements outside Q
        float r = 0.0f;
        bool first = true;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            if (Q & (1u << k)) continue;
            r = first ? m[k] : __fadd_rn(r, m[k]);
            first = false;
        }
        return r;
    };
    // four draws
    const uint32_t w4[4] = {words.x, words.y, words.z, words.w};
    unsigned removed = 0;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        float left = 0.0f;
        bool first = true;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            if (removed & (1u << k)) continue;
            left = first ? m[k] : __fadd_rn(left, m[k]);
            first = false;
        }
        const float thr = __fmul_rn(top24(w4[t]), __fmul_rn(left, 5.9604644775390625e-08f));
        float run = 0.0f;
        first = true;
        int pick = -1, last = -1;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            if (removed & (1u << k)) continue;
            last = k;
            if (pick >= 0) continue;
            run = first ? m[k] : __fadd_rn(run, m[k]);
            first = false;
            if (!(run <= thr)) pick = k;
        }
        if (pick < 0) pick = last;
        removed |= 1u << pick;
    }
    float p[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) p[i] = 1.0f;
    if (nnz > 4) {
        float u[256];                                       // only the 93 sets of at most three elements are ever touched
#pragma unroll
        for (int size = 0; size <= 3; ++size) {
#pragma unroll
            for (unsigned R = 0; R < 256; ++R) {
                if (popcount8_c(R) != size) continue;
                const float r = rest_of(R);
                const float inv = r == 0.0f ? 0.0f : __fdiv_rn(1.0f, r);
                float acc = 1.0f;                           // w({}) = 1
                bool first = true;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    if (!(R & (1u << k))) continue;
                    const float term = __fmul_rn(u[R & ~(1u << k)], m[k]);
                    acc = first ? term : __fadd_rn(acc, term);
                    first = false;
                }
                u[R] = size == 0 ? inv : __fmul_rn(acc, inv);
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float acc = 0.0f;
            bool first = true;
#pragma unroll
            for (int size = 0; size <= 3; ++size) {
#pragma unroll
                for (unsigned R = 0; R < 256; ++R) {
                    if (popcount8_c(R) != size || (R & (1u << i))) continue;
                    const float term = __fmul_rn(u[R], m[i]);
                    acc = first ? term : __fadd_rn(acc, term);
                    first = false;
                }
            }
            p[i] = acc;
        }
    }
    // survivors in ascending position
    float v[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    int n = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        if (!(removed & (1u << k))) continue;
        const float a = __uint_as_float(b[k]);
        const float val = (nnz > 4 && m[k] != 0.0f) ? __fdiv_rn(a, p[k]) : a;
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (e == n) v[e] = val;
        ++n;
    }
    out[0] = pack_bf16x2(v[0], v[1]);
    out[1] = pack_bf16x2(v[2], v[3]);
    return removed;
}

// Byte offset of the 16-bit metadata word of (row r of A, strip = k / 16) in the tensor-core order:
// blocks of 128 rows x 128 k (2 KiB, row-block major), inside a block 128 lanes of 16 bytes with
// lane = r % 8 + 8 * (strip % 2) + 16 * (r % 128 / 16), word = strip % 8 / 2, half-word = r / 8 % 2.
// This is the arrangement tcgen05.cp.128x128b moves verbatim into tensor memory for four MMAs.
__device__ __forceinline__ int64_t tc_meta_offset(int64_t r, int64_t strip, int64_t kblocks) {
    const int rl = (int)(r & 127), st = (int)(strip & 7);
    const int lane = (rl & 7) + 8 * (st & 1) + 16 * (rl >> 4);
    return ((r >> 7) * kblocks + (strip >> 3)) * 2048 + lane * 16 + (st >> 1) * 4 + ((rl >> 3) & 1) * 2;
}

// One work unit of bf16 input: raw[8] = 16 elements along K, two per word.
// kJoint selects the 2:4 estimator (0: App. A.2 table, 1: systematic sampling, 2: approx-MVUE of Sec. 4.4,
// which takes two words per block: one generator call per two blocks) or, with 3, MVUE 1:4; 1:2 has one law.
// The random words of unit number `unit` (16 consecutive elements along K).  kWords = 4: one word per block of four
// (2:4 with the pair table or systematic sampling, 1:4); kWords = 8: two per block (approx-MVUE) or one per pair (1:2).
// 32 bits per word: generator call `unit` (kWords = 4) or calls 2 unit, 2 unit + 1 (kWords = 8).
// kEps16: sixteen bits per word, handed over in the top half of a word whose low half is zero, so that one call serves
// eight words: call unit / 2, its first or second pair of words (kWords = 4), or call `unit` (kWords = 8).
template <int kWords, bool kEps16>
__device__ __forceinline__ void unit_words(uint64_t unit, const RoundKeys& rk, uint32_t (&w)[kWords]) {
    if (kWords == 4 && !kEps16) {
        const uint4 r = philox4x32_10(unit, rk);
        w[0] = r.x; w[1] = r.y; w[2] = r.z; w[3] = r.w;
    } else if (kWords == 4) {
        const uint4 r = philox4x32_10(unit >> 1, rk);
        const bool second = (unit & 1u) != 0;
        const uint32_t a = second ? r.z : r.x, b = second ? r.w : r.y;
        w[0] = a << 16; w[1] = a & 0xFFFF0000u; w[2] = b << 16; w[3] = b & 0xFFFF0000u;
    } else if (!kEps16) {
        const uint4 ra = philox4x32_10(2 * unit, rk), rb = philox4x32_10(2 * unit + 1, rk);
        w[0] = ra.x; w[1] = ra.y; w[2] = ra.z; w[3] = ra.w;
        w[kWords - 4] = rb.x; w[kWords - 3] = rb.y; w[kWords - 2] = rb.z; w[kWords - 1] = rb.w;
    } else {
        const uint4 r = philox4x32_10(unit, rk);
        const uint32_t x[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            w[2 * i % kWords] = x[i] << 16;
            w[(2 * i + 1) % kWords] = x[i] & 0xFFFF0000u;
        }
    }
}
// The words of the two consecutive units `unit` (even) and `unit + 1` at sixteen bits per word from their one shared call.
__device__ __forceinline__ void unit_pair_words16(uint64_t unit, const RoundKeys& rk, uint32_t (&w0)[4], uint32_t (&w1)[4]) {
    const uint4 r = philox4x32_10(unit >> 1, rk);
    w0[0] = r.x << 16; w0[1] = r.x & 0xFFFF0000u; w0[2] = r.y << 16; w0[3] = r.y & 0xFFFF0000u;
    w1[0] = r.z << 16; w1[1] = r.z & 0xFFFF0000u; w1[2] = r.w << 16; w1[3] = r.w & 0xFFFF0000u;
}

template <int M, int kJoint>
struct UnitWords { static constexpr int kCount = (M == 2 || kJoint == 2) ? 8 : 4; };

// One work unit with its random words given (UnitWords<M, kJoint>::kCount of them).
// kSR: survivors are rounded to bf16 stochastically; the unit's eight slots draw their 16 bits each from one more
// generator call, numbered by the unit itself on stream 1 (group j's two slots: word j).
template <int M, int kJoint, bool kSR>
__device__ __forceinline__ void prune_unit_bf16_w(const uint32_t (&raw)[8], const uint32_t (&words)[UnitWords<M, kJoint>::kCount],
                                                  uint64_t unit_index, const RoundKeys& rk, uint4* out_values,
                                                  uint32_t* out_meta) {
    uint32_t v[4];                                   // 8 survivors, two bf16 per word
    uint32_t meta = 0;
    uint32_t rnd[4] = {0u, 0u, 0u, 0u};
    if (kSR) {
        const uint4 r = philox4x32_10(unit_index, rk, 1u);
        rnd[0] = r.x; rnd[1] = r.y; rnd[2] = r.z; rnd[3] = r.w;
    }
    if (M == 4 && kJoint == 3) {                      // MVUE 1:4: one word per block, as for 2:4
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t nib;
            mvue_1of4_f32<kSR>(raw[2 * j] << 16, raw[2 * j] & 0xFFFF0000u, raw[2 * j + 1] << 16, raw[2 * j + 1] & 0xFFFF0000u,
                               words[j], &v[j], &nib, rnd[j]);
            meta += nib << (4 * j);
        }
    } else if (M == 4 && kJoint == 2) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t nib;
            mvue_2of4_approx_bf16<kSR>(raw[2 * j], raw[2 * j + 1], words[(2 * j) % UnitWords<M, kJoint>::kCount],
                                       words[(2 * j + 1) % UnitWords<M, kJoint>::kCount], &v[j], &nib, rnd[j]);
            meta += nib << (4 * j);
        }
    } else if (M == 4 && kJoint == 1) {                // systematic sampling: the unit's four blocks two at a time
        uint32_t nib[4];
        mvue_2of4_sys_bf16_x2<kSR>(raw[0], raw[1], raw[2], raw[3], words[0], words[1], &v[0], &v[1], &nib[0], &nib[1],
                                   rnd[0], rnd[1]);
        mvue_2of4_sys_bf16_x2<kSR>(raw[4], raw[5], raw[6], raw[7], words[2], words[3], &v[2], &v[3], &nib[2], &nib[3],
                                   rnd[2], rnd[3]);
        meta = nib[0] + (nib[1] << 4) + (nib[2] << 8) + (nib[3] << 12);
    } else if (M == 4) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t nib;
            mvue_2of4_bf16_gather<kSR>(raw[2 * j], raw[2 * j + 1], words[j], &v[j], &nib, rnd[j]);
            meta += nib << (4 * j);
        }
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t nib;
            mvue_1of2x2_bf16<kSR>(raw[2 * j], raw[2 * j + 1], words[(2 * j) % UnitWords<M, kJoint>::kCount],
                                  words[(2 * j + 1) % UnitWords<M, kJoint>::kCount], &v[j], &nib, rnd[j]);
            meta += nib << (4 * j);
        }
    }
    *out_values = make_uint4(v[0], v[1], v[2], v[3]);
    *out_meta = meta;
}

template <int M, int kJoint = 0, bool kSR = false, bool kEps16 = false>
__device__ __forceinline__ void prune_unit_bf16(const uint32_t (&raw)[8], uint64_t unit_index,
                                                const RoundKeys& rk, uint4* out_values,
                                                uint32_t* out_meta) {
    uint32_t words[UnitWords<M, kJoint>::kCount];
    unit_words<UnitWords<M, kJoint>::kCount, kEps16>(unit_index, rk, words);
    prune_unit_bf16_w<M, kJoint, kSR>(raw, words, unit_index, rk, out_values, out_meta);
}

// One work unit whose 16 elements are the half kHigh of 16 row words (K runs down the rows of g).
template <int M, bool kHigh, int kJoint = 0>
__device__ __forceinline__ void prune_unit_bf16_rows(const uint32_t (&w)[16], uint64_t unit_index,
                                                     const RoundKeys& rk, uint4* out_values, uint32_t* out_meta) {
    uint32_t v[4];
    uint32_t meta = 0;
    if (M == 4 && kJoint == 3) {
        const uint4 r = philox4x32_10(unit_index, rk);
        const uint32_t words[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t nib;
            auto widen = [](uint32_t x) { return kHigh ? (x & 0xFFFF0000u) : (x << 16); };
            mvue_1of4_f32(widen(w[4 * j]), widen(w[4 * j + 1]), widen(w[4 * j + 2]), widen(w[4 * j + 3]), words[j],
                          &v[j], &nib);
            meta += nib << (4 * j);
        }
    } else if (M == 4 && kJoint == 2) {
        const uint4 ra = philox4x32_10(2 * unit_index, rk);
        const uint4 rb = philox4x32_10(2 * unit_index + 1, rk);
        const uint32_t words[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t nib;
            auto widen = [](uint32_t x) { return kHigh ? (x & 0xFFFF0000u) : (x << 16); };
            mvue_2of4_approx_f32(widen(w[4 * j]), widen(w[4 * j + 1]), widen(w[4 * j + 2]), widen(w[4 * j + 3]),
                                 words[2 * j], words[2 * j + 1], &v[j], &nib);
            meta += nib << (4 * j);
        }
    } else if (M == 4) {
        const uint4 r = philox4x32_10(unit_index, rk);
        const uint32_t words[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t nib;
            if (kJoint == 0) {
                mvue_2of4_bf16<kHigh, kHigh, kHigh, kHigh>(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3],
                                                           words[j], &v[j], &nib);
            } else {   // the halves of two row words side by side: a0 | a1 << 16, a2 | a3 << 16
                const uint32_t x01 = __byte_perm(w[4 * j], w[4 * j + 1], kHigh ? 0x7632u : 0x5410u);
                const uint32_t x23 = __byte_perm(w[4 * j + 2], w[4 * j + 3], kHigh ? 0x7632u : 0x5410u);
                mvue_2of4_sys_bf16(x01, x23, words[j], &v[j], &nib);
            }
            meta += nib << (4 * j);
        }
    } else {
        const uint4 ra = philox4x32_10(2 * unit_index, rk);
        const uint4 rb = philox4x32_10(2 * unit_index + 1, rk);
        const uint32_t words[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t nib;
            mvue_1of2x2_bf16_rows<kHigh>(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3], words[2 * j],
                                         words[2 * j + 1], &v[j], &nib);
            meta += nib << (4 * j);
        }
    }
    *out_values = make_uint4(v[0], v[1], v[2], v[3]);
    *out_meta = meta;
}

}  // namespace mvue
