/*
 * CPU oracle for minimum-variance unbiased (MVUE) N:M pruning of a neural
 * gradient and for the matrix products that consume the pruned operand.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what
 * the method computes.  It shares no code with the CUDA library and must never
 * be linked into, imported by, or called from the product path.
 *
 * Every floating-point step of the selection is IEEE binary32, round to
 * nearest even, evaluated in exactly the order written.  Build with
 * -ffp-contract=off so the compiler never fuses a multiply with an add, and
 * without any fast-math option.
 *
 * Notation follows the paper: a block a = [a_1..a_M], theta(a) the pruned
 * block, p_i the probability that element i survives, p_ij the probability
 * that the pair (i, j) survives (indices refer to the block sorted by
 * magnitude, a_1 <= a_2 <= a_3 <= a_4).
 *
 * Parity pins (see tests): Philox against two independent implementations;
 * the 1:2 sampler against the closed form of Sec. 4.1; the 2:4 sampler against
 * the pair table of App. A.2 and the optimal marginals of Sec. 4.2 by an
 * exhaustive sweep over every value of the 24-bit uniform, and draw by draw
 * against oracle_mvue_2of4_cases, the appendix written out case by case in
 * binary64 (same pair on all but a handful of the 2^24 draws, same kept values
 * to binary32 rounding); the second 2:4 law
 * (systematic sampling) against the same optimal marginals, mean and minimal
 * variance by the same sweep, and against its interval-overlap law; bf16 rounding
 * against a library cast; the product against a library fp64 matmul; the
 * approx-MVUE sampler of Sec. 4.4 against the sequential-draw probabilities and the
 * inclusion-probability equation of that section by exhaustive sweeps of each draw.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

/* ------------------------------------------------------------------------
 * Counter-based random numbers: Philox4x32 with ten rounds (Salmon, Moraes,
 * Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3", SC'11).
 * The paper only asks for i.i.d. eps ~ U[0,1] (App. "Pruning Overhead",
 * Part 1); a counter-based generator keyed by (seed, block index) makes every
 * block's draw a pure function of its position.
 * ---------------------------------------------------------------------- */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint64_t mult0 = 0xD2511F53u;    /* multiplies counter word 0 */
    const uint64_t mult1 = 0xCD9E8D57u;    /* multiplies counter word 2 */
    const uint32_t bump0 = 0x9E3779B9u;    /* added to key word 0 after each round */
    const uint32_t bump1 = 0xBB67AE85u;    /* added to key word 1 after each round */
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t prod0 = mult0 * (uint64_t)c0;
        uint64_t prod1 = mult1 * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
        uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += bump0;
        k1 += bump1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 32-bit word that drives block number q (q counts blocks of the whole
 * operand, row by row): one generator call serves four consecutive blocks. */
uint32_t oracle_block_word(uint64_t seed, uint64_t q)
{
    uint64_t call = q >> 2;
    uint32_t ctr[4] = { (uint32_t)call, (uint32_t)(call >> 32), 0u, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    oracle_philox4x32_10(ctr, key, out);
    return out[q & 3u];
}

/* The two words of block number q for the estimator that draws twice per block
 * (Sec. 4.4): one generator call serves two consecutive blocks. */
void oracle_block_word_pair(uint64_t seed, uint64_t q, uint32_t words[2])
{
    uint64_t call = q >> 1;
    uint32_t ctr[4] = { (uint32_t)call, (uint32_t)(call >> 32), 0u, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    oracle_philox4x32_10(ctr, key, out);
    words[0] = out[2 * (q & 1u)];
    words[1] = out[2 * (q & 1u) + 1];
}

/* Sixteen random bits per block instead of thirty-two: one generator call then serves eight consecutive blocks
 * (sixteen elements of 1:2, thirty-two of 2:4 / 1:4).  Block number q takes the low (q even) or high (q odd) half
 * of word (q >> 1) & 3 of generator call q >> 3, and the sampler is handed those sixteen bits in the TOP half of a
 * 32-bit word whose low half is zero -- so the block samplers themselves are unchanged, only eps has a resolution of
 * 2^-16 (2^-15 for systematic sampling, which reads one bit less) instead of 2^-24 / 2^-23.  The paper asks only for
 * i.i.d. eps ~ U[0,1] (App. "Pruning Overhead", Part 1); every mask probability moves by at most that resolution,
 * still two hundred times finer than the bf16 grid the survivors are stored on. */
uint32_t oracle_block_word16(uint64_t seed, uint64_t q)
{
    uint64_t call = q >> 3;
    uint32_t ctr[4] = { (uint32_t)call, (uint32_t)(call >> 32), 0u, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    oracle_philox4x32_10(ctr, key, out);
    uint32_t w = out[(q >> 1) & 3u];
    return (q & 1u) ? (w & 0xFFFF0000u) : (w << 16);
}

/* The same economy for the estimator that draws twice per block (Sec. 4.4): block q takes word q & 3 of generator
 * call q >> 2 (one call serves four blocks instead of two), its low half for the first draw, its high half for the
 * second, each in the top half of a word. */
void oracle_block_word_pair16(uint64_t seed, uint64_t q, uint32_t words[2])
{
    uint64_t call = q >> 2;
    uint32_t ctr[4] = { (uint32_t)call, (uint32_t)(call >> 32), 0u, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    oracle_philox4x32_10(ctr, key, out);
    uint32_t w = out[q & 3u];
    words[0] = w << 16;
    words[1] = w & 0xFFFF0000u;
}

/* eps in [0,1): the top 24 bits of the word, exactly representable. */
float oracle_uniform24(uint32_t word)
{
    return (float)(word >> 8) * 5.9604644775390625e-08f;   /* 2^-24 */
}

/* ------------------------------------------------------------------------
 * bf16 storage: round a binary32 value to the nearest bfloat16, ties to even,
 * by integer arithmetic on the bit pattern.  Inputs are finite.
 * ---------------------------------------------------------------------- */
uint16_t oracle_bf16_rne(float x)
{
    uint32_t bits;
    memcpy(&bits, &x, 4);
    uint32_t lsb = (bits >> 16) & 1u;
    bits += 0x7FFFu + lsb;
    return (uint16_t)(bits >> 16);
}

float oracle_bf16_to_f32(uint16_t h)
{
    uint32_t bits = (uint32_t)h << 16;
    float x;
    memcpy(&x, &bits, 4);
    return x;
}

/* ------------------------------------------------------------------------
 * Stochastic rounding of a survivor to bf16 (Sec. 3 recalls that the neural
 * gradients want an unbiased quantiser "such as stochastic rounding"; App.
 * "Pruning Overhead" Part 1 names stochastic rounding as the sampling
 * primitive).  With round-to-nearest the stored survivor is a_i / p_i only up
 * to the bf16 grid, so E[stored] = a_i (1 + delta), |delta| <= 2^-9; rounding
 * stochastically makes the stored value itself unbiased:
 *     x lies between two neighbouring bf16 numbers lo <= x < hi (same sign);
 *     store hi with probability (x - lo) / (hi - lo), else lo.
 * On the bit pattern: the low 16 bits f of x are the numerator of that
 * probability over 2^16, and adding r, a uniform 16-bit integer, carries into
 * the upper half exactly when f + r >= 2^16, i.e. for f of the 2^16 values of r:
 *     stored = (bits(x) + r) >> 16.
 * A value already on the bf16 grid (f = 0) never moves; a carry out of the
 * mantissa lands on the next power of two, which is the correct neighbour.
 * Inputs are finite and below 2^127 in magnitude.
 * ---------------------------------------------------------------------- */
uint16_t oracle_bf16_sr(float x, uint16_t r)
{
    uint32_t bits;
    memcpy(&bits, &x, 4);
    return (uint16_t)((bits + (uint32_t)r) >> 16);
}

/* The 16 random bits that round survivor slot e (0..7) of unit number u (a unit
 * is 16 consecutive elements along K: four blocks of four, or eight pairs; its
 * eight survivors in packed order are the slots).  They come from a generator
 * call of their own, counter (lo32(u), hi32(u), 1, 0) under the same key -- the
 * selection draws all have third counter word 0 -- slot e taking the low (e even)
 * or high (e odd) half of word e / 2. */
uint16_t oracle_rounding_bits(uint64_t seed, uint64_t u, int e)
{
    uint32_t ctr[4] = { (uint32_t)u, (uint32_t)(u >> 32), 1u, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    oracle_philox4x32_10(ctr, key, out);
    uint32_t w = out[e >> 1];
    return (uint16_t)((e & 1) ? (w >> 16) : (w & 0xFFFFu));
}

/* ------------------------------------------------------------------------
 * MVUE 1:2 (Sec. 4.1, the estimator that closes that section; derivation in
 * App. A.1): keep a_1 with probability |a_1| / (|a_1| + |a_2|), else a_2; the
 * survivor becomes sign(a_i) (|a_1| + |a_2|).  The draw is the threshold test
 * eps < p_1 (App. "Pruning Overhead", Part 1) written without the division:
 * eps (|a_1|+|a_2|) < |a_1|, with eps = n / 2^24, n the top 24 bits of the
 * block's random word, evaluated as n * ((|a_1|+|a_2|) * 2^-24).
 * Zero rule (the paper leaves 0/0 open): a_2 = 0 always keeps a_1, so a zero
 * is never preferred to a non-zero; an all-zero block keeps a_1 (a signed zero).
 * Returns the kept index (0 or 1); *kept receives the new value.
 * ---------------------------------------------------------------------- */
int oracle_mvue_1of2(float a1, float a2, uint32_t word, float *kept)
{
    float m1 = fabsf(a1), m2 = fabsf(a2);
    float S = m1 + m2;
    float scale = S * 5.9604644775390625e-08f;            /* S * 2^-24, exact */
    float t = (float)(word >> 8) * scale;                 /* eps * S */
    int idx = (t < m1 || m2 == 0.0f) ? 0 : 1;
    *kept = copysignf(S, idx == 0 ? a1 : a2);
    return idx;
}

/* ------------------------------------------------------------------------
 * MVUE 2:4 (optimal marginals: Sec. 4.2; joint law over pairs: App. A.2).
 *
 * 1. Sort the magnitudes ascending, ties by original position:
 *      s_1 <= s_2 <= s_3 <= s_4  at original positions i_1..i_4.
 * 2. The appendix gives, for each of its three cases, the probability p_ij
 *    that the pair of ranks (i, j) survives.  The pair is drawn by walking the
 *    table in the fixed order 13, 14, 23, 24, 34: the first pair whose
 *    cumulative probability exceeds eps wins.  No division is needed: with
 *    d = s_4 - s_3 every case has the SAME cumulative numerators over the
 *    denominator D,
 *         C_13 = 2 s_1 - d                        (only case 1 has p_13 > 0)
 *         C_14 = 4 s_1
 *         C_23 = 4 s_1 + (2 s_2 - d) + min(2 s_1 - d, 0)
 *         C_24 = 4 (s_1 + s_2)
 *      case 1 (s_4 <= 2 s_1 + s_3):  D = 2 sum; the four numerators of the
 *              table are C_13, C_14 - C_13, C_23 - C_14, C_24 - C_23.
 *      case 2 (2 s_1 + s_3 <= s_4 <= s_1+s_2+s_3):  D = 2 sum; C_13 <= 0 is
 *              never hit (p_13 = 0) and C_23 = 2 (3 s_1 + s_2 - d)
 *              = 2 (2 s_1 + (s_1+s_2+s_3-s_4)), the table's p_14 + p_23.
 *      case 3 (s_4 >= s_1+s_2+s_3):  D = 4 (s_1+s_2+s_3); C_13 <= 0 and
 *              C_23 <= C_14 are never hit, leaving s_1 and s_1 + s_2 over
 *              s_1+s_2+s_3 for the partner of the dominant element.
 *    D = 2 (2 S3 + min(s_4 - S3, 0)) with S3 = s_1+s_2+s_3 covers all three
 *    (sum + sum in cases 1-2, 4 S3 in case 3).
 *    In case 3 the larger survivor is the dominant element whatever rounding
 *    does to C_23.
 * 3. Survivors become a_i / p_i (Sec. 4.2): sign(a_i) D/4 for every survivor
 *    with p_i < 1 (sum/2 in cases 1-2, S3 in case 3), and the dominant
 *    element of case 3 keeps its value: max(s_4, D/4).
 * Zero rule: an element of magnitude zero has zero-width intervals in the
 * walk, so it survives only if fewer than two non-zeros exist (pair 34 of the
 * (magnitude, position) order), as a signed zero.
 *
 * idx[0] < idx[1] are the surviving original positions, val[] their new
 * values in that order.
 * ---------------------------------------------------------------------- */
void oracle_mvue_2of4(const float a[4], uint32_t word, int idx[2], float val[2])
{
    float s[4];
    int   pos[4];
    /* insertion sort on (magnitude, position); strict '<' keeps ties stable */
    for (int i = 0; i < 4; ++i) {
        float m = fabsf(a[i]);
        int j = i;
        while (j > 0 && m < s[j - 1]) { s[j] = s[j - 1]; pos[j] = pos[j - 1]; --j; }
        s[j] = m; pos[j] = i;
    }
    const float s1 = s[0], s2 = s[1], s3 = s[2], s4 = s[3];
    const float S12 = s1 + s2;
    const float S3  = S12 + s3;
    const float d   = s4 - s3;
    const float x   = (s1 + s1) - d;                       /* 2 s_1 - d */
    const float y   = (s2 + s2) - d;                       /* 2 s_2 - d */
    const float C13 = x;
    const float C14 = 4.0f * s1;
    const float C23 = (C14 + y) + (x < 0.0f ? x : 0.0f);
    const float C24 = 4.0f * S12;
    const float e   = s4 - S3;                             /* >= 0: case 3 */
    const float Dh  = (S3 + S3) + (e < 0.0f ? e : 0.0f);   /* D / 2 */
    const float scale = Dh * 1.1920928955078125e-07f;      /* D * 2^-24, exact */
    const float t = (float)(word >> 8) * scale;            /* eps * D */

    int ka, kb;                                            /* sorted ranks (0..3) of the survivors */
    if      (t < C13) { ka = 0; kb = 2; }
    else if (t < C14) { ka = 0; kb = 3; }
    else if (t < C23) { ka = 1; kb = 2; }
    else if (t < C24) { ka = 1; kb = 3; }
    else              { ka = 2; kb = 3; }
    if (e >= 0.0f) kb = 3;                                 /* case 3: the dominant element always survives */

    const float quarter_D = 0.5f * Dh;
    const float va = copysignf(quarter_D, a[pos[ka]]);
    const float vb = copysignf(s4 > quarter_D ? s4 : quarter_D, a[pos[kb]]);
    if (pos[ka] < pos[kb]) { idx[0] = pos[ka]; idx[1] = pos[kb]; val[0] = va; val[1] = vb; }
    else                   { idx[0] = pos[kb]; idx[1] = pos[ka]; val[0] = vb; val[1] = va; }
}

/* ------------------------------------------------------------------------
 * MVUE 2:4 exactly as App. A.2 prints it, case by case, in binary64.
 *
 * This is the reference statement of the appendix and nothing else: sort the
 * magnitudes (ties by position), decide which of the three cases holds, form
 * that case's own six pair probabilities p_12 .. p_34 over that case's own
 * denominator with divisions, and draw the pair by the threshold test
 * eps < (cumulative p) of App. "Pruning Overhead" Part 1, walking the pairs in
 * the order the appendix lists them (12, 13, 14, 23, 24, 34), eps = n / 2^24.
 * A survivor becomes a_i / p_i (Sec. 4.2) with p_i the sum of the p_ij that
 * contain i.  No algebra is shared between the cases and nothing is rearranged
 * to avoid a division.
 *
 * oracle_mvue_2of4 above is the binary32, division-free evaluation that the GPU
 * must reproduce bit for bit; this function is what pins it to the appendix
 * (tests/test_oracle_mvue24.py sweeps every eps through both).  The two may
 * differ only where binary32 rounding moves a threshold: a handful of the 2^24
 * draws per block, and the last place of a kept value.
 *
 * The appendix assumes a_4 > a_3 > a_2 > a_1 > 0.  Ties and zeros among three
 * or more non-zeros are covered by its formulas as they stand (a zero gets
 * zero-width intervals).  With fewer than two non-zero elements every
 * denominator vanishes (0/0): the function then returns -1 and computes
 * nothing -- that situation is ruled by the zero rule stated above, not by the
 * appendix.  Returns the case number (1, 2 or 3) otherwise.
 * idx[0] < idx[1]: surviving original positions; val[]: their new values
 * (binary64).
 * ---------------------------------------------------------------------- */
int oracle_mvue_2of4_cases_planted(const float a[4], uint32_t word, int idx[2], double val[2], int mistake);

int oracle_mvue_2of4_cases(const float a[4], uint32_t word, int idx[2], double val[2])
{
    return oracle_mvue_2of4_cases_planted(a, word, idx, val, 0);
}

/* The same with one deliberate mistake planted (mistake = 1, 2, 3: in that case's formulas), so that the tests
 * can show that the comparison with the binary32 sampler would notice it.  mistake = 0 is the appendix. */
int oracle_mvue_2of4_cases_planted(const float a[4], uint32_t word, int idx[2], double val[2], int mistake)
{
    double s[4];
    int    pos[4];
    for (int i = 0; i < 4; ++i) {                           /* stable insertion sort by magnitude */
        double m = fabs((double)a[i]);
        int j = i;
        while (j > 0 && m < s[j - 1]) { s[j] = s[j - 1]; pos[j] = pos[j - 1]; --j; }
        s[j] = m; pos[j] = i;
    }
    const double a1 = s[0], a2 = s[1], a3 = s[2], a4 = s[3];
    if (a3 == 0.0) return -1;                               /* fewer than two non-zeros: 0/0 in every case */
    const double eps = (double)(word >> 8) / 16777216.0;    /* n / 2^24 */
    double p12, p13, p14, p23, p24, p34;
    int which;
    if (a4 >= a1 + a2 + a3) {
        /* case 3: a_4 is kept with probability 1, and one of a_1, a_2, a_3 with
         * probability a_i / (a_1 + a_2 + a_3) */
        which = 3;
        const double rest = a1 + a2 + a3;
        p12 = 0.0; p13 = 0.0; p23 = 0.0;
        p14 = a1 / rest;
        p24 = a2 / rest;
        p34 = a3 / rest;
        if (mistake == 3) { p14 = p24 = p34 = 1.0 / 3.0; }        /* planted: partner drawn uniformly */
    } else if (a4 <= 2.0 * a1 + a3) {
        /* case 1 */
        which = 1;
        const double sum = a1 + a2 + a3 + a4;
        p12 = 0.0;
        p13 = (2.0 * a1 + a3 - a4) / (2.0 * sum);
        p14 = (2.0 * a1 - a3 + a4) / (2.0 * sum);
        p23 = (2.0 * a2 + a3 - a4) / (2.0 * sum);
        p24 = (2.0 * a2 - a3 + a4) / (2.0 * sum);
        p34 = (-a1 - a2 + a3 + a4) / sum;
        if (mistake == 1) { double t = p13; p13 = p14; p14 = t; }  /* planted: a_3 and a_4 swapped in the first row */
    } else {
        /* case 2: 2 a_1 + a_3 <= a_4 <= a_1 + a_2 + a_3 */
        which = 2;
        const double sum = a1 + a2 + a3 + a4;
        p12 = 0.0;
        p13 = 0.0;
        p14 = (mistake == 2 ? 1.0 : 2.0) * a1 / sum;               /* planted: the factor two dropped */
        p23 = (a1 + a2 + a3 - a4) / sum;
        p24 = (-a1 + a2 - a3 + a4) / sum;
        p34 = (-a1 - a2 + a3 + a4) / sum;
    }
    /* threshold walk in the appendix's order */
    int ra, rb;                                             /* sorted ranks (0..3) of the survivors */
    double c = p12;
    if (eps < c) { ra = 0; rb = 1; }
    else if (eps < (c += p13)) { ra = 0; rb = 2; }
    else if (eps < (c += p14)) { ra = 0; rb = 3; }
    else if (eps < (c += p23)) { ra = 1; rb = 2; }
    else if (eps < (c += p24)) { ra = 1; rb = 3; }
    else { ra = 2; rb = 3; }
    /* survival probabilities of the four ranks: sums over the pairs that hold them */
    const double p[4] = { p12 + p13 + p14, p12 + p23 + p24, p13 + p23 + p34, p14 + p24 + p34 };
    const double va = copysign(s[ra] / p[ra], (double)a[pos[ra]]);
    const double vb = copysign(s[rb] / p[rb], (double)a[pos[rb]]);
    if (pos[ra] < pos[rb]) { idx[0] = pos[ra]; idx[1] = pos[rb]; val[0] = va; val[1] = vb; }
    else                   { idx[0] = pos[rb]; idx[1] = pos[ra]; val[0] = vb; val[1] = va; }
    return which;
}

/* Every eps through both statements of App. A.2 (the case-by-case binary64 one and
 * the binary32 one above): *pair_diff = the number of the 2^24 draws on which they
 * keep different pairs; *max_rel = the largest relative difference between their
 * kept values over the draws on which they keep the same pair (mistake: see
 * oracle_mvue_2of4_cases_planted; 0 for the appendix as printed).  Returns the case
 * number, or -1 (and touches nothing) for a block with fewer than two non-zeros. */
int oracle_sweep_2of4_cases(const float a[4], int mistake, uint64_t *pair_diff, double *max_rel)
{
    uint64_t diff = 0;
    double worst = 0.0;
    int which = -1;
    for (uint32_t n = 0; n < (1u << 24); ++n) {
        int ia[2], ib[2]; double va[2]; float vb[2];
        which = oracle_mvue_2of4_cases_planted(a, n << 8, ia, va, mistake);
        if (which < 0) return -1;
        oracle_mvue_2of4(a, n << 8, ib, vb);
        if (ia[0] != ib[0] || ia[1] != ib[1]) { diff += 1; continue; }
        for (int e = 0; e < 2; ++e) {
            double d = fabs(va[e] - (double)vb[e]);
            double ref = fabs(va[e]);
            double rel = ref > 0.0 ? d / ref : d;
            if (rel > worst) worst = rel;
        }
    }
    *pair_diff = diff;
    *max_rel = worst;
    return which;
}

/* ------------------------------------------------------------------------
 * MVUE 2:4 with a second joint law: systematic sampling.
 *
 * Sec. 4.2 shows that the block variance (its variance equation) is a function
 * of the marginals p_i alone, and that a 2:4 estimator is optimal exactly when
 * its marginals satisfy one of the two optimality criteria of that section
 * (all p_i = 2 a_i / sum, or one p_i = 1 and the rest a_k / sum of the rest).
 * App. A.2 is ONE joint law over pairs with those marginals.  This function
 * draws the pair from another law with the SAME marginals and the same kept
 * values a_i / p_i, hence the same expectation and the same (minimal)
 * variance, that needs no sort:
 *
 * 1. Work in the block's own order.  m_k = |a_k|, R_k = the sum of the other
 *    three magnitudes, and the weight e_k = min(m_k, R_k): an element heavier
 *    than the rest together is clipped to their sum (at most one element is
 *    clipped).  D = e_0+e_1+e_2+e_3, H = D/2; then e_k / H is exactly the
 *    optimal p_k of Sec. 4.2 in both of its cases (unclipped: H = sum/2;
 *    clipped element i: H = R_i, p_i = 1, p_k = m_k / R_i).
 * 2. Lay the weights end to end: element k owns [c_k, c_{k+1}) with c_0 = 0,
 *    c_1 = e_0, c_2 = c_1 + e_1, c_3 = c_2 + e_2.  Draw t = eps H in [0, H) and
 *    keep the owner of t and the owner of t + H.  Every interval is at most H
 *    long, so the two owners differ and element k is kept with probability
 *    e_k / H.
 * 3. A survivor becomes sign(a_k) max(m_k, H): H = m_k / p_k when p_k < 1, and
 *    the clipped element (p = 1, m_k >= H) keeps its value.
 *
 * Arithmetic (binary32, in the order written):
 *    q01 = (m0 + m1) + tiny,  q23 = (m2 + m3) + tiny,   tiny = 2^-149
 *    R0 = m1 + q23, R1 = m0 + q23, R2 = q01 + m3, R3 = q01 + m2
 *    eps = n / 2^23, n = the top 23 bits of the block's word;
 *    Hs = D 2^-24, H = D/2, t2 = (2^23 + n) Hs  (one rounding; H <= t2 < D), t = t2 - H
 *    (exact, since H <= t2 <= 2H): the two points are exactly H apart and 0 <= t < H
 *    i  = #{k in 1,2 : c_k <= t}
 *    j  = max(i + 1, #{k in 1,2,3 : c_k <= t2})
 * so that i < j are two valid positions for every input and every rounding.
 * Where a prefix sum is inexact a boundary sits one unit in the last place off
 * its exact position; the one or two draws (of 2^23) that fall into such a gap
 * resolve through the max above, which moves each survival probability by at
 * most 2^-22, the resolution of eps itself.
 * Zero rule: an element of magnitude zero owns an empty interval and is never
 * drawn.  tiny (the smallest positive binary32 number) leaves every R_k that is
 * a normal number unchanged and gives a lone non-zero element a non-empty
 * interval: then D = tiny, H and t round to zero, i is the number of zeros
 * before it (at most 2) and j = i + 1 or 3, so the non-zero survives with its own
 * value and a zero is kept beside it as a signed zero; an all-zero block keeps
 * positions 2 and 3.
 *
 * idx[0] < idx[1] are the surviving positions, val[] their new values.
 * ---------------------------------------------------------------------- */
void oracle_mvue_2of4_systematic(const float a[4], uint32_t word, int idx[2], float val[2])
{
    const float tiny = 1.401298464324817e-45f;             /* 2^-149 */
    const float m0 = fabsf(a[0]), m1 = fabsf(a[1]), m2 = fabsf(a[2]), m3 = fabsf(a[3]);
    const float q01 = (m0 + m1) + tiny;
    const float q23 = (m2 + m3) + tiny;
    const float R0 = m1 + q23, R1 = m0 + q23, R2 = q01 + m3, R3 = q01 + m2;
    const float e0 = m0 < R0 ? m0 : R0;
    const float e1 = m1 < R1 ? m1 : R1;
    const float e2 = m2 < R2 ? m2 : R2;
    const float e3 = m3 < R3 ? m3 : R3;
    const float c1 = e0;
    const float c2 = c1 + e1;
    const float c3 = c2 + e2;
    const float D  = c3 + e3;
    const float Hs = D * 5.9604644775390625e-08f;          /* D 2^-24 */
    const float H  = 0.5f * D;
    const float n2 = (float)((word >> 9) + (1u << 23));    /* 2^23 + n: 24 bits, exact */
    const float t2 = n2 * Hs;
    const float t  = t2 - H;
    int i = (c1 <= t) + (c2 <= t);
    int j = (c1 <= t2) + (c2 <= t2) + (c3 <= t2);
    if (j < i + 1) j = i + 1;
    const float m[4] = { m0, m1, m2, m3 };
    idx[0] = i; idx[1] = j;
    val[0] = copysignf(m[i] > H ? m[i] : H, a[i]);
    val[1] = copysignf(m[j] > H ? m[j] : H, a[j]);
}

/* ------------------------------------------------------------------------
 * Approximately optimal 2:4 (Sec. 4.4, "approx-MVUE"): two sequential draws
 * without replacement, each proportional to magnitude, and survivors divided by
 * their exact inclusion probability (the equation of Sec. 4.4), so the estimator
 * is unbiased; its variance is above the optimum of Sec. 4.2 by a factor the
 * paper's scan bounds below two.
 *
 * Steps (m_k = |a_k|, block order, no sort):
 * 1. First draw: element i with probability m_i / s, s = m_0+m_1+m_2+m_3, by the
 *    threshold test of App. "Pruning Overhead" Part 1 walked over the running
 *    sums c_1 = m_0, c_2 = c_1 + m_1, c_3 = c_2 + m_2, s = c_3 + m_3:
 *        t_1 = n_1 (s 2^-24),   i = #{k in 1,2,3 : c_k <= t_1},
 *    n_1 the top 24 bits of the block's first random word.
 * 2. Second draw among the other three, in position order r_0 < r_1 < r_2, with
 *    probability m_j / (s - m_i).  "s - m_i" is formed as the sum of the others,
 *    R_i = (m_{r0} + m_{r1}) + m_{r2}, never as a difference:
 *        d_1 = m_{r0}, d_2 = d_1 + m_{r1}, R_i = d_2 + m_{r2},
 *        t_2 = n_2 (R_i 2^-24),   j = r_{#{k in 1,2 : d_k <= t_2}},
 *    n_2 from the block's second random word.  i != j for every input.
 * 3. Inclusion probability (Sec. 4.4): p_k = m_k/s + sum_{l != k} (m_l/s)(m_k/R_l)
 *    = (m_k/s)(1 + T_k), T_k = sum_{l != k} vv_l, vv_l = m_l / R_l (Algorithm 1's vv;
 *    its q - vv_k is T_k, summed here directly so nothing cancels).  The survivor
 *    becomes a_k / p_k = sign(a_k) s / (1 + T_k): six divisions per block (the four
 *    vv_l, then one per survivor).  Sums of three run in position order, (x + y) + z.
 * Zero rules: an element of magnitude zero owns an empty interval in both walks.
 * If R_i = 0 (at most one non-zero in the block) both survivors keep their own
 * values (p = 1): the non-zero, if any, and a signed zero beside it; an all-zero
 * block keeps positions 3 and 2.
 *
 * first / second: the positions drawn first and second; v_first / v_second
 * their new values.
 * ---------------------------------------------------------------------- */
void oracle_mvue_2of4_approx_ordered(const float a[4], uint32_t word1, uint32_t word2,
                                     int *first, int *second, float *v_first, float *v_second)
{
    float m[4], R[4], vv[4];
    for (int k = 0; k < 4; ++k) m[k] = fabsf(a[k]);
    /* first draw */
    const float c1 = m[0];
    const float c2 = c1 + m[1];
    const float c3 = c2 + m[2];
    const float s  = c3 + m[3];
    const float t1 = (float)(word1 >> 8) * (s * 5.9604644775390625e-08f);
    const int i = (c1 <= t1) + (c2 <= t1) + (c3 <= t1);
    /* sums of the other three, in position order */
    for (int k = 0; k < 4; ++k) {
        int r[3], n = 0;
        for (int l = 0; l < 4; ++l) if (l != k) r[n++] = l;
        R[k] = (m[r[0]] + m[r[1]]) + m[r[2]];
    }
    /* second draw among the others */
    int r[3], n = 0;
    for (int l = 0; l < 4; ++l) if (l != i) r[n++] = l;
    const float d1 = m[r[0]];
    const float d2 = d1 + m[r[1]];
    const float t2 = (float)(word2 >> 8) * (R[i] * 5.9604644775390625e-08f);
    const int j = r[(d1 <= t2) + (d2 <= t2)];
    /* survivors */
    float vi, vj;
    if (R[i] == 0.0f) {
        vi = a[i]; vj = a[j];
    } else {
        for (int k = 0; k < 4; ++k) vv[k] = m[k] / R[k];
        float T[2];
        const int who[2] = { i, j };
        for (int e = 0; e < 2; ++e) {
            int o[3], c = 0;
            for (int l = 0; l < 4; ++l) if (l != who[e]) o[c++] = l;
            T[e] = (vv[o[0]] + vv[o[1]]) + vv[o[2]];
        }
        vi = copysignf(s / (1.0f + T[0]), a[i]);
        vj = copysignf(s / (1.0f + T[1]), a[j]);
    }
    *first = i; *second = j; *v_first = vi; *v_second = vj;
}

/* The same with the survivors in ascending position: idx[0] < idx[1], val[] their new values. */
void oracle_mvue_2of4_approx(const float a[4], uint32_t word1, uint32_t word2, int idx[2], float val[2])
{
    int i, j; float vi, vj;
    oracle_mvue_2of4_approx_ordered(a, word1, word2, &i, &j, &vi, &vj);
    if (i < j) { idx[0] = i; idx[1] = j; val[0] = vi; val[1] = vj; }
    else       { idx[0] = j; idx[1] = i; val[0] = vj; val[1] = vi; }
}

/* ------------------------------------------------------------------------
 * MVUE 1:4 (appendix "Additional sparsity results": like MVUE 1:2 for a block of
 * four): one element survives, element i with probability |a_i| / S,
 * S = |a_1|+|a_2|+|a_3|+|a_4|, and becomes sign(a_i) S.  This is Sec. 4.1's
 * argument for a block of M: an unbiased estimator that keeps one element has
 * theta_i = a_i / p_i, its variance sum_i a_i^2 / p_i - a_i^2 is least, under
 * sum_i p_i = 1, at p_i proportional to |a_i|, where it equals S^2 - sum a_i^2.
 * Draw: the threshold walk of App. "Pruning Overhead" Part 1 in the block's
 * own order over c_1 = m_1, c_2 = c_1 + m_2, c_3 = c_2 + m_3, S = c_3 + m_4:
 *     t = n (S 2^-24),   i = #{k in 1,2,3 : c_k <= t},
 * n the top 24 bits of the block's random word (one word per block, as for 2:4).
 * Zero rule: an element of magnitude zero owns an empty interval; an all-zero
 * block keeps its last element (a signed zero).
 * Returns the surviving position (0..3); *kept receives the new value.
 * ---------------------------------------------------------------------- */
int oracle_mvue_1of4(const float a[4], uint32_t word, float *kept)
{
    const float m0 = fabsf(a[0]), m1 = fabsf(a[1]), m2 = fabsf(a[2]), m3 = fabsf(a[3]);
    const float c1 = m0;
    const float c2 = c1 + m1;
    const float c3 = c2 + m2;
    const float S  = c3 + m3;
    const float t  = (float)(word >> 8) * (S * 5.9604644775390625e-08f);
    const int i = (c1 <= t) + (c2 <= t) + (c3 <= t);
    *kept = copysignf(S, a[i]);
    return i;
}

/* ------------------------------------------------------------------------
 * Approximately optimal 4:8 (appendix "Additional sparsity results": the
 * approximate 2:4 method of Sec. 4.4 carried to a block of eight with four
 * survivors; the paper gives no formulas).  Reading taken here: Sec. 4.4's
 * procedure with four draws instead of two -- each draw removes one of the
 * remaining elements with probability proportional to its magnitude -- and
 * Sec. 4.4's rule for the kept values, a_i / p_i with p_i the EXACT probability
 * that element i is among the four drawn, so that E[theta(a)] = a still holds.
 *
 * Inclusion probability.  The chance that the first |R| draws are the elements
 * of the set R, in any order, obeys
 *     w({}) = 1,   w(R) = sum_{k in R} w(R \ k) m_k / rest(R \ k),
 * rest(Q) = the sum of the magnitudes NOT in Q (what is left after Q was
 * removed), and element i is drawn at step |R| + 1 after R with probability
 * m_i / rest(R), so
 *     p_i = sum over R not containing i, |R| <= 3, of  w(R) m_i / rest(R).
 * For two draws from four this is the equation of Sec. 4.4.
 *
 * Arithmetic (binary32, in the order written; one IEEE division per set):
 *   rest(Q): the magnitudes outside Q added left to right in position order;
 *   inv(Q) = 1 / rest(Q), or 0 when rest(Q) = 0 (then nothing is left to draw);
 *   u(Q) = w(Q) inv(Q), so that m_k / rest(Q) times w(Q) is formed as u(Q) m_k:
 *     u({}) = inv({}),  w(R) = sum_{k in R} u(R \ k) m_k,  u(R) = w(R) inv(R),
 *     p_i = sum_{R not containing i, |R| <= 3} u(R) m_i;
 *   sets R are visited by size, then by increasing bit mask (bit k = element k);
 *   the sums over k in R and over R run in that order, first term first.
 * Draws: word t (t = 0..3) of the block's own generator call (block number q
 * of the operand counts blocks of eight: call q, four words) gives
 *   thr = n_t (rest(removed so far) 2^-24), n_t the word's top 24 bits; the
 *   running sums of the remaining magnitudes in position order are compared
 *   with thr and the draw is the remaining element number #{sums <= thr},
 *   capped at the last remaining one (the walk of App. "Pruning Overhead" Part 1).
 * Zero rules: an element of magnitude zero owns an empty interval.  A block
 * with at most four non-zeros keeps all of them with their own values (p = 1:
 * magnitude-proportional draws exhaust the non-zeros first), and fills up with
 * the zeros the walk lands on (the last remaining ones), as signed zeros.
 *
 * Contract: the non-zero magnitudes of a block lie within a factor 2^60 of each
 * other and sum to between 2^-100 and 2^100 (reciprocals and their products
 * then stay normal numbers); outside it the pattern is still a valid one, the
 * values are unspecified.
 *
 * idx[0..3]: surviving positions, ascending; val[]: their new values.
 * p_out (may be NULL) receives the eight inclusion probabilities as computed.
 * ---------------------------------------------------------------------- */
static int popcount8(unsigned x) { int c = 0; while (x) { c += (int)(x & 1u); x >>= 1; } return c; }

void oracle_approx_4of8_ordered(const float a[8], const uint32_t words[4], int idx[4], float val[4], float p_out[8],
                                int order_out[4]);

void oracle_approx_4of8(const float a[8], const uint32_t words[4], int idx[4], float val[4], float p_out[8])
{
    oracle_approx_4of8_ordered(a, words, idx, val, p_out, NULL);
}

/* The same; order_out (may be NULL) receives the four positions in the order they were drawn. */
void oracle_approx_4of8_ordered(const float a[8], const uint32_t words[4], int idx[4], float val[4], float p_out[8],
                                int order_out[4])
{
    float m[8];
    int nnz = 0;
    for (int k = 0; k < 8; ++k) { m[k] = fabsf(a[k]); nnz += m[k] != 0.0f; }
    /* rest(Q) and its reciprocal for every set Q of at most three elements */
    float rest[256], inv[256], u[256];
    for (unsigned Q = 0; Q < 256; ++Q) {
        if (popcount8(Q) > 3) continue;
        float r = 0.0f;
        int first = 1;
        for (int k = 0; k < 8; ++k) {
            if (Q & (1u << k)) continue;
            if (first) { r = m[k]; first = 0; } else r = r + m[k];
        }
        rest[Q] = r;
        inv[Q] = r == 0.0f ? 0.0f : 1.0f / r;
    }
    /* four draws */
    unsigned removed = 0;
    for (int t = 0; t < 4; ++t) {
        const float thr = (float)(words[t] >> 8) * (rest[removed] * 5.9604644775390625e-08f);
        float run = 0.0f;
        int first = 1, pick = -1, last = -1;
        for (int k = 0; k < 8; ++k) {
            if (removed & (1u << k)) continue;
            last = k;
            if (pick >= 0) continue;
            if (first) { run = m[k]; first = 0; } else run = run + m[k];
            if (!(run <= thr)) pick = k;                    /* first remaining element whose running sum exceeds thr */
        }
        if (pick < 0) pick = last;
        removed |= 1u << pick;
        if (order_out) order_out[t] = pick;
    }
    /* inclusion probabilities */
    float p[8];
    if (nnz > 4) {
        u[0] = inv[0];
        for (int size = 1; size <= 3; ++size) {
            for (unsigned R = 1; R < 256; ++R) {
                if (popcount8(R) != size) continue;
                float acc = 0.0f;
                int first = 1;
                for (int k = 0; k < 8; ++k) {
                    if (!(R & (1u << k))) continue;
                    const float term = u[R & ~(1u << k)] * m[k];
                    if (first) { acc = term; first = 0; } else acc = acc + term;
                }
                u[R] = acc * inv[R];
            }
        }
        for (int i = 0; i < 8; ++i) {
            float acc = 0.0f;
            int first = 1;
            for (int size = 0; size <= 3; ++size) {
                for (unsigned R = 0; R < 256; ++R) {
                    if (popcount8(R) != size || (R & (1u << i))) continue;
                    const float term = u[R] * m[i];
                    if (first) { acc = term; first = 0; } else acc = acc + term;
                }
            }
            p[i] = acc;
        }
    } else {
        for (int i = 0; i < 8; ++i) p[i] = m[i] != 0.0f ? 1.0f : 0.0f;
    }
    if (p_out) for (int i = 0; i < 8; ++i) p_out[i] = p[i];
    int n = 0;
    for (int k = 0; k < 8; ++k) {
        if (!(removed & (1u << k))) continue;
        idx[n] = k;
        val[n] = (nnz > 4 && m[k] != 0.0f) ? a[k] / p[k] : a[k];
        ++n;
    }
}

/* The four words of block-of-eight number q: generator call q. */
void oracle_block_words4(uint64_t seed, uint64_t q, uint32_t words[4])
{
    uint32_t ctr[4] = { (uint32_t)q, (uint32_t)(q >> 32), 0u, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    oracle_philox4x32_10(ctr, key, words);
}

/* Tensor-wide approx-4:8 prune (no tensor core reads this pattern: prune only).
 * Same operand view and block numbering as oracle_prune with blocks of eight:
 * block j of row r of A is number r (k_total / 8) + k_offset / 8 + j.
 * Output: values[Mrows x K/2] bf16 (nearest even), the four survivors of each
 * block in ascending position; mask[Mrows x K/8] bytes, bit k set iff element k
 * of the block survives (exactly four bits per byte). */
int oracle_prune_4of8(const void *g, int is_bf16, int64_t rows, int64_t cols, int64_t ld, int axis,
                      uint64_t seed, int64_t k_total, int64_t k_offset, uint16_t *values, uint8_t *mask,
                      int threads)
{
    const int64_t Mrows = axis == 1 ? rows : cols;
    const int64_t K     = axis == 1 ? cols : rows;
    if (K % 8 != 0 || k_total % 8 != 0 || k_offset % 8 != 0 || k_offset + K > k_total) return -1;
    (void)threads;
#pragma omp parallel for num_threads(threads) schedule(static)
    for (int64_t r = 0; r < Mrows; ++r) {
        for (int64_t j = 0; j < K / 8; ++j) {
            float a[8];
            for (int e = 0; e < 8; ++e) {
                int64_t k = 8 * j + e;
                int64_t off = axis == 1 ? r * ld + k : k * ld + r;
                a[e] = is_bf16 ? oracle_bf16_to_f32(((const uint16_t *)g)[off]) : ((const float *)g)[off];
            }
            uint64_t q = (uint64_t)r * (uint64_t)(k_total / 8) + (uint64_t)(k_offset / 8 + j);
            uint32_t words[4];
            oracle_block_words4(seed, q, words);
            int idx[4]; float val[4];
            oracle_approx_4of8(a, words, idx, val, NULL);
            uint8_t bits = 0;
            for (int e = 0; e < 4; ++e) {
                values[r * (K / 2) + 4 * j + e] = oracle_bf16_rne(val[e]);
                bits |= (uint8_t)(1u << idx[e]);
            }
            mask[r * (K / 8) + j] = bits;
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------
 * Tensor-wide prune and pack.
 *
 * g is a row-major [rows x cols] matrix with leading dimension ld, fp32
 * (is_bf16 = 0) or bf16 bit patterns (is_bf16 = 1; widened exactly).
 * The sparse operand is A[Mrows x K] with K the reduction axis of the GEMM
 * that will consume it: axis = 1 -> A = g (blocks along a row of g),
 * axis = 0 -> A = g^T (blocks run down a column of g).
 * Blocks are M contiguous elements along K (Sec. 1; Sec. 4).
 *
 * Block numbering: row r of A owns k_total/M consecutive numbers; k_offset is
 * the global K position of this tensor's first element (0 unless the K axis
 * is sharded), so a shard draws the same words as the whole tensor would.
 *
 * Output (canonical packed form):
 *   values[Mrows x K/2]  bf16, the survivors in ascending position;
 *   meta  [Mrows x K/8]  bytes; each nibble = idx0 | idx1 << 2 for one group
 *                        of four, low nibble = even group.
 * A 1:2 result is written as a valid 2:4 pattern: the pair (4j, 4j+1) gives
 * idx0 in {0,1}, the pair (4j+2, 4j+3) gives idx1 in {2,3}.  A 1:4 result
 * (n = 1, m = 4) is written as the survivor beside a +0 partner: positions
 * (i, 3) for i < 3, (2, 3) for i = 3.
 * joint selects the 2:4 estimator: 0 = the pair table of App. A.2,
 * 1 = systematic sampling, 2 = approx-MVUE of Sec. 4.4 (above; two random words
 * per block); 1:2 has a single law and ignores it.
 * Returns 0, or -1 for an unsupported shape.
 * ---------------------------------------------------------------------- */
static float load_elem(const void *g, int is_bf16, int64_t off)
{
    if (is_bf16) return oracle_bf16_to_f32(((const uint16_t *)g)[off]);
    return ((const float *)g)[off];
}

int oracle_prune_opts(const void *g, int is_bf16, int64_t rows, int64_t cols, int64_t ld,
                      int n, int m, int axis, uint64_t seed, int64_t k_total, int64_t k_offset,
                      uint16_t *values, uint8_t *meta, int threads, int joint, int stochastic_rounding, int eps16);

int oracle_prune_rounded(const void *g, int is_bf16, int64_t rows, int64_t cols, int64_t ld,
                         int n, int m, int axis, uint64_t seed, int64_t k_total, int64_t k_offset,
                         uint16_t *values, uint8_t *meta, int threads, int joint, int stochastic_rounding)
{
    return oracle_prune_opts(g, is_bf16, rows, cols, ld, n, m, axis, seed, k_total, k_offset, values, meta, threads,
                             joint, stochastic_rounding, 0);
}

int oracle_prune(const void *g, int is_bf16, int64_t rows, int64_t cols, int64_t ld,
                 int n, int m, int axis, uint64_t seed, int64_t k_total, int64_t k_offset,
                 uint16_t *values, uint8_t *meta, int threads, int joint)
{
    return oracle_prune_rounded(g, is_bf16, rows, cols, ld, n, m, axis, seed, k_total, k_offset, values, meta,
                                threads, joint, 0);
}

/* The same with the rounding of the survivors chosen: stochastic_rounding = 0 rounds to the nearest bf16 (ties to
 * even), 1 rounds stochastically (oracle_bf16_sr) with the bits of oracle_rounding_bits: the survivor stored at
 * values[r][8 t + e] is slot e of unit number r (k_total / 16) + k_offset / 16 + t.  Needs K, k_total, k_offset
 * multiples of 16 then. */
/* eps16 = 1: the blocks draw sixteen random bits each (oracle_block_word16 / oracle_block_word_pair16). */
int oracle_prune_opts(const void *g, int is_bf16, int64_t rows, int64_t cols, int64_t ld,
                      int n, int m, int axis, uint64_t seed, int64_t k_total, int64_t k_offset,
                      uint16_t *values, uint8_t *meta, int threads, int joint, int stochastic_rounding, int eps16)
{
    const int64_t Mrows = axis == 1 ? rows : cols;
    const int64_t K     = axis == 1 ? cols : rows;
    if (!((n == 1 && m == 2) || (n == 2 && m == 4) || (n == 1 && m == 4))) return -1;
    if (K % 8 != 0 || k_total % 8 != 0 || k_offset % 8 != 0 || k_offset + K > k_total) return -1;
    if (joint < 0 || joint > 2) return -1;
    if (stochastic_rounding && (K % 16 != 0 || k_total % 16 != 0 || k_offset % 16 != 0)) return -1;
    (void)threads;
#pragma omp parallel for num_threads(threads) schedule(static)
    for (int64_t r = 0; r < Mrows; ++r) {
        for (int64_t j = 0; j < K / 4; ++j) {           /* j: group of four along K */
            float a[4];
            for (int e = 0; e < 4; ++e) {
                int64_t k = 4 * j + e;
                int64_t off = axis == 1 ? r * ld + k : k * ld + r;
                a[e] = load_elem(g, is_bf16, off);
            }
            int idx[2]; float val[2];
            if (m == 4 && n == 1) {
                /* one survivor, stored in the 2:4 container beside a +0: positions (i, 3), or (2, 3) when i = 3 */
                uint64_t q = (uint64_t)r * (uint64_t)(k_total / 4) + (uint64_t)(k_offset / 4 + j);
                float kept;
                int i = oracle_mvue_1of4(a, eps16 ? oracle_block_word16(seed, q) : oracle_block_word(seed, q), &kept);
                if (i < 3) { idx[0] = i; idx[1] = 3; val[0] = kept; val[1] = 0.0f; }
                else       { idx[0] = 2; idx[1] = 3; val[0] = 0.0f; val[1] = kept; }
            } else if (m == 4) {
                uint64_t q = (uint64_t)r * (uint64_t)(k_total / 4) + (uint64_t)(k_offset / 4 + j);
                const uint32_t word = joint == 2 ? 0u : eps16 ? oracle_block_word16(seed, q) : oracle_block_word(seed, q);
                if (joint == 0)      oracle_mvue_2of4(a, word, idx, val);
                else if (joint == 1) oracle_mvue_2of4_systematic(a, word, idx, val);
                else {
                    uint32_t w[2];
                    if (eps16) oracle_block_word_pair16(seed, q, w);
                    else       oracle_block_word_pair(seed, q, w);
                    oracle_mvue_2of4_approx(a, w[0], w[1], idx, val);
                }
            } else {
                for (int half = 0; half < 2; ++half) {
                    uint64_t q = (uint64_t)r * (uint64_t)(k_total / 2)
                               + (uint64_t)(k_offset / 2 + 2 * j + half);
                    idx[half] = 2 * half + oracle_mvue_1of2(a[2 * half], a[2 * half + 1],
                                                            eps16 ? oracle_block_word16(seed, q)
                                                                  : oracle_block_word(seed, q), &val[half]);
                }
            }
            if (stochastic_rounding) {
                uint64_t u = (uint64_t)r * (uint64_t)(k_total / 16) + (uint64_t)(k_offset / 16 + j / 4);
                int slot = 2 * (int)(j % 4);
                values[r * (K / 2) + 2 * j]     = oracle_bf16_sr(val[0], oracle_rounding_bits(seed, u, slot));
                values[r * (K / 2) + 2 * j + 1] = oracle_bf16_sr(val[1], oracle_rounding_bits(seed, u, slot + 1));
            } else {
                values[r * (K / 2) + 2 * j]     = oracle_bf16_rne(val[0]);
                values[r * (K / 2) + 2 * j + 1] = oracle_bf16_rne(val[1]);
            }
            uint8_t nib = (uint8_t)(idx[0] | (idx[1] << 2));
            uint8_t *byte = &meta[r * (K / 8) + j / 2];
            if (j % 2 == 0) *byte = (uint8_t)((*byte & 0xF0u) | nib);
            else            *byte = (uint8_t)((*byte & 0x0Fu) | (nib << 4));
        }
    }
    return 0;
}

/* Expand the canonical packed form back to a dense fp32 A[Mrows x K]. */
void oracle_unpack(const uint16_t *values, const uint8_t *meta, int64_t Mrows, int64_t K,
                   float *dense)
{
    for (int64_t r = 0; r < Mrows; ++r) {
        for (int64_t j = 0; j < K / 4; ++j) {
            uint8_t byte = meta[r * (K / 8) + j / 2];
            uint8_t nib = (j % 2 == 0) ? (byte & 0x0Fu) : (byte >> 4);
            float *out = &dense[r * K + 4 * j];
            out[0] = out[1] = out[2] = out[3] = 0.0f;
            /* written in this order so that a malformed nibble with equal
             * indices still yields a defined result (second value wins) */
            out[nib & 3u]        = oracle_bf16_to_f32(values[r * (K / 2) + 2 * j]);
            out[(nib >> 2) & 3u] = oracle_bf16_to_f32(values[r * (K / 2) + 2 * j + 1]);
        }
    }
}

/* ------------------------------------------------------------------------
 * Matrix product that consumes the pruned operand (Sec. 1: the update
 * dC/dW_l = g_l h_{l-1}^T and the backward product W^T g).
 *   C[M x N] = A[M x K] . B[K x N]  (+ elementwise * E[M x N] if E != NULL)
 * A is the dense expansion of the packed operand (fp32), B and E hold bf16 bit
 * patterns, row-major with leading dimensions ldb / lde.  Plain triple loop,
 * accumulated in binary64.  Update: A = theta(g)^T, B = h.  Backward:
 * A = theta(g), B = W, E = f'(z).
 * ---------------------------------------------------------------------- */
void oracle_gemm(const float *A, int64_t M, int64_t K, const uint16_t *B, int64_t N, int64_t ldb,
                 const uint16_t *E, int64_t lde, double *C, int threads)
{
    (void)threads;
#pragma omp parallel for num_threads(threads) schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k)
                acc += (double)A[i * K + k] * (double)oracle_bf16_to_f32(B[k * ldb + j]);
            if (E) acc *= (double)oracle_bf16_to_f32(E[i * lde + j]);
            C[i * N + j] = acc;
        }
    }
}

/* One output entry of the same product, for sampled checks at sizes where the
 * full triple loop is too slow. */
double oracle_gemm_entry(const float *A_row, int64_t K, const uint16_t *B, int64_t ldb, int64_t j)
{
    double acc = 0.0;
    for (int64_t k = 0; k < K; ++k)
        acc += (double)A_row[k] * (double)oracle_bf16_to_f32(B[k * ldb + j]);
    return acc;
}

/* ------------------------------------------------------------------------
 * Exhaustive sweep helper for the pins: run the block sampler for every one
 * of the 2^24 values eps can take and count how often each outcome occurs.
 * 2:4: counts[6] over the position pairs (0,1),(0,2),(0,3),(1,2),(1,3),(2,3)
 * of the ORIGINAL block (joint: 0 = App. A.2 table, 1 = systematic sampling, which reads
 * 23 of the 24 bits, so every outcome is counted twice); sum_val[4] accumulates theta(a) per position;
 * sum_sq accumulates |theta(a) - a|^2.  1:2: counts[0..1], sum_val[0..1].
 * ---------------------------------------------------------------------- */
void oracle_sweep_2of4(const float a[4], int joint, uint64_t counts[6], double sum_val[4], double *sum_sq)
{
    static const int pair_id[4][4] = { { -1, 0, 1, 2 }, { 0, -1, 3, 4 }, { 1, 3, -1, 5 }, { 2, 4, 5, -1 } };
    for (int i = 0; i < 6; ++i) counts[i] = 0;
    for (int i = 0; i < 4; ++i) sum_val[i] = 0.0;
    *sum_sq = 0.0;
    for (uint32_t n = 0; n < (1u << 24); ++n) {
        int idx[2]; float val[2];
        if (joint == 0) oracle_mvue_2of4(a, n << 8, idx, val);
        else            oracle_mvue_2of4_systematic(a, n << 8, idx, val);
        counts[pair_id[idx[0]][idx[1]]] += 1;
        double th[4] = { 0, 0, 0, 0 };
        th[idx[0]] = val[0]; th[idx[1]] = val[1];
        for (int i = 0; i < 4; ++i) {
            sum_val[i] += th[i];
            double d = th[i] - (double)a[i];
            *sum_sq += d * d;
        }
    }
}

void oracle_sweep_1of2(float a1, float a2, uint64_t counts[2], double sum_val[2], double *sum_sq)
{
    counts[0] = counts[1] = 0; sum_val[0] = sum_val[1] = 0.0; *sum_sq = 0.0;
    for (uint32_t n = 0; n < (1u << 24); ++n) {
        float kept;
        int idx = oracle_mvue_1of2(a1, a2, n << 8, &kept);
        counts[idx] += 1;
        double th[2] = { 0, 0 };
        th[idx] = kept;
        sum_val[0] += th[0]; sum_val[1] += th[1];
        *sum_sq += (th[0] - (double)a1) * (th[0] - (double)a1) + (th[1] - (double)a2) * (th[1] - (double)a2);
    }
}

/* Sweeps for the approx-MVUE sampler (Sec. 4.4), one draw at a time:
 * first[i]      = how many of the 2^24 values of the first uniform draw element i first;
 * second[i][j]  = with a first uniform that draws i (if none exists the row stays zero), how
 *                 many of the 2^24 values of the second uniform draw j second;
 * val[k]        = the value element k takes when it survives (it does not depend on the
 *                 partner); NaN if k was never seen to survive. */
void oracle_sweep_approx24(const float a[4], uint64_t first[4], uint64_t second[4][4], float val[4])
{
    uint32_t rep[4]; int have[4] = { 0, 0, 0, 0 };
    for (int i = 0; i < 4; ++i) { first[i] = 0; val[i] = NAN; for (int j = 0; j < 4; ++j) second[i][j] = 0; }
    for (uint32_t n = 0; n < (1u << 24); ++n) {
        int i, j; float vi, vj;
        oracle_mvue_2of4_approx_ordered(a, n << 8, 0u, &i, &j, &vi, &vj);
        first[i] += 1;
        if (!have[i]) { have[i] = 1; rep[i] = n << 8; }
    }
    for (int i = 0; i < 4; ++i) {
        if (!have[i]) continue;
        for (uint32_t n = 0; n < (1u << 24); ++n) {
            int i2, j; float vi, vj;
            oracle_mvue_2of4_approx_ordered(a, rep[i], n << 8, &i2, &j, &vi, &vj);
            second[i][j] += 1;
            val[i2] = vi; val[j] = vj;
        }
    }
}

void oracle_sweep_1of4(const float a[4], uint64_t counts[4], double sum_val[4], double *sum_sq)
{
    for (int i = 0; i < 4; ++i) { counts[i] = 0; sum_val[i] = 0.0; }
    *sum_sq = 0.0;
    for (uint32_t n = 0; n < (1u << 24); ++n) {
        float kept;
        int i = oracle_mvue_1of4(a, n << 8, &kept);
        counts[i] += 1;
        sum_val[i] += kept;
        for (int k = 0; k < 4; ++k) {
            double d = (k == i ? (double)kept : 0.0) - (double)a[k];
            *sum_sq += d * d;
        }
    }
}
