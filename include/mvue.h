/*
 * mvue.h -- C ABI of the B200 (sm_100a) library for minimum-variance unbiased
 * (MVUE) N:M pruning of neural gradients and the 2:4-sparse matrix products that
 * consume the pruned gradient.
 *
 * Method: Chmiel, Hubara, Banner, Soudry, "Minimum Variance Unbiased N:M
 * Sparsity for the Neural Gradients" (arXiv 2203.10991).  Citations below name
 * the paper's sections, equations and appendices.
 *
 * General rules for every call
 *  - All tensor pointers are DEVICE pointers unless an argument says "host".
 *    The caller owns every buffer; the library never allocates or frees device
 *    memory and keeps no device state -- with one exception, the fixed scratch
 *    array of mvue_sparse_update_gemm_noalloc (described at its declaration).
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *    stream).  Calls enqueue work on that stream and return without waiting.
 *  - The return value is an mvue_status.  Argument errors are detected on the
 *    host before anything is launched; nothing is written in that case.
 *    Nothing throws, aborts or traps across this boundary.
 *  - Matrices are row-major; leading dimensions are in ELEMENTS.
 *  - The device must be compute capability 10.x; otherwise MVUE_ERR_ARCH.
 *  - Inputs must be finite with |x| <= 2^125; other values give unspecified
 *    results but never an out-of-bounds access.
 */
#ifndef MVUE_H_
#define MVUE_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define MVUE_API __attribute__((visibility("default")))
#else
#define MVUE_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MVUE_OK = 0,
    MVUE_ERR_NULL = -1,           /* a required pointer is NULL */
    MVUE_ERR_NM = -2,             /* only (N,M) = (1,2), (2,4) and (1,4) exist (the fused product: the first two) */
    MVUE_ERR_SHAPE = -3,          /* non-positive / non-multiple extents, ld < cols, bad axis or K shard */
    MVUE_ERR_ALIGN = -4,          /* base pointer or leading dimension not 16-byte aligned */
    MVUE_ERR_DTYPE = -5,
    MVUE_ERR_LAYOUT = -6,
    MVUE_ERR_WORKSPACE = -7,      /* workspace NULL or smaller than mvue_gemm_workspace_bytes */
    MVUE_ERR_ARCH = -8,           /* current device is not sm_100 */
    MVUE_ERR_CUDA = -9,           /* a CUDA runtime/driver call failed; text in mvue_last_cuda_error() */
    MVUE_ERR_DEVICE_TIMEOUT = -10,/* only ever written to a device status word: a bounded wait expired */
    MVUE_ERR_JOINT = -11,         /* unknown mvue_joint */
    MVUE_ERR_OPTION = -12         /* unknown bit in the options of mvue_prune_opts */
} mvue_status;

typedef enum { MVUE_F32 = 0, MVUE_BF16 = 1 } mvue_dtype;

/* The joint law over pairs from which a 2:4 block's two survivors are drawn.  Sec. 4.2 fixes
 * only the marginals p_i (the block variance is a function of them alone); both laws below have
 * exactly those marginals and the kept values a_i / p_i, hence E[theta(a)] = a and the same,
 * minimal, variance.  They draw different pairs for the same seed.
 * MVUE_JOINT_TABLE:      the pair table of App. A.2 (sorts the block by magnitude).
 * MVUE_JOINT_SYSTEMATIC: systematic sampling in the block's own order, no sort: element k owns an
 *   interval of length e_k = min(|a_k|, sum of the other three) of [0, D), D = sum e_k; the owners
 *   of t and t + D/2 survive, t = eps D/2 (eps: the top 23 bits of the block's random word);
 *   a survivor becomes sign(a_k) max(|a_k|, D/2).  About a fifth fewer instructions per block.
 * MVUE_JOINT_APPROX:     not a law with the optimal marginals but the approximate estimator of
 *   Sec. 4.4 ("approx-MVUE", the one the paper's 2:4 accuracy tables were run with): element i is
 *   drawn with probability |a_i| / sum, then j among the other three with probability
 *   |a_j| / (sum - |a_i|), in the block's own order; a survivor becomes a_k / p_k with p_k the
 *   inclusion probability given by that section's equation, so E[theta(a)] = a still holds, with a
 *   block variance the paper's scan bounds below twice the optimum.  It takes TWO random words per
 *   block: block q reads words 2 (q & 1) and 2 (q & 1) + 1 of generator call q >> 1 (same key).
 *   Arithmetic, binary32 in this order: m_k = |a_k|; c_1 = m_0, c_2 = c_1 + m_1, c_3 = c_2 + m_2,
 *   s = c_3 + m_3; t_1 = n_1 (s 2^-24), i = #{c_k <= t_1}; R_k = the sum of the other three
 *   magnitudes in position order, (x + y) + z; the second draw walks the others' running sums d_1,
 *   d_2 with t_2 = n_2 (R_i 2^-24); vv_k = m_k / R_k; T_k = the sum of the other three vv in position
 *   order; survivor k becomes sign(a_k) s / (1 + T_k) (IEEE divisions).  If R_i = 0 (at most one
 *   non-zero) both survivors keep their own values.  Blocks whose non-zero magnitudes span more than
 *   2^100, or sum to less than 2^-100, are outside the contract (valid pattern, unspecified values).
 *   On this hardware the six divisions make it the slowest of the three, not the cheapest.
 * 1:2 has a single law (Sec. 4.1) and ignores the choice. */
typedef enum { MVUE_JOINT_TABLE = 0, MVUE_JOINT_SYSTEMATIC = 1, MVUE_JOINT_APPROX = 2 } mvue_joint;

/* Packed operand layouts.
 * MVUE_LAYOUT_CANONICAL: for the sparse operand A[Mrows x K] (K = pruned axis)
 *   values: bf16 [Mrows x K/2] row-major -- the two survivors of each group of
 *           four consecutive k, in ascending k;
 *   meta:   bytes [Mrows x K/8] row-major -- one nibble per group,
 *           idx0 | idx1 << 2 with idx0 < idx1 the survivors' positions in the
 *           group, low nibble = even group.  (The 2-bit-per-survivor encoding
 *           of 2:4 sparse tensor cores.)
 * MVUE_LAYOUT_TC: same values; the metadata in the order the sparse tensor cores
 *   read it, so that the GEMMs move it with one bulk copy per K block and no
 *   rearrangement: blocks of 128 rows x 128 k (2048 bytes; row-block major, rows
 *   padded to a multiple of 128), inside a block 128 "lanes" of 16 bytes,
 *   lane = r%8 + 8*((k/16)%2) + 16*((r%128)/16); the 32-bit word (k%128)/32 of a
 *   lane holds the 16-bit nibble string of k%32 in [0,16) or [16,32) for row r
 *   (low half, (r/8)%2 = 0) and row r+8 (high half).  Needs K a multiple of 128.
 *   This is what the GEMM entry points consume; canonical is the interchange
 *   and checking form (mvue_unpack reads both). */
typedef enum { MVUE_LAYOUT_CANONICAL = 0, MVUE_LAYOUT_TC = 1 } mvue_layout;

/* Bytes of the packed outputs of mvue_prune for a [rows x cols] input.
 * values_bytes / meta_bytes are HOST pointers (either may be NULL). */
MVUE_API int mvue_packed_sizes(int64_t rows, int64_t cols, int n, int m, int axis, int layout,
                      size_t* values_bytes, size_t* meta_bytes);

/* MVUE N:M prune + pack of a neural gradient g in one pass.
 *
 * What it computes.  Each block of M elements that are contiguous along the
 * reduction axis K of the GEMM that will consume g is replaced by an unbiased,
 * minimum-variance N:M-sparse block theta(a), E[theta(a)] = a:
 *   (1,2): Sec. 4.1, closing equation (derivation App. A.1): a_1 survives with
 *          probability |a_1|/(|a_1|+|a_2|), else a_2; the survivor becomes
 *          sign(a_i)(|a_1|+|a_2|).
 *   (2,4): Sec. 4.2 (optimal survival probabilities p_i, survivors a_i/p_i) with
 *          the joint law over pairs of App. A.2 (three cases on the sorted
 *          magnitudes), drawn by walking the cumulative pair table in the order
 *          13, 14, 23, 24, 34.
 *   (1,4): the paper's "MVUE 1:4" (appendix "Additional sparsity results": like MVUE 1:2 for a
 *          block of four; Sec. 4.1's argument with one survivor of M): element i survives with
 *          probability |a_i| / S, S the sum of the block's magnitudes, and becomes sign(a_i) S;
 *          running sums in the block's own order, i = #{c_k <= eps S}.  One random word per
 *          block, numbered as for (2,4).  The survivor is stored in the 2:4 container beside a
 *          +0 partner -- positions (i, 3), or (2, 3) when i = 3 -- so the products below consume
 *          it unchanged (at the 2:4 rate: no tensor core runs 1:4).
 * The draw is the threshold test eps < p of App. "Pruning Overhead" (Part 1)
 * with eps = (w >> 8) * 2^-24, w the 32-bit word of block number q:
 *   w = Philox4x32-10(counter = (lo32(q>>2), hi32(q>>2), 0, 0),
 *                     key = (lo32(seed), hi32(seed)))[q & 3],
 *   q = r * (k_total / M) + (k_offset / M + j) for block j of row r of A.
 * All selection arithmetic is IEEE binary32 in a fixed order without fused
 * multiply-add; survivors are rounded once to bf16 (nearest even).  Zeros: an
 * element of magnitude zero owns a zero-width interval of every threshold walk,
 * so it survives only when fewer than N non-zeros exist, as a signed zero (its
 * own sign bit).  Which zero then fills the pattern: (2,4) with the pair table
 * keeps the top ranks of the (magnitude, position) order -- a lone non-zero
 * beside position 3, or beside position 2 if it is itself at 3; an all-zero block
 * keeps positions 2 and 3; (1,2) keeps a_1 whenever a_2 = 0; (1,4) keeps the last
 * element of an all-zero block.  A (1,2) result is emitted as a valid 2:4 pattern
 * (pair 0 -> position 0/1, pair 1 -> position 2/3).
 * The same (g, n, m, axis, seed, k_total, k_offset) always gives the same bits.
 *
 * Arguments.
 *   g        [rows x cols], leading dimension ld, dtype MVUE_F32 or MVUE_BF16.
 *   axis     1: A = g      (Mrows = rows, K = cols; blocks along a row of g;
 *                            the backward product's operand),
 *            0: A = g^T    (Mrows = cols, K = rows; blocks down a column of g;
 *                            the update product's operand).
 *   k_total  K of the whole (unsharded) operand, k_offset the global k of this
 *            tensor's first element; pass K and 0 unless K is sharded.
 *   values, meta   outputs in `layout`, sizes from mvue_packed_sizes.
 * Preconditions (else MVUE_ERR_SHAPE / MVUE_ERR_ALIGN): K, k_total and k_offset
 * multiples of 16; Mrows a multiple of 8; ld >= cols; g, values, meta and
 * ld * sizeof(element) 16-byte aligned; K <= 65535 * 256 for axis 1, Mrows <=
 * 65535 * 64 for axis 0. */
MVUE_API int mvue_prune(const void* g, int dtype, int64_t rows, int64_t cols, int64_t ld, int n, int m,
               int axis, uint64_t seed, int64_t k_total, int64_t k_offset, void* values,
               void* meta, int layout, void* stream);

/* mvue_prune with the 2:4 estimator chosen by the caller (an mvue_joint; mvue_prune itself uses
 * MVUE_JOINT_TABLE).  Everything else -- block numbering, random words, packed layouts, arguments,
 * preconditions, errors -- is as for mvue_prune; an unknown joint gives MVUE_ERR_JOINT. */
MVUE_API int mvue_prune_joint(const void* g, int dtype, int64_t rows, int64_t cols, int64_t ld, int n, int m,
                     int axis, uint64_t seed, int64_t k_total, int64_t k_offset, void* values,
                     void* meta, int layout, int joint, void* stream);

/* mvue_prune_joint with options (a bitwise OR of mvue_prune_option; an unknown bit gives MVUE_ERR_OPTION).
 *
 * MVUE_OPT_STOCHASTIC_ROUNDING: the survivors are rounded to bf16 stochastically instead of to the nearest bf16
 *   (Sec. 3: the neural gradients want an unbiased quantiser such as stochastic rounding; App. "Pruning Overhead",
 *   Part 1, names stochastic rounding as the sampling primitive).  Round-to-nearest stores a_i / p_i only up to the
 *   bf16 grid, E[stored] = a_i (1 + delta) with |delta| <= 2^-9; with this option the stored value itself is unbiased:
 *   a binary32 survivor x between the neighbouring bf16 numbers lo <= |x| < hi is stored as hi with probability
 *   (|x| - lo) / (hi - lo), else lo -- on the bit pattern, stored = (bits(x) + r) >> 16 with r a uniform 16-bit
 *   integer.  Masks and metadata are those of the same call without the option; survivors already on the bf16 grid
 *   (every survivor that keeps its own bf16 value) never move.  The bits r: unit u = r_A (k_total / 16) + k_offset / 16
 *   + t (16 consecutive k of row r_A of A) makes one more generator call, Philox4x32-10 with counter
 *   (lo32(u), hi32(u), 1, 0) under the same key (the selection draws all have third counter word 0); the survivor stored
 *   at values[r_A][8 t + e] takes the low (e even) or high (e odd) half of word e / 2.  About 15 more instructions per
 *   block of four.
 * MVUE_OPT_EPS16: sixteen random bits per block instead of thirty-two, so that one generator call serves eight
 *   blocks (App. "Pruning Overhead", Part 1, asks only for i.i.d. eps ~ U[0,1]; the generator is a fifth of the
 *   instructions of the prune).  Block q takes the low (q even) or high (q odd) half of word (q >> 1) & 3 of call
 *   q >> 3; approx-MVUE, which draws twice per block, takes word q & 3 of call q >> 2, low half first.  The sixteen
 *   bits are used as the top half of a word whose low half is zero, so every formula above stands with eps on a grid
 *   of 2^-16 (2^-15 for systematic sampling): each mask probability moves by at most that, two hundred times below
 *   the bf16 grid of the survivors.  Masks differ from those of the same call without the option. */
typedef enum { MVUE_OPT_NONE = 0, MVUE_OPT_STOCHASTIC_ROUNDING = 1, MVUE_OPT_EPS16 = 2 } mvue_prune_option;
MVUE_API int mvue_prune_opts(const void* g, int dtype, int64_t rows, int64_t cols, int64_t ld, int n, int m,
                    int axis, uint64_t seed, int64_t k_total, int64_t k_offset, void* values,
                    void* meta, int layout, int joint, unsigned options, void* stream);

/* Approx-4:8 prune (appendix "Additional sparsity results": the approximate 2:4 method of Sec. 4.4 carried to four
 * survivors of eight; the paper prints no formulas).  Prune only: no tensor core reads a 4:8 pattern, so there is no
 * product that consumes this output.
 * What it computes, per block of eight elements contiguous along K (operand view, axis, k_total, k_offset as for
 * mvue_prune; block j of row r of A is number q = r (k_total / 8) + k_offset / 8 + j): four sequential draws, each
 * removing one of the remaining elements with probability proportional to its magnitude (threshold walk in position
 * order with eps = the top 24 bits of word t of Philox4x32-10(counter (lo32(q), hi32(q), 0, 0), key = seed), t = 0..3);
 * a survivor becomes a_i / p_i with p_i the exact probability that i is among the four drawn, so E[theta(a)] = a:
 *   rest(Q) = the magnitudes outside the set Q added left to right, inv(Q) = 1 / rest(Q) (0 if rest(Q) = 0),
 *   u({}) = inv({}), w(R) = sum_{k in R} u(R \ k) |a_k|, u(R) = w(R) inv(R),
 *   p_i = sum over R not containing i, |R| <= 3, of u(R) |a_i|
 * (binary32, sets by size then by increasing bit mask, sums first term first; for two draws of four this is the
 * inclusion probability printed in Sec. 4.4).  A block with at most four non-zeros keeps them all with their own
 * values.  Values are specified for blocks whose non-zero magnitudes lie within 2^60 of each other and sum to between
 * 2^-100 and 2^100; the pattern is valid for every input.
 * Output: values bf16 [Mrows x K/2] (nearest even), the four survivors of each block in ascending position;
 *         mask  bytes [Mrows x K/8], bit k of a byte set iff element k of that block survives.
 * Preconditions: K, k_total, k_offset multiples of 8; g and ld * sizeof(element) 16-byte aligned, values 8-byte. */
MVUE_API int mvue_prune_4of8(const void* g, int dtype, int64_t rows, int64_t cols, int64_t ld, int axis, uint64_t seed,
                    int64_t k_total, int64_t k_offset, void* values, void* mask, void* stream);

/* Expand a packed operand back to dense bf16 A[Mrows x K] (row-major, ld = K).
 * A checking aid: the inverse of the pack step, no arithmetic. */
MVUE_API int mvue_unpack(const void* values, const void* meta, int layout, int64_t mrows, int64_t K,
                void* dense_bf16, void* stream);

/* Update product with the pruned gradient as the 2:4-sparse operand
 * (Sec. 1, update equation dC/dW_l = g_l h_{l-1}^T):
 *   dW[out x in] (+)= theta(g)^T[out x T] . h[T x in]
 * values/meta: packed theta(g)^T (mvue_prune with axis 0 on g[T x out]);
 * h: bf16 [T x in], ld ldh; dW: MVUE_F32 or MVUE_BF16 [out x in], ld lddW;
 * accumulate != 0 adds into dW (MVUE_F32 only).  bf16 x bf16 products, fp32
 * accumulation on the sparse tensor cores.
 * workspace: mvue_gemm_workspace_bytes(0, out, in, T) bytes (may be 0, then
 * NULL is accepted), 16-byte aligned, contents scratch: small outputs with a long
 * reduction are split along K and summed in a second, deterministic pass (without
 * that workspace: MVUE_ERR_WORKSPACE); large fp32 outputs whose last round of tiles
 * would leave most of the GPU idle have those tiles split along K in the same way
 * (with a smaller or NULL workspace they are simply computed whole).  dev_status: optional device int, receives
 * MVUE_ERR_DEVICE_TIMEOUT if a bounded pipeline wait expires (then dW is
 * unspecified); otherwise left untouched.
 * Preconditions: T a multiple of 128; out, in multiples of 8; pointers and
 * leading dimensions (in bytes) 16-byte aligned; act_grad needs a bf16 or
 * MVUE_F32 output without accumulate. */
MVUE_API int mvue_sparse_update_gemm(const void* values, const void* meta, int layout, int64_t out,
                            int64_t T, const void* h, int64_t in, int64_t ldh, void* dW,
                            int dW_dtype, int64_t lddW, int accumulate, void* workspace,
                            size_t workspace_bytes, int* dev_status, void* stream);

/* Backward product with the pruned gradient as the 2:4-sparse operand
 * (Sec. 1, backward equation g_l = Diag(f'(z_l)) W_{l+1}^T g_{l+1}, written for
 * a batch of T rows):
 *   dh[T x in] = (theta(g)[T x out] . W[out x in]) (* act_grad[T x in])
 * values/meta: packed theta(g) (mvue_prune with axis 1 on g[T x out]);
 * W: bf16 [out x in]; act_grad: optional bf16 [T x in] (f'(z)), ld = lddh,
 * multiplied elementwise in the epilogue, or NULL; dh: MVUE_F32 or MVUE_BF16.
 * Workspace, dev_status and preconditions as above with K = out. */
MVUE_API int mvue_sparse_backward_gemm(const void* values, const void* meta, int layout, int64_t T,
                              int64_t out, const void* W, int64_t in, int64_t ldW,
                              const void* act_grad, void* dh, int dh_dtype, int64_t lddh,
                              void* workspace, size_t workspace_bytes, int* dev_status,
                              void* stream);

/* The backward product that hands its result on already pruned (Sec. 1, backward equation: the g_l it produces is
 * the gradient the next layer down prunes again for its own backward product):
 *   dh[T x in] = (theta(g)[T x out] . W[out x in]) * act_grad[T x in]            (bf16, as mvue_sparse_backward_gemm)
 *   (next_values, next_meta) = mvue_prune_opts(dh, 2:4, axis 1, next_seed, k_total = in, k_offset = 0,
 *                                              MVUE_LAYOUT_TC, next_joint, next_options)
 * in ONE launch: in the epilogue a thread holds one row of the output tile, 128 consecutive columns as bf16 -- eight
 * prune units in the form they have when K is contiguous -- and prunes them in registers before the dense tile is
 * stored, so dh is not read back for this prune.  The packed output is bit-identical to the separate call on the
 * stored dh.  dh itself is still written (the update product's prune, down the token axis, needs it).
 * next_joint: MVUE_JOINT_TABLE or MVUE_JOINT_SYSTEMATIC; next_options: mvue_prune_option bits (another bit:
 * MVUE_ERR_OPTION).  act_grad is required; in must be a multiple of 128.
 * When the product has to be split along K (small outputs, see mvue_gemm_workspace_bytes), T is not a multiple of
 * 128, or MVUE_OPT_STOCHASTIC_ROUNDING is asked for, the entry point runs the two steps one after the other instead
 * -- same results.  The epilogue costs ~2000
 * instructions per thread and tile: it hides under main loops of K = out >= 4096 and slows products with a short K,
 * where the separate calls are the better choice.  Other arguments, workspace, dev_status and errors as
 * mvue_sparse_backward_gemm. */
MVUE_API int mvue_sparse_backward_gemm_pruned(const void* values, const void* meta, int layout, int64_t T,
                                              int64_t out, const void* W, int64_t in, int64_t ldW,
                                              const void* act_grad, void* dh, int64_t lddh, uint64_t next_seed,
                                              int next_joint, unsigned next_options, void* next_values,
                                              void* next_meta, void* workspace, size_t workspace_bytes,
                                              int* dev_status, void* stream);

/* Prune fused into the update product (Sec. 4.1 / 4.2 + App. A.2 applied to g along the
 * token axis, then the update equation of Sec. 1) in ONE kernel:
 *   dW[out x in] (+)= theta(g)^T h,   g bf16 [T x out] (ld ldg), h bf16 [T x in]
 * The packed operand is never written to memory.  The random words are those of mvue_prune(g, n, m, axis 0, seed)
 * (mvue_prune_joint with `joint` for the _joint form: MVUE_JOINT_TABLE or MVUE_JOINT_SYSTEMATIC), so the result equals
 * that prune followed by mvue_sparse_update_gemm with the same seed (up to fp32 summation order across K splits).
 * One thread block per 128 x 256 output tile; up to four blocks whose tiles are neighbours along `in` form a cluster
 * and share every pruned stage through each other's shared memory, so a row tile of g is read and pruned once per 1024
 * output columns (when in / 256 is a multiple of 4; once per 512 / 256 columns when it is only even / odd).  The prune
 * then hides under the tensor-core time of wide layers; on narrow layers (in <= 256) the prune is the whole cost and the
 * kernel ties with the separate calls.  Its use is when memory for the packed operand is not available.
 * dtype must be MVUE_BF16 (else MVUE_ERR_DTYPE); (n, m) = (1,2) or (2,4).  workspace: mvue_gemm_workspace_bytes(2, out,
 * in, T) bytes.  Other arguments, preconditions and errors as mvue_sparse_update_gemm. */
MVUE_API int mvue_fused_update_gemm(const void* g, int dtype, int64_t T, int64_t out, int64_t ldg, int n,
                                    int m, uint64_t seed, const void* h, int64_t in, int64_t ldh,
                                    void* dW, int dW_dtype, int64_t lddW, int accumulate,
                                    void* workspace, size_t workspace_bytes, int* dev_status,
                                    void* stream);
MVUE_API int mvue_fused_update_gemm_joint(const void* g, int dtype, int64_t T, int64_t out, int64_t ldg, int n,
                                          int m, int joint, uint64_t seed, const void* h, int64_t in, int64_t ldh,
                                          void* dW, int dW_dtype, int64_t lddW, int accumulate,
                                          void* workspace, size_t workspace_bytes, int* dev_status,
                                          void* stream);

/* Scratch bytes the product C[M x N] = A[M x K] . B[K x N] needs
 * (which: 0 update, 1 backward, 2 fused update).  bytes is a HOST pointer. */
MVUE_API int mvue_gemm_workspace_bytes(int which, int64_t M, int64_t N, int64_t K, size_t* bytes);

/* The update product for callers that cannot allocate device memory.
 * (The paper has no counterpart; this is a convenience of this library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plugin inside a host
 * application that owns the allocator and hands out only input and output buffers, a
 * real-time or certified loop in which allocation calls are forbidden after start-up, a
 * callback running where the CUDA allocator may not be entered.  Such a caller cannot
 * supply the split-K workspace that mvue_sparse_update_gemm asks for on small outputs
 * with a long reduction.
 *
 * Same arguments as mvue_sparse_update_gemm, minus the workspace, and the same product (equal
 * up to the order of the fp32 sums over K, see below): the scratch is a fixed 8 MiB
 * (MVUE_NOALLOC_SCRATCH_BYTES) array inside the library's device image.  Every GPU on which
 * the library is loaded holds those bytes until the process exits.  The call itself allocates
 * nothing, on the host side or the device side.
 *  - Arguments are checked first, as for mvue_sparse_update_gemm, before anything else happens.
 *  - Only the split of a long reduction over a small output NEEDS scratch.  A problem whose
 *    split needs more than the array (the K-split part of mvue_gemm_workspace_bytes(0, out, in,
 *    T), which is all of it whenever the split applies) is refused with MVUE_ERR_WORKSPACE;
 *    nothing is launched.
 *  - Large fp32 outputs use scratch only optionally, to cut the tiles of a mostly idle last
 *    round along K: that happens here when those partial tiles fit the array, and otherwise the
 *    tiles are computed whole, exactly as mvue_sparse_update_gemm does when it is given no
 *    workspace.  So the array may be in use (and the race described below applies) for every
 *    shape, and the result can differ from mvue_sparse_update_gemm with a full workspace in
 *    the last bits of those tiles (a different summation order over K).
 *  - The first call on each device looks up the array's device address (that device must
 *    be current, as for every call).  Make that first call outside any stream capture.
 *  - All calls on a device share the one array, and it keeps whatever the last call left.
 *    The kernel overwrites every scratch element it later reads, so nothing has to be
 *    cleared in between; but two calls that overlap on the GPU (different streams) race
 *    on it.  Keep calls to this entry point on one stream, or order them with events. */
#define MVUE_NOALLOC_SCRATCH_BYTES (8u << 20)
MVUE_API int mvue_sparse_update_gemm_noalloc(const void* values, const void* meta, int layout,
                                             int64_t out, int64_t T, const void* h, int64_t in,
                                             int64_t ldh, void* dW, int dW_dtype, int64_t lddW,
                                             int accumulate, int* dev_status, void* stream);

/* Measurement aid (the paper has no counterpart): the rate at which this GPU retires the sparse tensor-core
 * instruction of the products above when nothing has to be loaded.  One launch: every resident pair of thread blocks
 * issues iters x 4 tcgen05.mma.sp (M = 256, N = 256, K = 32, bf16, fp32 accumulate) back to back on one
 * shared-memory stage of zeros.  Time the launch with events on `stream`; *flops (HOST pointer, may be NULL) receives
 * the dense-equivalent floating-point operations of the launch (2 M N K per instruction, as the products are
 * counted), *pairs (HOST, may be NULL) the number of pairs.  1 <= iters <= 2^20, else MVUE_ERR_SHAPE.  dev_status as
 * for the products (the one wait of the kernel is bounded).  Reads and writes no caller memory. */
MVUE_API int mvue_probe_sparse_mma(int iters, int* pairs, double* flops, int* dev_status, void* stream);

/* Self-test of the bounded-wait exit that every pipeline wait of the products shares (the paper has no counterpart).
 * One launch of the probe's blocks with nothing issued: no copy, no tensor-core instruction and no caller memory is in
 * flight, and nobody ever arrives on the barrier each block waits for, so that wait gives up after `polls` polls
 * (1 <= polls <= 65536, else MVUE_ERR_SHAPE; a few thousand polls take well under a millisecond).  Every block then
 * leaves the ordinary way: MVUE_ERR_DEVICE_TIMEOUT is written to *dev_status (device int, required), the pair of
 * blocks meets at its cluster barrier and tensor memory is handed back.  Nothing traps or faults; the context stays
 * usable and the next product call must be correct.  Returns MVUE_OK when the launch was enqueued. */
MVUE_API int mvue_selftest_wait_timeout(int polls, int* dev_status, void* stream);

MVUE_API const char* mvue_status_string(int status);
/* Text of the last CUDA error seen by the calling thread ("" if none). */
MVUE_API const char* mvue_last_cuda_error(void);
MVUE_API int mvue_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MVUE_H_ */
