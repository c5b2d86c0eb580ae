// 2:4-sparse GEMM on the 5th-generation tensor cores (tcgen05.mma.sp), sm_100a.
//
//   C[M x N] = A[M x K] . B[K x N]
// A is the MVUE-pruned gradient in packed form: bf16 survivors [M x K/2] (K-major) plus
// the position nibbles in tensor-core order (MVUE_LAYOUT_TC).  B is dense bf16, row-major
// [K x N] (N contiguous): the activations h for the update product g^T h, the weights W
// for the backward product g W (Sec. 1 of the paper).
//
// A cluster of two thread blocks computes one 256 x 256 output tile over a range of K with
// tcgen05.mma.sp.cta_group::2: block r of the pair loads its own 128 rows of A (and their
// metadata) and its own 128 columns of B, the leader (r = 0) issues the MMAs for both, and
// each block keeps the fp32 accumulator of its 128 rows in its own tensor memory.  Per block
// and 128-deep K step that is 50 KiB of TMA traffic for 16.8 MFLOP, three times less L2
// traffic per flop than a single-SM 128 x 256 tile.
//   warp 0      TMA producer: A tile (128 x 64 bf16, 128-byte swizzle), two 64 x 128 boxes
//               of B (128-byte swizzle), one 2 KiB metadata block; all complete on the
//               leader's "full" barrier of the stage
//   warp 1      (leader) per stage: tcgen05.cp of the metadata into tensor memory, four
//               tcgen05.mma.sp of K = 32, commit to both blocks' "empty" barrier
//   warp 2      allocates / frees tensor memory
//   warps 4-7   epilogue: tcgen05.ld -> registers -> global, one quarter of the lanes each
// Every wait on an mbarrier is bounded; when a bound expires the block records
// MVUE_ERR_DEVICE_TIMEOUT in the caller's status word and drains.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>

#include "../../include/mvue.h"
#include "mvue_device.cuh"
#include "mvue_internal.h"
#include "mvue_tma.h"

namespace mvue {
namespace {

constexpr int BM = 128;                    // rows of A per thread block (256 per pair)
constexpr int BN = 256;
constexpr int BK = 128;                    // logical K per pipeline stage (four MMAs of K = 32)
constexpr int kStages = 4;
constexpr int kABytes = BM * (BK / 2) * 2; // 16 KiB: 128 rows x 128 bytes of survivors
constexpr int kBBoxBytes = 64 * BK * 2;    // 16 KiB: 128 k-rows x 128 bytes (64 columns)
constexpr int kBBytes = (BN / 2 / 64) * kBBoxBytes;   // this block's 128 columns
constexpr int kEBytes = BM * 16;           // 2 KiB: 16 bytes per tensor-memory lane
constexpr int kStageBytes = kABytes + kBBytes + kEBytes;
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int kThreads = 352;            // pair kernel: producer, MMA, allocator and 8 epilogue warps
constexpr int kEpiWarps = 8;
constexpr int kBandTiles = 8;              // row tiles per band of the tile order
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemECol = 256;        // metadata columns start after the accumulator
constexpr uint32_t kSpinLimit = 1u << 22;  // bounded waits: ~4M polls with back-off

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// The same test with acquire semantics at cluster scope: for a barrier that the peer block arrives on.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t spin = 0; spin < (1u << 22); ++spin) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if (*abort_flag) return false;
        if (spin > 64) __nanosleep(spin > 4096 ? 256 : 32);
    }
    *abort_flag = 1;
    return false;
}
// Bounded wait.  Returns false (and raises the block's abort flag) when the bound expires
// or another role has already given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          uint32_t limit = kSpinLimit) {
    for (uint32_t spin = 0; spin < limit; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (spin > 64) __nanosleep(spin > 4096 ? 256 : 32);
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (64 bits): start address, leading / stride byte offsets
// (all >> 4), descriptor version 1, swizzle mode in the top three bits.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes,
                                                   uint32_t swizzle_code) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | ((uint64_t)swizzle_code << 61);
}
constexpr uint32_t kSwizzleNone = 0, kSwizzle128B = 2;

// Instruction descriptor of tcgen05.mma.sp.cta_group::2.kind::f16: sparse, fp32 accumulate,
// bf16 x bf16, A K-major, B N-major, N = 256, M = 256 (128 rows in each block of the pair).
constexpr uint32_t kInstrDesc2 = (1u << 2) /*sparse*/ | (1u << 4) /*D = f32*/ | (1u << 7) /*A = bf16*/ |
                                 (1u << 10) /*B = bf16*/ | (0u << 15) /*A K-major*/ | (1u << 16) /*B N-major*/ |
                                 ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);

struct GemmParams {
    int64_t M, N, K;
    int64_t k_steps_per_split;
    float* partial;           // split-K workspace [splits x M x N] (splits > 1) else unused
    void* C;                  // output when splits == 1
    int64_t ldc;
    const __nv_bfloat16* scale;  // optional elementwise multiplier [M x N], ld = ldc (splits == 1 path)
    int c_is_bf16;
    int accumulate;
    int splits;
    int64_t n_work;           // work items of the pair kernel: tiles x splits, or n_main + tail_rem x tail_splits
    int64_t n_main;           // work items below this number are whole tiles (or tiles of a K split)
    int tail_rem, tail_splits;   // the last tail_rem tiles are cut into tail_splits parts along K (0, 1: not)
    float* tail_partial;      // [tail_splits x tail_rem] tiles of 256 x 256 fp32
    int* dev_status;
    // modes 5 / 6: the bf16 output tile is also pruned along its own columns (MVUE 2:4, the next product's reduction
    // axis) and packed, as mvue_prune(output, axis 1, next_seed, tensor-core order) would
    uint4* next_values;       // [M x N/2] bf16 survivors of the pruned output
    uint8_t* next_meta;       // its metadata in tensor-core order
    RoundKeys next_rk;
};

// Epilogue of one thread: its accumulator row (32 columns at a time from tensor memory) goes to the
// split-K workspace, or through the optional elementwise scale / accumulate / bf16 conversion to C.
// kPre: the row's scale factors were loaded into registers (sc[c / 8] = columns c .. c + 7) while the main loop
// ran, so the drain never waits on memory; the column loop is then unrolled so that sc[] stays in registers.
template <bool kPre>
__device__ __forceinline__ void epilogue_rows(const GemmParams& p, int split, int64_t row, int64_t n0,
                                              uint32_t tmem_rows, bool have_acc, const uint4* sc_pre) {
#pragma unroll(kPre ? BN / 32 : 1)
    for (int c = 0; c < BN; c += 32) {
        uint32_t v[32];
        if (have_acc) {
            tmem_ld_32x32b_x32(tmem_rows + (uint32_t)c, v);
            tmem_ld_wait();
        } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) v[e] = 0u;
        }
        if (row < p.M) {
            const int64_t col0 = n0 + c;
            if (p.splits > 1) {
                float* dst = p.partial + ((int64_t)split * p.M + row) * p.N + col0;
#pragma unroll
                for (int e = 0; e < 32; e += 4)
                    if (col0 + e < p.N)
                        *reinterpret_cast<uint4*>(dst + e) = make_uint4(v[e], v[e + 1], v[e + 2], v[e + 3]);
            } else {
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                    if (col0 + e >= p.N) break;
                    float f[8];
#pragma unroll
                    for (int t = 0; t < 8; ++t) f[t] = __uint_as_float(v[e + t]);
                    if (kPre || p.scale) {
                        const uint4 sc = kPre ? sc_pre[(c + e) / 8]
                                              : *reinterpret_cast<const uint4*>(p.scale + row * p.ldc + col0 + e);
                        const uint32_t sw[4] = {sc.x, sc.y, sc.z, sc.w};
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            f[2 * t] *= __uint_as_float(sw[t] << 16);
                            f[2 * t + 1] *= __uint_as_float(sw[t] & 0xFFFF0000u);
                        }
                    }
                    if (p.c_is_bf16) {
                        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.C) + row * p.ldc + col0 + e;
                        uint32_t o[4];
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            __nv_bfloat162 pr = __floats2bfloat162_rn(f[2 * t], f[2 * t + 1]);
                            o[t] = *reinterpret_cast<uint32_t*>(&pr);
                        }
                        *reinterpret_cast<uint4*>(dst) = make_uint4(o[0], o[1], o[2], o[3]);
                    } else {
                        float* dst = reinterpret_cast<float*>(p.C) + row * p.ldc + col0 + e;
                        if (p.accumulate) {
                            const float4 c0 = *reinterpret_cast<const float4*>(dst);
                            const float4 c1 = *reinterpret_cast<const float4*>(dst + 4);
                            f[0] += c0.x; f[1] += c0.y; f[2] += c0.z; f[3] += c0.w;
                            f[4] += c1.x; f[5] += c1.y; f[6] += c1.z; f[7] += c1.w;
                        }
                        if ((reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {     // one full 32-byte sector per store
                            asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                                         ::"l"(dst), "f"(f[0]), "f"(f[1]), "f"(f[2]), "f"(f[3]), "f"(f[4]), "f"(f[5]),
                                           "f"(f[6]), "f"(f[7]) : "memory");
                        } else {
                            *reinterpret_cast<float4*>(dst) = make_float4(f[0], f[1], f[2], f[3]);
                            *reinterpret_cast<float4*>(dst + 4) = make_float4(f[4], f[5], f[6], f[7]);
                        }
                    }
                }
            }
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_copy_128x128b(uint32_t tmem_addr, uint64_t smem_desc) {
    asm volatile("tcgen05.cp.cta_group::1.128x128b [%0], %1;" ::"r"(tmem_addr), "l"(smem_desc) : "memory");
}
__device__ __forceinline__ void tc_mma_sp_bf16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc,
                                               uint32_t tmem_meta, uint32_t idesc, uint32_t accumulate) {
    const uint32_t zero = 0u;                 // no output lane is disabled
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::1.kind::f16 [%0], %1, %2, [%3], %4, {%6, %6, %6, %6}, p;\n\t}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(tmem_meta), "r"(idesc), "r"(accumulate), "r"(zero) : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t out;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(smem_addr), "r"(rank));
    return out;
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// TMA load whose completion bytes are counted on a barrier of the pair's leader.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y,
                                                 uint32_t leader_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(leader_bar) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {      // arrives on `bar` in both blocks
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void tc_copy_128x128b_pair(uint32_t tmem_addr, uint64_t smem_desc) {
    asm volatile("tcgen05.cp.cta_group::2.128x128b [%0], %1;" ::"r"(tmem_addr), "l"(smem_desc) : "memory");
}
__device__ __forceinline__ void tc_mma_sp_bf16_pair(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc,
                                                    uint32_t tmem_meta, uint32_t idesc, uint32_t accumulate) {
    const uint32_t zero = 0u;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%3], %4, {%6, %6, %6, %6, %6, %6, %6, %6}, p;\n\t}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(tmem_meta), "r"(idesc), "r"(accumulate), "r"(zero) : "memory");
}

// One work item of the persistent pair kernel: an output tile (of one K split).
struct WorkItem {
    int64_t m_block, m0, n0;      // this block's 128-row block of A, its first row, the pair's first column
    int split;
    int tail_slot;                // >= 0: part * tail_rem + tile of a tail tile cut along K; -1 otherwise
    int64_t step_begin, n_steps;
};

// Tiles go in bands of kBandTiles row tiles, row tile fastest inside a band, so that the pairs running at the
// same time cover a compact block of the output and share their A and B tiles in L2.
__device__ __forceinline__ void tile_of(int64_t M, int64_t N, int64_t pair_id, int64_t* tile_m, int64_t* tile_n) {
    const int64_t tiles_m = (M + 2 * BM - 1) / (2 * BM), tiles_n = (N + BN - 1) / BN;
    const int64_t band = pair_id / (kBandTiles * tiles_n);
    const int64_t band_h = tiles_m - band * kBandTiles < kBandTiles ? tiles_m - band * kBandTiles : kBandTiles;
    const int64_t in_band = pair_id - band * kBandTiles * tiles_n;
    *tile_m = band * kBandTiles + in_band % band_h;
    *tile_n = in_band / band_h;
}

// Work items are numbered split-major (K splits of small outputs), or, for outputs of many tiles whose last round
// would leave most pairs idle: first the n_main tiles of the full rounds, then the remaining tail_rem tiles cut
// into tail_splits parts along K (part-major), whose fp32 partial tiles a second pass sums.
__device__ __forceinline__ WorkItem decode_work(const GemmParams& p, int64_t w, uint32_t rank) {
    const int64_t tiles_m = (p.M + 2 * BM - 1) / (2 * BM), tiles_n = (p.N + BN - 1) / BN;
    const int64_t n_tiles = tiles_m * tiles_n;
    const int64_t total_steps = p.K / BK;
    WorkItem it;
    int64_t pair_id, per_part;
    int part;
    if (w >= p.n_main) {                                  // a part of a tail tile
        const int64_t j = w - p.n_main;
        part = (int)(j / p.tail_rem);
        const int tile = (int)(j - (int64_t)part * p.tail_rem);
        pair_id = p.n_main + tile;
        it.split = 0;
        it.tail_slot = part * p.tail_rem + tile;
        per_part = (total_steps + p.tail_splits - 1) / p.tail_splits;
    } else {
        it.split = (int)(w / n_tiles);
        pair_id = w - (int64_t)it.split * n_tiles;
        it.tail_slot = -1;
        part = it.split;
        per_part = p.k_steps_per_split;
    }
    int64_t tile_m, tile_n;
    tile_of(p.M, p.N, pair_id, &tile_m, &tile_n);
    it.m_block = tile_m * 2 + rank;
    it.m0 = it.m_block * BM;
    it.n0 = tile_n * BN;
    it.step_begin = (int64_t)part * per_part;
    int64_t step_end = it.step_begin + per_part;
    if (step_end > total_steps) step_end = total_steps;
    it.n_steps = step_end > it.step_begin ? step_end - it.step_begin : 0;
    return it;
}

// 8 values of one row to 32-byte-aligned memory in one store where the address allows, else two 16-byte stores.
__device__ __forceinline__ void store8_b32(void* dst, const uint32_t* v) {
    if ((reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                     ::"l"(dst), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                     : "memory");
    } else {
        reinterpret_cast<uint4*>(dst)[0] = make_uint4(v[0], v[1], v[2], v[3]);
        reinterpret_cast<uint4*>(dst)[1] = make_uint4(v[4], v[5], v[6], v[7]);
    }
}

// 4 x 4 transpose of 16-word cells among the four lanes of a quad.  v[] is one row of 64 words seen as eight
// 32-byte chunks; cell c = chunks c and c + 4 (words 8 c .. 8 c + 7 and 32 + 8 c .. 32 + 8 c + 7).  On entry a lane
// holds the cells of its own row; on exit its cell c is cell (lane % 4) of the row of quad lane c, so that the four
// lanes of a quad together hold whole 128-byte lines of each of the quad's four rows and a warp-wide 32-byte access
// touches 8 lines instead of 32.  The transpose is its own inverse.
__device__ __forceinline__ void quad_transpose(uint32_t (&v)[64], int lane) {
#pragma unroll
    for (int m = 1; m <= 2; m <<= 1) {
        const bool up = (lane & m) != 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if (c & m) continue;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int lo = (i < 8 ? 0 : 32) + 8 * c + (i & 7), hi = lo + 8 * m;   // cell c and cell c + m
                const uint32_t send = up ? v[lo] : v[hi];
                const uint32_t recv = __shfl_xor_sync(0xFFFFFFFFu, send, m);
                if (up) v[lo] = recv;
                else v[hi] = recv;
            }
        }
    }
}

// Persistent kernel: every pair of thread blocks walks the work items pair, pair + #pairs, ...
//   warp 0      TMA producer (both blocks); runs ahead into the next tile while the current one drains
//   warp 1      metadata copy + MMA issue (leader block only)
//   warp 2      tensor-memory allocation
//   warps 3-10  epilogue: warp w drains lanes 32 (w % 4) .. of columns 128 ((w - 3) / 4) .. into registers,
//               hands the accumulator back to the MMA warp at once, and only then converts and stores, so the
//               stores of one tile overlap the main loop of the next
// kMode fixes the output path at compile time so that the drained tile fits the register file:
//   0: fp32 (C, C +=, or the split-K workspace)   1: bf16   2: bf16 times p.scale   3: fp32 times p.scale
//   4: as 0 with the small-footprint epilogue (64 registers per thread), for work items with long main loops
//   5, 6: as 2, and the drained bf16 tile -- one row per lane, 128 consecutive columns: eight prune units in the form a
//         unit has when K is contiguous -- is pruned in registers (5: systematic sampling, 6: App. A.2 table) and its
//         survivors and metadata stored before the dense tile goes out: the output of the backward product (Sec. 1,
//         backward equation) leaves already pruned along the next backward product's reduction axis
//   7, 8: as 5, 6 with sixteen random bits per block (two units share one generator call)
// The scale factors of a row are fetched into registers under the main loop.
template <int kMode>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kMode == 4 ? 1024 : kThreads, 1)
sparse_gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                        const __grid_constant__ CUtensorMap map_e, const GemmParams p) {
    grid_dependency_wait();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t bar_base = smem_base + kStages * kStageBytes;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };                 // used in the leader only
    auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
    const uint32_t acc_bar = bar_base + 8u * (2 * kStages);                   // accumulators complete (both blocks)
    const uint32_t acc_free_bar = bar_base + 8u * (2 * kStages + 1);          // accumulators drained (leader only)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + kStages * kStageBytes + 8 * (2 * kStages + 2));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int64_t n_pairs = gridDim.x >> 1, first = blockIdx.x >> 1;
    const int64_t total_steps = p.K / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar(s), 1);       // the leader's producer arrives once, expecting both blocks' bytes
            mbar_init(empty_bar(s), 1);      // the leader's tcgen05.commit
        }
        mbar_init(acc_bar, 1);
        mbar_init(acc_free_bar, 2 * kEpiWarps);   // one arrival per epilogue warp of both blocks
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();                          // the peer's barriers exist before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both blocks)
        if (lane == 0) {
            uint32_t g = 0;                                  // stages filled so far, over all work items
            bool ok = true;
            for (int64_t w = first; w < p.n_work && ok; w += n_pairs) {
                const WorkItem it = decode_work(p, w, rank);
                const bool rows_exist = it.m0 < p.M;         // a pair may hang over the last row block
                for (int64_t i = 0; i < it.n_steps; ++i, ++g) {
                    const int s = (int)(g % kStages);
                    const uint32_t use = g / kStages;
                    if (use > 0 && !mbar_wait(empty_bar(s), (use - 1) & 1u, abort_flag)) { ok = false; break; }
                    const uint32_t a_dst = smem_base + s * kStageBytes;
                    const uint32_t b_dst = a_dst + kABytes;
                    const uint32_t e_dst = b_dst + kBBytes;
                    const int64_t step = it.step_begin + i;
                    const int k = (int)(step * BK);
                    const uint32_t leader_full = map_to_cta(full_bar(s), 0);
                    // only the leader arrives, and locally: a cluster-scope release from the peer on every stage
                    // would wait out the copies already in flight and serialise the pipeline
                    if (rank == 0) mbar_expect_tx(full_bar(s), 2 * kStageBytes);
                    // rows past M read as zeros (out-of-range boxes are zero-filled); the metadata of a row
                    // block that does not exist is taken from block 0 -- any valid pattern is harmless there
                    tma_load_2d_pair(a_dst, &map_a, k / 2, (int)it.m0, leader_full);
#pragma unroll
                    for (int j = 0; j < BN / 2 / 64; ++j)
                        tma_load_2d_pair(b_dst + j * kBBoxBytes, &map_b, (int)it.n0 + (int)rank * (BN / 2) + 64 * j, k,
                                         leader_full);
                    const int64_t e_block = (rows_exist ? it.m_block : 0) * total_steps + step;
                    tma_load_2d_pair(e_dst, &map_e, 0, (int)(e_block * 8), leader_full);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader only)
        if (rank == 0 && lane == 0) {
            uint32_t g = 0, tiles_done = 0;
            bool ok = true;
            for (int64_t w = first; w < p.n_work && ok; w += n_pairs) {
                const WorkItem it = decode_work(p, w, rank);
                if (it.n_steps == 0) continue;
                if (tiles_done > 0) {                        // the previous tile has left tensor memory
                    ok = mbar_wait_cluster(acc_free_bar, (tiles_done - 1) & 1u, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                }
                for (int64_t i = 0; i < it.n_steps; ++i, ++g) {
                    const int s = (int)(g % kStages);
                    const uint32_t use = g / kStages;
                    ok = mbar_wait(full_bar(s), use & 1u, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + s * kStageBytes;
                    const uint32_t b_addr = a_addr + kABytes;
                    const uint32_t e_addr = b_addr + kBBytes;
                    const uint32_t tmem_e = tmem_base + kTmemECol + 4u * s;
                    // 128 lanes x 16 bytes of metadata -> tensor-memory columns tmem_e .. tmem_e + 3 (both blocks)
                    tc_copy_128x128b_pair(tmem_e, make_smem_desc(e_addr, 16, 128, kSwizzleNone));
#pragma unroll
                    for (int kb = 0; kb < BK / 32; ++kb) {
                        // A: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart; 32 bytes per K = 32 block
                        const uint64_t a_desc = make_smem_desc(a_addr + kb * 32, 16, 1024, kSwizzle128B);
                        // B: N-major, 128-byte swizzle; 64-column blocks kBBoxBytes apart (leading), 8-row
                        //    groups 1024 bytes apart (stride); 32 k-rows per K = 32 block = 4096 bytes
                        const uint64_t b_desc = make_smem_desc(b_addr + kb * 4096, kBBoxBytes, 1024, kSwizzle128B);
                        // metadata of K block kb: column pair (kb & ~1) of the stage's four, selector kb & 1
                        tc_mma_sp_bf16_pair(tmem_base, a_desc, b_desc, tmem_e + (uint32_t)(kb & ~1),
                                            kInstrDesc2 | (uint32_t)(kb & 1), (i > 0 || kb > 0) ? 1u : 0u);
                    }
                    tc_commit_pair(empty_bar(s));    // frees the stage in both blocks when the MMAs retire
                }
                if (!ok) break;
                tc_commit_pair(acc_bar);             // accumulators complete
                ++tiles_done;
            }
        }
    } else if (warp >= 3) {
        // ------------------------------------------------------------ epilogue (both blocks, own rows)
        const int q = warp & 3;                                  // tensor-memory lanes 32 q .. 32 q + 31 (a warp's quarter)
        const int c_off = 128 * ((warp - 3) >> 2);               // this warp's half of the tile's columns
        const uint32_t tmem_rows = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)c_off;
        const uint32_t leader_free = map_to_cta(acc_free_bar, 0);
        uint32_t tiles_done = 0;
        for (int64_t w = first; w < p.n_work; w += n_pairs) {
            const WorkItem it = decode_work(p, w, rank);
            const int64_t row = it.m0 + 32 * q + lane;
            const int64_t col0 = it.n0 + c_off;
            const bool row_ok = row < p.M;
            if constexpr (kMode == 4) {
                // fp32 output, small register footprint: 32 columns at a time from tensor memory straight to their
                // destination, tensor memory handed back after the last store has been issued.  Next to a main loop
                // of dozens of stages the longer hold is nothing, and at 64 registers per thread the block leaves
                // two thirds of the SM's register file to other kernels' blocks.
                const bool have_acc = it.n_steps > 0;
                if (have_acc) {
                    if (!__all_sync(0xFFFFFFFFu, mbar_wait(acc_bar, tiles_done & 1u, abort_flag))) break;
                    tc_fence_after();
                }
                float* dst;
                int64_t cols_here;                               // columns of this warp's 128 that exist
                bool plain = false;                              // the final output (may accumulate), not a partial
                if (it.tail_slot >= 0) {
                    dst = p.tail_partial + (((int64_t)it.tail_slot * (2 * BM) + (int64_t)rank * BM + 32 * q + lane) * BN) + c_off;
                    cols_here = 128;
                } else if (p.splits > 1) {
                    dst = p.partial + ((int64_t)it.split * p.M + row) * p.N + col0;
                    cols_here = p.N - col0;
                } else {
                    dst = reinterpret_cast<float*>(p.C) + row * p.ldc + col0;
                    cols_here = p.N - col0;
                    plain = true;
                }
#pragma unroll 1
                for (int c = 0; c < 128; c += 32) {
                    uint32_t v[32];
                    if (have_acc) {
                        tmem_ld_32x32b_x32(tmem_rows + (uint32_t)c, v);
                        tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = 0u;
                    }
                    if (row_ok) {
#pragma unroll
                        for (int e = 0; e < 32; e += 8) {
                            if (c + e >= cols_here) break;       // N is a multiple of 8
                            if (plain && p.accumulate) {
                                const float4 c0 = *reinterpret_cast<const float4*>(dst + c + e);
                                const float4 c1 = *reinterpret_cast<const float4*>(dst + c + e + 4);
                                v[e] = __float_as_uint(__uint_as_float(v[e]) + c0.x);
                                v[e + 1] = __float_as_uint(__uint_as_float(v[e + 1]) + c0.y);
                                v[e + 2] = __float_as_uint(__uint_as_float(v[e + 2]) + c0.z);
                                v[e + 3] = __float_as_uint(__uint_as_float(v[e + 3]) + c0.w);
                                v[e + 4] = __float_as_uint(__uint_as_float(v[e + 4]) + c1.x);
                                v[e + 5] = __float_as_uint(__uint_as_float(v[e + 5]) + c1.y);
                                v[e + 6] = __float_as_uint(__uint_as_float(v[e + 6]) + c1.z);
                                v[e + 7] = __float_as_uint(__uint_as_float(v[e + 7]) + c1.w);
                            }
                            store8_b32(dst + c + e, &v[e]);
                        }
                    }
                }
                if (have_acc) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0)
                        asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(leader_free) : "memory");
                    ++tiles_done;
                }
                continue;
            }
            // bf16 x scale keeps the row's factors in registers; fp32 x scale has no room for them beside 128
            // fp32 results and applies them after tensor memory has been handed back
            constexpr bool kPrune = kMode >= 5 && kMode <= 8;             // 5, 7: systematic sampling; 6, 8: App. A.2 table
            constexpr int kPruneJoint = (kMode == 5 || kMode == 7) ? 1 : 0;
            constexpr bool kPruneEps16 = kMode >= 7;                       // 7, 8: sixteen random bits per block
            constexpr bool kScale = kMode == 2 || kPrune, kLateScale = kMode == 3, kToBf16 = kMode == 1 || kScale;
            // bf16 outputs and their factors move in the quad-transposed arrangement (quad_transpose): lane
            // 4 a + b reads / writes, for c = 0..3 and k = 0, 1, the 32-byte chunk b + 4 k of row 4 a + c of the warp's
            // 32 rows, i.e. the quad covers whole 128-byte lines.
            const int64_t row_q = it.m0 + 32 * q + 4 * (lane >> 2);      // first row of this lane's quad
            const int64_t col_q = col0 + 16 * (lane & 3);                // this lane's chunk (k = 0) of those rows
            uint32_t scw[kScale ? 64 : 1];
            if constexpr (kScale) {                              // the factors, fetched under the main loop
#pragma unroll
                for (int c = 0; c < 4; ++c) {
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        uint32_t* d = &scw[32 * k + 8 * c];
#pragma unroll
                        for (int t = 0; t < 8; ++t) d[t] = 0u;
                        const int64_t cc = col_q + 64 * k;
                        if (row_q + c >= p.M) continue;
                        const __nv_bfloat16* src = p.scale + (row_q + c) * p.ldc + cc;
                        if (cc + 8 < p.N && (reinterpret_cast<uintptr_t>(src) & 31u) == 0) {   // one whole 32-byte sector
                            asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                                         : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]), "=r"(d[4]), "=r"(d[5]),
                                           "=r"(d[6]), "=r"(d[7])
                                         : "l"(src));
                        } else {
                            if (cc < p.N) {
                                const uint4 v4 = __ldg(reinterpret_cast<const uint4*>(src));
                                d[0] = v4.x; d[1] = v4.y; d[2] = v4.z; d[3] = v4.w;
                            }
                            if (cc + 8 < p.N) {
                                const uint4 v4 = __ldg(reinterpret_cast<const uint4*>(src + 8));
                                d[4] = v4.x; d[5] = v4.y; d[6] = v4.z; d[7] = v4.w;
                            }
                        }
                    }
                }
                quad_transpose(scw, lane);                       // back to one row per lane, as the drain multiplies
            }
            uint32_t r[kToBf16 ? 64 : 128];                      // packed bf16 pairs, or fp32 bit patterns
            if (it.n_steps > 0) {
                // (warp-uniform: the lanes shuffle with each other further down)
                if (!__all_sync(0xFFFFFFFFu, mbar_wait(acc_bar, tiles_done & 1u, abort_flag))) break;
                tc_fence_after();
#pragma unroll
                for (int half = 0; half < 2; ++half) {           // 64 columns at a time
                    uint32_t t0[32], t1[32];
                    tmem_ld_32x32b_x32(tmem_rows + (uint32_t)(64 * half), t0);
                    tmem_ld_32x32b_x32(tmem_rows + (uint32_t)(64 * half + 32), t1);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 64; e += 2) {
                        float f0 = __uint_as_float(e < 32 ? t0[e] : t1[e - 32]);
                        float f1 = __uint_as_float(e < 32 ? t0[e + 1] : t1[e - 31]);
                        if (kScale) {
                            const uint32_t sw = scw[(64 * half + e) / 2];
                            f0 *= __uint_as_float(sw << 16);
                            f1 *= __uint_as_float(sw & 0xFFFF0000u);
                        }
                        if (kToBf16) {
                            __nv_bfloat162 pr = __floats2bfloat162_rn(f0, f1);
                            r[(64 * half + e) / 2] = *reinterpret_cast<uint32_t*>(&pr);
                        } else {
                            r[64 * half + e] = __float_as_uint(f0);
                            r[64 * half + e + 1] = __float_as_uint(f1);
                        }
                    }
                }
                // the accumulator is in registers (tcgen05.wait::ld has returned in every lane): give tensor
                // memory back before touching global memory.  The arrival orders nothing but that, so it is
                // relaxed: a release at cluster scope would first wait out the previous tile's global stores.
                tc_fence_before();
                __syncwarp();
                if (lane == 0)
                    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(leader_free) : "memory");
                ++tiles_done;
            } else {
#pragma unroll
                for (int e = 0; e < (kToBf16 ? 64 : 128); ++e) r[e] = 0u;
            }
            if constexpr (kPrune) {
                // r[8 t .. 8 t + 7] = columns col0 + 16 t .. + 15 of this lane's row as bf16 pairs: prune unit t of the row
                if (row_ok && col0 < p.N) {                              // (N is a multiple of 128: all eight units exist)
                    const int64_t upr = p.N >> 4, strip0 = col0 >> 4;
                    uint4* vdst = p.next_values + row * upr + strip0;
#pragma unroll
                    for (int t = 0; t < 8; t += 2) {                     // units 2i, 2i + 1 (strip0 + t is even)
                        uint32_t raw0[8], raw1[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) { raw0[e] = r[8 * t + e]; raw1[e] = r[8 * t + 8 + e]; }
                        const uint64_t unit = (uint64_t)(row * upr + strip0 + t);
                        uint4 v0, v1;
                        uint32_t mt0, mt1;
                        if constexpr (kPruneEps16) {                      // the two units share one generator call
                            uint32_t w0[4], w1[4];
                            unit_pair_words16(unit, p.next_rk, w0, w1);
                            prune_unit_bf16_w<4, kPruneJoint, false>(raw0, w0, unit, p.next_rk, &v0, &mt0);
                            prune_unit_bf16_w<4, kPruneJoint, false>(raw1, w1, unit + 1, p.next_rk, &v1, &mt1);
                        } else {
                            prune_unit_bf16<4, kPruneJoint>(raw0, unit, p.next_rk, &v0, &mt0);
                            prune_unit_bf16<4, kPruneJoint>(raw1, unit + 1, p.next_rk, &v1, &mt1);
                        }
                        vdst[t] = v0;
                        vdst[t + 1] = v1;
                        *reinterpret_cast<uint16_t*>(p.next_meta + tc_meta_offset(row, strip0 + t, p.N >> 7)) = (uint16_t)mt0;
                        *reinterpret_cast<uint16_t*>(p.next_meta + tc_meta_offset(row, strip0 + t + 1, p.N >> 7)) = (uint16_t)mt1;
                    }
                }
            }
            if constexpr (kToBf16) {
                quad_transpose(r, lane);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        const int64_t cc = col_q + 64 * k;
                        if (row_q + c >= p.M) continue;
                        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.C) + (row_q + c) * p.ldc + cc;
                        const uint32_t* v = &r[32 * k + 8 * c];
                        if (cc + 8 < p.N) store8_b32(dst, v);
                        else if (cc < p.N) *reinterpret_cast<uint4*>(dst) = make_uint4(v[0], v[1], v[2], v[3]);
                    }
                }
                continue;
            }
            if (!row_ok) continue;
            if (!kToBf16 && it.tail_slot >= 0) {             // a K part of a tail tile: unscaled fp32 partial tile
                float* dst = p.tail_partial + (((int64_t)it.tail_slot * (2 * BM) + (int64_t)rank * BM + 32 * q + lane) * BN) + c_off;
#pragma unroll
                for (int e = 0; e < 128; e += 8) store8_b32(dst + e, &r[e]);
            } else if (kToBf16) {
                __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.C) + row * p.ldc + col0;
#pragma unroll
                for (int e = 0; e < 128; e += 16) {
                    if (col0 + e + 8 < p.N) store8_b32(dst + e, &r[e / 2]);
                    else if (col0 + e < p.N)
                        *reinterpret_cast<uint4*>(dst + e) = make_uint4(r[e / 2], r[e / 2 + 1], r[e / 2 + 2], r[e / 2 + 3]);
                }
            } else if (kMode == 0 && p.splits > 1) {
                float* dst = p.partial + ((int64_t)it.split * p.M + row) * p.N + col0;
#pragma unroll
                for (int e = 0; e < 128; e += 8)
                    if (col0 + e < p.N) store8_b32(dst + e, &r[e]);
            } else {
                float* dst = reinterpret_cast<float*>(p.C) + row * p.ldc + col0;
#pragma unroll
                for (int e = 0; e < 128; e += 8) {
                    if (col0 + e >= p.N) break;
                    if (kLateScale) {
                        const uint4 s4 = __ldg(reinterpret_cast<const uint4*>(p.scale + row * p.ldc + col0 + e));
                        const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            r[e + 2 * t] = __float_as_uint(__uint_as_float(r[e + 2 * t]) * __uint_as_float(sw[t] << 16));
                            r[e + 2 * t + 1] =
                                __float_as_uint(__uint_as_float(r[e + 2 * t + 1]) * __uint_as_float(sw[t] & 0xFFFF0000u));
                        }
                    }
                    if (kMode == 0 && p.accumulate) {
                        const float4 c0 = *reinterpret_cast<const float4*>(dst + e);
                        const float4 c1 = *reinterpret_cast<const float4*>(dst + e + 4);
                        r[e] = __float_as_uint(__uint_as_float(r[e]) + c0.x);
                        r[e + 1] = __float_as_uint(__uint_as_float(r[e + 1]) + c0.y);
                        r[e + 2] = __float_as_uint(__uint_as_float(r[e + 2]) + c0.z);
                        r[e + 3] = __float_as_uint(__uint_as_float(r[e + 3]) + c0.w);
                        r[e + 4] = __float_as_uint(__uint_as_float(r[e + 4]) + c1.x);
                        r[e + 5] = __float_as_uint(__uint_as_float(r[e + 5]) + c1.y);
                        r[e + 6] = __float_as_uint(__uint_as_float(r[e + 6]) + c1.z);
                        r[e + 7] = __float_as_uint(__uint_as_float(r[e + 7]) + c1.w);
                    }
                    store8_b32(dst + e, &r[e]);
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) {
        // give copies that may still be in flight a bounded chance to land before the pair exits
        for (int s = 0; s < kStages; ++s)
            for (uint32_t spin = 0; spin < 4096 && !mbar_try_wait(full_bar(s), 0) && !mbar_try_wait(full_bar(s), 1); ++spin)
                __nanosleep(64);
        if (p.dev_status) *p.dev_status = MVUE_ERR_DEVICE_TIMEOUT;
    }
    cluster_sync();                          // neither block leaves while the other may still touch it
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// =============================================================================
// Prune fused into the update product: dW[out x in] = theta(g)^T h with g read once per cluster and the
// packed operand never written to memory.  One thread block per 128 x 256 output tile
// (tcgen05.mma.sp.cta_group::1, M = 128), two stages of K = 128; C = 1, 2 or 4 blocks whose tiles are neighbours
// along `in` form a cluster and SHARE the pruned stage: every block prunes 1 / C of the stage's 1024 units (a unit =
// one row of A x 16 tokens) and writes each result -- 16 bytes of survivors at their 128-byte-swizzled place in the
// A tile, 2 bytes of metadata at their tensor-core lane / word -- into the shared memory of all C blocks
// (st.shared::cluster), so a row tile of g is pruned in / (256 C) times instead of in / 256 times.
//   warp 0      TMA producer of the block's own B tile (four 64-column boxes of h)
//   warp 1      tcgen05.cp of the stage's metadata, four MMAs, commit -- arriving on the "empty" barrier of ALL
//               blocks of the cluster: a stage is rewritten only when every block has consumed it
//   warp 2      tensor-memory allocation
//   warps 4-7   epilogue
//   warps 8-15  prune: warp w of block r owns strip (8 / C) r + w / C of the stage and the rows
//               (128 / C) (w % C) + lane + 32 i, i < 4 / C; a lane reads its column of g for the strip's 16 tokens
//               (a warp reads 64 contiguous bytes per token), prunes the unit with the same unit function and the
//               same global block numbers as mvue_prune, stores to every block, fences the writes for the
//               tensor cores' asynchronous reads and arrives on every block's "full" barrier (1 + 8 C arrivals).
// No block leaves before all have (cluster barrier): peers write into its shared memory until the last stage.
// =============================================================================
constexpr int kFStages = 2;
constexpr int kFBBytes = (BN / 64) * kBBoxBytes;                 // 64 KiB: all 256 columns
constexpr int kFStageBytes = kABytes + kFBBytes + kEBytes;       // 82 KiB
constexpr int kFSmemBytes = kFStages * kFStageBytes + 1024 + 256;
constexpr int kFThreads = 512;
constexpr int kFPruneWarps = 8;
constexpr uint32_t kInstrDesc1 = (1u << 2) | (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                                 ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

struct FusedParams {
    const uint16_t* g;        // bf16 [T x out]
    int64_t ldg;              // leading dimension of g in elements
    RoundKeys rk;
    GemmParams gemm;          // M = out, N = in, K = T
};

__device__ __forceinline__ void st_cluster_v4(uint32_t addr, uint4 v) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void st_cluster_u16(uint32_t addr, uint16_t v) {
    asm volatile("st.shared::cluster.b16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t remote_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
__device__ __forceinline__ void tc_commit_cluster(uint32_t bar, uint16_t mask) {   // arrives on `bar` in every block of the mask
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}

// NM: 2 (1:2) or 4 (2:4); kJoint: the 2:4 law (0 App. A.2 table, 1 systematic sampling).
template <int NM, int kJoint, int kC>
__global__ void __launch_bounds__(kFThreads, 1)
fused_update_kernel(const __grid_constant__ CUtensorMap map_b, const FusedParams fp) {
    const GemmParams& p = fp.gemm;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t bar_base = smem_base + kFStages * kFStageBytes;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kFStages + s); };
    const uint32_t acc_bar = bar_base + 8u * (2 * kFStages);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + kFStages * kFStageBytes + 8 * (2 * kFStages + 1));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t C = kC;                                               // blocks of a cluster differ in blockIdx.x only
    const uint32_t rank = cluster_ctarank();
    const int64_t m0 = (int64_t)blockIdx.y * BM;
    const int64_t n0 = (int64_t)blockIdx.x * BN;
    const int split = blockIdx.z;
    const int64_t total_steps = p.K / BK;
    const int64_t step_begin = (int64_t)split * p.k_steps_per_split;
    int64_t step_end = step_begin + p.k_steps_per_split;
    if (step_end > total_steps) step_end = total_steps;
    const int64_t n_steps = step_end > step_begin ? step_end - step_begin : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kFStages; ++s) {
            mbar_init(full_bar(s), 1 + kFPruneWarps * C);   // B bytes + one arrival per prune warp of every block
            mbar_init(empty_bar(s), C);                     // every block's MMA warp has consumed the stage
        }
        mbar_init(acc_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();                          // the peers' barriers exist before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            for (int64_t i = 0; i < n_steps; ++i) {
                const int s = (int)(i % kFStages);
                const uint32_t use = (uint32_t)(i / kFStages);
                if (use > 0 && !mbar_wait_cluster(empty_bar(s), (use - 1) & 1u, abort_flag)) break;
                const uint32_t b_dst = smem_base + s * kFStageBytes + kABytes;
                const int k = (int)((step_begin + i) * BK);
                mbar_expect_tx(full_bar(s), kFBBytes);
#pragma unroll
                for (int j = 0; j < BN / 64; ++j)
                    tma_load_2d(b_dst + j * kBBoxBytes, &map_b, (int)n0 + 64 * j, k, full_bar(s));
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = true;
            const uint16_t all = (uint16_t)((1u << C) - 1u);
            for (int64_t i = 0; i < n_steps && ok; ++i) {
                const int s = (int)(i % kFStages);
                const uint32_t use = (uint32_t)(i / kFStages);
                ok = mbar_wait_cluster(full_bar(s), use & 1u, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_addr = smem_base + s * kFStageBytes;
                const uint32_t b_addr = a_addr + kABytes;
                const uint32_t e_addr = b_addr + kFBBytes;
                const uint32_t tmem_e = tmem_base + kTmemECol + 4u * s;
                tc_copy_128x128b(tmem_e, make_smem_desc(e_addr, 16, 128, kSwizzleNone));
#pragma unroll
                for (int kb = 0; kb < BK / 32; ++kb) {
                    const uint64_t a_desc = make_smem_desc(a_addr + kb * 32, 16, 1024, kSwizzle128B);
                    const uint64_t b_desc = make_smem_desc(b_addr + kb * 4096, kBBoxBytes, 1024, kSwizzle128B);
                    tc_mma_sp_bf16(tmem_base, a_desc, b_desc, tmem_e + (uint32_t)(kb & ~1),
                                   kInstrDesc1 | (uint32_t)(kb & 1), (i > 0 || kb > 0) ? 1u : 0u);
                }
                tc_commit_cluster(empty_bar(s), all);
            }
            tc_commit(acc_bar);
        }
    } else if (warp >= 4 && warp < 8) {
        const int q = warp - 4;
        const bool acc_ok = n_steps > 0 ? mbar_wait(acc_bar, 0, abort_flag) : true;
        tc_fence_after();
        const int64_t row = m0 + 32 * q + lane;
        if (acc_ok && n0 < p.N)
            epilogue_rows<false>(p, split, row, n0, tmem_base + ((uint32_t)(32 * q) << 16), n_steps > 0, nullptr);
    } else if (warp >= 8) {
        // ------------------------------------------------------------ prune warps
        const int pw = warp - 8;
        constexpr int kStripsOwn = 8 / kC, kUnits = 4 / kC;         // strips of a stage per block, units per lane
        const int strip_l = kStripsOwn * (int)rank + pw / kC;       // 16-token strip of the stage
        const int row_base = (128 / kC) * (pw % kC) + lane;         // first of this lane's rows of the A tile
        const int64_t units_per_row = p.K / 16;
        // the lane's columns of g for one stage: 16 tokens each; the next stage's are requested before this one is pruned
        auto load_stage = [&](int64_t i, uint32_t (&dst)[kUnits][16]) {
            const int64_t k0 = (step_begin + i) * BK + 16 * strip_l;
#pragma unroll
            for (int u = 0; u < kUnits; ++u) {
                const int64_t col = m0 + row_base + 32 * u;                 // row of A = column of g
                const uint16_t* src = fp.g + k0 * fp.ldg + col;
#pragma unroll
                for (int r = 0; r < 16; ++r) dst[u][r] = col < p.M ? (uint32_t)__ldg(src + r * fp.ldg) : 0u;
            }
        };
        constexpr bool kPrefetch = kUnits <= 2;                      // (four units per lane leave no registers for a second set)
        uint32_t cur[kUnits][16], nxt[kPrefetch ? kUnits : 1][16];
        if (kPrefetch && n_steps > 0) load_stage(0, cur);
        bool ok = true;
        for (int64_t i = 0; i < n_steps && ok; ++i) {
            const int s = (int)(i % kFStages);
            const uint32_t use = (uint32_t)(i / kFStages);
            const int64_t k0 = (step_begin + i) * BK + 16 * strip_l;        // first token of the strip
            if constexpr (kPrefetch) {
                if (i + 1 < n_steps) load_stage(i + 1, nxt);
            } else {
                load_stage(i, cur);
            }
            if (use > 0) ok = mbar_wait_cluster(empty_bar(s), (use - 1) & 1u, abort_flag);
            if (!ok) break;
            const uint32_t a_tile = smem_base + s * kFStageBytes;
            const uint32_t e_tile = a_tile + kABytes + kFBBytes;
#pragma unroll
            for (int u = 0; u < kUnits; ++u) {
                const int m_l = row_base + 32 * u;                          // row of the A tile
                const int64_t col = m0 + m_l;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                uint32_t mt = 0x4444u;
                if (col < p.M) {
                    uint32_t raw[8];                                         // the unit as it is when K is contiguous
#pragma unroll
                    for (int e = 0; e < 8; ++e) raw[e] = cur[u][2 * e] | (cur[u][2 * e + 1] << 16);
                    const uint64_t unit = (uint64_t)col * (uint64_t)units_per_row + (uint64_t)(k0 >> 4);
                    prune_unit_bf16<NM, kJoint>(raw, unit, fp.rk, &v, &mt);
                }
                // A tile: row m_l is 128 bytes; the strip's 8 survivors are chunk strip_l, swizzled by the row;
                // metadata: lane / word / half-word of the tensor-core order.  Same place in every block of the cluster.
                const uint32_t a_off = a_tile + (uint32_t)(m_l * 128 + ((strip_l ^ (m_l & 7)) << 4));
                const int tc_lane = (m_l & 7) + 8 * (strip_l & 1) + 16 * (m_l >> 4);
                const uint32_t e_off = e_tile + (uint32_t)(tc_lane * 16 + (strip_l >> 1) * 4 + ((m_l >> 3) & 1) * 2);
#pragma unroll
                for (uint32_t d = 0; d < C; ++d) {
                    st_cluster_v4(map_to_cta(a_off, d), v);
                    st_cluster_u16(map_to_cta(e_off, d), (uint16_t)mt);
                }
            }
            asm volatile("fence.proxy.async.shared::cluster;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
#pragma unroll
                for (uint32_t d = 0; d < C; ++d) mbar_arrive_cluster(map_to_cta(full_bar(s), d));
            }
            if constexpr (kPrefetch) {
#pragma unroll
                for (int u = 0; u < kUnits; ++u) {
#pragma unroll
                    for (int r = 0; r < 16; ++r) cur[u][r] = nxt[u][r];
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) {
            for (int s = 0; s < kFStages; ++s)
                for (uint32_t spin = 0; spin < 4096 && !mbar_try_wait(full_bar(s), 0) && !mbar_try_wait(full_bar(s), 1); ++spin)
                    __nanosleep(64);
            if (p.dev_status) *p.dev_status = MVUE_ERR_DEVICE_TIMEOUT;
        }
        __syncthreads();
    }
    cluster_sync();                          // no block leaves while a peer may still write to it or signal it
    if (warp == 2) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// Second pass of split-K: sums the partial tiles in a fixed order (deterministic) and applies the
// same epilogue as the single-pass path.
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float* __restrict__ partial, int splits, int64_t M, int64_t N, void* C, int64_t ldc,
                     const __nv_bfloat16* __restrict__ scale, int c_is_bf16, int accumulate) {
    const int64_t n4 = N / 4;
    const int64_t total = M * n4;
    grid_dependency_wait();
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / n4, c = (i - r * n4) * 4;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s = 0; s < splits; ++s) {
            const float4 v = *reinterpret_cast<const float4*>(partial + ((int64_t)s * M + r) * N + c);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        if (scale) {
            const uint2 sc = *reinterpret_cast<const uint2*>(scale + r * ldc + c);
            acc.x *= __uint_as_float(sc.x << 16); acc.y *= __uint_as_float(sc.x & 0xFFFF0000u);
            acc.z *= __uint_as_float(sc.y << 16); acc.w *= __uint_as_float(sc.y & 0xFFFF0000u);
        }
        if (c_is_bf16) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
            *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(C) + r * ldc + c) =
                make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
        } else {
            float* dst = reinterpret_cast<float*>(C) + r * ldc + c;
            if (accumulate) {
                const float4 o = *reinterpret_cast<const float4*>(dst);
                acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w;
            }
            *reinterpret_cast<float4*>(dst) = acc;
        }
    }
}

// Sums the K parts of the tail tiles (see decode_work) into C: one block per row of a tail tile.
__global__ void __launch_bounds__(64)
tail_reduce_kernel(const float* __restrict__ partial, int rem, int parts, int64_t n_main, int64_t M, int64_t N,
                   float* __restrict__ C, int64_t ldc, const __nv_bfloat16* __restrict__ scale, int accumulate) {
    grid_dependency_wait();
    const int tile = blockIdx.x / (2 * BM), lr = blockIdx.x % (2 * BM);
    int64_t tile_m, tile_n;
    tile_of(M, N, n_main + tile, &tile_m, &tile_n);
    const int64_t row = tile_m * (2 * BM) + lr, col = tile_n * BN + 4 * threadIdx.x;
    if (row >= M || col >= N) return;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int part = 0; part < parts; ++part) {
        const float4 v = *reinterpret_cast<const float4*>(
            partial + (((int64_t)(part * rem + tile) * (2 * BM) + lr) * BN) + 4 * threadIdx.x);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    if (scale) {
        const uint2 sc = *reinterpret_cast<const uint2*>(scale + row * ldc + col);
        acc.x *= __uint_as_float(sc.x << 16); acc.y *= __uint_as_float(sc.x & 0xFFFF0000u);
        acc.z *= __uint_as_float(sc.y << 16); acc.w *= __uint_as_float(sc.y & 0xFFFF0000u);
    }
    float* dst = C + row * ldc + col;
    if (accumulate) {
        const float4 o = *reinterpret_cast<const float4*>(dst);
        acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w;
    }
    *reinterpret_cast<float4*>(dst) = acc;
}

// =============================================================================
// Issue-rate probe: what the sparse tensor cores deliver when nothing has to be loaded.  Every pair fills ONE
// pipeline stage with zeros and a valid metadata pattern and its leader issues `iters` x 4 of the very
// tcgen05.mma.sp.cta_group::2 instructions of the product kernel (M = 256, N = 256, K = 32 each) on that stage, back to
// back, one commit at the end.  The time of this launch is the ceiling any tiling of the product can approach.
// =============================================================================
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(128, 1)
sparse_mma_issue_probe_kernel(int iters, uint32_t spin_limit, int* dev_status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t done_bar = smem_base + kStageBytes;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + kStageBytes + 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();

    for (int i = threadIdx.x; i < kStageBytes / 16; i += blockDim.x) {       // A and B zero, metadata "positions 0 and 1"
        const uint32_t w = i * 16 >= kABytes + kBBytes ? 0x44444444u : 0u;
        reinterpret_cast<uint4*>(smem_gen)[i] = make_uint4(w, w, w, w);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");             // the tensor cores read what the lanes wrote
    if (threadIdx.x == 0) {
        mbar_init(done_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // iters = 0 issues nothing and commits nothing: nobody ever arrives on done_bar, so the wait below runs out after
    // spin_limit polls and both blocks leave through the ordinary exit (the self-test of the bounded-wait path)
    if (iters > 0 && rank == 0 && warp == 1 && lane == 0) {
        const uint32_t a_addr = smem_base, b_addr = a_addr + kABytes, e_addr = b_addr + kBBytes;
        const uint32_t tmem_e = tmem_base + kTmemECol;
        tc_copy_128x128b_pair(tmem_e, make_smem_desc(e_addr, 16, 128, kSwizzleNone));
        for (int i = 0; i < iters; ++i) {
#pragma unroll
            for (int kb = 0; kb < BK / 32; ++kb) {
                const uint64_t a_desc = make_smem_desc(a_addr + kb * 32, 16, 1024, kSwizzle128B);
                const uint64_t b_desc = make_smem_desc(b_addr + kb * 4096, kBBoxBytes, 1024, kSwizzle128B);
                tc_mma_sp_bf16_pair(tmem_base, a_desc, b_desc, tmem_e + (uint32_t)(kb & ~1), kInstrDesc2 | (uint32_t)(kb & 1),
                                    (i > 0 || kb > 0) ? 1u : 0u);
            }
        }
        tc_commit_pair(done_bar);                                            // both blocks' barriers, when the MMAs retire
    }
    const bool ok = mbar_wait(done_bar, 0u, abort_flag, spin_limit);         // bounded
    tc_fence_after();
    __syncthreads();
    if (!ok && threadIdx.x == 0 && dev_status) *dev_status = MVUE_ERR_DEVICE_TIMEOUT;
    tc_fence_before();
    cluster_sync();
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ---- host side ----------------------------------------------------------------
}  // namespace

int gemm_split_count(int64_t M, int64_t N, int64_t K, int sm_count) {
    // thread blocks one split launches: two per 256 x 256 tile
    const int64_t blocks = 2 * ((M + 2 * BM - 1) / (2 * BM)) * ((N + BN - 1) / BN);
    const int64_t steps = K / BK;
    if (blocks >= sm_count || steps < 8) return 1;
    int64_t splits = sm_count / blocks;
    if (splits > steps / 4) splits = steps / 4;      // at least 4 stages (K = 512) per split
    if (splits > 64) splits = 64;
    return (int)(splits < 1 ? 1 : splits);
}

size_t gemm_required_workspace_bytes(int64_t M, int64_t N, int64_t K, int sm_count) {
    const int splits = gemm_split_count(M, N, K, sm_count);
    return splits > 1 ? (size_t)splits * (size_t)M * (size_t)N * sizeof(float) : 0;
}

namespace {

// The instantiations of the pair kernel, their shared-memory attribute, and how many pairs fit the GPU at
// once (one block per SM): the size of the persistent grid.  Looked up once per device.
struct PairKernelSetup {
    PerDeviceOnce once;
    int max_pairs[kMaxDevices] = {};
};
PairKernelSetup& pair_setup() {
    static PairKernelSetup st;
    return st;
}
cudaError_t pair_kernel_setup() {
    PairKernelSetup& st = pair_setup();
    return once_per_device(st.once, [&st](int dev) {
        const void* kernels[9] = {reinterpret_cast<const void*>(sparse_gemm_pair_kernel<0>),
                                  reinterpret_cast<const void*>(sparse_gemm_pair_kernel<1>),
                                  reinterpret_cast<const void*>(sparse_gemm_pair_kernel<2>),
                                  reinterpret_cast<const void*>(sparse_gemm_pair_kernel<3>),
                                  reinterpret_cast<const void*>(sparse_gemm_pair_kernel<4>),
                                  reinterpret_cast<const void*>(sparse_gemm_pair_kernel<5>),
                                  reinterpret_cast<const void*>(sparse_gemm_pair_kernel<6>),
                                  reinterpret_cast<const void*>(sparse_gemm_pair_kernel<7>),
                                  reinterpret_cast<const void*>(sparse_gemm_pair_kernel<8>)};
        cudaError_t err = cudaSuccess;
        for (int i = 0; i < 9 && err == cudaSuccess; ++i)
            err = cudaFuncSetAttribute(kernels[i], cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2, 1, 1);
        cfg.blockDim = dim3(kThreads, 1, 1);
        cfg.dynamicSmemBytes = kSmemBytes;
        int n = 0;
        if (err == cudaSuccess && cudaOccupancyMaxActiveClusters(&n, sparse_gemm_pair_kernel<0>, &cfg) == cudaSuccess)
            st.max_pairs[dev] = n;
        (void)cudaGetLastError();
        return err;
    });
}
int resident_pairs(int sm_count) {
    int dev = 0, n = 0;
    if (pair_kernel_setup() == cudaSuccess && cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices)
        n = pair_setup().max_pairs[dev];
    return n > 0 ? n : (sm_count / 2 > 0 ? sm_count / 2 : 1);
}

// When the output has more tiles than resident pairs and the last round would keep at most half of them busy,
// the tiles of that round are cut along K into `parts` so that the round is short and full.
struct TailPlan {
    int rem = 0, parts = 0;
    int64_t n_main = 0;       // tiles (times splits) handled whole
};
TailPlan tail_plan(int64_t M, int64_t N, int64_t K, int splits, int n_pairs) {
    const int64_t n_tiles = ((M + 2 * BM - 1) / (2 * BM)) * ((N + BN - 1) / BN);
    const int64_t steps = K / BK;
    TailPlan t;
    t.n_main = n_tiles * splits;
    if (splits != 1 || n_tiles <= n_pairs) return t;
    const int64_t rem = n_tiles % n_pairs;
    if (rem == 0 || rem > n_pairs / 2 || steps < 16) return t;
    int64_t parts = n_pairs / rem;
    if (parts > steps / 8) parts = steps / 8;             // at least 8 stages (K = 1024) per part
    if (parts > 16) parts = 16;
    if (parts < 2) return t;
    t.rem = (int)rem;
    t.parts = (int)parts;
    t.n_main = n_tiles - rem;
    return t;
}

}  // namespace

size_t gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int sm_count) {
    const size_t required = gemm_required_workspace_bytes(M, N, K, sm_count);
    if (required > 0) return required;
    const TailPlan t = tail_plan(M, N, K, 1, resident_pairs(sm_count));
    return (size_t)t.rem * (size_t)t.parts * (size_t)(2 * BM) * (size_t)BN * sizeof(float);
}

// ---- library-owned split-K scratch --------------------------------------------------
// Scratch for callers that have no way to allocate device memory.  It lives in the library's
// device image: every GPU that loads the library carries these bytes until the process exits.
// The name below is only a host-side handle; the device address is looked up once per device.
__device__ __align__(256) static unsigned char g_static_scratch[kStaticScratchBytes];

int static_scratch(void** ptr, size_t* bytes) {
    static std::mutex mu;
    static void* addr[kMaxDevices] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { set_cuda_error(e, "cudaGetDevice"); return MVUE_ERR_CUDA; }
    if (dev < 0 || dev >= kMaxDevices) return MVUE_ERR_ARCH;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void* q = nullptr;
        e = cudaGetSymbolAddress(&q, g_static_scratch);      // the current device's copy of the array
        if (e != cudaSuccess || !q) { set_cuda_error(e, "cudaGetSymbolAddress"); return MVUE_ERR_CUDA; }
        addr[dev] = q;
    }
    *ptr = addr[dev];
    *bytes = kStaticScratchBytes;
    return MVUE_OK;
}

int fused_split_count(int64_t M, int64_t N, int64_t K, int sm_count) {
    const int64_t blocks = ((M + BM - 1) / BM) * ((N + BN - 1) / BN);
    const int64_t steps = K / BK;
    if (blocks >= sm_count || steps < 8) return 1;
    int64_t splits = sm_count / blocks;
    if (splits > steps / 4) splits = steps / 4;
    if (splits > 64) splits = 64;
    return (int)(splits < 1 ? 1 : splits);
}

size_t fused_workspace_bytes(int64_t M, int64_t N, int64_t K, int sm_count) {
    const int splits = fused_split_count(M, N, K, sm_count);
    return splits > 1 ? (size_t)splits * (size_t)M * (size_t)N * sizeof(float) : 0;
}

template <int NM, int kJoint, int kC>
cudaError_t launch_fused_c(const CUtensorMap& map_b, const FusedParams& fp, dim3 grid, cudaStream_t stream) {
    constexpr unsigned cluster = kC;
    static PerDeviceOnce once;
    const cudaError_t attr_err = once_per_device(once, [](int) {
        return cudaFuncSetAttribute(fused_update_kernel<NM, kJoint, kC>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFSmemBytes);
    });
    if (attr_err != cudaSuccess) return attr_err;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kFThreads, 1, 1);
    cfg.dynamicSmemBytes = kFSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fused_update_kernel<NM, kJoint, kC>, map_b, fp);
}
template <int NM, int kJoint>
cudaError_t launch_fused_t(const CUtensorMap& map_b, const FusedParams& fp, dim3 grid, unsigned cluster, cudaStream_t stream) {
    if (cluster == 4) return launch_fused_c<NM, kJoint, 4>(map_b, fp, grid, stream);
    if (cluster == 2) return launch_fused_c<NM, kJoint, 2>(map_b, fp, grid, stream);
    return launch_fused_c<NM, kJoint, 1>(map_b, fp, grid, stream);
}

int launch_fused_update(const FusedArgs& f, cudaStream_t stream) {
    const SparseGemmArgs& a = f.gemm;
    CUtensorMap map_b;
    if (!make_map_2d(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, a.B, (uint64_t)a.N, (uint64_t)a.K,
                     (uint64_t)a.ldb * 2, 64, BK, CU_TENSOR_MAP_SWIZZLE_128B)) {
        set_cuda_error(cudaErrorUnknown, "cuTensorMapEncodeTiled");
        return MVUE_ERR_CUDA;
    }
    const int splits = fused_split_count(a.M, a.N, a.K, a.sm_count);
    const int64_t steps = a.K / BK;
    FusedParams fp;
    fp.g = reinterpret_cast<const uint16_t*>(f.g);
    fp.ldg = f.ldg;
    fp.rk = make_round_keys(f.seed);
    GemmParams& p = fp.gemm;
    p.M = a.M; p.N = a.N; p.K = a.K;
    p.k_steps_per_split = (steps + splits - 1) / splits;
    p.partial = reinterpret_cast<float*>(a.workspace);
    p.C = a.C; p.ldc = a.ldc;
    p.scale = nullptr;
    p.c_is_bf16 = a.c_is_bf16; p.accumulate = a.accumulate; p.splits = splits;
    p.n_work = p.n_main = 0; p.tail_rem = p.tail_splits = 0; p.tail_partial = nullptr;   // pair kernel only
    p.next_values = nullptr; p.next_meta = nullptr; p.next_rk = fp.rk;
    p.dev_status = a.dev_status;
    // blocks whose tiles are neighbours along N share the pruned stage: clusters of 4, 2 or 1 along the first grid axis
    const unsigned tiles_n = (unsigned)((a.N + BN - 1) / BN);
    const unsigned cluster = tiles_n % 4 == 0 ? 4u : (tiles_n % 2 == 0 ? 2u : 1u);
    dim3 grid(tiles_n, (unsigned)((a.M + BM - 1) / BM), (unsigned)splits);
    cudaError_t e;
    if (f.m == 2)          e = launch_fused_t<2, 0>(map_b, fp, grid, cluster, stream);
    else if (f.joint == 1) e = launch_fused_t<4, 1>(map_b, fp, grid, cluster, stream);
    else                   e = launch_fused_t<4, 0>(map_b, fp, grid, cluster, stream);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e == cudaSuccess && splits > 1) {
        const int64_t total = a.M * (a.N / 4);
        const int64_t want = (total + 255) / 256;
        const int blocks = (int)(want < (int64_t)a.sm_count * 8 ? want : (int64_t)a.sm_count * 8);
        splitk_reduce_kernel<<<blocks, 256, 0, stream>>>(p.partial, splits, a.M, a.N, a.C, a.ldc, nullptr,
                                                         a.c_is_bf16, a.accumulate);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) { set_cuda_error(e, "fused update launch"); return MVUE_ERR_CUDA; }
    return MVUE_OK;
}

int launch_sparse_mma_probe(int iters, uint32_t spin_limit, int sm_count, int* pairs_out, int* dev_status,
                            cudaStream_t stream) {
    static PerDeviceOnce once;
    const cudaError_t attr_err = once_per_device(once, [](int) {
        return cudaFuncSetAttribute(sparse_mma_issue_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    });
    if (attr_err != cudaSuccess) { set_cuda_error(attr_err, "cudaFuncSetAttribute"); return MVUE_ERR_CUDA; }
    const int pairs = resident_pairs(sm_count);
    if (pairs_out) *pairs_out = pairs;
    // the product kernel's shared-memory request, so that one block lands on each SM as it does there
    sparse_mma_issue_probe_kernel<<<dim3((unsigned)(2 * pairs)), 128, kSmemBytes, stream>>>(
        iters, spin_limit == 0 ? kSpinLimit : spin_limit, dev_status);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e, "sparse MMA probe launch"); return MVUE_ERR_CUDA; }
    return MVUE_OK;
}

int launch_sparse_gemm(const SparseGemmArgs& a, cudaStream_t stream) {
    CUtensorMap map_a, map_b, map_e;
    const uint64_t e_blocks = (uint64_t)((a.M + BM - 1) / BM) * (uint64_t)(a.K / BK);
    if (!make_map_2d(&map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, a.values, (uint64_t)(a.K / 2), (uint64_t)a.M,
                     (uint64_t)(a.K / 2) * 2, BK / 2, BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, a.B, (uint64_t)a.N, (uint64_t)a.K,
                     (uint64_t)a.ldb * 2, 64, BK, CU_TENSOR_MAP_SWIZZLE_128B) ||
        // metadata blocks of 2 KiB seen as 8 rows of 256 bytes
        !make_map_2d(&map_e, CU_TENSOR_MAP_DATA_TYPE_UINT8, a.meta, 256, e_blocks * 8, 256, 256, 8,
                     CU_TENSOR_MAP_SWIZZLE_NONE)) {
        set_cuda_error(cudaErrorUnknown, "cuTensorMapEncodeTiled");
        return MVUE_ERR_CUDA;
    }
    const cudaError_t setup_err = pair_kernel_setup();
    if (setup_err != cudaSuccess) { set_cuda_error(setup_err, "cudaFuncSetAttribute"); return MVUE_ERR_CUDA; }

    const int splits = gemm_split_count(a.M, a.N, a.K, a.sm_count);
    const int64_t steps = a.K / BK;
    GemmParams p;
    p.M = a.M; p.N = a.N; p.K = a.K;
    p.k_steps_per_split = (steps + splits - 1) / splits;
    p.partial = reinterpret_cast<float*>(a.workspace);
    p.C = a.C; p.ldc = a.ldc;
    p.scale = reinterpret_cast<const __nv_bfloat16*>(a.scale);
    p.c_is_bf16 = a.c_is_bf16; p.accumulate = a.accumulate; p.splits = splits;
    p.dev_status = a.dev_status;
    p.next_values = reinterpret_cast<uint4*>(a.next_values);
    p.next_meta = reinterpret_cast<uint8_t*>(a.next_meta);
    p.next_rk = make_round_keys(a.next_seed);
    const int resident = resident_pairs(a.sm_count);
    TailPlan tail = tail_plan(a.M, a.N, a.K, splits, resident);
    const size_t tail_bytes = (size_t)tail.rem * (size_t)tail.parts * (size_t)(2 * BM) * (size_t)BN * sizeof(float);
    // the tail split needs fp32 output and room for its partial tiles; without either the tiles simply stay whole
    if (tail.parts < 2 || a.c_is_bf16 || a.workspace == nullptr || a.workspace_bytes < tail_bytes) {
        tail = TailPlan();
        tail.n_main = ((a.M + 2 * BM - 1) / (2 * BM)) * ((a.N + BN - 1) / BN) * splits;
    }
    p.n_main = tail.n_main;
    p.tail_rem = tail.rem;
    p.tail_splits = tail.parts;
    p.tail_partial = reinterpret_cast<float*>(a.workspace);
    p.n_work = tail.n_main + (int64_t)tail.rem * tail.parts;
    int64_t n_pairs = resident;
    if (n_pairs > p.n_work) n_pairs = p.n_work;
    if (n_pairs < 1) n_pairs = 1;
    dim3 grid((unsigned)(2 * n_pairs), 1u, 1u);
    const bool scaled = p.scale != nullptr && splits == 1, to_bf16 = p.c_is_bf16 && splits == 1;
    // main loops of at least 32 stages (K = 4096) per work item: the small-footprint epilogue costs nothing there
    const int64_t item_steps = tail.parts > 1 ? steps / tail.parts : p.k_steps_per_split;
    const bool long_items = item_steps >= 32;
    using PairKernel = void (*)(CUtensorMap, CUtensorMap, CUtensorMap, GemmParams);
    PairKernel kernel;
    if (a.next_values != nullptr) {
        if (!(scaled && to_bf16)) return MVUE_ERR_SHAPE;         // (the caller routes split products elsewhere)
        kernel = a.next_joint == 1 ? (a.next_eps16 ? sparse_gemm_pair_kernel<7> : sparse_gemm_pair_kernel<5>)
                                   : (a.next_eps16 ? sparse_gemm_pair_kernel<8> : sparse_gemm_pair_kernel<6>);
    } else {
        kernel = scaled && to_bf16 ? sparse_gemm_pair_kernel<2>
               : scaled            ? sparse_gemm_pair_kernel<3>
               : to_bf16           ? sparse_gemm_pair_kernel<1>
               : long_items        ? sparse_gemm_pair_kernel<4> : sparse_gemm_pair_kernel<0>;
    }
    cudaError_t e = launch_dependent(kernel, grid, dim3(kThreads), kSmemBytes, stream, map_a, map_b, map_e, p);
    if (e == cudaSuccess && tail.parts > 1) {
        e = launch_dependent(tail_reduce_kernel, dim3((unsigned)(tail.rem * 2 * BM)), dim3(BN / 4), 0, stream,
                             p.tail_partial, tail.rem, tail.parts, tail.n_main, a.M, a.N, reinterpret_cast<float*>(a.C),
                             a.ldc, reinterpret_cast<const __nv_bfloat16*>(a.scale), a.accumulate);
    }
    if (e == cudaSuccess && splits > 1) {
        const int64_t total = a.M * (a.N / 4);
        const int64_t want = (total + 255) / 256;
        const int blocks = (int)(want < (int64_t)a.sm_count * 8 ? want : (int64_t)a.sm_count * 8);
        e = launch_dependent(splitk_reduce_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, p.partial, splits, a.M,
                             a.N, a.C, a.ldc, p.scale, a.c_is_bf16, a.accumulate);
    }
    if (e != cudaSuccess) { set_cuda_error(e, "sparse GEMM launch"); return MVUE_ERR_CUDA; }
    return MVUE_OK;
}

}  // namespace mvue
