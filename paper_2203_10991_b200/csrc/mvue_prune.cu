// MVUE N:M prune + pack kernels (memory-bound: one pass over g, packed bf16
// survivors and 2-bit position metadata written in the same pass).
//
// Work unit: 16 consecutive elements along the pruned axis K.  For 2:4 that is
// four blocks sharing one generator call; for 1:2 it is eight pairs using two.
//   axis 1 (K contiguous in memory): one thread owns one unit = 32 contiguous
//           bytes of bf16 (64 of fp32); a warp reads 1 KiB (2 KiB) contiguous.
//   axis 0 (K runs down the rows of g): bf16 tiles arrive by TMA and are handed to
//           the lanes transposed (one lane = 16 rows of one column); binary32 is read
//           with plain loads, one lane owning a strip of 16 rows by two columns.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstring>
#include <mutex>

#include "mvue_device.cuh"
#include "mvue_internal.h"
#include "mvue_tma.h"

namespace mvue {
namespace {

__device__ __forceinline__ uint4 ldg128(const void* p) {
    return __ldg(reinterpret_cast<const uint4*>(p));
}

// One work unit of binary32 input: b[16] = bit patterns of 16 elements along K.
template <int M, int kJoint = 0, bool kSR = false, bool kEps16 = false>
__device__ __forceinline__ void prune_unit_f32(const uint32_t (&b)[16], uint64_t unit_index,
                                               const RoundKeys& rk, uint4* out_values,
                                               uint32_t* out_meta) {
    constexpr int kW = UnitWords<M, kJoint>::kCount;
    uint32_t v[4];
    uint32_t meta = 0;
    uint32_t rnd[4] = {0u, 0u, 0u, 0u};              // stochastic rounding: 16 bits per survivor slot, stream 1 of the unit
    if (kSR) {
        const uint4 r = philox4x32_10(unit_index, rk, 1u);
        rnd[0] = r.x; rnd[1] = r.y; rnd[2] = r.z; rnd[3] = r.w;
    }
    uint32_t words[kW];
    unit_words<kW, kEps16>(unit_index, rk, words);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint32_t nib;
        if (M == 4 && kJoint == 3) {
            mvue_1of4_f32<kSR>(b[4 * j], b[4 * j + 1], b[4 * j + 2], b[4 * j + 3], words[j], &v[j], &nib, rnd[j]);
        } else if (M == 4 && kJoint == 2) {
            mvue_2of4_approx_f32<kSR>(b[4 * j], b[4 * j + 1], b[4 * j + 2], b[4 * j + 3], words[(2 * j) % kW],
                                      words[(2 * j + 1) % kW], &v[j], &nib, rnd[j]);
        } else if (M == 4 && kJoint == 1) {
            mvue_2of4_sys_f32<kSR>(b[4 * j], b[4 * j + 1], b[4 * j + 2], b[4 * j + 3], words[j], &v[j], &nib, rnd[j]);
        } else if (M == 4) {
            mvue_2of4_f32<kSR>(b[4 * j], b[4 * j + 1], b[4 * j + 2], b[4 * j + 3], words[j], &v[j], &nib, rnd[j]);
        } else {
            float v0, v1;
            const bool k0 = mvue_1of2(__uint_as_float(b[4 * j]), __uint_as_float(b[4 * j + 1]), words[(2 * j) % kW], &v0);
            const bool k1 = mvue_1of2(__uint_as_float(b[4 * j + 2]), __uint_as_float(b[4 * j + 3]), words[(2 * j + 1) % kW], &v1);
            v[j] = pack_out<kSR>(v0, v1, rnd[j]);
            nib = (k0 ? 0u : 1u) | (k1 ? 8u : 12u);
        }
        meta |= nib << (4 * j);
    }
    *out_values = make_uint4(v[0], v[1], v[2], v[3]);
    *out_meta = meta;
}

// ---- axis 1 ---------------------------------------------------------------
// K is contiguous: a unit is 32 contiguous bytes of bf16 (64 of binary32).  A thread block owns 16 rows of A
// by 16 units; thread = (row % 8, unit) and handles rows r and r + 8 of its unit, whose 16-bit nibble strings
// share one 32-bit word in the tensor-core order.  A warp reads full 128-byte lines (8 rows x 4 units) and no
// index needs a division.
constexpr int kA1Units = 16;                          // units per block along K

// 32 bytes in one load where the address allows (whole sectors, nothing kept in L1), else two 16-byte loads.
__device__ __forceinline__ void ldg256(const char* p, uint32_t (&v)[8]) {
    if ((reinterpret_cast<uintptr_t>(p) & 31u) == 0) {
        asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                     : "l"(p));
    } else {
        const uint4 a = ldg128(p), b = ldg128(p + 16);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    }
}

template <int M, bool kBf16, bool kTC, int kJoint, bool kSR, bool kEps16>
__global__ void __launch_bounds__(8 * kA1Units, kBf16 ? 12 : 8)
prune_axis1_kernel(const void* __restrict__ g, int64_t n_rows, int units_per_row, int64_t ld,
                   int64_t units_per_row_total, int64_t unit_offset, RoundKeys rk,
                   uint4* __restrict__ values, uint16_t* __restrict__ meta) {
    grid_dependency_wait();
    const int j = threadIdx.x & 7;
    const int c = blockIdx.y * kA1Units + (threadIdx.x >> 3);
    if (c >= units_per_row) return;
    const int64_t r0 = (int64_t)blockIdx.x * 16 + j;
    uint32_t meta_pair = 0;
    if (kBf16) {
        // The short selections (1:2, 1:4) are bound by bytes in flight: both rows' units are requested before either
        // is pruned (64 bytes per thread).  The 2:4 selections are bound by instruction issue at 40 registers and
        // keep the second row's load behind the first row's arithmetic.
        constexpr bool kBothFirst = M == 2 || kJoint == 3;
        uint32_t raw[2][8];
        if (kBothFirst) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int64_t r = r0 + 8 * h;
                if (r < n_rows) {
                    ldg256(reinterpret_cast<const char*>(g) + (r * ld + (int64_t)c * 16) * 2, raw[h]);
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) raw[h][i] = 0u;
                }
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int64_t r = r0 + 8 * h;
            uint32_t mt = 0x4444u;                    // rows that pad A to a multiple of 128 keep a valid pattern
            if (r < n_rows) {
                if (!kBothFirst) ldg256(reinterpret_cast<const char*>(g) + (r * ld + (int64_t)c * 16) * 2, raw[h]);
                const uint64_t unit = (uint64_t)r * (uint64_t)units_per_row_total + (uint64_t)(unit_offset + c);
                uint4 v;
                prune_unit_bf16<M, kJoint, kSR, kEps16>(raw[h], unit, rk, &v, &mt);
                values[r * units_per_row + c] = v;
                if (!kTC) meta[r * units_per_row + c] = (uint16_t)mt;
            }
            meta_pair |= mt << (16 * h);
        }
    } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int64_t r = r0 + 8 * h;
            uint32_t mt = 0x4444u;
            if (r < n_rows) {
                const char* p = reinterpret_cast<const char*>(g) + (r * ld + (int64_t)c * 16) * 4;
                uint32_t lo[8], hi[8];
                ldg256(p, lo);
                ldg256(p + 32, hi);
                const uint32_t b[16] = {lo[0], lo[1], lo[2], lo[3], lo[4], lo[5], lo[6], lo[7],
                                        hi[0], hi[1], hi[2], hi[3], hi[4], hi[5], hi[6], hi[7]};
                const uint64_t unit = (uint64_t)r * (uint64_t)units_per_row_total + (uint64_t)(unit_offset + c);
                uint4 v;
                prune_unit_f32<M, kJoint, kSR, kEps16>(b, unit, rk, &v, &mt);
                values[r * units_per_row + c] = v;
                if (!kTC) meta[r * units_per_row + c] = (uint16_t)mt;
            }
            meta_pair |= mt << (16 * h);
        }
    }
    if (kTC)   // (r0, c) is the low half of its word; r0 % 16 < 8
        *reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(meta) + tc_meta_offset(r0, c, units_per_row >> 3)) = meta_pair;
}

// ---- axis 1, bf16, whole blocks ---------------------------------------------------
// For tensors whose rows are a multiple of 16 and whose K is a multiple of 512 elements, 32-byte aligned (the packed
// operands of the backward products); a narrower K of 32, 64, 128 or 256 elements is taken too, the block then owning
// 16, 8, 4 or 2 groups of 16 rows (`pair_shift` = log2 of the unit pairs of a row that one block covers, 4 for wide K).
// A thread block owns 16 rows of A by 32 units; thread = (row % 8, unit pair)
// handles the two consecutive units 2 c, 2 c + 1 of rows r and r + 8: 64 contiguous bytes per row (both rows requested
// before either is pruned), a 32-byte store of survivors per row, two whole metadata words in tensor-core order.  No
// bounds checks, half the addressing per unit, and with sixteen bits per block the two units of a row share one
// generator call.  A warp reads 8 rows x 256 contiguous bytes.
constexpr int kA1PairsPerBlock = 16;

__device__ __forceinline__ void ldg256_aligned(const char* p, uint32_t (&v)[8]) {
    asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "l"(p));
}

// Resident blocks per SM: eight (64 registers) where the arithmetic is short enough to fit them without spills that
// cost more than the extra warps bring; six for the App. A.2 table and for 1:2 with its two generator calls per unit.
template <int M, int kJoint, bool kEps16>
constexpr int a1_pairs_min_blocks() { return ((M == 4 && kJoint == 0) || (M == 2 && !kEps16)) ? 6 : 8; }

template <int M, bool kTC, int kJoint, bool kSR, bool kEps16>
__global__ void __launch_bounds__(8 * kA1PairsPerBlock, a1_pairs_min_blocks<M, kJoint, kEps16>())
prune_axis1_bf16_pairs_kernel(const void* __restrict__ g, int units_per_row, int64_t ld, int64_t units_per_row_total,
                              int64_t unit_offset, RoundKeys rk, uint4* __restrict__ values, uint16_t* __restrict__ meta,
                              int pair_shift) {
    grid_dependency_wait();
    const int j = threadIdx.x & 7, q = threadIdx.x >> 3;
    const int c = 2 * (blockIdx.y * kA1PairsPerBlock + (q & ((1 << pair_shift) - 1)));   // first unit of the pair
    const int64_t r0 = ((((int64_t)blockIdx.x) << (4 - pair_shift)) + (q >> pair_shift)) * 16 + j;
    uint32_t raw[2][2][8];                                                    // [row h][unit][8 words]
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const char* p = reinterpret_cast<const char*>(g) + ((r0 + 8 * h) * ld + (int64_t)c * 16) * 2;
        ldg256_aligned(p, raw[h][0]);
        ldg256_aligned(p + 32, raw[h][1]);
    }
    uint32_t meta_pair[2] = {0u, 0u};                                         // unit 2 c and 2 c + 1: rows r (low), r + 8 (high)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int64_t r = r0 + 8 * h;
        const uint64_t unit = (uint64_t)r * (uint64_t)units_per_row_total + (uint64_t)(unit_offset + c);
        uint4 v[2];
        uint32_t mt[2];
        if (kEps16 && UnitWords<M, kJoint>::kCount == 4) {                    // unit is even: the two units share one call
            uint32_t w0[4], w1[4];
            unit_pair_words16(unit, rk, w0, w1);
            prune_unit_bf16_w<M, kJoint, kSR>(raw[h][0], reinterpret_cast<const uint32_t (&)[UnitWords<M, kJoint>::kCount]>(w0),
                                              unit, rk, &v[0], &mt[0]);
            prune_unit_bf16_w<M, kJoint, kSR>(raw[h][1], reinterpret_cast<const uint32_t (&)[UnitWords<M, kJoint>::kCount]>(w1),
                                              unit + 1, rk, &v[1], &mt[1]);
        } else {
#pragma unroll
            for (int e = 0; e < 2; ++e) prune_unit_bf16<M, kJoint, kSR, kEps16>(raw[h][e], unit + e, rk, &v[e], &mt[e]);
        }
        uint4* dst = values + r * units_per_row + c;
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                     ::"l"(dst), "r"(v[0].x), "r"(v[0].y), "r"(v[0].z), "r"(v[0].w), "r"(v[1].x), "r"(v[1].y),
                       "r"(v[1].z), "r"(v[1].w) : "memory");
        if (!kTC) *reinterpret_cast<uint32_t*>(meta + r * units_per_row + c) = mt[0] | (mt[1] << 16);
        meta_pair[0] |= mt[0] << (16 * h);
        meta_pair[1] |= mt[1] << (16 * h);
    }
    if (kTC) {
        char* base = reinterpret_cast<char*>(meta);
        *reinterpret_cast<uint32_t*>(base + tc_meta_offset(r0, c, units_per_row >> 3)) = meta_pair[0];
        *reinterpret_cast<uint32_t*>(base + tc_meta_offset(r0, c + 1, units_per_row >> 3)) = meta_pair[1];
    }
}

// ---- axis 0 ---------------------------------------------------------------
// g is [K x C] row-major; A = g^T.  A thread block owns a tile of 256 rows (16
// strips of 16, one warp per strip) by 64 columns (two per lane).  Each lane reads
// its two columns of every row of the strip (a warp reads one 128-byte line of
// bf16, two of binary32, per row), prunes both columns, and stages the packed
// outputs in shared memory (values: per column 16 slots of 16 bytes, slot index
// XOR lane to avoid bank conflicts; metadata: per column 16 x 2 bytes) so that
// the tile leaves as contiguous runs of 256 / 32 bytes per column of g.
constexpr int kTileStrips = 16;
constexpr int kTileCols = 64;
constexpr int kMetaPitch = 36;                       // bytes per staged metadata row

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// (Used for binary32 input; bf16 input takes prune_axis0_bf16_kernel below.)
template <int M, bool kBf16, bool kTC, int kJoint, bool kSR, bool kEps16>
__global__ void __launch_bounds__(kTileStrips * 32, kBf16 ? 3 : 2)
prune_axis0_kernel(const void* __restrict__ g, int64_t n_strips, int64_t n_cols, int64_t ld,
                   int64_t units_per_row_total, int64_t unit_offset, RoundKeys rk,
                   uint4* __restrict__ values, uint16_t* __restrict__ meta) {
    grid_dependency_wait();
    constexpr int ES = kBf16 ? 2 : 4;
    constexpr int NT = kTileStrips * 32;
    __shared__ uint4 s_val[kTileCols * kTileStrips];
    __shared__ __align__(16) unsigned char s_meta[kTileCols * kMetaPitch];   // >= 2048 bytes

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int strip_l = tid >> 5;
    const int64_t strip0 = (int64_t)blockIdx.x * kTileStrips;
    const int64_t col0 = (int64_t)blockIdx.y * kTileCols;
    const int64_t strip = strip0 + strip_l;
    const int64_t col = col0 + 2 * lane;             // this lane's first column (n_cols is even)
    if (kTC) {                                       // padding rows of A keep a valid pattern
        for (int i = tid; i < 2048 / 4; i += NT) reinterpret_cast<uint32_t*>(s_meta)[i] = 0x44444444u;
    }
    if (kTC) __syncthreads();

    if (strip < n_strips && col < n_cols) {
        const char* p = reinterpret_cast<const char*>(g) + ((strip * 16) * ld + col) * ES;
        uint32_t w[16][kBf16 ? 1 : 2];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            if (kBf16) {
                w[i][0] = __ldg(reinterpret_cast<const uint32_t*>(p + (int64_t)i * ld * ES));
            } else {
                const uint2 t = __ldg(reinterpret_cast<const uint2*>(p + (int64_t)i * ld * ES));
                w[i][0] = t.x;
                w[i][kBf16 ? 0 : 1] = t.y;
            }
        }
        const uint64_t unit_base = (uint64_t)(unit_offset + strip);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int col_l = 2 * lane + e;          // column inside the tile = row of A
            const uint64_t unit = (uint64_t)(col + e) * (uint64_t)units_per_row_total + unit_base;
            uint4 v;
            uint32_t mt;
            if (kBf16) {
                uint32_t rw[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) rw[i] = w[i][0];
                if (e == 0) prune_unit_bf16_rows<M, false, kJoint>(rw, unit, rk, &v, &mt);
                else        prune_unit_bf16_rows<M, true, kJoint>(rw, unit, rk, &v, &mt);
            } else {
                uint32_t b[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) b[i] = w[i][kBf16 ? 0 : e];
                prune_unit_f32<M, kJoint, kSR, kEps16>(b, unit, rk, &v, &mt);
            }
            s_val[col_l * kTileStrips + (strip_l ^ (lane & 15))] = v;
            if (kTC) {
                // staged as [k-block 0/1][lane of this 64-row quarter x2][16 bytes], ready to leave as 1 KiB runs
                const int tc_lane = (col_l & 7) + 8 * (strip_l & 1) + 16 * (col_l >> 4);
                const int off = (strip_l >> 3) * 1024 + tc_lane * 16 + ((strip_l & 7) >> 1) * 4 + ((col_l >> 3) & 1) * 2;
                *reinterpret_cast<uint16_t*>(&s_meta[off]) = (uint16_t)mt;
            } else {
                *reinterpret_cast<uint16_t*>(&s_meta[col_l * kMetaPitch + strip_l * 2]) = (uint16_t)mt;
            }
        }
    }
    __syncthreads();

    const int64_t strips_here = n_strips - strip0 < kTileStrips ? n_strips - strip0 : kTileStrips;
    // values: 64 columns x 16 slots of 16 bytes; 16 consecutive threads write one column's run
#pragma unroll
    for (int it = 0; it < kTileCols * kTileStrips / NT; ++it) {
        const int idx = it * NT + tid;
        const int col_l = idx >> 4, j = idx & 15;
        const int64_t c = col0 + col_l;
        if (j < strips_here && c < n_cols)
            values[c * n_strips + strip0 + j] = s_val[col_l * kTileStrips + (j ^ ((col_l >> 1) & 15))];
    }
    if (kTC) {
        // metadata: per 128-k block one contiguous 1 KiB run (64 rows x 16 bytes of lanes)
        if (tid < 128) {
            const int kb = tid >> 6;
            if (8 * kb < strips_here) {
                const int64_t block = (col0 >> 7) * (n_strips >> 3) + (strip0 >> 3) + kb;
                char* dst = reinterpret_cast<char*>(meta) + block * 2048 + ((col0 & 64) ? 1024 : 0) + (tid & 63) * 16;
                *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(&s_meta[kb * 1024 + (tid & 63) * 16]);
            }
        }
    } else {
        // metadata: 64 columns x 32 bytes; 8 consecutive threads write one column's run as words
        const int col_l = tid >> 3, wd = tid & 7;
        const int64_t c = col0 + col_l;
        if (c < n_cols) {
            const uint32_t word = *reinterpret_cast<const uint32_t*>(&s_meta[col_l * kMetaPitch + wd * 4]);
            uint16_t* dst = meta + c * n_strips + strip0 + 2 * wd;
            const bool word_ok = (reinterpret_cast<uintptr_t>(dst) & 3u) == 0;   // odd K/16 misaligns rows
            if (2 * wd + 1 < strips_here && word_ok) {
                *reinterpret_cast<uint32_t*>(dst) = word;
            } else {
                if (2 * wd < strips_here) dst[0] = (uint16_t)word;
                if (2 * wd + 1 < strips_here) dst[1] = (uint16_t)(word >> 16);
            }
        }
    }
}

// ---- axis 0, bf16 -----------------------------------------------------------
// A thread block owns a tile of kStrips strips of 16 rows of g by 64 columns, one warp per strip.  The tile
// arrives by ONE TMA box copy through the 4-D view of make_map_strips, which lays it out so that two
// transposing 8x8 matrix loads hand a lane the 16 consecutive rows of one column as eight words of two bf16
// -- exactly the form a unit has when K is contiguous -- with no bank conflict, no byte shuffles and no
// address arithmetic per element.  A warp covers 4 strips x 8 columns per step (lane = 4 (column % 8) +
// strip % 4) and takes two steps whose columns are 8 apart, so in the tensor-core order the two 16-bit nibble
// strings of a lane share one 32-bit word.  Packed survivors go straight from registers to memory: the four
// lanes of a column write 64 contiguous bytes.  Small tiles (4 strips, two warps, 24 blocks per SM) keep
// the copy of one block hidden behind the arithmetic of the others.
constexpr int kA0Cols = 64;
template <int kStrips, int kWarps> struct A0 {                   // kStrips: strips of 16 rows per tile (4, 8 or 16)
    static constexpr int kRows = 16 * kStrips, kThreads = 32 * kWarps;
    static constexpr int kTileBytes = kRows * kA0Cols * 2;
    static constexpr int kSmemBytes = kTileBytes + 1024 + 16;     // alignment slack + one mbarrier
    static constexpr int kBlocksPerSM = 1536 / kThreads < 24 ? 1536 / kThreads : 24;
};

// Plain-load replacement of the box copy (same shared-memory arrangement), used only if the copy never landed.
template <int kStrips, int kWarps>
__device__ __noinline__ void fill_tile_bf16(const char* g, int64_t ld, int64_t n_rows, int64_t n_cols, int64_t row0,
                                            int64_t col0, unsigned char* tile) {
    for (int i = threadIdx.x; i < A0<kStrips, kWarps>::kRows * 8; i += A0<kStrips, kWarps>::kThreads) {   // 16-byte chunks
        const int line = i >> 3, chunk = i & 7;
        const int k8 = line / (2 * kStrips), strip = (line >> 1) % kStrips, k2 = line & 1;
        const int64_t r = row0 + 16 * strip + 2 * k8 + k2, c = col0 + 8 * chunk;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (r < n_rows && c < n_cols) v = ldg128(g + (r * ld + c) * 2);     // n_cols is a multiple of 8
        *reinterpret_cast<uint4*>(tile + line * 128 + ((chunk ^ (line & 7)) << 4)) = v;
    }
}

template <int M, bool kTC, int kJoint, bool kSR, bool kEps16, int kStrips, int kWarps>
__global__ void __launch_bounds__(32 * kWarps, A0<kStrips, kWarps>::kBlocksPerSM)
prune_axis0_bf16_kernel(const __grid_constant__ CUtensorMap map_g, const void* __restrict__ g, int64_t n_strips,
                        int64_t n_cols, int64_t ld, int64_t units_per_row_total, int64_t unit_offset, RoundKeys rk,
                        uint4* __restrict__ values, uint16_t* __restrict__ meta) {
    grid_dependency_wait();
    constexpr int kTileBytes = A0<kStrips, kWarps>::kTileBytes;
    constexpr int kQuads = kStrips / 4;                                      // groups of 4 strips per tile
    constexpr int kPairStride = kWarps / kQuads;                             // warps that share a group of 4 strips
    static_assert(kWarps % kQuads == 0 && 4 % kPairStride == 0, "warps must tile the 4 x kQuads steps");
    extern __shared__ unsigned char s_raw[];
    const uint32_t tile = (smem_addr(s_raw) + 1023u) & ~1023u;              // the 128-byte swizzle needs 1 KiB alignment
    const uint32_t bar = tile + kTileBytes;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t strip0 = (int64_t)blockIdx.x * kStrips;
    const int64_t col0 = (int64_t)blockIdx.y * kA0Cols;
    const bool has_input = col0 < n_cols;                                    // false only for tiles that pad A's rows

    if (has_input) {
        if (tid == 0) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kTileBytes) : "memory");
            asm volatile(
                "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
                ::"r"(tile), "l"(&map_g), "r"((int)col0), "r"(0), "r"((int)strip0), "r"(0), "r"(bar) : "memory");
        }
        __syncthreads();
        bool landed = false;
        for (uint32_t spin = 0; spin < (1u << 20) && !landed; ++spin) {      // bounded wait
            uint32_t ok;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\t"
                         "selp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(bar) : "memory");
            landed = ok != 0;
        }
        if (__syncthreads_or(!landed)) {
            fill_tile_bf16<kStrips, kWarps>(reinterpret_cast<const char*>(g), ld, n_strips * 16, n_cols, strip0 * 16, col0,
                                    s_raw + (tile - smem_addr(s_raw)));
            __syncthreads();
        }
    }

    // this lane's units: strip = strip0 + 4 (warp % kQuads) + lane % 4; columns col0 + 16 pair + lane / 4 and
    // + 8, for pair = warp / kQuads, + kPairStride, ... < 4
    const int quad = warp % kQuads, p = lane & 3;
    const int64_t strip = strip0 + 4 * quad + p;
    const bool strip_ok = strip < n_strips;
    // address this lane supplies to the matrix loads: matrix lane / 8 (= k8, +4 for the second load), line lane % 8
    const uint32_t ld_base = tile + (uint32_t)(((lane >> 3) * (2 * kStrips) + 8 * quad + (lane & 7)) * 128);
#pragma unroll
    for (int pair = warp / kQuads; pair < 4; pair += kPairStride) {
        uint32_t meta_pair = 0;
#pragma unroll
        for (int step = 0; step < 2; ++step) {
            const int cb = 2 * pair + step;                                  // 8-column block inside the tile
            const int64_t c = col0 + 8 * cb + (lane >> 2);
            uint32_t mt = 0x4444u;                                           // rows that pad A keep a valid pattern
            if (has_input) {
                const uint32_t addr = ld_base + (uint32_t)((cb ^ (lane & 7)) << 4);
                uint32_t raw[8];
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                             : "=r"(raw[0]), "=r"(raw[1]), "=r"(raw[2]), "=r"(raw[3]) : "r"(addr));
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                             : "=r"(raw[4]), "=r"(raw[5]), "=r"(raw[6]), "=r"(raw[7])
                             : "r"(addr + 4u * (2 * kStrips) * 128u));
                if (strip_ok && c < n_cols) {
                    const uint64_t unit = (uint64_t)c * (uint64_t)units_per_row_total + (uint64_t)(unit_offset + strip);
                    uint4 v;
                    prune_unit_bf16<M, kJoint, kSR, kEps16>(raw, unit, rk, &v, &mt);
                    values[c * n_strips + strip] = v;
                    if (!kTC) meta[c * n_strips + strip] = (uint16_t)mt;
                }
            }
            meta_pair |= mt << (16 * step);
        }
        if (kTC && strip_ok) {
            // rows c and c + 8 share the 32-bit word (k % 128) / 32 of lane c % 8 + 8 (strip % 2) + 16 (c % 128 / 16)
            const int64_t c = col0 + 16 * pair + (lane >> 2);
            const int rl = (int)(c & 127);
            const int tc_lane = (rl & 7) + 8 * (p & 1) + 16 * (rl >> 4);
            const int64_t block = (c >> 7) * (n_strips >> 3) + (strip >> 3);
            const int word = 2 * ((int)(strip >> 2) & 1) + (p >> 1);
            *reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(meta) + block * 2048 + tc_lane * 16 + word * 4) = meta_pair;
        }
    }
}

// ---- axis 0, bf16, whole tiles ------------------------------------------------
// For tensors made of whole tiles of 128 rows x 64 columns (every packed operand in tensor-core order is: K is a multiple
// of 128 there).  One TMA box copy through the 5-D view of make_map_strip_pairs; four warps, warp w owns the 16 columns
// 16 w .. 16 w + 15 of the tile, lane l the columns 16 w + l / 4 and + 8 and, of each, the two consecutive strips
// 2 (l % 4) and 2 (l % 4) + 1 of the tile's eight: four units per lane, the two strips of a column leave as ONE 32-byte
// store of survivors, and rows c and c + 8 of A share their metadata words as in the kernel above.  Against that kernel:
// half as many blocks, barriers and copies per byte, no bounds checks, and the addressing of a unit pair shared.
constexpr int kWTRows = 128, kWTCols = 64, kWTBytes = kWTRows * kWTCols * 2, kWTWarps = 4;

template <int kDummy>
__device__ __noinline__ void fill_whole_tile_bf16(const char* g, int64_t ld, int64_t row0, int64_t col0, unsigned char* tile) {
    for (int i = threadIdx.x; i < kWTRows * 8; i += 32 * kWTWarps) {         // 16-byte chunks; line = 16 k8 + 8 h + 2 pair + k2
        const int line = i >> 3, chunk = i & 7;
        const int k8 = line >> 4, h = (line >> 3) & 1, pair = (line >> 1) & 3, k2 = line & 1;
        const int64_t r = row0 + 32 * pair + 16 * h + 2 * k8 + k2, c = col0 + 8 * chunk;
        *reinterpret_cast<uint4*>(tile + line * 128 + ((chunk ^ (line & 7)) << 4)) = ldg128(g + (r * ld + c) * 2);
    }
}

template <int M, bool kTC, int kJoint, bool kSR, bool kEps16>
__global__ void __launch_bounds__(32 * kWTWarps, 12)
prune_axis0_bf16_whole_tiles_kernel(const __grid_constant__ CUtensorMap map_g, const void* __restrict__ g, int64_t n_strips,
                                    int64_t ld, int64_t units_per_row_total, int64_t unit_offset, RoundKeys rk,
                                    uint4* __restrict__ values, uint16_t* __restrict__ meta, int walk) {
    grid_dependency_wait();
    __shared__ __align__(1024) unsigned char s_tile[kWTBytes];                // the 128-byte swizzle needs 1 KiB alignment
    __shared__ __align__(8) uint64_t s_bar;
    const uint32_t tile = smem_addr(s_tile), bar = smem_addr(&s_bar);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // walk < 0: column tiles fastest (a narrow g: the blocks that run together then read whole rows of g between them
    // instead of one 128-byte piece of every row).  walk = s >= 0: groups of 2^s column tiles, column tile fastest
    // inside a group, then row tiles, then groups: the blocks that run together then touch a few hundred 2 MiB pages
    // of g and of the survivors instead of a thousand (row tiles fastest, s = 0, reads 128 rows 8 KiB apart per block
    // and a different megabyte of g in every block: 76 % of the copy bandwidth on a 4 GiB g against 99 % with s = 3)
    const int64_t row_tile = walk < 0 ? blockIdx.y : (blockIdx.x >> walk);
    const int64_t col_tile = walk < 0 ? blockIdx.x : (((int64_t)blockIdx.y << walk) + (blockIdx.x & ((1u << walk) - 1u)));
    const int64_t strip0 = row_tile * 8;
    const int64_t col0 = col_tile * kWTCols;

    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kWTBytes) : "memory");
        asm volatile(
            "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
            ::"r"(tile), "l"(&map_g), "r"((int)col0), "r"(0), "r"((int)(strip0 >> 1)), "r"(0), "r"(0), "r"(bar) : "memory");
    }
    __syncthreads();
    bool landed = false;
    for (uint32_t spin = 0; spin < (1u << 20) && !landed; ++spin) {           // bounded wait
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(bar) : "memory");
        landed = ok != 0;
    }
    if (__syncthreads_or(!landed)) {                                         // the copy never landed: plain loads instead
        fill_whole_tile_bf16<0>(reinterpret_cast<const char*>(g), ld, strip0 * 16, col0, s_tile);
        __syncthreads();
    }

    const int p = lane & 3, cq = lane >> 2;
    // address this lane supplies to the matrix loads: matrix lane / 8 = k8 (+ 4 for the second load), line
    // 16 k8 + 8 h + lane % 8, 16-byte chunk (column block) ^ (lane % 8)
    const uint32_t ld_base = tile + (uint32_t)((16 * (lane >> 3) + (lane & 7)) * 128 + ((lane & 7) << 4));
    const int64_t strip = strip0 + 2 * p;                                    // this lane's first strip (even)
    uint32_t meta_h[2] = {0u, 0u};                                           // strip parity h: rows c (low half) and c + 8 (high)
#pragma unroll
    for (int step = 0; step < 2; ++step) {
        const int cb = 2 * warp + step;                                      // 8-column block inside the tile
        const int64_t c = col0 + 8 * cb + cq;
        const uint64_t unit = (uint64_t)c * (uint64_t)units_per_row_total + (uint64_t)(unit_offset + strip);
        uint32_t raw[2][8];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t addr = (ld_base ^ (uint32_t)(cb << 4)) + (uint32_t)(h * 8 * 128);
            asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                         : "=r"(raw[h][0]), "=r"(raw[h][1]), "=r"(raw[h][2]), "=r"(raw[h][3]) : "r"(addr));
            asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                         : "=r"(raw[h][4]), "=r"(raw[h][5]), "=r"(raw[h][6]), "=r"(raw[h][7]) : "r"(addr + 64u * 128u));
        }
        uint4 v[2];
        uint32_t mt[2];
        if (kEps16 && UnitWords<M, kJoint>::kCount == 4) {    // the lane's two units share one generator call (unit is even)
            uint32_t w0[4], w1[4];
            unit_pair_words16(unit, rk, w0, w1);
            prune_unit_bf16_w<M, kJoint, kSR>(raw[0], reinterpret_cast<const uint32_t (&)[UnitWords<M, kJoint>::kCount]>(w0),
                                              unit, rk, &v[0], &mt[0]);
            prune_unit_bf16_w<M, kJoint, kSR>(raw[1], reinterpret_cast<const uint32_t (&)[UnitWords<M, kJoint>::kCount]>(w1),
                                              unit + 1, rk, &v[1], &mt[1]);
        } else {
#pragma unroll
            for (int h = 0; h < 2; ++h) prune_unit_bf16<M, kJoint, kSR, kEps16>(raw[h], unit + h, rk, &v[h], &mt[h]);
        }
        uint4* dst = values + c * n_strips + strip;                          // 32-byte aligned: n_strips and strip are even
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                     ::"l"(dst), "r"(v[0].x), "r"(v[0].y), "r"(v[0].z), "r"(v[0].w), "r"(v[1].x), "r"(v[1].y),
                       "r"(v[1].z), "r"(v[1].w) : "memory");
        if (!kTC) *reinterpret_cast<uint32_t*>(meta + c * n_strips + strip) = mt[0] | (mt[1] << 16);
        meta_h[0] |= mt[0] << (16 * step);
        meta_h[1] |= mt[1] << (16 * step);
    }
    if (kTC) {
        // rows c and c + 8 share the 32-bit word (k % 128) / 32 = p of lane c % 8 + 8 h + 16 (c % 128 / 16)
        const int64_t c = col0 + 16 * warp + cq;
        const int rl = (int)(c & 127);
        const int64_t block = (c >> 7) * (n_strips >> 3) + (strip0 >> 3);
        char* base = reinterpret_cast<char*>(meta) + block * 2048 + ((rl & 7) + 16 * (rl >> 4)) * 16 + p * 4;
        *reinterpret_cast<uint32_t*>(base) = meta_h[0];
        *reinterpret_cast<uint32_t*>(base + 128) = meta_h[1];
    }
}

// ---- approx-4:8 (prune only) ---------------------------------------------------
// One thread per block of eight.  Row r of A and block j along K; threads run along K for axis 1 (8 contiguous
// elements per thread) and along the rows of A for axis 0 (8 rows of g, neighbouring threads on neighbouring columns),
// so that the loads of a warp coalesce either way.  The arithmetic (93 reciprocals and a few hundred multiply-adds per
// block) is what bounds this kernel, not memory.
template <bool kBf16>
__global__ void __launch_bounds__(128)
prune_4of8_kernel(const void* __restrict__ g, int64_t mrows, int64_t kblocks, int64_t ld, int axis,
                  int64_t kblocks_total, int64_t kblock_offset, RoundKeys rk, uint2* __restrict__ values,
                  uint8_t* __restrict__ mask) {
    const int64_t n = mrows * kblocks;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = axis == 1 ? i / kblocks : i % mrows;
        const int64_t j = axis == 1 ? i % kblocks : i / mrows;
        uint32_t b[8];
        if (axis == 1) {
            if (kBf16) {
                const uint4 x = ldg128(reinterpret_cast<const char*>(g) + (r * ld + 8 * j) * 2);
                const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) { b[2 * e] = w[e] << 16; b[2 * e + 1] = w[e] & 0xFFFF0000u; }
            } else {
                const uint4 x = ldg128(reinterpret_cast<const char*>(g) + (r * ld + 8 * j) * 4);
                const uint4 y = ldg128(reinterpret_cast<const char*>(g) + (r * ld + 8 * j) * 4 + 16);
                b[0] = x.x; b[1] = x.y; b[2] = x.z; b[3] = x.w; b[4] = y.x; b[5] = y.y; b[6] = y.z; b[7] = y.w;
            }
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int64_t off = (8 * j + e) * ld + r;
                b[e] = kBf16 ? (uint32_t)__ldg(reinterpret_cast<const uint16_t*>(g) + off) << 16
                             : __ldg(reinterpret_cast<const uint32_t*>(g) + off);
            }
        }
        const uint64_t q = (uint64_t)r * (uint64_t)kblocks_total + (uint64_t)(kblock_offset + j);
        uint32_t out[2];
        const uint32_t bits = approx_4of8(b, philox4x32_10(q, rk), out);
        values[r * kblocks + j] = make_uint2(out[0], out[1]);
        mask[r * kblocks + j] = (uint8_t)bits;
    }
}

// ---- unpack ---------------------------------------------------------------
// One thread expands one unit: a 16-bit metadata word (four groups) and its 8 survivors
// become 16 dense elements (32 bytes).
template <bool kTC>
__global__ void __launch_bounds__(256)
unpack_kernel(const uint4* __restrict__ values, const uint16_t* __restrict__ meta, int64_t n_units,
              int64_t units_per_row, uint4* __restrict__ dense) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_units; i += stride) {
        uint32_t mw;
        if (kTC) {
            const int64_t r = i / units_per_row, c = i - r * units_per_row;
            mw = *reinterpret_cast<const uint16_t*>(reinterpret_cast<const char*>(meta) +
                                                    tc_meta_offset(r, c, units_per_row >> 3));
        } else {
            mw = meta[i];
        }
        const uint4 v = values[i];
        const uint32_t vw[4] = {v.x, v.y, v.z, v.w};
        uint32_t out[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t i0 = (mw >> (4 * j)) & 3u, i1 = (mw >> (4 * j + 2)) & 3u;
            const uint32_t lo = vw[j] & 0xFFFFu, hi = vw[j] >> 16;
            uint32_t e[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int t = 0; t < 4; ++t) e[t] = (i1 == (uint32_t)t) ? hi : ((i0 == (uint32_t)t) ? lo : 0u);
            out[2 * j] = e[0] | (e[1] << 16);
            out[2 * j + 1] = e[2] | (e[3] << 16);
        }
        dense[2 * i] = make_uint4(out[0], out[1], out[2], out[3]);
        dense[2 * i + 1] = make_uint4(out[4], out[5], out[6], out[7]);
    }
}

template <int M, bool kBf16, bool kTC, int kJoint, bool kSR, bool kEps16>
cudaError_t launch_prune_t(const PruneArgs& a, cudaStream_t stream) {
    const RoundKeys rk = make_round_keys(a.seed);
    const int64_t upr_total = a.k_total / 16, uoff = a.k_offset / 16;
    uint4* values = reinterpret_cast<uint4*>(a.values);
    uint16_t* meta = reinterpret_cast<uint16_t*>(a.meta);
    if (a.axis == 1) {
        const int64_t upr = a.cols / 16;
        // in tensor-core order the rows of A are padded to 128: the blocks past the last row write only metadata
        const int64_t cover_rows = kTC ? ((a.rows + 127) / 128) * 128 : a.rows;
        // whole blocks of 16 rows x 32 units, 32-byte aligned rows and outputs, no padding rows of A to cover, and (for
        // sixteen bits per block) unit pairs that start on even unit numbers: the kernel without bounds checks
        int pair_shift = 4;                                  // unit pairs of a row per block = 2^pair_shift
        if (upr == 2 || upr == 4 || upr == 8 || upr == 16) pair_shift = upr == 2 ? 0 : upr == 4 ? 1 : upr == 8 ? 2 : 3;
        const int64_t rows_per_block = 16 << (4 - pair_shift);
        const bool whole = kBf16 && a.rows % rows_per_block == 0 && upr % (2 << pair_shift) == 0 && cover_rows == a.rows &&
                           (a.ld * 2) % 32 == 0 && reinterpret_cast<uintptr_t>(a.g) % 32 == 0 &&
                           reinterpret_cast<uintptr_t>(a.values) % 32 == 0 &&
                           (!kEps16 || UnitWords<M, kJoint>::kCount != 4 || (uoff % 2 == 0 && upr_total % 2 == 0));
        if (whole) {
            dim3 grid_p((unsigned)(a.rows / rows_per_block), (unsigned)(upr / (2 << pair_shift)));
            launch_dependent(prune_axis1_bf16_pairs_kernel<M, kTC, kJoint, kSR, kEps16>, dim3(grid_p),
                             dim3(8 * kA1PairsPerBlock), 0, stream, a.g, (int)upr, a.ld, upr_total, uoff, rk, values,
                             meta, pair_shift);
        } else {
            dim3 grid((unsigned)((cover_rows + 15) / 16), (unsigned)((upr + kA1Units - 1) / kA1Units));
            launch_dependent(prune_axis1_kernel<M, kBf16, kTC, kJoint, kSR, kEps16>, dim3(grid), dim3(8 * kA1Units),
                             0, stream, a.g, a.rows, (int)upr, a.ld, upr_total, uoff, rk, values, meta);
        }
    } else {
        const int64_t n_strips = a.rows / 16;
        // in tensor-core order the rows of A are padded to 128: cover the padding with (load-free) tiles
        const int64_t cover_cols = kTC ? ((a.cols + 127) / 128) * 128 : a.cols;
        dim3 grid((unsigned)((n_strips + kTileStrips - 1) / kTileStrips),
                  (unsigned)((cover_cols + kTileCols - 1) / kTileCols));
        // whole tiles of 128 rows x 64 columns (and no padding rows of A to cover): the kernel without bounds checks
        // (with sixteen bits per block a lane's two units share a generator call: they must be units 2 i, 2 i + 1)
        const bool pairs_aligned = !kEps16 || UnitWords<M, kJoint>::kCount != 4 || (uoff % 2 == 0 && upr_total % 2 == 0);
        if (kBf16 && a.rows % kWTRows == 0 && a.cols % kWTCols == 0 && cover_cols == a.cols && pairs_aligned &&
            reinterpret_cast<uintptr_t>(a.values) % 32 == 0) {
            CUtensorMap map_g;
            memset(&map_g, 0, sizeof(map_g));
            if (!make_map_strip_pairs(&map_g, a.g, (uint64_t)a.cols, (uint64_t)a.rows, (uint64_t)a.ld * 2))
                return cudaErrorInvalidValue;
            const unsigned row_tiles = (unsigned)(a.rows / kWTRows), col_tiles = (unsigned)(a.cols / kWTCols);
            const bool col_fast = col_tiles <= 8 && row_tiles <= 65535u;    // (the second grid dimension is 16 bits wide)
            // otherwise groups of 8, 4 or 2 column tiles (whichever divides their number), or row tiles fastest
            const int shift = row_tiles > (1u << 27) ? 0
                            : col_tiles % 8 == 0 ? 3 : col_tiles % 4 == 0 ? 2 : col_tiles % 2 == 0 ? 1 : 0;
            const dim3 grid_w = col_fast ? dim3(col_tiles, row_tiles) : dim3(row_tiles << shift, col_tiles >> shift);
            launch_dependent(prune_axis0_bf16_whole_tiles_kernel<M, kTC, kJoint, kSR, kEps16>, dim3(grid_w),
                             dim3(32 * kWTWarps), 0, stream, map_g, a.g, n_strips, a.ld, upr_total, uoff, rk, values,
                             meta, col_fast ? -1 : shift);
        } else if (kBf16) {
            CUtensorMap map_g;
            memset(&map_g, 0, sizeof(map_g));
            constexpr int kS = 4, kW = 2;                                    // strips per tile, warps per block
            if (!make_map_strips(&map_g, a.g, (uint64_t)a.cols, (uint64_t)a.rows, (uint64_t)a.ld * 2, kS))
                return cudaErrorInvalidValue;
            static PerDeviceOnce once;
            const cudaError_t attr_err = once_per_device(once, [](int) {
                return cudaFuncSetAttribute(prune_axis0_bf16_kernel<M, kTC, kJoint, kSR, kEps16, kS, kW>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, A0<kS, kW>::kSmemBytes);
            });
            if (attr_err != cudaSuccess) return attr_err;
            dim3 grid_b((unsigned)((n_strips + kS - 1) / kS), (unsigned)((cover_cols + kA0Cols - 1) / kA0Cols));
            launch_dependent(prune_axis0_bf16_kernel<M, kTC, kJoint, kSR, kEps16, kS, kW>, dim3(grid_b),
                             dim3(A0<kS, kW>::kThreads), A0<kS, kW>::kSmemBytes, stream, map_g, a.g, n_strips, a.cols,
                             a.ld, upr_total, uoff, rk, values, meta);
        } else {
            launch_dependent(prune_axis0_kernel<M, false, kTC, kJoint, kSR, kEps16>, dim3(grid),
                             dim3(kTileStrips * 32), 0, stream, a.g, n_strips, a.cols, a.ld, upr_total, uoff, rk,
                             values, meta);
        }
    }
    return cudaGetLastError();
}

template <int M, int kJoint, bool kSR, bool kEps16>
cudaError_t launch_prune_r(const PruneArgs& a, cudaStream_t stream) {
    if (a.tc_layout)
        return a.is_bf16 ? launch_prune_t<M, true, true, kJoint, kSR, kEps16>(a, stream)
                         : launch_prune_t<M, false, true, kJoint, kSR, kEps16>(a, stream);
    return a.is_bf16 ? launch_prune_t<M, true, false, kJoint, kSR, kEps16>(a, stream)
                     : launch_prune_t<M, false, false, kJoint, kSR, kEps16>(a, stream);
}

template <int M, int kJoint>
cudaError_t launch_prune_m(const PruneArgs& a, cudaStream_t stream) {
    if (a.eps16)
        return a.stochastic_rounding ? launch_prune_r<M, kJoint, true, true>(a, stream)
                                     : launch_prune_r<M, kJoint, false, true>(a, stream);
    return a.stochastic_rounding ? launch_prune_r<M, kJoint, true, false>(a, stream)
                                 : launch_prune_r<M, kJoint, false, false>(a, stream);
}

}  // namespace

cudaError_t launch_prune(const PruneArgs& a, cudaStream_t stream) {
    if (a.m == 2) return launch_prune_m<2, 0>(a, stream);
    if (a.joint == 3) return launch_prune_m<4, 3>(a, stream);          // MVUE 1:4
    if (a.joint == 2) return launch_prune_m<4, 2>(a, stream);
    return a.joint == 1 ? launch_prune_m<4, 1>(a, stream) : launch_prune_m<4, 0>(a, stream);
}

cudaError_t launch_prune_4of8(const PruneArgs& a, cudaStream_t stream) {
    const int64_t mrows = a.axis == 1 ? a.rows : a.cols, K = a.axis == 1 ? a.cols : a.rows;
    const int64_t n = mrows * (K / 8);
    const int64_t want = (n + 127) / 128;
    const int grid = (int)(want < (int64_t)a.sm_count * 16 ? want : (int64_t)a.sm_count * 16);
    const RoundKeys rk = make_round_keys(a.seed);
    if (a.is_bf16)
        prune_4of8_kernel<true><<<grid, 128, 0, stream>>>(a.g, mrows, K / 8, a.ld, a.axis, a.k_total / 8, a.k_offset / 8, rk,
                                                         reinterpret_cast<uint2*>(a.values), reinterpret_cast<uint8_t*>(a.meta));
    else
        prune_4of8_kernel<false><<<grid, 128, 0, stream>>>(a.g, mrows, K / 8, a.ld, a.axis, a.k_total / 8, a.k_offset / 8, rk,
                                                          reinterpret_cast<uint2*>(a.values), reinterpret_cast<uint8_t*>(a.meta));
    return cudaGetLastError();
}

cudaError_t launch_unpack(const void* values, const void* meta, bool tc_layout, int64_t mrows, int64_t K,
                          void* dense, int sm_count, cudaStream_t stream) {
    const int64_t n_units = mrows * (K / 16);
    const int64_t want = (n_units + 255) / 256;
    const int grid = (int)(want < (int64_t)sm_count * 32 ? want : (int64_t)sm_count * 32);
    if (tc_layout)
        unpack_kernel<true><<<grid, 256, 0, stream>>>(reinterpret_cast<const uint4*>(values),
                                                      reinterpret_cast<const uint16_t*>(meta), n_units, K / 16,
                                                      reinterpret_cast<uint4*>(dense));
    else
        unpack_kernel<false><<<grid, 256, 0, stream>>>(reinterpret_cast<const uint4*>(values),
                                                       reinterpret_cast<const uint16_t*>(meta), n_units, K / 16,
                                                       reinterpret_cast<uint4*>(dense));
    return cudaGetLastError();
}

}  // namespace mvue
