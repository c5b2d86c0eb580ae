// MVUE N:M prune + pack kernels (memory-bound: one pass over g, packed bf16
// survivors and 2-bit position metadata written in the same pass).
//
// Work unit: 16 consecutive elements along the pruned axis K.  For 2:4 that is
// four blocks sharing one generator call; for 1:2 it is eight pairs using two.
//   axis 1 (K contiguous in memory): one thread owns one unit = 32 contiguous
//           bytes of bf16 (64 of fp32); a warp reads 1 KiB (2 KiB) contiguous.
//   axis 0 (K runs down the rows of g): one thread owns a strip of 16 rows by
//           16 bytes of columns; a warp reads 512 contiguous bytes per row.
#include <cuda_runtime.h>

#include "mvue_device.cuh"
#include "mvue_internal.h"

namespace mvue {
namespace {

__device__ __forceinline__ uint4 ldg128(const void* p) {
    return __ldg(reinterpret_cast<const uint4*>(p));
}

// One work unit of bf16 input: raw[8] = 16 elements along K, two per word.
template <int M>
__device__ __forceinline__ void prune_unit_bf16(const uint32_t (&raw)[8], uint64_t unit_index,
                                                const RoundKeys& rk, uint4* out_values,
                                                uint32_t* out_meta) {
    uint32_t v[4];                                   // 8 survivors, two bf16 per word
    uint32_t meta = 0;
    if (M == 4) {
        const uint4 w = philox4x32_10(unit_index, rk);
        const uint32_t words[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t nib;
            mvue_2of4_bf16(raw[2 * j], raw[2 * j + 1], words[j], &v[j], &nib);
            meta += nib << (4 * j);
        }
    } else {
        const uint4 wa = philox4x32_10(2 * unit_index, rk);
        const uint4 wb = philox4x32_10(2 * unit_index + 1, rk);
        const uint32_t words[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t nib;
            mvue_1of2x2_bf16(raw[2 * j], raw[2 * j + 1], words[2 * j], words[2 * j + 1], &v[j], &nib);
            meta += nib << (4 * j);
        }
    }
    *out_values = make_uint4(v[0], v[1], v[2], v[3]);
    *out_meta = meta;
}

// One work unit of binary32 input: b[16] = bit patterns of 16 elements along K.
template <int M>
__device__ __forceinline__ void prune_unit_f32(const uint32_t (&b)[16], uint64_t unit_index,
                                               const RoundKeys& rk, uint4* out_values,
                                               uint32_t* out_meta) {
    uint32_t v[4];
    uint32_t meta = 0;
    if (M == 4) {
        const uint4 w = philox4x32_10(unit_index, rk);
        const uint32_t words[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t nib;
            mvue_2of4_f32(b[4 * j], b[4 * j + 1], b[4 * j + 2], b[4 * j + 3], words[j], &v[j], &nib);
            meta |= nib << (4 * j);
        }
    } else {
        const uint4 wa = philox4x32_10(2 * unit_index, rk);
        const uint4 wb = philox4x32_10(2 * unit_index + 1, rk);
        const uint32_t words[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float v0, v1;
            const bool k0 = mvue_1of2(__uint_as_float(b[4 * j]), __uint_as_float(b[4 * j + 1]), words[2 * j], &v0);
            const bool k1 = mvue_1of2(__uint_as_float(b[4 * j + 2]), __uint_as_float(b[4 * j + 3]), words[2 * j + 1], &v1);
            v[j] = pack_bf16x2(v0, v1);
            meta |= (k0 ? 0u : (1u << (4 * j))) | (k1 ? (8u << (4 * j)) : (12u << (4 * j)));
        }
    }
    *out_values = make_uint4(v[0], v[1], v[2], v[3]);
    *out_meta = meta;
}

// ---- axis 1 ---------------------------------------------------------------
// slot = r * units_per_row + c.  kLinear: the tensor is contiguous and unsharded,
// so the input offset and the generator call number are linear in the slot.
template <int M, bool kBf16, bool kLinear>
__global__ void __launch_bounds__(256, kBf16 ? 6 : 4)
prune_axis1_kernel(const void* __restrict__ g, int64_t n_slots, int64_t units_per_row, int64_t ld,
                   int64_t units_per_row_total, int64_t unit_offset, RoundKeys rk,
                   uint4* __restrict__ values, uint16_t* __restrict__ meta) {
    constexpr int U = 1;                              // units per thread per trip, loads issued first
    constexpr int LW = kBf16 ? 2 : 4;                 // 16-byte loads per unit
    const int64_t trip = (int64_t)blockDim.x * U;
    for (int64_t base = (int64_t)blockIdx.x * trip; base < n_slots; base += (int64_t)gridDim.x * trip) {
        uint4 in[U][LW];
        uint64_t unit[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t slot = base + (int64_t)u * blockDim.x + threadIdx.x;
            if (slot < n_slots) {
                int64_t elem_off;
                if (kLinear) {
                    elem_off = slot * 16;
                    unit[u] = (uint64_t)slot;
                } else {
                    const int64_t r = slot / units_per_row;
                    const int64_t c = slot - r * units_per_row;
                    elem_off = r * ld + c * 16;
                    unit[u] = (uint64_t)r * (uint64_t)units_per_row_total + (uint64_t)(unit_offset + c);
                }
                const char* p = reinterpret_cast<const char*>(g) + elem_off * (kBf16 ? 2 : 4);
#pragma unroll
                for (int i = 0; i < LW; ++i) in[u][i] = ldg128(p + 16 * i);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t slot = base + (int64_t)u * blockDim.x + threadIdx.x;
            if (slot < n_slots) {
                uint4 v;
                uint32_t mt;
                if (kBf16) {
                    const uint32_t raw[8] = {in[u][0].x, in[u][0].y, in[u][0].z, in[u][0].w,
                                             in[u][1].x, in[u][1].y, in[u][1].z, in[u][1].w};
                    prune_unit_bf16<M>(raw, unit[u], rk, &v, &mt);
                } else {
                    uint32_t b[16];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        b[4 * i] = (&in[u][i].x)[0]; b[4 * i + 1] = (&in[u][i].x)[1];
                        b[4 * i + 2] = (&in[u][i].x)[2]; b[4 * i + 3] = (&in[u][i].x)[3];
                    }
                    prune_unit_f32<M>(b, unit[u], rk, &v, &mt);
                }
                values[slot] = v;
                meta[slot] = (uint16_t)mt;
            }
        }
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

template <int M, bool kBf16>
__global__ void __launch_bounds__(kTileStrips * 32, kBf16 ? 3 : 2)
prune_axis0_kernel(const void* __restrict__ g, int64_t n_strips, int64_t n_cols, int64_t ld,
                   int64_t units_per_row_total, int64_t unit_offset, RoundKeys rk,
                   uint4* __restrict__ values, uint16_t* __restrict__ meta) {
    constexpr int ES = kBf16 ? 2 : 4;
    constexpr int NT = kTileStrips * 32;
    __shared__ uint4 s_val[kTileCols * kTileStrips];
    __shared__ __align__(16) unsigned char s_meta[kTileCols * kMetaPitch];

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int strip_l = tid >> 5;
    const int64_t strip0 = (int64_t)blockIdx.x * kTileStrips;
    const int64_t col0 = (int64_t)blockIdx.y * kTileCols;
    const int64_t strip = strip0 + strip_l;
    const int64_t col = col0 + 2 * lane;             // this lane's first column (n_cols is even)

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
                uint32_t raw[8];
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    raw[j] = __byte_perm(w[2 * j][0], w[2 * j + 1][0], e ? 0x7632 : 0x5410);
                prune_unit_bf16<M>(raw, unit, rk, &v, &mt);
            } else {
                uint32_t b[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) b[i] = w[i][kBf16 ? 0 : e];
                prune_unit_f32<M>(b, unit, rk, &v, &mt);
            }
            s_val[col_l * kTileStrips + (strip_l ^ (lane & 15))] = v;
            *reinterpret_cast<uint16_t*>(&s_meta[col_l * kMetaPitch + strip_l * 2]) = (uint16_t)mt;
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
    // metadata: 64 columns x 32 bytes; 8 consecutive threads write one column's run as words
    {
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

// ---- unpack ---------------------------------------------------------------
// One thread expands one metadata byte (two groups = 8 dense elements = 16 bytes).
__global__ void __launch_bounds__(256)
unpack_kernel(const uint32_t* __restrict__ values, const uint8_t* __restrict__ meta, int64_t n_bytes,
              uint4* __restrict__ dense) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_bytes; i += stride) {
        const uint32_t mb = meta[i];
        const uint32_t va = values[2 * i], vb = values[2 * i + 1];
        uint16_t out[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        out[mb & 3u] = (uint16_t)va;
        out[(mb >> 2) & 3u] = (uint16_t)(va >> 16);
        out[4 + ((mb >> 4) & 3u)] = (uint16_t)vb;
        out[4 + ((mb >> 6) & 3u)] = (uint16_t)(vb >> 16);
        dense[i] = make_uint4(out[0] | ((uint32_t)out[1] << 16), out[2] | ((uint32_t)out[3] << 16),
                              out[4] | ((uint32_t)out[5] << 16), out[6] | ((uint32_t)out[7] << 16));
    }
}

template <int M, bool kBf16>
cudaError_t launch_prune_t(const PruneArgs& a, cudaStream_t stream) {
    const RoundKeys rk = make_round_keys(a.seed);
    const int64_t upr_total = a.k_total / 16, uoff = a.k_offset / 16;
    uint4* values = reinterpret_cast<uint4*>(a.values);
    uint16_t* meta = reinterpret_cast<uint16_t*>(a.meta);
    if (a.axis == 1) {
        const int64_t upr = a.cols / 16;
        const int64_t n_slots = a.rows * upr;
        const bool linear = (a.ld == a.cols) && (a.k_total == a.cols) && (a.k_offset == 0);
        const int64_t want = (n_slots + 255) / 256;
        const int grid = (int)(want < (int64_t)a.sm_count * 48 ? want : (int64_t)a.sm_count * 48);
        if (linear)
            prune_axis1_kernel<M, kBf16, true><<<grid, 256, 0, stream>>>(a.g, n_slots, upr, a.ld, upr_total, uoff, rk, values, meta);
        else
            prune_axis1_kernel<M, kBf16, false><<<grid, 256, 0, stream>>>(a.g, n_slots, upr, a.ld, upr_total, uoff, rk, values, meta);
    } else {
        const int64_t n_strips = a.rows / 16;
        dim3 grid((unsigned)((n_strips + kTileStrips - 1) / kTileStrips),
                  (unsigned)((a.cols + kTileCols - 1) / kTileCols));
        prune_axis0_kernel<M, kBf16><<<grid, kTileStrips * 32, 0, stream>>>(a.g, n_strips, a.cols, a.ld, upr_total, uoff, rk, values, meta);
    }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prune(const PruneArgs& a, cudaStream_t stream) {
    if (a.m == 4) return a.is_bf16 ? launch_prune_t<4, true>(a, stream) : launch_prune_t<4, false>(a, stream);
    return a.is_bf16 ? launch_prune_t<2, true>(a, stream) : launch_prune_t<2, false>(a, stream);
}

cudaError_t launch_unpack(const void* values, const void* meta, int64_t mrows, int64_t K, void* dense,
                          int sm_count, cudaStream_t stream) {
    const int64_t n_bytes = mrows * (K / 8);
    const int64_t want = (n_bytes + 255) / 256;
    const int grid = (int)(want < (int64_t)sm_count * 32 ? want : (int64_t)sm_count * 32);
    unpack_kernel<<<grid, 256, 0, stream>>>(reinterpret_cast<const uint32_t*>(values),
                                            reinterpret_cast<const uint8_t*>(meta), n_bytes,
                                            reinterpret_cast<uint4*>(dense));
    return cudaGetLastError();
}

}  // namespace mvue
