// C ABI of the library: argument validation on the host, then one launch on the
// caller's stream.  No allocation, no synchronisation, no exceptions.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <mutex>

#include "../../include/mvue.h"
#include "mvue_internal.h"

namespace mvue {

static thread_local char g_cuda_error[256] = "";

void set_cuda_error(cudaError_t e, const char* where) {
    std::snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s (%s)", where, cudaGetErrorName(e),
                  cudaGetErrorString(e));
}

int current_device_info(DeviceInfo* info) {
    static std::mutex mu;
    static DeviceInfo cache[64];
    static bool known[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { set_cuda_error(e, "cudaGetDevice"); return MVUE_ERR_CUDA; }
    if (dev < 0 || dev >= 64) return MVUE_ERR_ARCH;
    std::lock_guard<std::mutex> lock(mu);
    if (!known[dev]) {
        DeviceInfo d;
        e = cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) { set_cuda_error(e, "cudaDeviceGetAttribute"); return MVUE_ERR_CUDA; }
        cache[dev] = d;
        known[dev] = true;
    }
    *info = cache[dev];
    return info->cc_major == 10 ? MVUE_OK : MVUE_ERR_ARCH;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_nm(int n, int m) {
    return ((n == 1 && m == 2) || (n == 2 && m == 4) || (n == 1 && m == 4)) ? MVUE_OK : MVUE_ERR_NM;
}

// Host-side checks shared by the product entry points; fills *dev for the current device.
static int check_gemm(const void* values, const void* meta, int layout, int64_t M, int64_t N, int64_t K,
                      const void* B, int64_t ldb, const void* scale, void* C, int c_dtype, int64_t ldc,
                      int accumulate, DeviceInfo* dev) {
    if (!values || !meta || !B || !C) return MVUE_ERR_NULL;
    if (layout != MVUE_LAYOUT_TC) return MVUE_ERR_LAYOUT;
    if (c_dtype != MVUE_F32 && c_dtype != MVUE_BF16) return MVUE_ERR_DTYPE;
    if (accumulate && c_dtype != MVUE_F32) return MVUE_ERR_DTYPE;
    if (accumulate && scale) return MVUE_ERR_DTYPE;
    if (M <= 0 || N <= 0 || K <= 0 || K % 128 != 0 || M % 8 != 0 || N % 8 != 0) return MVUE_ERR_SHAPE;
    if (ldb < N || ldc < N) return MVUE_ERR_SHAPE;
    if (M > 0x7FFFFFFF || N > 0x7FFFFFFF || K > 0x7FFFFFFF) return MVUE_ERR_SHAPE;
    const int64_t c_esz = c_dtype == MVUE_BF16 ? 2 : 4;
    if (!aligned16(values) || !aligned16(meta) || !aligned16(B) || !aligned16(C) || (ldb * 2) % 16 != 0 ||
        (ldc * c_esz) % 16 != 0 || (scale && (!aligned16(scale) || (ldc * 2) % 16 != 0)))
        return MVUE_ERR_ALIGN;
    return current_device_info(dev);
}

static int run_gemm(const void* values, const void* meta, int layout, int64_t M, int64_t N, int64_t K,
                    const void* B, int64_t ldb, const void* scale, void* C, int c_dtype, int64_t ldc,
                    int accumulate, void* workspace, size_t workspace_bytes, int* dev_status, void* stream) {
    DeviceInfo dev;
    if (int s = check_gemm(values, meta, layout, M, N, K, B, ldb, scale, C, c_dtype, ldc, accumulate, &dev)) return s;
    // the split of a long K needs its workspace; the K split of the last round's tiles is skipped without it
    const size_t need = gemm_required_workspace_bytes(M, N, K, dev.sm_count);
    if (need > 0 && (!workspace || workspace_bytes < need)) return MVUE_ERR_WORKSPACE;
    if (workspace && !aligned16(workspace)) return MVUE_ERR_WORKSPACE;
    SparseGemmArgs a{values, meta, M, N, K, B, ldb, C, ldc, c_dtype == MVUE_BF16, accumulate, scale,
                     workspace, workspace ? workspace_bytes : 0, dev_status, dev.sm_count};
    return launch_sparse_gemm(a, reinterpret_cast<cudaStream_t>(stream));
}

}  // namespace mvue

using namespace mvue;

extern "C" {

int mvue_version(void) { return 140; }   // 1.4: prune options on the backward product that prunes its own output

const char* mvue_status_string(int status) {
    switch (status) {
        case MVUE_OK: return "ok";
        case MVUE_ERR_NULL: return "null pointer";
        case MVUE_ERR_NM: return "unsupported N:M (only 1:2, 2:4 and 1:4; the fused product: 1:2 and 2:4)";
        case MVUE_ERR_SHAPE: return "bad shape, axis, leading dimension or K shard";
        case MVUE_ERR_ALIGN: return "pointer or leading dimension not 16-byte aligned";
        case MVUE_ERR_DTYPE: return "unsupported dtype";
        case MVUE_ERR_LAYOUT: return "unsupported layout";
        case MVUE_ERR_WORKSPACE: return "workspace missing or too small";
        case MVUE_ERR_ARCH: return "device is not compute capability 10.x";
        case MVUE_ERR_CUDA: return "CUDA call failed (see mvue_last_cuda_error)";
        case MVUE_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
        case MVUE_ERR_JOINT: return "unknown 2:4 estimator (App. A.2 table, systematic sampling or approx-MVUE)";
        case MVUE_ERR_OPTION: return "unknown prune option bit";
        default: return "unknown status";
    }
}

const char* mvue_last_cuda_error(void) { return g_cuda_error; }

int mvue_packed_sizes(int64_t rows, int64_t cols, int n, int m, int axis, int layout,
                      size_t* values_bytes, size_t* meta_bytes) {
    if (int s = check_nm(n, m)) return s;
    if (layout != MVUE_LAYOUT_CANONICAL && layout != MVUE_LAYOUT_TC) return MVUE_ERR_LAYOUT;
    if (axis != 0 && axis != 1) return MVUE_ERR_SHAPE;
    if (rows <= 0 || cols <= 0) return MVUE_ERR_SHAPE;
    const int64_t mrows = axis == 1 ? rows : cols;
    const int64_t K = axis == 1 ? cols : rows;
    if (K % 16 != 0 || mrows % 8 != 0) return MVUE_ERR_SHAPE;
    if (layout == MVUE_LAYOUT_TC && K % 128 != 0) return MVUE_ERR_SHAPE;
    const int64_t meta_rows = layout == MVUE_LAYOUT_TC ? (mrows + 127) / 128 * 128 : mrows;
    if (values_bytes) *values_bytes = (size_t)mrows * (size_t)(K / 2) * 2;
    if (meta_bytes) *meta_bytes = (size_t)meta_rows * (size_t)(K / 8);
    return MVUE_OK;
}

int mvue_prune(const void* g, int dtype, int64_t rows, int64_t cols, int64_t ld, int n, int m,
               int axis, uint64_t seed, int64_t k_total, int64_t k_offset, void* values,
               void* meta, int layout, void* stream) {
    return mvue_prune_joint(g, dtype, rows, cols, ld, n, m, axis, seed, k_total, k_offset, values, meta, layout,
                            MVUE_JOINT_TABLE, stream);
}

int mvue_prune_joint(const void* g, int dtype, int64_t rows, int64_t cols, int64_t ld, int n, int m,
                     int axis, uint64_t seed, int64_t k_total, int64_t k_offset, void* values,
                     void* meta, int layout, int joint, void* stream) {
    return mvue_prune_opts(g, dtype, rows, cols, ld, n, m, axis, seed, k_total, k_offset, values, meta, layout, joint,
                           MVUE_OPT_NONE, stream);
}

int mvue_prune_opts(const void* g, int dtype, int64_t rows, int64_t cols, int64_t ld, int n, int m,
                    int axis, uint64_t seed, int64_t k_total, int64_t k_offset, void* values,
                    void* meta, int layout, int joint, unsigned options, void* stream) {
    if (!g || !values || !meta) return MVUE_ERR_NULL;
    if (options & ~(unsigned)(MVUE_OPT_STOCHASTIC_ROUNDING | MVUE_OPT_EPS16)) return MVUE_ERR_OPTION;
    if (joint != MVUE_JOINT_TABLE && joint != MVUE_JOINT_SYSTEMATIC && joint != MVUE_JOINT_APPROX) return MVUE_ERR_JOINT;
    if (dtype != MVUE_F32 && dtype != MVUE_BF16) return MVUE_ERR_DTYPE;
    if (int s = mvue_packed_sizes(rows, cols, n, m, axis, layout, nullptr, nullptr)) return s;
    const int64_t K = axis == 1 ? cols : rows;
    if (ld < cols) return MVUE_ERR_SHAPE;
    // launch-grid limits: 65535 blocks of 256 k (axis 1) or of 64 rows of A (axis 0) in the second grid dimension
    if (axis == 1 ? K > 65535ll * 256 : cols > 65535ll * 64) return MVUE_ERR_SHAPE;
    if (k_total % 16 != 0 || k_offset % 16 != 0 || k_offset < 0 || k_offset + K > k_total) return MVUE_ERR_SHAPE;
    const int64_t esz = dtype == MVUE_BF16 ? 2 : 4;
    if (!aligned16(g) || !aligned16(values) || !aligned16(meta) || (ld * esz) % 16 != 0) return MVUE_ERR_ALIGN;
    DeviceInfo dev;
    if (int s = current_device_info(&dev)) return s;
    PruneArgs a{g, dtype == MVUE_BF16, rows, cols, ld, m, axis, seed, k_total, k_offset, values, meta, dev.sm_count,
                layout == MVUE_LAYOUT_TC, (n == 1 && m == 4) ? 3 : joint,      // one survivor of four has a single law
                (options & MVUE_OPT_STOCHASTIC_ROUNDING) != 0, (options & MVUE_OPT_EPS16) != 0};
    cudaError_t e = launch_prune(a, reinterpret_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { set_cuda_error(e, "mvue_prune launch"); return MVUE_ERR_CUDA; }
    return MVUE_OK;
}

int mvue_prune_4of8(const void* g, int dtype, int64_t rows, int64_t cols, int64_t ld, int axis, uint64_t seed,
                    int64_t k_total, int64_t k_offset, void* values, void* mask, void* stream) {
    if (!g || !values || !mask) return MVUE_ERR_NULL;
    if (dtype != MVUE_F32 && dtype != MVUE_BF16) return MVUE_ERR_DTYPE;
    if (axis != 0 && axis != 1) return MVUE_ERR_SHAPE;
    if (rows <= 0 || cols <= 0 || ld < cols) return MVUE_ERR_SHAPE;
    const int64_t K = axis == 1 ? cols : rows;
    if (K % 8 != 0 || k_total % 8 != 0 || k_offset % 8 != 0 || k_offset < 0 || k_offset + K > k_total) return MVUE_ERR_SHAPE;
    const int64_t esz = dtype == MVUE_BF16 ? 2 : 4;
    if (!aligned16(g) || (reinterpret_cast<uintptr_t>(values) & 7u) != 0 || (ld * esz) % 16 != 0) return MVUE_ERR_ALIGN;
    DeviceInfo dev;
    if (int s = current_device_info(&dev)) return s;
    PruneArgs a{g, dtype == MVUE_BF16, rows, cols, ld, 8, axis, seed, k_total, k_offset, values, mask, dev.sm_count,
                false, 0};
    cudaError_t e = launch_prune_4of8(a, reinterpret_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { set_cuda_error(e, "mvue_prune_4of8 launch"); return MVUE_ERR_CUDA; }
    return MVUE_OK;
}

int mvue_unpack(const void* values, const void* meta, int layout, int64_t mrows, int64_t K,
                void* dense_bf16, void* stream) {
    if (!values || !meta || !dense_bf16) return MVUE_ERR_NULL;
    if (layout != MVUE_LAYOUT_CANONICAL && layout != MVUE_LAYOUT_TC) return MVUE_ERR_LAYOUT;
    if (mrows <= 0 || K <= 0 || K % 16 != 0) return MVUE_ERR_SHAPE;
    if (layout == MVUE_LAYOUT_TC && K % 128 != 0) return MVUE_ERR_SHAPE;
    if (!aligned16(values) || !aligned16(meta) || !aligned16(dense_bf16)) return MVUE_ERR_ALIGN;
    DeviceInfo dev;
    if (int s = current_device_info(&dev)) return s;
    cudaError_t e = launch_unpack(values, meta, layout == MVUE_LAYOUT_TC, mrows, K, dense_bf16, dev.sm_count,
                                  reinterpret_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { set_cuda_error(e, "mvue_unpack launch"); return MVUE_ERR_CUDA; }
    return MVUE_OK;
}

int mvue_gemm_workspace_bytes(int which, int64_t M, int64_t N, int64_t K, size_t* bytes) {
    if (!bytes) return MVUE_ERR_NULL;
    if (which != 0 && which != 1 && which != 2) return MVUE_ERR_SHAPE;
    if (M <= 0 || N <= 0 || K <= 0 || K % 128 != 0) return MVUE_ERR_SHAPE;
    DeviceInfo dev;
    if (int s = current_device_info(&dev)) return s;
    *bytes = which == 2 ? fused_workspace_bytes(M, N, K, dev.sm_count) : gemm_workspace_bytes(M, N, K, dev.sm_count);
    return MVUE_OK;
}

int mvue_sparse_update_gemm(const void* values, const void* meta, int layout, int64_t out, int64_t T,
                            const void* h, int64_t in, int64_t ldh, void* dW, int dW_dtype, int64_t lddW,
                            int accumulate, void* workspace, size_t workspace_bytes, int* dev_status,
                            void* stream) {
    return run_gemm(values, meta, layout, out, in, T, h, ldh, nullptr, dW, dW_dtype, lddW, accumulate,
                    workspace, workspace_bytes, dev_status, stream);
}

int mvue_sparse_backward_gemm(const void* values, const void* meta, int layout, int64_t T, int64_t out,
                              const void* W, int64_t in, int64_t ldW, const void* act_grad, void* dh,
                              int dh_dtype, int64_t lddh, void* workspace, size_t workspace_bytes,
                              int* dev_status, void* stream) {
    return run_gemm(values, meta, layout, T, in, out, W, ldW, act_grad, dh, dh_dtype, lddh, 0, workspace,
                    workspace_bytes, dev_status, stream);
}

int mvue_sparse_backward_gemm_pruned(const void* values, const void* meta, int layout, int64_t T, int64_t out,
                                     const void* W, int64_t in, int64_t ldW, const void* act_grad, void* dh,
                                     int64_t lddh, uint64_t next_seed, int next_joint, unsigned next_options,
                                     void* next_values, void* next_meta, void* workspace, size_t workspace_bytes,
                                     int* dev_status, void* stream) {
    if (!act_grad || !next_values || !next_meta) return MVUE_ERR_NULL;
    if (next_joint != MVUE_JOINT_TABLE && next_joint != MVUE_JOINT_SYSTEMATIC) return MVUE_ERR_JOINT;
    if (next_options & ~(unsigned)(MVUE_OPT_STOCHASTIC_ROUNDING | MVUE_OPT_EPS16)) return MVUE_ERR_OPTION;
    const bool next_sr = (next_options & MVUE_OPT_STOCHASTIC_ROUNDING) != 0, next_eps16 = (next_options & MVUE_OPT_EPS16) != 0;
    if (in % 128 != 0) return MVUE_ERR_SHAPE;                      // K of the next product, tensor-core order
    if (!aligned16(next_values) || !aligned16(next_meta)) return MVUE_ERR_ALIGN;
    DeviceInfo dev;
    if (int s = check_gemm(values, meta, layout, T, in, out, W, ldW, act_grad, dh, MVUE_BF16, lddh, 0, &dev)) return s;
    const size_t need = gemm_required_workspace_bytes(T, in, out, dev.sm_count);
    if (need > 0 && (!workspace || workspace_bytes < need)) return MVUE_ERR_WORKSPACE;
    if (workspace && !aligned16(workspace)) return MVUE_ERR_WORKSPACE;
    SparseGemmArgs a{values, meta, T, in, out, W, ldW, dh, lddh, 1, 0, act_grad, workspace,
                     workspace ? workspace_bytes : 0, dev_status, dev.sm_count};
    if (need == 0 && T % 128 == 0 && !next_sr) {                    // one launch: the prune rides in the epilogue
        a.next_values = next_values;
        a.next_meta = next_meta;
        a.next_seed = next_seed;
        a.next_joint = next_joint;
        a.next_eps16 = next_eps16;
        return launch_sparse_gemm(a, reinterpret_cast<cudaStream_t>(stream));
    }
    // a product split along K (its tiles are partial sums), a ragged last row block, or stochastic rounding (its extra
    // generator call per unit has no room in the epilogue's registers): the two steps one after the other
    if (int s = launch_sparse_gemm(a, reinterpret_cast<cudaStream_t>(stream))) return s;
    if (T % 8 != 0) return MVUE_ERR_SHAPE;
    PruneArgs pa{dh, true, T, in, lddh, 4, 1, next_seed, in, 0, next_values, next_meta, dev.sm_count, true, next_joint};
    pa.stochastic_rounding = next_sr;
    pa.eps16 = next_eps16;
    cudaError_t e = launch_prune(pa, reinterpret_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { set_cuda_error(e, "mvue_sparse_backward_gemm_pruned prune launch"); return MVUE_ERR_CUDA; }
    return MVUE_OK;
}

int mvue_fused_update_gemm(const void* g, int dtype, int64_t T, int64_t out, int64_t ldg, int n, int m,
                           uint64_t seed, const void* h, int64_t in, int64_t ldh, void* dW, int dW_dtype,
                           int64_t lddW, int accumulate, void* workspace, size_t workspace_bytes,
                           int* dev_status, void* stream) {
    return mvue_fused_update_gemm_joint(g, dtype, T, out, ldg, n, m, MVUE_JOINT_TABLE, seed, h, in, ldh, dW, dW_dtype, lddW,
                                        accumulate, workspace, workspace_bytes, dev_status, stream);
}

int mvue_fused_update_gemm_joint(const void* g, int dtype, int64_t T, int64_t out, int64_t ldg, int n, int m, int joint,
                                 uint64_t seed, const void* h, int64_t in, int64_t ldh, void* dW, int dW_dtype,
                                 int64_t lddW, int accumulate, void* workspace, size_t workspace_bytes,
                                 int* dev_status, void* stream) {
    if (!g || !h || !dW) return MVUE_ERR_NULL;
    if (joint != MVUE_JOINT_TABLE && joint != MVUE_JOINT_SYSTEMATIC) return MVUE_ERR_JOINT;
    if (int s = check_nm(n, m)) return s;
    if (n == 1 && m == 4) return MVUE_ERR_NM;                      // the fused path prunes to 1:2 and 2:4 only
    if (dtype != MVUE_BF16) return MVUE_ERR_DTYPE;                 // the fused path takes bf16 gradients only
    if (dW_dtype != MVUE_F32 && dW_dtype != MVUE_BF16) return MVUE_ERR_DTYPE;
    if (accumulate && dW_dtype != MVUE_F32) return MVUE_ERR_DTYPE;
    if (T <= 0 || out <= 0 || in <= 0 || T % 128 != 0 || out % 8 != 0 || in % 8 != 0) return MVUE_ERR_SHAPE;
    if (ldg < out || ldh < in || lddW < in) return MVUE_ERR_SHAPE;
    if (T > 0x7FFFFFFF || out > 0x7FFFFFFF || in > 0x7FFFFFFF) return MVUE_ERR_SHAPE;
    const int64_t c_esz = dW_dtype == MVUE_BF16 ? 2 : 4;
    if (!aligned16(g) || !aligned16(h) || !aligned16(dW) || (ldg * 2) % 16 != 0 || (ldh * 2) % 16 != 0 ||
        (lddW * c_esz) % 16 != 0)
        return MVUE_ERR_ALIGN;
    DeviceInfo dev;
    if (int s = current_device_info(&dev)) return s;
    const size_t need = fused_workspace_bytes(out, in, T, dev.sm_count);
    if (need > 0 && (!workspace || workspace_bytes < need || !aligned16(workspace))) return MVUE_ERR_WORKSPACE;
    FusedArgs f{g, ldg, m, seed,
                SparseGemmArgs{nullptr, nullptr, out, in, T, h, ldh, dW, lddW, dW_dtype == MVUE_BF16, accumulate,
                               nullptr, workspace, workspace ? workspace_bytes : 0, dev_status, dev.sm_count},
                joint};
    return launch_fused_update(f, reinterpret_cast<cudaStream_t>(stream));
}

int mvue_probe_sparse_mma(int iters, int* pairs, double* flops, int* dev_status, void* stream) {
    if (iters <= 0 || iters > (1 << 20)) return MVUE_ERR_SHAPE;
    DeviceInfo dev;
    if (int s = current_device_info(&dev)) return s;
    int n_pairs = 0;
    if (int s = launch_sparse_mma_probe(iters, 0u, dev.sm_count, &n_pairs, dev_status, reinterpret_cast<cudaStream_t>(stream)))
        return s;
    if (pairs) *pairs = n_pairs;
    if (flops) *flops = (double)n_pairs * (double)iters * 4.0 * 2.0 * 256.0 * 256.0 * 32.0;
    return MVUE_OK;
}

int mvue_selftest_wait_timeout(int polls, int* dev_status, void* stream) {
    if (!dev_status) return MVUE_ERR_NULL;
    if (polls <= 0 || polls > (1 << 16)) return MVUE_ERR_SHAPE;
    DeviceInfo dev;
    if (int s = current_device_info(&dev)) return s;
    return launch_sparse_mma_probe(0, (uint32_t)polls, dev.sm_count, nullptr, dev_status,
                                   reinterpret_cast<cudaStream_t>(stream));
}

int mvue_sparse_update_gemm_noalloc(const void* values, const void* meta, int layout, int64_t out, int64_t T,
                                    const void* h, int64_t in, int64_t ldh, void* dW, int dW_dtype,
                                    int64_t lddW, int accumulate, int* dev_status, void* stream) {
    // every argument is checked before the scratch array's address is looked up (a CUDA call on first use)
    DeviceInfo dev;
    if (int s = check_gemm(values, meta, layout, out, in, T, h, ldh, nullptr, dW, dW_dtype, lddW, accumulate, &dev))
        return s;
    const size_t need = gemm_required_workspace_bytes(out, in, T, dev.sm_count);
    if (need > kStaticScratchBytes) return MVUE_ERR_WORKSPACE;     // beyond what the library carries
    void* scratch = nullptr;
    size_t scratch_bytes = 0;
    if (int s = static_scratch(&scratch, &scratch_bytes)) return s;
    return run_gemm(values, meta, layout, out, in, T, h, ldh, nullptr, dW, dW_dtype, lddW, accumulate,
                    scratch, scratch_bytes, dev_status, stream);
}

}  // extern "C"
