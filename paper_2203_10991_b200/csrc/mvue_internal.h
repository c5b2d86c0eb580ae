// Host-side declarations shared by the translation units of the library.
#pragma once
#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>
#include <mutex>

namespace mvue {

struct PruneArgs {
    const void* g;
    bool is_bf16;
    int64_t rows, cols, ld;
    int m;               // 2 or 4 (n is implied: 1 or 2; one survivor of four is joint = 3)
    int axis;            // 0 or 1
    uint64_t seed;
    int64_t k_total, k_offset;
    void* values;
    void* meta;
    int sm_count;
    bool tc_layout;      // metadata in tensor-core order instead of canonical rows
    int joint;           // 2:4 estimator: 0 = App. A.2 table, 1 = systematic sampling, 2 = approx-MVUE (Sec. 4.4); 3 = MVUE 1:4
    bool stochastic_rounding = false;   // survivors rounded to bf16 stochastically (unbiased storage) instead of to nearest
    bool eps16 = false;                 // sixteen random bits per block: one generator call per eight blocks
};

cudaError_t launch_prune(const PruneArgs& a, cudaStream_t stream);
cudaError_t launch_prune_4of8(const PruneArgs& a, cudaStream_t stream);   // approx-4:8, prune only (meta = mask bytes)
cudaError_t launch_unpack(const void* values, const void* meta, bool tc_layout, int64_t mrows, int64_t K,
                          void* dense, int sm_count, cudaStream_t stream);

struct SparseGemmArgs {
    const void* values;   // packed survivors [M x K/2] bf16
    const void* meta;     // position nibbles in tensor-core order (MVUE_LAYOUT_TC)
    int64_t M, N, K;
    const void* B;        // dense bf16 [K x N], leading dimension ldb
    int64_t ldb;
    void* C;              // [M x N] fp32 or bf16, leading dimension ldc
    int64_t ldc;
    int c_is_bf16;
    int accumulate;
    const void* scale;    // optional bf16 [M x N] (ld = ldc) multiplied into the result, or nullptr
    void* workspace;
    size_t workspace_bytes;
    int* dev_status;
    int sm_count;
    // optional: the bf16 output pruned along its columns in the epilogue (needs scale, bf16 output, no K split)
    void* next_values = nullptr;
    void* next_meta = nullptr;
    uint64_t next_seed = 0;
    int next_joint = 0;   // 0 = App. A.2 table, 1 = systematic sampling
    bool next_eps16 = false;   // sixteen random bits per block for that prune
};
int launch_sparse_gemm(const SparseGemmArgs& a, cudaStream_t stream);     // returns an mvue_status
// iters = 0: nothing is issued and the kernel's one wait expires after spin_limit polls (0: the default bound)
int launch_sparse_mma_probe(int iters, uint32_t spin_limit, int sm_count, int* pairs_out, int* dev_status,
                            cudaStream_t stream);                           // mvue_status
int gemm_split_count(int64_t M, int64_t N, int64_t K, int sm_count);
size_t gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int sm_count);            // what lets every path run
size_t gemm_required_workspace_bytes(int64_t M, int64_t N, int64_t K, int sm_count);   // the split along K alone

struct FusedArgs {
    const void* g;        // dense bf16 gradient [T x out]
    int64_t ldg;          // leading dimension in elements
    int m;                // 2 or 4
    uint64_t seed;
    SparseGemmArgs gemm;  // M = out, N = in, K = T; values / meta unused
    int joint = 0;        // the 2:4 law: 0 = App. A.2 table, 1 = systematic sampling
};
int launch_fused_update(const FusedArgs& f, cudaStream_t stream);         // returns an mvue_status
size_t fused_workspace_bytes(int64_t M, int64_t N, int64_t K, int sm_count);

// Split-K scratch that the library itself carries (see mvue_sparse_update_gemm_noalloc).
constexpr size_t kStaticScratchBytes = 8u << 20;
int static_scratch(void** ptr, size_t* bytes);   // returns an mvue_status; device address for the current device

// Per-device facts, looked up once.
struct DeviceInfo {
    int cc_major = 0;
    int sm_count = 0;
};
int current_device_info(DeviceInfo* info);   // returns an mvue_status
void set_cuda_error(cudaError_t e, const char* where);

// Function attributes (the dynamic shared-memory limit) and occupancy figures belong to a device, not to the
// process: a set-up step guarded by this runs once on every device that a call arrives on, with that device current.
constexpr int kMaxDevices = 64;
struct PerDeviceOnce {
    std::mutex mu;
    bool done[kMaxDevices] = {};
    cudaError_t err[kMaxDevices] = {};
};
template <typename F>
cudaError_t once_per_device(PerDeviceOnce& st, F&& setup) {
    int dev = 0;
    const cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(st.mu);
    if (!st.done[dev]) {
        st.err[dev] = setup(dev);
        st.done[dev] = true;
    }
    return st.err[dev];
}

// Launches `kernel` as a programmatic dependent of whatever precedes it on the stream: its blocks may be set up while
// that work drains (the launch no longer waits for the predecessor's completion to be reported), which takes one to
// two microseconds off every kernel of a chain.  The kernel must call grid_dependency_wait() (mvue_device.cuh)
// before it touches global memory; until then it has read nothing the predecessor wrote and written nothing the
// predecessor reads.
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                             Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace mvue
