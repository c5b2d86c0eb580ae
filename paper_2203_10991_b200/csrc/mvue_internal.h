// Host-side declarations shared by the translation units of the library.
#pragma once
#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>

namespace mvue {

struct PruneArgs {
    const void* g;
    bool is_bf16;
    int64_t rows, cols, ld;
    int m;               // 2 or 4 (n is implied: 1 or 2)
    int axis;            // 0 or 1
    uint64_t seed;
    int64_t k_total, k_offset;
    void* values;
    void* meta;
    int sm_count;
};

cudaError_t launch_prune(const PruneArgs& a, cudaStream_t stream);
cudaError_t launch_unpack(const void* values, const void* meta, int64_t mrows, int64_t K, void* dense,
                          int sm_count, cudaStream_t stream);

// Per-device facts, looked up once.
struct DeviceInfo {
    int cc_major = 0;
    int sm_count = 0;
};
int current_device_info(DeviceInfo* info);   // returns an mvue_status
void set_cuda_error(cudaError_t e, const char* where);

}  // namespace mvue
