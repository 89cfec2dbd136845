// Internal launch interface between the C-ABI layer and the kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace tf {

constexpr int kGemvMaxThreads = 256;

struct GemvPlan {
    int cluster;        // CTAs per cluster = K split factor (1, 2, 4 or 8)
    int tiles_per_cta;  // k-tiles each CTA of a cluster walks
    int threads;        // CTA size
    int strips;         // grid.y
    int ktiles;
};

GemvPlan plan_gemv(int K, int N, int sm_count);
cudaError_t launch_gemv(int bits, const GemvPlan& plan, const void* blob, const void* a, void* y,
                        int M, int K, int N, void* status, cudaStream_t stream);

cudaError_t launch_unpack_w4(const void* blob, uint8_t* q, uint8_t* z, uint16_t* s, int K, int N,
                             int group_size, cudaStream_t stream);
cudaError_t launch_unpack_w8(const void* blob, int8_t* q, uint16_t* s, int K, int N, int group_size,
                             cudaStream_t stream);

// Prefill GEMM (tcgen05).  `workspace` starts with the DeviceStatus word.
size_t gemm_workspace_bytes(int M, int K, int N);
cudaError_t launch_gemm(int bits, const void* blob, const void* a, void* y, int M, int K, int N,
                        void* workspace, size_t workspace_bytes, int sm_count, cudaStream_t stream);

}  // namespace tf
