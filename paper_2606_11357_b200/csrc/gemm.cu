#include "common.cuh"
#include "kernels.h"
namespace tf {
size_t gemm_workspace_bytes(int M, int K, int N) { return 256; }
cudaError_t launch_gemm(int, const void*, const void*, void*, int, int, int, void*, size_t, int, cudaStream_t) {
    return cudaErrorNotSupported;
}
}
