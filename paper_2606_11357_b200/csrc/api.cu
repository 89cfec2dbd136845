// C-ABI entry points: argument validation and kernel launches.  No allocation, no retained state
// other than a per-device cache of immutable device attributes.
#include <cuda_runtime.h>

#include <atomic>

#include "../../include/tilefuse.h"
#include "kernels.h"
#include "layout.h"

namespace {

struct DeviceInfo {
    int known;      // 1 = ok (cc 10.x), -1 = wrong architecture
    int sm_count;
};
// Per device: 0 = not queried yet, else (sm_count << 2) | (2 = compute capability 10.x, 1 = another architecture).
// One atomic word per device, so a host thread either sees nothing or a complete entry; two threads that query at the
// same time store the same value.
std::atomic<int> g_devices[64];
std::atomic<uint32_t> g_debug_word{0};

// Device attributes of the current device (cached after the first call on that device).
tf_status device_info(DeviceInfo* out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return TF_ERR_CUDA; }
    if (dev < 0 || dev >= 64) return TF_ERR_CUDA;
    int word = g_devices[dev].load(std::memory_order_acquire);
    if (word == 0) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError();
            return TF_ERR_CUDA;
        }
        word = (sms << 2) | (major == 10 ? 2 : 1);
        g_devices[dev].store(word, std::memory_order_release);
    }
    if ((word & 3) != 2) return TF_ERR_ARCH;
    out->known = 1;
    out->sm_count = word >> 2;
    return TF_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

tf_status check_linear_args(int bits, const void* packed, const void* a, void* y, int M, int K, int N,
                            int max_m, int group_size) {
    if (!packed || !a || !y) return TF_ERR_NULL;
    if (M < 1 || M > max_m) return TF_ERR_SHAPE;
    if (tf_packed_size(bits, K, N, group_size) == 0) return TF_ERR_SHAPE;
    if (!aligned16(packed) || !aligned16(a) || !aligned16(y)) return TF_ERR_ALIGN;
    return TF_OK;
}

tf_status gemv(int bits, const void* packed, const void* a, void* y, int M, int K, int N, void* workspace,
               size_t workspace_bytes, void* stream, int group_size = tf::kTileK) {
    tf_status st = check_linear_args(bits, packed, a, y, M, K, N, TF_MAX_M_GEMV, group_size);
    if (st != TF_OK) return st;
    if (workspace == nullptr || workspace_bytes < tf::kGemvWorkspaceBytes) return TF_ERR_WORKSPACE;
    if (!aligned16(workspace)) return TF_ERR_ALIGN;
    DeviceInfo dev;
    st = device_info(&dev);
    if (st != TF_OK) return st;
    if (dev.sm_count > tf::kGemvMaxGrid) dev.sm_count = tf::kGemvMaxGrid;
    const tf::GemvPlan plan = tf::plan_gemv(bits, M, K, N, dev.sm_count, tf::groups_per_tile(group_size));
    cudaError_t e = tf::launch_gemv(bits, plan, packed, a, y, M, K, N, workspace, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { cudaGetLastError(); return TF_ERR_CUDA; }
    return TF_OK;
}

tf_status gemm(int bits, const void* packed, const void* a, void* y, int M, int K, int N, void* workspace,
               size_t workspace_bytes, void* stream, int group_size = tf::kTileK) {
    tf_status st = check_linear_args(bits, packed, a, y, M, K, N, TF_MAX_M_GEMM, group_size);
    if (st != TF_OK) return st;
    const size_t need = tf_workspace_size(bits == 4 ? TF_OP_GEMM_W4A16 : TF_OP_GEMM_W8A16, M, K, N);
    if (workspace == nullptr || workspace_bytes < need) return TF_ERR_WORKSPACE;
    if (!aligned16(workspace)) return TF_ERR_ALIGN;
    DeviceInfo dev;
    st = device_info(&dev);
    if (st != TF_OK) return st;
    cudaError_t e = tf::launch_gemm(bits, packed, a, y, M, K, N, workspace, workspace_bytes, dev.sm_count,
                                    static_cast<cudaStream_t>(stream), tf::groups_per_tile(group_size));
    if (e != cudaSuccess) { cudaGetLastError(); return TF_ERR_CUDA; }
    return TF_OK;
}

}  // namespace

namespace tf {
uint32_t debug_word() { return g_debug_word.load(std::memory_order_relaxed); }
void set_debug_word(uint32_t word) { g_debug_word.store(word, std::memory_order_relaxed); }
}  // namespace tf

extern "C" __attribute__((visibility("default"))) tf_status tf_debug_inject(unsigned wait_limit_kcycles, int drop_weight_copies) {
    if (wait_limit_kcycles >= (1u << 24)) return TF_ERR_SHAPE;
    tf::set_debug_word((wait_limit_kcycles << 8) | (drop_weight_copies ? 1u : 0u));
    return TF_OK;
}

extern "C" __attribute__((visibility("default"))) tf_status tf_gemv_w4a16(const void* packed, const void* a, void* y, int M, int K, int N,
                                   void* workspace, size_t workspace_bytes, void* stream) {
    return gemv(4, packed, a, y, M, K, N, workspace, workspace_bytes, stream);
}
extern "C" __attribute__((visibility("default"))) tf_status tf_gemv_w8a16(const void* packed, const void* a, void* y, int M, int K, int N,
                                   void* workspace, size_t workspace_bytes, void* stream) {
    return gemv(8, packed, a, y, M, K, N, workspace, workspace_bytes, stream);
}
extern "C" __attribute__((visibility("default"))) tf_status tf_gemm_w4a16(const void* packed, const void* a, void* y, int M, int K, int N,
                                   void* workspace, size_t workspace_bytes, void* stream) {
    return gemm(4, packed, a, y, M, K, N, workspace, workspace_bytes, stream);
}
extern "C" __attribute__((visibility("default"))) tf_status tf_gemm_w8a16(const void* packed, const void* a, void* y, int M, int K, int N,
                                   void* workspace, size_t workspace_bytes, void* stream) {
    return gemm(8, packed, a, y, M, K, N, workspace, workspace_bytes, stream);
}

extern "C" __attribute__((visibility("default"))) tf_status tf_gemv_w4a16_grouped(const void* packed, const void* a, void* y, int M, int K,
                                   int N, int group_size, void* workspace, size_t workspace_bytes, void* stream) {
    return gemv(4, packed, a, y, M, K, N, workspace, workspace_bytes, stream, group_size);
}
extern "C" __attribute__((visibility("default"))) tf_status tf_gemm_w4a16_grouped(const void* packed, const void* a, void* y, int M, int K,
                                   int N, int group_size, void* workspace, size_t workspace_bytes, void* stream) {
    return gemm(4, packed, a, y, M, K, N, workspace, workspace_bytes, stream, group_size);
}

extern "C" __attribute__((visibility("default"))) tf_status tf_gemv_plan(int bits, int M, int K, int N, int sm_count, int* out) {
    if (!out) return TF_ERR_NULL;
    if (bits != 4 && bits != 8) return TF_ERR_SHAPE;
    if (M < 1 || M > TF_MAX_M_GEMV || tf_packed_size(bits, K, N, tf::kTileK) == 0) return TF_ERR_SHAPE;
    if (sm_count <= 0) {
        DeviceInfo dev;
        tf_status st = device_info(&dev);
        if (st != TF_OK) return st;
        sm_count = dev.sm_count;
    }
    if (sm_count > tf::kGemvMaxGrid) sm_count = tf::kGemvMaxGrid;
    const tf::GemvPlan p = tf::plan_gemv(bits, M, K, N, sm_count);
    out[0] = p.grid; out[1] = p.threads; out[2] = p.consumers; out[3] = p.stages;
    out[4] = p.full ? 1 : 0; out[5] = p.i8 ? (p.piece_tab > 0 ? 2 : 1) : 0; out[6] = p.cluster; out[7] = p.nclusters;
    return TF_OK;
}

extern "C" __attribute__((visibility("default"))) size_t tf_workspace_size(int op, int M, int K, int N) {
    const int bits = (op == TF_OP_GEMV_W4A16 || op == TF_OP_GEMM_W4A16) ? 4 : 8;
    if (op < TF_OP_GEMV_W4A16 || op > TF_OP_GEMM_W8A16) return 0;
    if (tf_packed_size(bits, K, N, tf::kTileK) == 0) return 0;
    if (op == TF_OP_GEMV_W4A16 || op == TF_OP_GEMV_W8A16)
        return (M >= 1 && M <= TF_MAX_M_GEMV) ? tf::kGemvWorkspaceBytes : 0;
    if (M < 1 || M > TF_MAX_M_GEMM) return 0;
    return tf::gemm_workspace_bytes(M, K, N);
}

static tf_status unpack_common(int bits, const void* packed, void* q, void* z, uint16_t* s, int K, int N,
                               int group_size, void* stream) {
    if (!packed) return TF_ERR_NULL;
    if (tf_packed_size(bits, K, N, group_size) == 0) return TF_ERR_SHAPE;
    if (!aligned16(packed)) return TF_ERR_ALIGN;
    DeviceInfo dev;
    tf_status st = device_info(&dev);
    if (st != TF_OK) return st;
    cudaError_t e = bits == 4
        ? tf::launch_unpack_w4(packed, static_cast<uint8_t*>(q), static_cast<uint8_t*>(z), s, K, N, group_size,
                               static_cast<cudaStream_t>(stream))
        : tf::launch_unpack_w8(packed, static_cast<int8_t*>(q), s, K, N, group_size,
                               static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { cudaGetLastError(); return TF_ERR_CUDA; }
    return TF_OK;
}

extern "C" __attribute__((visibility("default"))) tf_status tf_unpack_w4(const void* packed, uint8_t* q, uint8_t* z, uint16_t* s, int K, int N,
                                  int group_size, void* stream) {
    return unpack_common(4, packed, q, z, s, K, N, group_size, stream);
}
extern "C" __attribute__((visibility("default"))) tf_status tf_unpack_w8(const void* packed, int8_t* q, uint16_t* s, int K, int N, int group_size,
                                  void* stream) {
    return unpack_common(8, packed, q, nullptr, s, K, N, group_size, stream);
}

extern "C" __attribute__((visibility("default"))) tf_status tf_dequant_bf16(const void* packed, void* w_bf16, int bits, int K, int N,
                                                                           void* stream) {
    if (!packed || !w_bf16) return TF_ERR_NULL;
    if (tf_packed_size(bits, K, N, tf::kTileK) == 0) return TF_ERR_SHAPE;
    if (!aligned16(packed) || !aligned16(w_bf16)) return TF_ERR_ALIGN;
    DeviceInfo dev;
    tf_status st = device_info(&dev);
    if (st != TF_OK) return st;
    if (tf::launch_dequant(bits, packed, w_bf16, K, N, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        cudaGetLastError();
        return TF_ERR_CUDA;
    }
    return TF_OK;
}

extern "C" __attribute__((visibility("default"))) size_t tf_gemv_awq_raw_workspace_size(int M, int K, int N, int group_size) {
    if (M < 1 || M > TF_MAX_M_GEMV || N < 8 || N > TF_MAX_DIM || N % 8 != 0) return 0;
    if (group_size != 32 && group_size != 64 && group_size != 128) return 0;
    if (K < group_size || K > TF_MAX_DIM || K % group_size != 0) return 0;
    DeviceInfo dev;
    if (device_info(&dev) != TF_OK) return 0;
    return tf::gemv_raw_workspace_bytes(M, N, dev.sm_count);
}

extern "C" __attribute__((visibility("default"))) tf_status tf_gemv_awq_raw(const uint32_t* qweight, const uint16_t* scales,
                                                                            const uint32_t* qzeros, const void* a, void* y,
                                                                            int M, int K, int N, int group_size,
                                                                            void* workspace, size_t workspace_bytes,
                                                                            void* stream) {
    if (!qweight || !scales || !qzeros || !a || !y) return TF_ERR_NULL;
    if (M < 1 || M > TF_MAX_M_GEMV || N < 8 || N > TF_MAX_DIM || N % 8 != 0) return TF_ERR_SHAPE;
    if (group_size != 32 && group_size != 64 && group_size != 128) return TF_ERR_SHAPE;
    if (K < group_size || K > TF_MAX_DIM || K % group_size != 0) return TF_ERR_SHAPE;
    if (!aligned16(qweight) || !aligned16(scales) || !aligned16(qzeros) || !aligned16(a) || !aligned16(y))
        return TF_ERR_ALIGN;
    DeviceInfo dev;
    tf_status st = device_info(&dev);
    if (st != TF_OK) return st;
    if (workspace == nullptr || workspace_bytes < tf::gemv_raw_workspace_bytes(M, N, dev.sm_count)) return TF_ERR_WORKSPACE;
    if (!aligned16(workspace)) return TF_ERR_ALIGN;
    const tf::RawGemvPlan plan = tf::plan_gemv_raw(M, K, N, group_size, dev.sm_count);
    cudaError_t e = tf::launch_gemv_raw(plan, qweight, scales, qzeros, a, y, M, K, N, group_size, workspace,
                                        static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { cudaGetLastError(); return TF_ERR_CUDA; }
    return TF_OK;
}

extern "C" __attribute__((visibility("default"))) tf_status tf_pack_awq_device(const uint32_t* qweight, const uint16_t* scales,
                                                                               const uint32_t* qzeros, int K, int N, int group_size,
                                                                               void* out, size_t out_bytes, void* stream) {
    if (!qweight || !scales || !qzeros || !out) return TF_ERR_NULL;
    const size_t total = tf_packed_size(4, K, N, group_size);
    if (total == 0) return TF_ERR_SHAPE;
    if (out_bytes < total) return TF_ERR_WORKSPACE;
    if (!aligned16(qweight) || !aligned16(scales) || !aligned16(qzeros) || !aligned16(out)) return TF_ERR_ALIGN;
    DeviceInfo dev;
    tf_status st = device_info(&dev);
    if (st != TF_OK) return st;
    if (tf::launch_repack_awq(qweight, scales, qzeros, out, K, N, group_size, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        cudaGetLastError();
        return TF_ERR_CUDA;
    }
    return TF_OK;
}

// scratch of the raw-layout GEMM: the re-tiled blob (rounded up to 256 bytes), then the GEMM's own workspace
static size_t raw_gemm_blob_bytes(int K, int N, int group_size) {
    return (tf_packed_size(4, K, N, group_size) + 255) / 256 * 256;
}

extern "C" __attribute__((visibility("default"))) size_t tf_gemm_awq_raw_workspace_size(int M, int K, int N, int group_size) {
    if (M < 1 || M > TF_MAX_M_GEMM || tf_packed_size(4, K, N, group_size) == 0) return 0;
    return raw_gemm_blob_bytes(K, N, group_size) + tf::gemm_workspace_bytes(M, K, N);
}

extern "C" __attribute__((visibility("default"))) tf_status tf_gemm_awq_raw(const uint32_t* qweight, const uint16_t* scales,
                                                                            const uint32_t* qzeros, const void* a, void* y,
                                                                            int M, int K, int N, int group_size,
                                                                            void* workspace, size_t workspace_bytes, void* stream) {
    if (!qweight || !scales || !qzeros || !a || !y) return TF_ERR_NULL;
    if (M < 1 || M > TF_MAX_M_GEMM) return TF_ERR_SHAPE;
    const size_t need = tf_gemm_awq_raw_workspace_size(M, K, N, group_size);
    if (need == 0) return TF_ERR_SHAPE;
    if (workspace == nullptr || workspace_bytes < need) return TF_ERR_WORKSPACE;
    if (!aligned16(workspace)) return TF_ERR_ALIGN;
    const size_t blob_bytes = raw_gemm_blob_bytes(K, N, group_size);
    uint8_t* gemm_ws = static_cast<uint8_t*>(workspace);                 // the GEMM's workspace first: its head holds the status word
    uint8_t* blob = gemm_ws + tf::gemm_workspace_bytes(M, K, N);
    tf_status st = tf_pack_awq_device(qweight, scales, qzeros, K, N, group_size, blob, blob_bytes, stream);
    if (st != TF_OK) return st;
    return gemm(4, blob, a, y, M, K, N, gemm_ws, tf::gemm_workspace_bytes(M, K, N), stream, group_size);
}

extern "C" __attribute__((visibility("default"))) tf_status tf_device_status(const void* workspace, void* stream) {
    if (!workspace) return TF_ERR_NULL;
    uint32_t word[4] = {0, 0, 0, 0};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(word, workspace, sizeof(word), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return TF_ERR_CUDA;
    }
    return word[0] <= TF_ERR_TIMEOUT ? static_cast<tf_status>(word[0]) : TF_ERR_CUDA;
}

extern "C" __attribute__((visibility("default"))) const char* tf_status_string(tf_status status) {
    switch (status) {
        case TF_OK: return "ok";
        case TF_ERR_NULL: return "a required pointer is NULL";
        case TF_ERR_SHAPE: return "illegal M, K, N or group size";
        case TF_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case TF_ERR_BLOB: return "packed blob header does not match the arguments";
        case TF_ERR_WORKSPACE: return "workspace or output buffer too small";
        case TF_ERR_ARCH: return "device is not compute capability 10.x (B200)";
        case TF_ERR_CUDA: return "CUDA runtime call or kernel launch failed";
        case TF_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    }
    return "unknown status";
}

extern "C" __attribute__((visibility("default"))) int tf_version(void) { return 100; }
