// tf_gemv_w4a16_static: the W4A16 decode GEMV for callers that may not allocate device memory.
//
// Some hosts of this library cannot hand it a workspace: a plug-in inside a serving process whose memory
// pool is owned (and already fully reserved) by another framework, a real-time thread that must never enter
// the allocator, or code between cudaStreamBeginCapture and EndCapture, where cudaMalloc is not allowed.
// For them the scratch the GEMV needs (the status word + one fp32 partial-sum slot per persistent CTA for strips cut
// between CTAs) lives in a fixed array in this library's own device image.  The entry point calls
// no cudaMalloc / cudaFree and no library routine that allocates.
//
// The array exists once per GPU that loads the library and stays until the process exits
// (kStaticScratchBytes, 675,840 bytes).  All calls share it and it keeps whatever the last call left: the status
// word is cleared on the stream before every launch, the partial-sum slots are zero when the library is loaded and
// every kernel that completes normally puts the zeros back (tf_gemv_w4a16_static_status clears the whole array when it
// reports an error), and two calls that overlap on the GPU (different streams, or graphs run concurrently) would race
// on it -- serialise them.
#include <cuda_runtime.h>

#include <atomic>

#include "../../include/tilefuse.h"
#include "kernels.h"
#include "layout.h"

namespace {

constexpr int kStaticMaxGrid = 160;                       // persistent CTAs the scratch has room for
constexpr size_t kStaticScratchBytes = tf::kGemvPartialOffset + (size_t)kStaticMaxGrid * tf::kGemvSlotBytes;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct PerDevice {
    std::atomic<int> state;   // 0 = not set up, 1 = ready, -1 = wrong architecture; published after the fields below
    int sm_count;
    void* scratch;            // device address of g_static_scratch on this device
};
PerDevice g_dev[64];

// In host code `g_static_scratch` is only a handle for the symbol, not a device address: the address the
// kernel needs comes from cudaGetSymbolAddress, asked once per device while that device is current.  The same
// first call does every other one-time step a GEMV launch can need (function attributes of every kernel variant,
// occupancy queries), so that later calls of any shape do nothing but launch.  Two host threads that make their
// first call at the same time both do the set-up and store the same values; `state` is written last (release), so
// a thread that sees 1 also sees the address.
tf_status setup_current_device(PerDevice** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return TF_ERR_CUDA; }
    PerDevice& d = g_dev[dev];
    int state = d.state.load(std::memory_order_acquire);
    if (state == 0) {
        int major = 0, sms = 0;
        void* ptr = nullptr;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError();
            return TF_ERR_CUDA;
        }
        if (major != 10) {
            state = -1;
        } else {
            if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
                cudaGetLastError();
                return TF_ERR_CUDA;
            }
            if (tf::configure_gemv_kernels() != cudaSuccess) { cudaGetLastError(); return TF_ERR_CUDA; }
            d.scratch = ptr;
            d.sm_count = sms;
            state = 1;
        }
        d.state.store(state, std::memory_order_release);
    }
    if (state != 1) return TF_ERR_ARCH;
    *out = &d;
    return TF_OK;
}

}  // namespace

extern "C" __attribute__((visibility("default")))
tf_status tf_gemv_w4a16_static(const void* packed, const void* a_bf16, void* y_bf16, int M, int K, int N,
                               void* cuda_stream) {
    if (!packed || !a_bf16 || !y_bf16) return TF_ERR_NULL;
    if (M < 1 || M > TF_MAX_M_GEMV) return TF_ERR_SHAPE;                       // beyond the scratch's stated maximum
    if (tf_packed_size(4, K, N, tf::kTileK) == 0) return TF_ERR_SHAPE;         // K, N > 32768 or not a legal shape
    const uintptr_t align = reinterpret_cast<uintptr_t>(packed) | reinterpret_cast<uintptr_t>(a_bf16) |
                            reinterpret_cast<uintptr_t>(y_bf16);
    if (align & 15u) return TF_ERR_ALIGN;
    PerDevice* dev = nullptr;
    tf_status st = setup_current_device(&dev);
    if (st != TF_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // status word and arrival counters must start at zero; the partial sums are always written before read
    if (cudaMemsetAsync(dev->scratch, 0, tf::kGemvStatusBytes, stream) != cudaSuccess) { cudaGetLastError(); return TF_ERR_CUDA; }
    const int ctas = dev->sm_count < kStaticMaxGrid ? dev->sm_count : kStaticMaxGrid;
    const tf::GemvPlan plan = tf::plan_gemv(4, M, K, N, ctas);
    if (tf::launch_gemv(4, plan, packed, a_bf16, y_bf16, M, K, N, dev->scratch, stream) != cudaSuccess) {
        cudaGetLastError();
        return TF_ERR_CUDA;
    }
    return TF_OK;
}

// The status word of the last tf_gemv_w4a16_static call on this device (every such call clears it before it
// launches): synchronises `cuda_stream` and reads the first word of the fixed scratch array.
extern "C" __attribute__((visibility("default")))
tf_status tf_gemv_w4a16_static_status(void* cuda_stream) {
    PerDevice* dev = nullptr;
    tf_status st = setup_current_device(&dev);
    if (st != TF_OK) return st;
    st = tf_device_status(dev->scratch, cuda_stream);
    if (st != TF_OK) {
        // a kernel that gave up may have left partial sums behind: the next call needs the slots zero again
        cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
        if (cudaMemsetAsync(dev->scratch, 0, kStaticScratchBytes, stream) != cudaSuccess || cudaStreamSynchronize(stream) != cudaSuccess) {
            cudaGetLastError();
            return TF_ERR_CUDA;
        }
    }
    return st;
}
