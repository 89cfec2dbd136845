// Pre-tiling on the GPU (Section 4.2 done at run time instead of offline), and the GEMM arm of the layout ablation
// (Section 5.5): the fused GEMM computed from the AWQ arrays as the quantizer wrote them, i.e. re-tiled on the fly
// into scratch memory by the kernel below and then multiplied by the pre-tiled GEMM.  What the paper's offline
// pre-tiling saves is exactly this pass per call.  The device packer writes, byte for byte, what tf_pack_awq writes.
#include <cuda_runtime.h>

#include "../../include/tilefuse.h"
#include "kernels.h"
#include "layout.h"

namespace tf {

namespace {

__device__ __forceinline__ uint32_t awq_code_dev(const uint32_t* __restrict__ words, size_t row_words, int r, int c) {
    // nibble position of column c % 8 in the AWQ order 0,2,4,6,1,3,5,7: positions 0,4,1,5,2,6,3,7
    const int pos = ((c & 1) << 2) | ((c & 7) >> 1);
    return (__ldg(words + (size_t)r * row_words + (c >> 3)) >> (4 * pos)) & 0xFu;
}

// One thread per 32-bit word of the output blob's tiles (weights, scale pairs, zero words), plus the header.
__global__ void __launch_bounds__(256) repack_awq_kernel(const uint32_t* __restrict__ qweight, const uint16_t* __restrict__ scales,
                                                         const uint32_t* __restrict__ qzeros, uint8_t* __restrict__ out, int K, int N,
                                                         int group_size, int ktiles, int strips, long long total_words) {
    const int G = groups_per_tile(group_size);
    const int tile_words = w4_tile_bytes(G) / 4;
    const long long item = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (item == 0) {
        tf_blob_header h = {};
        h.magic = kMagic; h.version = kBlobVersion; h.bits = 4; h.K = (uint32_t)K; h.N = (uint32_t)N;
        h.group_size = (uint32_t)group_size; h.n_padded = (uint32_t)(strips * kTileN); h.strips = (uint32_t)strips;
        h.ktiles = (uint32_t)ktiles; h.tile_bytes = (uint32_t)w4_tile_bytes(G); h.tiles_offset = kHeaderBytes;
        h.total_bytes = (uint64_t)kHeaderBytes + (uint64_t)strips * ktiles * w4_tile_bytes(G);
        *reinterpret_cast<tf_blob_header*>(out) = h;
    }
    if (item >= total_words) return;
    const long long tile_id = item / tile_words;
    const int wi = (int)(item - tile_id * tile_words);
    const int T = (int)(tile_id % ktiles), S = (int)(tile_id / ktiles);
    const int k0 = T * kTileK, n0 = S * kTileN;
    const size_t row_words = (size_t)N / 8;
    uint32_t word = 0;
    if (wi < kW4WeightBytes / 4) {
        const int w = wi & 3, lane = (wi >> 2) & 31, kb = wi >> 7;
        const int g = lane >> 2, t = lane & 3;
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            const int reg = p & 3, el = p >> 2;
            const int k = k0 + 16 * kb + 4 * t + 2 * (reg >> 1) + el;
            const int n = n0 + 16 * w + g + 8 * (reg & 1);
            const uint32_t code = n < N ? awq_code_dev(qweight, row_words, k, n) : 0u;     // padded columns: q = z = 0, s = 0
            word |= code << (4 * p);
        }
    } else if (wi < (kW4WeightBytes + G * kScaleBytes) / 4) {
        const int si = wi - kW4WeightBytes / 4;                       // scale pair index: [group][g][w] -> (2w, 2w+1) = columns +0, +8
        const int gr = si / (kScaleBytes / 4), rest = si % (kScaleBytes / 4);
        const int g = rest >> 2, w = rest & 3;
        const int grp = G > 1 ? T * G + gr : k0 / group_size;
        const int n = n0 + 16 * w + g;
        const uint32_t lo = n < N ? __ldg(scales + (size_t)grp * N + n) : 0u;
        const uint32_t hi = n + 8 < N ? __ldg(scales + (size_t)grp * N + n + 8) : 0u;
        word = lo | (hi << 16);
    } else {
        const int zi = wi - (kW4WeightBytes + G * kScaleBytes) / 4;   // zero word index: [group][g]
        const int gr = zi / (kZeroBytes / 4), g = zi % (kZeroBytes / 4);
        const int grp = G > 1 ? T * G + gr : k0 / group_size;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int n = n0 + 16 * (i & 3) + g + 8 * (i >> 2);
            const uint32_t code = n < N ? awq_code_dev(qzeros, row_words, grp, n) : 0u;
            word |= code << (4 * i);
        }
    }
    reinterpret_cast<uint32_t*>(out + kHeaderBytes)[item] = word;
}

}  // namespace

cudaError_t launch_repack_awq(const uint32_t* qweight, const uint16_t* scales, const uint32_t* qzeros, void* out, int K, int N,
                              int group_size, cudaStream_t stream) {
    const int strips = (N + kTileN - 1) / kTileN, ktiles = K / kTileK;
    const long long words = (long long)strips * ktiles * (w4_tile_bytes(groups_per_tile(group_size)) / 4);
    const long long blocks = (words + 255) / 256;
    repack_awq_kernel<<<(unsigned)blocks, 256, 0, stream>>>(qweight, scales, qzeros, static_cast<uint8_t*>(out), K, N, group_size,
                                                            ktiles, strips, words);
    return cudaGetLastError();
}

}  // namespace tf
