// Blob -> plain arrays, on the GPU, through the same unpack helpers the GEMV / GEMM use
// (the "unpacking" step of Section 4.3).  Bit-exact by construction of the helpers: the values
// 128 + q (4-bit) and q (int8) are exact in bf16 and are turned back into integers here.
#include "common.cuh"
#include "kernels.h"

namespace tf {

__device__ __forceinline__ int bf16_bits_to_int(uint32_t bits16) {
    return (int)__uint_as_float(bits16 << 16);
}

// One thread per packed word (W4) / per pair of words (W8): thread id -> (strip, ktile, kb, lane, w).
template <int BITS>
__global__ void unpack_kernel(const uint8_t* __restrict__ blob, uint8_t* __restrict__ q,
                              uint8_t* __restrict__ z, uint16_t* __restrict__ s, int K, int N,
                              int group_size, int ktiles, long long total_items) {
    constexpr int kWeightBytes = BITS == 4 ? kW4WeightBytes : kW8WeightBytes;
    if (!header_matches(blob, BITS, (uint32_t)K, (uint32_t)N) || header_group_size(blob) != (uint32_t)group_size) return;
    const int G = groups_per_tile(group_size);                       // groups inside one tile (4-bit, group size 64 / 32)
    const int kTileBytes = tile_bytes(BITS, G);
    const long long item = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (item >= total_items) return;
    const int w = item & 3, lane = (item >> 2) & 31, kb = (item >> 7) & 7;
    const long long tile_id = item >> 10;
    const int T = (int)(tile_id % ktiles), S = (int)(tile_id / ktiles);
    const int g = lane >> 2, t = lane & 3;
    const uint8_t* tile = blob + kHeaderBytes + (size_t)tile_id * kTileBytes;
    const int k0 = T * kTileK, n0 = S * kTileN;

    uint32_t r[4];
    if (BITS == 4) {
        const uint32_t x = reinterpret_cast<const uint32_t*>(tile)[(kb * 32 + lane) * 4 + w];
#pragma unroll
        for (int i = 0; i < 4; ++i) r[i] = bf16x2_sub(w4_reg_biased(x, i), 0x43004300u);   // exact q
    } else {
        const uint32_t* v = reinterpret_cast<const uint32_t*>(tile) + ((kb * 2 + (w >> 1)) * 32 + lane) * 4 + 2 * (w & 1);
        w8_word_to_regs(v[0], r[0], r[1]);
        w8_word_to_regs(v[1], r[2], r[3]);
    }
    if (q != nullptr) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int el = 0; el < 2; ++el) {
                const int k = k0 + 16 * kb + 4 * t + 2 * (i >> 1) + el;
                const int n = n0 + 16 * w + g + 8 * (i & 1);
                const int val = bf16_bits_to_int(el ? (r[i] >> 16) : (r[i] & 0xFFFFu));
                if (n < N) q[(size_t)k * N + n] = (uint8_t)val;
            }
    }
    // metadata: the threads with t == 0 of k-block gr < G write group gr of the tile (of the first tile of a group
    // that spans several tiles)
    if (kb < G && t == 0 && (G > 1 || (k0 % group_size) == 0)) {
        const int gr = kb;
        const int grp = G > 1 ? T * G + gr : k0 / group_size;
        const uint16_t* sc = reinterpret_cast<const uint16_t*>(tile + kWeightBytes + gr * kScaleBytes) + g * 8;
        uint32_t zg[4], zg8[4];
        if (BITS == 4) {
            const uint32_t zword = reinterpret_cast<const uint32_t*>(tile + w4_zero_offset(G, gr))[g];
            w4_zero_regs(zword, zg, zg8);
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int n = n0 + 16 * w + g + 8 * h;
            if (n >= N) continue;
            if (s != nullptr) s[(size_t)grp * N + n] = sc[2 * w + h];
            if (BITS == 4 && z != nullptr) {
                const uint32_t pair = h ? zg8[0 + w] : zg[0 + w];     // (128 + z) duplicated
                z[(size_t)grp * N + n] = (uint8_t)(bf16_bits_to_int(pair & 0xFFFFu) - 128);
            }
        }
    }
}

template <int BITS>
static cudaError_t launch_unpack(const void* blob, uint8_t* q, uint8_t* z, uint16_t* s, int K, int N,
                                 int group_size, cudaStream_t stream) {
    const int strips = (N + kTileN - 1) / kTileN, ktiles = K / kTileK;
    const long long items = (long long)strips * ktiles * 1024;
    const int threads = 256;
    const long long blocks = (items + threads - 1) / threads;
    unpack_kernel<BITS><<<(unsigned)blocks, threads, 0, stream>>>(static_cast<const uint8_t*>(blob), q, z, s, K, N,
                                                                 group_size, ktiles, items);
    return cudaGetLastError();
}

cudaError_t launch_unpack_w4(const void* blob, uint8_t* q, uint8_t* z, uint16_t* s, int K, int N,
                             int group_size, cudaStream_t stream) {
    return launch_unpack<4>(blob, q, z, s, K, N, group_size, stream);
}
cudaError_t launch_unpack_w8(const void* blob, int8_t* q, uint16_t* s, int K, int N, int group_size,
                             cudaStream_t stream) {
    return launch_unpack<8>(blob, reinterpret_cast<uint8_t*>(q), nullptr, s, K, N, group_size, stream);
}

// Blob -> the full-precision weight matrix in global memory, w[k][n] = bf16((q - z) * s): the "dequantize into memory,
// then multiply" arrangement that the fused kernels exist to avoid (Section 4.1), kept as the baseline of the
// ablation (Section 5.5).  (q - z) * s is exact in fp32 (at most 8 x 11 significant bits), so the only rounding is
// the one to bf16.  One CTA per tile; the tile is assembled in shared memory and stored as whole 128-byte rows.
template <int BITS>
__global__ void __launch_bounds__(256) dequant_kernel(const uint8_t* __restrict__ blob, __nv_bfloat16* __restrict__ wout, int K,
                                                      int N, int ktiles) {
    constexpr int kWeightBytes = BITS == 4 ? kW4WeightBytes : kW8WeightBytes;
    constexpr int kRow = kTileN + 8;                                 // padded row of the staging tile (bf16 elements)
    __shared__ __align__(16) __nv_bfloat16 stage[kTileK * kRow];
    if (!header_matches(blob, BITS, (uint32_t)K, (uint32_t)N)) return;
    const int G = groups_per_tile((int)header_group_size(blob));
    const int kTileBytes = tile_bytes(BITS, G);
    const int tile_id = blockIdx.x;
    const int T = tile_id % ktiles, S = tile_id / ktiles;
    const uint8_t* tile = blob + kHeaderBytes + (size_t)tile_id * kTileBytes;
    for (int item = threadIdx.x; item < 1024; item += 256) {
        const int w = item & 3, lane = (item >> 2) & 31, kb = item >> 7;
        const int g = lane >> 2, t = lane & 3;
        const int gr = kb / (8 / G);                                 // the group of this k-block inside the tile
        const uint16_t* scales = reinterpret_cast<const uint16_t*>(tile + kWeightBytes + gr * kScaleBytes);
        uint32_t r[4];
        if (BITS == 4) {
            const uint32_t x = reinterpret_cast<const uint32_t*>(tile)[(kb * 32 + lane) * 4 + w];
            const uint32_t zword = reinterpret_cast<const uint32_t*>(tile + w4_zero_offset(G, gr))[g];
            const uint32_t pair = w4_reg_biased(zword, w);                         // (128 + z[row g], 128 + z[row g+8])
            const uint32_t zg = __byte_perm(pair, 0, 0x1010), zg8 = __byte_perm(pair, 0, 0x3232);
#pragma unroll
            for (int i = 0; i < 4; ++i) r[i] = bf16x2_sub(w4_reg_biased(x, i), (i & 1) ? zg8 : zg);   // exact q - z
        } else {
            const uint32_t* v = reinterpret_cast<const uint32_t*>(tile) + ((kb * 2 + (w >> 1)) * 32 + lane) * 4 + 2 * (w & 1);
            w8_word_to_regs(v[0], r[0], r[1]);
            w8_word_to_regs(v[1], r[2], r[3]);
        }
        const float s_g = fp16_bits_to_float(scales[g * 8 + 2 * w]), s_g8 = fp16_bits_to_float(scales[g * 8 + 2 * w + 1]);
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int el = 0; el < 2; ++el) {
                const int k = 16 * kb + 4 * t + 2 * (i >> 1) + el;
                const int n = 16 * w + g + 8 * (i & 1);
                const float v = __uint_as_float(el ? (r[i] & 0xFFFF0000u) : (r[i] << 16)) * ((i & 1) ? s_g8 : s_g);
                stage[k * kRow + n] = __float2bfloat16_rn(v);
            }
    }
    __syncthreads();
    const int k0 = T * kTileK, n0 = S * kTileN;
    for (int item = threadIdx.x; item < kTileK * 8; item += 256) {
        const int row = item >> 3, chunk = item & 7;
        const int n = n0 + 8 * chunk;
        if (n < N)                                                   // N % 8 == 0: a group of 8 columns is in or out
            *reinterpret_cast<uint4*>(wout + (size_t)(k0 + row) * N + n) = *reinterpret_cast<const uint4*>(stage + row * kRow + 8 * chunk);
    }
}

cudaError_t launch_dequant(int bits, const void* blob, void* w_bf16, int K, int N, cudaStream_t stream) {
    const int strips = (N + kTileN - 1) / kTileN, ktiles = K / kTileK;
    if (bits == 4)
        dequant_kernel<4><<<strips * ktiles, 256, 0, stream>>>(static_cast<const uint8_t*>(blob), static_cast<__nv_bfloat16*>(w_bf16), K, N, ktiles);
    else
        dequant_kernel<8><<<strips * ktiles, 256, 0, stream>>>(static_cast<const uint8_t*>(blob), static_cast<__nv_bfloat16*>(w_bf16), K, N, ktiles);
    return cudaGetLastError();
}

}  // namespace tf
