// Fused W4A16 GEMV on the weights as the quantizer wrote them -- no offline pre-tiling.
//
// Section 5.5 of the paper separates two gains: fusing dequantization into the multiplication, and re-tiling
// the weights offline so that a worker streams exactly what it needs.  This kernel is the first without the
// second: it reads the AWQ arrays directly (qweight [K][N/8] u32 with eight columns per word in nibble order
// 0,2,4,6,1,3,5,7; scales [K/g][N] fp16; qzeros [K/g][N/8] u32 in the same nibble order), dequantizes in
// registers and accumulates in fp32.  The row-major layout has eight neighbouring *columns* in a word, while
// the tensor-core operand wants neighbouring *k*; without a transposition the products run on the fp32 pipe.
//
// Mapping: a lane owns one word column (eight output columns), a warp 32 of them (256 columns), the eight
// warps of a CTA split the rows of a quantization group between them, and the CTAs of one 256-column block
// split the groups (split-K).  Each CTA adds its warps' sums in warp order and writes an fp32 partial; a second
// kernel adds the partials in split order and rounds to bf16 once.  No atomics: results do not depend on timing.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "kernels.h"

namespace tf {
namespace {

constexpr int kRawWarps = 8;
constexpr int kRawThreads = 32 * kRawWarps;
constexpr int kRawColumns = 256;   // output columns of a CTA: 32 lanes x 8 columns of a word

__device__ __forceinline__ uint32_t ldg_nc_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

// The four bf16 pairs 128 + q of a word, pair i = columns (2i, 2i + 1) of the word's eight: the nibble order
// of the format puts columns 2i and 2i + 1 sixteen bits apart, so one mask per pair does it.
__device__ __forceinline__ void biased_pairs(uint32_t x, uint32_t (&p)[4]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) p[i] = ((x >> (4 * i)) & 0x000F000Fu) | 0x43004300u;
}

__device__ __forceinline__ uint32_t sub_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// MT tokens per pass, R = g / 8 rows of a group per warp.
template <int MT, int R>
__global__ void __launch_bounds__(kRawThreads)
gemv_awq_raw_kernel(const uint32_t* __restrict__ qweight, const uint16_t* __restrict__ scales,
                    const uint32_t* __restrict__ qzeros, const __nv_bfloat16* __restrict__ a,
                    float* __restrict__ partial, int M, int K, int N, int groups, int groups_per_cta) {
    extern __shared__ float red[];                      // [warps][MT][256]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int words = N >> 3;
    const int word = blockIdx.x * 32 + lane;
    const bool live = word < words;
    const int m0 = blockIdx.z * MT;
    const int g_begin = blockIdx.y * groups_per_cta;
    const int g_end = min(groups, g_begin + groups_per_cta);
    constexpr int kGroup = 8 * R;

    float acc[MT][8];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[m][c] = 0.f;

    for (int grp = g_begin; grp < g_end; ++grp) {
        const int k0 = grp * kGroup + warp * R;
        uint32_t x[R];
        if (live) {
#pragma unroll
            for (int r = 0; r < R; ++r) x[r] = ldg_nc_u32(qweight + (size_t)(k0 + r) * words + word);
        } else {
#pragma unroll
            for (int r = 0; r < R; ++r) x[r] = 0u;
        }
        uint32_t zp[4];
        float s[8];
        if (live) {
            biased_pairs(__ldg(qzeros + (size_t)grp * words + word), zp);
            const uint4 sv = __ldg(reinterpret_cast<const uint4*>(scales + (size_t)grp * N) + word);
            const uint32_t sw[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&sw[i]));
                s[2 * i] = f.x;
                s[2 * i + 1] = f.y;
            }
        } else {
            biased_pairs(0u, zp);
#pragma unroll
            for (int c = 0; c < 8; ++c) s[c] = 0.f;
        }
        float part[MT][8];
#pragma unroll
        for (int m = 0; m < MT; ++m)
#pragma unroll
            for (int c = 0; c < 8; ++c) part[m][c] = 0.f;
#pragma unroll
        for (int rb = 0; rb < R; rb += 4) {
            float av[MT][4];
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                uint2 raw = make_uint2(0u, 0u);
                if (m0 + m < M) raw = __ldg(reinterpret_cast<const uint2*>(a + (size_t)(m0 + m) * K + k0 + rb));
                av[m][0] = __uint_as_float(raw.x << 16);
                av[m][1] = __uint_as_float(raw.x & 0xFFFF0000u);
                av[m][2] = __uint_as_float(raw.y << 16);
                av[m][3] = __uint_as_float(raw.y & 0xFFFF0000u);
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                uint32_t qp[4];
                biased_pairs(x[rb + r], qp);
                float w[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t d = sub_bf16x2(qp[i], zp[i]);          // q - z, exact
                    w[2 * i] = __uint_as_float(d << 16);
                    w[2 * i + 1] = __uint_as_float(d & 0xFFFF0000u);
                }
#pragma unroll
                for (int m = 0; m < MT; ++m)
#pragma unroll
                    for (int c = 0; c < 8; ++c) part[m][c] = fmaf(av[m][r], w[c], part[m][c]);
            }
        }
#pragma unroll
        for (int m = 0; m < MT; ++m)
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[m][c] = fmaf(s[c], part[m][c], acc[m][c]);
    }

    // warps -> CTA, in warp order
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        float4* dst = reinterpret_cast<float4*>(red + ((size_t)warp * MT + m) * kRawColumns + lane * 8);
        dst[0] = make_float4(acc[m][0], acc[m][1], acc[m][2], acc[m][3]);
        dst[1] = make_float4(acc[m][4], acc[m][5], acc[m][6], acc[m][7]);
    }
    __syncthreads();
    const int n = blockIdx.x * kRawColumns + threadIdx.x;
    if (n < N) {
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            if (m0 + m >= M) break;
            float sum = 0.f;
#pragma unroll
            for (int w = 0; w < kRawWarps; ++w) sum += red[((size_t)w * MT + m) * kRawColumns + threadIdx.x];
            partial[((size_t)blockIdx.y * M + m0 + m) * N + n] = sum;
        }
    }
}

__global__ void __launch_bounds__(256)
gemv_awq_raw_finish_kernel(const float* __restrict__ partial, __nv_bfloat16* __restrict__ y, int MN, int splits) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= MN) return;
    float sum = 0.f;
    for (int s = 0; s < splits; ++s) sum += partial[(size_t)s * MN + i];
    y[i] = __float2bfloat16_rn(sum);
}

template <int MT, int R>
cudaError_t launch_raw(const RawGemvPlan& p, const uint32_t* qweight, const uint16_t* scales, const uint32_t* qzeros,
                       const void* a, float* partial, int M, int K, int N, cudaStream_t stream) {
    const int smem = kRawWarps * MT * kRawColumns * (int)sizeof(float);
    if (smem > 48 * 1024) {   // per device and cheap, so set on every launch rather than remembered
        cudaError_t e = cudaFuncSetAttribute(gemv_awq_raw_kernel<MT, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
    }
    dim3 grid(p.col_blocks, p.splits, (M + MT - 1) / MT);
    gemv_awq_raw_kernel<MT, R><<<grid, kRawThreads, smem, stream>>>(
        qweight, scales, qzeros, static_cast<const __nv_bfloat16*>(a), partial, M, K, N, p.groups, p.groups_per_cta);
    return cudaGetLastError();
}

template <int MT>
cudaError_t launch_raw_rows(const RawGemvPlan& p, int group_size, const uint32_t* qweight, const uint16_t* scales,
                            const uint32_t* qzeros, const void* a, float* partial, int M, int K, int N,
                            cudaStream_t stream) {
    switch (group_size) {
        case 32: return launch_raw<MT, 4>(p, qweight, scales, qzeros, a, partial, M, K, N, stream);
        case 64: return launch_raw<MT, 8>(p, qweight, scales, qzeros, a, partial, M, K, N, stream);
        default: return launch_raw<MT, 16>(p, qweight, scales, qzeros, a, partial, M, K, N, stream);
    }
}

}  // namespace

RawGemvPlan plan_gemv_raw(int K, int N, int group_size, int sm_count) {
    RawGemvPlan p;
    p.groups = K / group_size;
    p.col_blocks = (N / 8 + 31) / 32;
    // four CTAs per SM in flight is what the register budget allows; more splits only add partial sums
    const int want = (4 * sm_count + p.col_blocks - 1) / p.col_blocks;
    const int splits = want < p.groups ? want : p.groups;
    p.groups_per_cta = (p.groups + splits - 1) / splits;
    p.splits = (p.groups + p.groups_per_cta - 1) / p.groups_per_cta;
    return p;
}

size_t gemv_raw_workspace_bytes(int M, int N, int sm_count) {
    const int col_blocks = (N / 8 + 31) / 32;
    const size_t max_splits = (size_t)(4 * sm_count + col_blocks - 1) / col_blocks;
    return max_splits * (size_t)M * N * sizeof(float);
}

cudaError_t launch_gemv_raw(const RawGemvPlan& p, const uint32_t* qweight, const uint16_t* scales,
                            const uint32_t* qzeros, const void* a, void* y, int M, int K, int N, int group_size,
                            void* workspace, cudaStream_t stream) {
    float* partial = static_cast<float*>(workspace);
    note_whole_sm_launch(stream);   // not a half-SM GEMV: the next one must not assume it follows one
    cudaError_t e;
    if (M == 1) e = launch_raw_rows<1>(p, group_size, qweight, scales, qzeros, a, partial, M, K, N, stream);
    else if (M == 2) e = launch_raw_rows<2>(p, group_size, qweight, scales, qzeros, a, partial, M, K, N, stream);
    else if (M <= 4) e = launch_raw_rows<4>(p, group_size, qweight, scales, qzeros, a, partial, M, K, N, stream);
    else e = launch_raw_rows<8>(p, group_size, qweight, scales, qzeros, a, partial, M, K, N, stream);
    if (e != cudaSuccess) return e;
    const int MN = M * N;
    gemv_awq_raw_finish_kernel<<<(MN + 255) / 256, 256, 0, stream>>>(partial, static_cast<__nv_bfloat16*>(y), MN, p.splits);
    return cudaGetLastError();
}

}  // namespace tf
