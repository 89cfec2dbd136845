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
constexpr int kRawFp32MaxM = 8;    // up to this many tokens the fp32 pipe is the cheaper one (measured, see below)

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

// ---- the same arm on the tensor cores (9 to 16 tokens) -----------------------------------------------------
// The fp32 kernel above costs 8 multiply-adds per word and token, so its time grows with the number of tokens.
// The alternative is to pay for the transposition: in `mma.sync.m16n8k16` with the tokens as the 16-row operand
// the weights are the 16 (k) x 8 (n) operand, and 8 columns is exactly one word.  Lane (g, t) of the fragment
// holds column g at four values of k, so it needs the word at rows 4t .. 4t + 3 and picks nibble g out of every
// one: one rotate per word, then a select and a mask per pair.  A warp brings a 16-row x 8-word block into a ring
// in shared memory with one coalesced 512-byte asynchronous copy, six blocks ahead, and every lane reads its 32
// words from there (the eight g-lanes share each address).  About 170 instructions per lane and block whatever
// the number of tokens; measured on 4096 x 14336 it takes 53 us for 1 to 16 tokens (the zero points, scales and
// activations of a block are fetched when it is processed, and that latency is what bounds it), where the fp32
// kernel takes 18 us for one token, 50 us for eight and 89 us for sixteen.  Hence: fp32 up to 8 tokens, this above.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f), "f"(0.f), "f"(0.f), "f"(0.f));
}

// Eight consecutive words of a row; `vec`: the row segment is 16-byte aligned and entirely inside the row.
__device__ __forceinline__ void load_words8(const uint32_t* p, bool vec, int valid, uint32_t (&x)[8]) {
    if (vec) {
        const uint4 lo = __ldg(reinterpret_cast<const uint4*>(p)), hi = __ldg(reinterpret_cast<const uint4*>(p) + 1);
        x[0] = lo.x; x[1] = lo.y; x[2] = lo.z; x[3] = lo.w; x[4] = hi.x; x[5] = hi.y; x[6] = hi.z; x[7] = hi.w;
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) x[j] = j < valid ? __ldg(p + j) : 0u;
    }
}

constexpr int kRawMmaColumns = 64;        // output columns of a CTA: eight words
constexpr int kRawMmaStages = 7;          // per-warp ring of 16-row x 8-word blocks (six in flight)
constexpr int kRawMmaStageBytes = 576;    // 16 rows x 32 bytes, 16 bytes of padding after every four rows
constexpr int kRawMmaRingBytes = 4096;    // per warp, >= 7 x 576
static_assert(kRawMmaStages * kRawMmaStageBytes <= kRawMmaRingBytes, "ring");
static_assert(kRawWarps * kRawMmaRingBytes <= kRawWarps * 16 * kRawMmaColumns * 4, "the ring lives where the reduction buffer is");

// Byte offset of (row, 16-byte half) inside a stage: the padding puts the rows 4t + r of the four t-groups of a
// fragment on different banks, so the eight-lane broadcast reads below are conflict-free.
__device__ __forceinline__ uint32_t raw_stage_offset(int row, int half) { return row * 32 + (row >> 2) * 16 + half * 16; }

__global__ void __launch_bounds__(kRawThreads, 2)
gemv_awq_raw_mma_kernel(const uint32_t* __restrict__ qweight, const uint16_t* __restrict__ scales,
                        const uint32_t* __restrict__ qzeros, const __nv_bfloat16* __restrict__ a,
                        float* __restrict__ partial, int M, int K, int N, int group_size, int blocks_per_cta) {
    __shared__ __align__(16) unsigned char smem[kRawWarps * 16 * kRawMmaColumns * 4];
    float (*red)[16][kRawMmaColumns] = reinterpret_cast<float (*)[16][kRawMmaColumns]>(smem);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int words = N >> 3;
    const int word0 = blockIdx.x * 8;
    const int valid = min(8, words - word0);
    const bool vec = (words & 3) == 0 && valid == 8;
    // nibble position of column g in a word (order 0,2,4,6,1,3,5,7), as rotate amounts that bring it to bit 0 / bit 16
    const int sh = 4 * ((g >> 1) + 4 * (g & 1));
    const int rot_lo = sh, rot_hi = (sh + 16) & 31;
    const int kblocks = K >> 4;
    const int b_begin = blockIdx.y * blocks_per_cta;
    const int b_end = min(kblocks, b_begin + blocks_per_cta);
    unsigned char* ring = smem + warp * kRawMmaRingBytes;
    const uint32_t ring_s = static_cast<uint32_t>(__cvta_generic_to_shared(ring));

    // lane L moves the 16 bytes (row L >> 1, half L & 1) of a block: one coalesced 512-byte request per warp
    const int my_row = lane >> 1, my_half = lane & 1;
    auto issue = [&](int b, int stage) {
        if (b < b_end) {
            const uint32_t* src = qweight + (size_t)(16 * b + my_row) * words + word0 + 4 * my_half;
            const uint32_t off = stage * kRawMmaStageBytes + raw_stage_offset(my_row, my_half);
            if (vec) {
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(ring_s + off), "l"(src) : "memory");
            } else {
                uint4 v;
                v.x = 4 * my_half + 0 < valid ? __ldg(src + 0) : 0u;
                v.y = 4 * my_half + 1 < valid ? __ldg(src + 1) : 0u;
                v.z = 4 * my_half + 2 < valid ? __ldg(src + 2) : 0u;
                v.w = 4 * my_half + 3 < valid ? __ldg(src + 3) : 0u;
                *reinterpret_cast<uint4*>(ring + off) = v;
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    float acc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[j][i] = 0.f;

#pragma unroll
    for (int s = 0; s < kRawMmaStages - 1; ++s) issue(b_begin + warp + s * kRawWarps, s);
    int stage = 0;
    for (int b = b_begin + warp; b < b_end; b += kRawWarps) {
        const int ahead = stage == 0 ? kRawMmaStages - 1 : stage - 1;        // the stage read in the previous iteration
        issue(b + (kRawMmaStages - 1) * kRawWarps, ahead);
        asm volatile("cp.async.wait_group %0;" :: "n"(kRawMmaStages - 1) : "memory");
        __syncwarp();
        const int k0 = 16 * b + 4 * t;
        const int grp = (16 * b) / group_size;
        uint32_t zw[8];
        load_words8(qzeros + (size_t)grp * words + word0, vec, valid, zw);
        uint32_t af[4];
        {
            uint2 lo = make_uint2(0u, 0u), hi = make_uint2(0u, 0u);
            if (g < M) lo = __ldg(reinterpret_cast<const uint2*>(a + (size_t)g * K + k0));
            if (g + 8 < M) hi = __ldg(reinterpret_cast<const uint2*>(a + (size_t)(g + 8) * K + k0));
            af[0] = lo.x; af[1] = hi.x; af[2] = lo.y; af[3] = hi.y;
        }
        const unsigned char* st = ring + stage * kRawMmaStageBytes;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            uint32_t x[4][4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const uint4 v = *reinterpret_cast<const uint4*>(st + raw_stage_offset(4 * t + r, half));
                x[r][0] = v.x; x[r][1] = v.y; x[r][2] = v.z; x[r][3] = v.w;
            }
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int j = 4 * half + jj;
                const uint32_t zr = __funnelshift_r(zw[j], zw[j], rot_lo) & 0xFu;
                const uint32_t zp = zr | (zr << 16) | 0x43004300u;
                uint32_t bq[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t lo = __funnelshift_r(x[2 * h][jj], x[2 * h][jj], rot_lo);
                    const uint32_t hi = __funnelshift_r(x[2 * h + 1][jj], x[2 * h + 1][jj], rot_hi);
                    const uint32_t both = (hi & 0xFFFF0000u) | (lo & 0x0000FFFFu);
                    bq[h] = sub_bf16x2((both & 0x000F000Fu) | 0x43004300u, zp);      // q - z, exact
                }
                float d[4];
                mma_bf16_16816(d, af, bq[0], bq[1]);
                float2 s = make_float2(0.f, 0.f);
                if (j < valid)
                    s = __half22float2(__ldg(reinterpret_cast<const __half2*>(scales + (size_t)grp * N + (size_t)(word0 + j) * 8) + t));
                acc[j][0] = fmaf(s.x, d[0], acc[j][0]);
                acc[j][1] = fmaf(s.y, d[1], acc[j][1]);
                acc[j][2] = fmaf(s.x, d[2], acc[j][2]);
                acc[j][3] = fmaf(s.y, d[3], acc[j][3]);
            }
        }
        __syncwarp();                                   // every lane is done with this stage before it is refilled
        stage = stage + 1 == kRawMmaStages ? 0 : stage + 1;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();                                    // the rings are dead: their memory becomes the reduction buffer

#pragma unroll
    for (int j = 0; j < 8; ++j) {
        *reinterpret_cast<float2*>(&red[warp][g][8 * j + 2 * t]) = make_float2(acc[j][0], acc[j][1]);
        *reinterpret_cast<float2*>(&red[warp][g + 8][8 * j + 2 * t]) = make_float2(acc[j][2], acc[j][3]);
    }
    __syncthreads();
    for (int o = threadIdx.x; o < 16 * kRawMmaColumns; o += kRawThreads) {
        const int m = o >> 6, c = o & 63;
        const int n = blockIdx.x * kRawMmaColumns + c;
        if (m >= M || n >= N) continue;
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < kRawWarps; ++w) sum += red[w][m][c];
        partial[((size_t)blockIdx.y * M + m) * N + n] = sum;
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

RawGemvPlan plan_gemv_raw(int M, int K, int N, int group_size, int sm_count) {
    RawGemvPlan p;
    p.mma = M > kRawFp32MaxM;
    if (p.mma) {
        // units of 16 rows; two CTAs per SM fit (registers), and every warp of a CTA should get a block
        const int kblocks = K / 16;
        p.groups = kblocks;
        p.col_blocks = (N + kRawMmaColumns - 1) / kRawMmaColumns;
        int want = (2 * sm_count + p.col_blocks - 1) / p.col_blocks;
        const int most = (kblocks + kRawWarps - 1) / kRawWarps;
        if (want > most) want = most;
        p.groups_per_cta = (kblocks + want - 1) / want;
        p.splits = (kblocks + p.groups_per_cta - 1) / p.groups_per_cta;
        return p;
    }
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
    const int col_blocks = M > kRawFp32MaxM ? (N + kRawMmaColumns - 1) / kRawMmaColumns : (N / 8 + 31) / 32;
    const size_t max_splits = (size_t)((M > kRawFp32MaxM ? 2 : 4) * sm_count + col_blocks - 1) / col_blocks;
    return max_splits * (size_t)M * N * sizeof(float);
}

cudaError_t launch_gemv_raw(const RawGemvPlan& p, const uint32_t* qweight, const uint16_t* scales,
                            const uint32_t* qzeros, const void* a, void* y, int M, int K, int N, int group_size,
                            void* workspace, cudaStream_t stream) {
    float* partial = static_cast<float*>(workspace);
    note_whole_sm_launch(stream);   // not a half-SM GEMV: the next one must not assume it follows one
    cudaError_t e;
    if (p.mma) {
        dim3 grid(p.col_blocks, p.splits, 1);
        gemv_awq_raw_mma_kernel<<<grid, kRawThreads, 0, stream>>>(qweight, scales, qzeros, static_cast<const __nv_bfloat16*>(a),
                                                                  partial, M, K, N, group_size, p.groups_per_cta);
        e = cudaGetLastError();
    } else if (M == 1) e = launch_raw_rows<1>(p, group_size, qweight, scales, qzeros, a, partial, M, K, N, stream);
    else if (M == 2) e = launch_raw_rows<2>(p, group_size, qweight, scales, qzeros, a, partial, M, K, N, stream);
    else if (M <= 4) e = launch_raw_rows<4>(p, group_size, qweight, scales, qzeros, a, partial, M, K, N, stream);
    else e = launch_raw_rows<8>(p, group_size, qweight, scales, qzeros, a, partial, M, K, N, stream);
    if (e != cudaSuccess) return e;
    const int MN = M * N;
    gemv_awq_raw_finish_kernel<<<(MN + 255) / 256, 256, 0, stream>>>(partial, static_cast<__nv_bfloat16*>(y), MN, p.splits);
    return cudaGetLastError();
}

}  // namespace tf
