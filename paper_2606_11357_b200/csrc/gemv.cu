// Decode-phase fused GEMV, M = 1..16 tokens (Sections 4.3 "GEMV microkernel" and 4.4).
//
// Work split: a CTA cluster owns one strip of 64 output columns for all K (the paper's rule that
// each worker owns distinct outputs and partial sums never travel between workers, Section 4.4);
// the cluster's CTAs and their warps split K tile by tile.  A warp streams whole packed tiles
// (128 k x 64 n, one contiguous payload with its scales and zeros) with 128-bit loads, turns
// the codes into exact small-integer bf16 values (q - z), and contracts them with the
// activations on the warp-level tensor-core MMA (weights = the 16x16 operand, up to 8 tokens =
// the 16x8 operand), so the cost per weight does not grow with M.  The fp16 scale multiplies the
// fp32 per-group sum once per 128 weights.  Partials are reduced through shared memory inside a
// CTA and through distributed shared memory inside the cluster, in a fixed order.
#include <cooperative_groups.h>

#include "common.cuh"
#include "kernels.h"

namespace cg = cooperative_groups;

namespace tf {

template <int BITS, int MT>
__global__ void __launch_bounds__(kGemvMaxThreads)
gemv_kernel(const uint8_t* __restrict__ blob, const __nv_bfloat16* __restrict__ a,
            __nv_bfloat16* __restrict__ y, int M, int K, int N, int ktiles, int tiles_per_cta,
            int cluster_size, DeviceStatus* status) {
    constexpr int kTileBytes = BITS == 4 ? kW4TileBytes : kW8TileBytes;
    constexpr int kWeightBytes = BITS == 4 ? kW4WeightBytes : kW8WeightBytes;
    constexpr int kTok = 8 * MT;                 // token slots per warp tile
    constexpr int kVecPerKb = BITS == 4 ? 1 : 2;  // 16-byte vectors per lane per k-block

    __shared__ __align__(16) float red[kGemvMaxThreads / 32][kTok][kTileN];

    const int strip = blockIdx.y;
    const int kx = blockIdx.x;                    // rank inside the cluster (cluster spans x)
    const int nwarps = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;

    const bool header_ok = header_matches(blob, BITS, (uint32_t)K, (uint32_t)N);

    const int t_begin = kx * tiles_per_cta;
    const int t_end = min(ktiles, t_begin + tiles_per_cta);
    const uint8_t* strip_base = blob + kHeaderBytes + (size_t)strip * ktiles * kTileBytes;

    float acc[4][MT][4];
#pragma unroll
    for (int w = 0; w < 4; ++w)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[w][mt][i] = 0.f;

    for (int T = t_begin + warp; T < t_end; T += nwarps) {
        const uint8_t* tile = strip_base + (size_t)T * kTileBytes;
        // ---- issue every load of the tile --------------------------------------------------
        uint4 wv[8 * kVecPerKb];
#pragma unroll
        for (int i = 0; i < 8 * kVecPerKb; ++i)
            wv[i] = ldg_stream(tile + ((size_t)i * 32 + lane) * 16);
        const uint4 sc = __ldg(reinterpret_cast<const uint4*>(tile + kWeightBytes) + g);
        uint32_t zword = 0;
        if (BITS == 4) zword = __ldg(reinterpret_cast<const uint32_t*>(tile + kWeightBytes + kScaleBytes) + g);
        uint4 av[MT][2][2];                       // [token tile][64-k chunk][half]
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            const int m = g + 8 * mt;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                if (m < M) {
                    const uint4* ap = reinterpret_cast<const uint4*>(a + (size_t)m * K + T * kTileK + 64 * c + 16 * t);
                    av[mt][c][0] = __ldg(ap);
                    av[mt][c][1] = __ldg(ap + 1);
                } else {
                    av[mt][c][0] = make_uint4(0, 0, 0, 0);
                    av[mt][c][1] = make_uint4(0, 0, 0, 0);
                }
            }
        }
        // ---- contract the 128 k of this group -------------------------------------------------
        uint32_t zg[4], zg8[4];
        if (BITS == 4) w4_zero_regs(zword, zg, zg8);
        float gacc[4][MT][4];
#pragma unroll
        for (int w = 0; w < 4; ++w)
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) gacc[w][mt][i] = 0.f;

#pragma unroll
        for (int kb = 0; kb < 8; ++kb) {
            uint32_t b0[MT], b1[MT];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const uint4 v = av[mt][kb >> 2][(kb & 3) >> 1];
                b0[mt] = (kb & 1) ? v.z : v.x;
                b1[mt] = (kb & 1) ? v.w : v.y;
            }
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                uint32_t r0, r1, r2, r3;
                if (BITS == 4) {
                    const uint4 v = wv[kb];
                    const uint32_t x = w == 0 ? v.x : w == 1 ? v.y : w == 2 ? v.z : v.w;
                    r0 = bf16x2_sub(w4_reg_biased(x, 0), zg[w]);
                    r1 = bf16x2_sub(w4_reg_biased(x, 1), zg8[w]);
                    r2 = bf16x2_sub(w4_reg_biased(x, 2), zg[w]);
                    r3 = bf16x2_sub(w4_reg_biased(x, 3), zg8[w]);
                } else {
                    const uint4 v = wv[kb * 2 + (w >> 1)];
                    w8_word_to_regs((w & 1) ? v.z : v.x, r0, r1);
                    w8_word_to_regs((w & 1) ? v.w : v.y, r2, r3);
                }
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) mma_bf16_16816(gacc[w][mt], r0, r1, r2, r3, b0[mt], b1[mt]);
            }
        }
        // ---- apply the group's scales in fp32 (Eq. 1 / Eq. 2 factored per group) ---------------
        const uint32_t sw[4] = {sc.x, sc.y, sc.z, sc.w};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float s_g = fp16_bits_to_float((uint16_t)(sw[w] & 0xFFFFu));
            const float s_g8 = fp16_bits_to_float((uint16_t)(sw[w] >> 16));
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                acc[w][mt][0] = fmaf(s_g, gacc[w][mt][0], acc[w][mt][0]);
                acc[w][mt][1] = fmaf(s_g, gacc[w][mt][1], acc[w][mt][1]);
                acc[w][mt][2] = fmaf(s_g8, gacc[w][mt][2], acc[w][mt][2]);
                acc[w][mt][3] = fmaf(s_g8, gacc[w][mt][3], acc[w][mt][3]);
            }
        }
    }

    // ---- reduce over the warps of this CTA (fixed order) ------------------------------------------
#pragma unroll
    for (int w = 0; w < 4; ++w)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            const int tok = 8 * mt + 2 * t;
            red[warp][tok][16 * w + g] = acc[w][mt][0];
            red[warp][tok + 1][16 * w + g] = acc[w][mt][1];
            red[warp][tok][16 * w + g + 8] = acc[w][mt][2];
            red[warp][tok + 1][16 * w + g + 8] = acc[w][mt][3];
        }
    __syncthreads();
    float* part = &red[0][0][0];                  // CTA partial, [token][n]
    for (int e = threadIdx.x; e < kTok * kTileN; e += blockDim.x) {
        float s = part[e];
        for (int w = 1; w < nwarps; ++w) s += (&red[w][0][0])[e];
        part[e] = s;                              // element e is touched by this thread only
    }

    // ---- reduce over the cluster through distributed shared memory, rank 0 stores -----------------
    if (cluster_size > 1) {
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();
        if (kx == 0 && header_ok) {
            for (int e = threadIdx.x; e < M * kTileN; e += blockDim.x) {
                float s = part[e];
                for (int r = 1; r < cluster_size; ++r) s += cluster.map_shared_rank(part, r)[e];
                const int m = e / kTileN, n = strip * kTileN + (e % kTileN);
                if (n < N) y[(size_t)m * N + n] = __float2bfloat16_rn(s);
            }
        }
        cluster.sync();                           // peers' shared memory stays alive until read
    } else if (header_ok) {
        __syncthreads();
        for (int e = threadIdx.x; e < M * kTileN; e += blockDim.x) {
            const int m = e / kTileN, n = strip * kTileN + (e % kTileN);
            if (n < N) y[(size_t)m * N + n] = __float2bfloat16_rn(part[e]);
        }
    }
    if (!header_ok && status != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
        status->code = TF_ERR_BLOB;
        status->detail = 1;
    }
}

// Shape -> launch geometry.  Aim for a few warps per SM sub-partition on all 148 SMs while
// keeping at least one whole tile per warp.
GemvPlan plan_gemv(int K, int N, int sm_count) {
    GemvPlan p;
    const int strips = (N + kTileN - 1) / kTileN, ktiles = K / kTileK;
    int cluster = 1;
    // grow the K split until there are about 4 CTAs per SM or a CTA would drop below 4 tiles
    while (cluster < 8 && strips * cluster < 4 * sm_count && ktiles / (cluster * 2) >= 4) cluster *= 2;
    const int tiles_per_cta = (ktiles + cluster - 1) / cluster;
    int warps = tiles_per_cta < 8 ? tiles_per_cta : 8;
    if (warps < 1) warps = 1;
    p.cluster = cluster;
    p.tiles_per_cta = tiles_per_cta;
    p.threads = warps * 32;
    p.strips = strips;
    p.ktiles = ktiles;
    return p;
}

template <int BITS, int MT>
static cudaError_t launch_one(const GemvPlan& p, const void* blob, const void* a, void* y, int M, int K,
                              int N, void* status, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.cluster, p.strips, 1);
    cfg.blockDim = dim3(p.threads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = p.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_kernel<BITS, MT>, static_cast<const uint8_t*>(blob),
                              static_cast<const __nv_bfloat16*>(a), static_cast<__nv_bfloat16*>(y), M, K, N,
                              p.ktiles, p.tiles_per_cta, p.cluster, static_cast<DeviceStatus*>(status));
}

cudaError_t launch_gemv(int bits, const GemvPlan& p, const void* blob, const void* a, void* y, int M, int K,
                        int N, void* status, cudaStream_t stream) {
    if (bits == 4) {
        return M <= 8 ? launch_one<4, 1>(p, blob, a, y, M, K, N, status, stream)
                      : launch_one<4, 2>(p, blob, a, y, M, K, N, status, stream);
    }
    return M <= 8 ? launch_one<8, 1>(p, blob, a, y, M, K, N, status, stream)
                  : launch_one<8, 2>(p, blob, a, y, M, K, N, status, stream);
}

}  // namespace tf
