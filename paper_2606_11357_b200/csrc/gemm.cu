// Prefill-phase fused GEMM (Section 4.3 "GEMM microkernel"), 1 <= M <= 4096 tokens.
//
// Output tile of one CTA: 128 weight columns (n) x BT tokens, computed "swapped": the dequantized
// weights are the 128-row operand of the tensor-core instruction, the activations the BT-column one,
//     D[n, token] = sum_k W[n, k] * A[token, k]          (tcgen05.mma, bf16 x bf16 -> fp32 in TMEM)
// so that each packed weight is unpacked and dequantized exactly once per CTA tile and then reused by
// all BT token rows (the dequantize-once rule of Section 4.1) and the dequant cost is as small as it
// can be relative to the MMA work.
//
// Persistent, warp-specialised CTA (512 threads):
//   warp 0      producer: bulk (TMA) copies of packed weight tiles (payload = weights + their scales
//               and zeros, Section 4.2) and tiled TMA loads of the activation tile (128B swizzle).
//   warp 1      one thread issues tcgen05.mma (4 per 64-wide k-step) and tcgen05.commit.
//   warp 2      allocates / frees tensor memory (two accumulators: epilogue overlaps the next tile).
//   warps 4-11  dequantize: packed words -> (q - z) exact in bf16 -> times bf16 scale -> bf16 operand
//               in shared memory in the K-major 128B-swizzled layout the MMA reads.
//   warps 12-15 epilogue: tcgen05.ld accumulator -> bf16 -> y.
// Every mbarrier wait is bounded; on a timeout all roles leave, TMEM is freed, the status word is set.
#include <cuda.h>

#include "async.cuh"
#include "common.cuh"
#include "kernels.h"

namespace tf {

namespace {

constexpr int kGemmThreads = 512;
constexpr int kBN = 128;                  // weight columns per CTA tile (two packed strips)
constexpr int kBK = 64;                   // k per pipeline step (one 128-byte swizzled row)
constexpr int kStages = 4;                // activation / dequantized-weight ring depth
constexpr int kAStageBytes = kBN * kBK * 2;            // 16 KB of dequantized weights per k-step
constexpr int kMaxWpStages = 3;

// packed-weight ring: one stage = the two strip tiles of one k-tile (= two k-steps)
__host__ __device__ constexpr int wp_strip_bytes(int bits) { return bits == 4 ? 4352 : 8320; }
__host__ __device__ constexpr int wp_stages(int bits) { return bits == 4 ? 3 : 2; }
__host__ __device__ constexpr int act_stage_bytes(int bt) { return bt * kBK * 2; }
__host__ __device__ constexpr int gemm_smem_bytes(int bits, int bt) {
    return 1024 /*alignment slack*/ + kStages * (act_stage_bytes(bt) + kAStageBytes) +
           wp_stages(bits) * 2 * wp_strip_bytes(bits) + 1024;
}

struct GemmBarriers {
    uint64_t act_full[kStages];
    uint64_t w_full[kStages];
    uint64_t ab_empty[kStages];
    uint64_t wp_full[kMaxWpStages];
    uint64_t wp_empty[kMaxWpStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    uint32_t abort_flag;
};

__device__ __forceinline__ uint32_t bf16_dup(float v) {
    const uint32_t b = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v));
    return b | (b << 16);
}

}  // namespace

template <int BITS, int BT>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap act_map, const uint8_t* __restrict__ blob,
            __nv_bfloat16* __restrict__ y, int M, int K, int N, int ktiles, int n_tiles, int m_tiles,
            uint8_t* __restrict__ workspace) {
    constexpr int kTileBytes = BITS == 4 ? kW4TileBytes : kW8TileBytes;
    constexpr int kWeightBytes = BITS == 4 ? kW4WeightBytes : kW8WeightBytes;
    constexpr int kActStage = act_stage_bytes(BT);
    constexpr int kWpStages = wp_stages(BITS);
    constexpr int kWpStripBytes = wp_strip_bytes(BITS);
    constexpr int kWpStageBytes = 2 * kWpStripBytes;
    constexpr uint32_t kTmemCols = 2 * BT < 32 ? 32 : 2 * BT;
    constexpr uint32_t kIdesc = umma_idesc_bf16(kBN, BT);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* act_ring = smem;                                        // kStages x kActStage   (1024-aligned)
    uint8_t* a_ring = act_ring + kStages * kActStage;                // kStages x 16 KB        (1024-aligned)
    uint8_t* wp_ring = a_ring + kStages * kAStageBytes;              // kWpStages x packed tiles
    GemmBarriers* bars = reinterpret_cast<GemmBarriers*>(wp_ring + kWpStages * kWpStageBytes);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = n_tiles * m_tiles;
    const int strips = (N + kTileN - 1) / kTileN;
    const bool header_ok = header_matches(blob, BITS, (uint32_t)K, (uint32_t)N);
    DeviceStatus* status = reinterpret_cast<DeviceStatus*>(workspace);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&bars->act_full[s]), 1);
            mbar_init(smem_u32(&bars->w_full[s]), 4);        // the four dequant warps of one k-half
            mbar_init(smem_u32(&bars->ab_empty[s]), 1);      // tcgen05.commit
        }
        for (int s = 0; s < kWpStages; ++s) {
            mbar_init(smem_u32(&bars->wp_full[s]), 1);
            mbar_init(smem_u32(&bars->wp_empty[s]), 8);      // all eight dequant warps
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bars->acc_full[b]), 1);
            mbar_init(smem_u32(&bars->acc_empty[b]), 4);     // four epilogue warps
        }
        bars->abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 2) {
        tmem_alloc(smem_u32(&bars->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (header_ok) {
        if (warp == 0 && lane == 0) {
            // ================= producer ====================================================================
            prefetch_tensormap(&act_map);
            uint32_t it = 0, wit = 0;
            for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
                const int n_tile = tile / m_tiles, m_tile = tile - n_tile * m_tiles;
                const int strip0 = 2 * n_tile;
                const int nstrips = (strip0 + 1 < strips) ? 2 : 1;
                bool ok = true;
                for (int T = 0; T < ktiles && ok; ++T, ++wit) {
                    const int ws = wit % kWpStages;
                    ok = mbar_wait(smem_u32(&bars->wp_empty[ws]), ((wit / kWpStages) & 1) ^ 1, abort_flag, 0x300 + ws);
                    if (!ok) break;
                    mbar_arrive_expect_tx(smem_u32(&bars->wp_full[ws]), nstrips * kTileBytes);
                    for (int q = 0; q < nstrips; ++q)
                        bulk_copy_g2s(smem_u32(wp_ring + ws * kWpStageBytes + q * kWpStripBytes),
                                      blob + kHeaderBytes + ((size_t)(strip0 + q) * ktiles + T) * kTileBytes, kTileBytes,
                                      smem_u32(&bars->wp_full[ws]));
                    for (int half = 0; half < 2; ++half, ++it) {
                        const int s = it % kStages;
                        ok = mbar_wait(smem_u32(&bars->ab_empty[s]), ((it / kStages) & 1) ^ 1, abort_flag, 0x310 + s);
                        if (!ok) break;
                        mbar_arrive_expect_tx(smem_u32(&bars->act_full[s]), kActStage);
                        tma_load_2d(smem_u32(act_ring + s * kActStage), &act_map, T * kTileK + half * kBK, m_tile * BT,
                                    smem_u32(&bars->act_full[s]));
                    }
                }
                if (!ok) break;
            }
        } else if (warp == 1 && lane == 0) {
            // ================= MMA issuer ==================================================================
            uint32_t it = 0, tile_it = 0;
            for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++tile_it) {
                const int buf = tile_it & 1;
                if (!mbar_wait(smem_u32(&bars->acc_empty[buf]), ((tile_it >> 1) & 1) ^ 1, abort_flag, 0x400 + buf)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BT;
                bool ok = true;
                for (int ks = 0; ks < 2 * ktiles; ++ks, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1;
                    ok = mbar_wait(smem_u32(&bars->w_full[s]), ph, abort_flag, 0x410 + s) &&
                         mbar_wait(smem_u32(&bars->act_full[s]), ph, abort_flag, 0x420 + s);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t a_desc = umma_desc_k_sw128(smem_u32(a_ring + s * kAStageBytes));
                    const uint64_t b_desc = umma_desc_k_sw128(smem_u32(act_ring + s * kActStage));
#pragma unroll
                    for (int j = 0; j < kBK / 16; ++j)       // 16 k per instruction = 32 bytes along the swizzled row
                        tc_mma_f16(d_tmem, a_desc + 2 * j, b_desc + 2 * j, kIdesc, (ks | j) != 0 ? 1u : 0u);
                    tc_commit(smem_u32(&bars->ab_empty[s]));
                }
                if (!ok) break;
                tc_commit(smem_u32(&bars->acc_full[buf]));
            }
        } else if (warp >= 4 && warp < 12) {
            // ================= dequantize: packed tile -> bf16 MMA operand ===================================
            const int dw = warp - 4;
            const int half = dw >> 2, strip_sel = (dw >> 1) & 1, kpl = dw & 1;
            const int kp = 2 * half + kpl;                   // k-block pair (kb = 2kp, 2kp+1) of the 128-k tile
            const int g = lane >> 2, t = lane & 3;
            const int chunk = 2 * t + kpl;                   // 16-byte chunk of the 128-byte row: k = 8*chunk .. +7
            uint32_t wit = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                const int n_tile = tile / m_tiles;
                const bool strip_exists = 2 * n_tile + strip_sel < strips;
                for (int T = 0; T < ktiles; ++T, ++wit) {
                    const int ws = wit % kWpStages;
                    ok = mbar_wait(smem_u32(&bars->wp_full[ws]), (wit / kWpStages) & 1, abort_flag, 0x500 + ws);
                    if (!ok) break;
                    const uint8_t* tile_smem = wp_ring + ws * kWpStageBytes + strip_sel * kWpStripBytes;
                    // operands of this thread: rows 16w+g and 16w+g+8 (w = 0..3), 8 consecutive k
                    uint32_t lo_g[4][2], lo_g8[4][2], hi_g[4][2], hi_g8[4][2];   // [w][k-pair] for k 0..3 / 4..7
                    const uint4 sc = *(reinterpret_cast<const uint4*>(tile_smem + kWeightBytes) + g);
                    if (BITS == 4) {
                        const uint4 x0 = *reinterpret_cast<const uint4*>(tile_smem + ((2 * kp) * 32 + lane) * 16);
                        const uint4 x1 = *reinterpret_cast<const uint4*>(tile_smem + ((2 * kp + 1) * 32 + lane) * 16);
                        const uint32_t zword = *(reinterpret_cast<const uint32_t*>(tile_smem + kWeightBytes + kScaleBytes) + g);
                        uint32_t zg[4], zg8[4];
                        w4_zero_regs(zword, zg, zg8);
                        const uint32_t xs0[4] = {x0.x, x0.y, x0.z, x0.w}, xs1[4] = {x1.x, x1.y, x1.z, x1.w};
#pragma unroll
                        for (int w = 0; w < 4; ++w) {
                            lo_g[w][0] = bf16x2_sub(w4_reg_biased(xs0[w], 0), zg[w]);
                            lo_g8[w][0] = bf16x2_sub(w4_reg_biased(xs0[w], 1), zg8[w]);
                            lo_g[w][1] = bf16x2_sub(w4_reg_biased(xs0[w], 2), zg[w]);
                            lo_g8[w][1] = bf16x2_sub(w4_reg_biased(xs0[w], 3), zg8[w]);
                            hi_g[w][0] = bf16x2_sub(w4_reg_biased(xs1[w], 0), zg[w]);
                            hi_g8[w][0] = bf16x2_sub(w4_reg_biased(xs1[w], 1), zg8[w]);
                            hi_g[w][1] = bf16x2_sub(w4_reg_biased(xs1[w], 2), zg[w]);
                            hi_g8[w][1] = bf16x2_sub(w4_reg_biased(xs1[w], 3), zg8[w]);
                        }
                    } else {
#pragma unroll
                        for (int h2 = 0; h2 < 2; ++h2) {
                            const uint4 x0 = *reinterpret_cast<const uint4*>(tile_smem + (((2 * kp) * 2 + h2) * 32 + lane) * 16);
                            const uint4 x1 = *reinterpret_cast<const uint4*>(tile_smem + (((2 * kp + 1) * 2 + h2) * 32 + lane) * 16);
                            w8_word_to_regs(x0.x, lo_g[2 * h2][0], lo_g8[2 * h2][0]);
                            w8_word_to_regs(x0.y, lo_g[2 * h2][1], lo_g8[2 * h2][1]);
                            w8_word_to_regs(x0.z, lo_g[2 * h2 + 1][0], lo_g8[2 * h2 + 1][0]);
                            w8_word_to_regs(x0.w, lo_g[2 * h2 + 1][1], lo_g8[2 * h2 + 1][1]);
                            w8_word_to_regs(x1.x, hi_g[2 * h2][0], hi_g8[2 * h2][0]);
                            w8_word_to_regs(x1.y, hi_g[2 * h2][1], hi_g8[2 * h2][1]);
                            w8_word_to_regs(x1.z, hi_g[2 * h2 + 1][0], hi_g8[2 * h2 + 1][0]);
                            w8_word_to_regs(x1.w, hi_g[2 * h2 + 1][1], hi_g8[2 * h2 + 1][1]);
                        }
                    }
                    // the packed stage is in registers now
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars->wp_empty[ws]));

                    // wait until the MMAs that read this operand stage (kStages steps ago) are done
                    const uint32_t it = 2 * wit + half;
                    const int s = it % kStages;
                    ok = mbar_wait(smem_u32(&bars->ab_empty[s]), ((it / kStages) & 1) ^ 1, abort_flag, 0x510 + s);
                    if (!ok) break;
                    uint8_t* a_stage = a_ring + s * kAStageBytes;
                    if (strip_exists) {
                        const uint32_t sw[4] = {sc.x, sc.y, sc.z, sc.w};
#pragma unroll
                        for (int w = 0; w < 4; ++w) {
                            const uint32_t s_g = bf16_dup(fp16_bits_to_float((uint16_t)(sw[w] & 0xFFFFu)));
                            const uint32_t s_g8 = bf16_dup(fp16_bits_to_float((uint16_t)(sw[w] >> 16)));
                            const int row = 64 * strip_sel + 16 * w + g;                  // row & 7 == g
                            uint4 v;
                            v.x = bf16x2_mul(lo_g[w][0], s_g);
                            v.y = bf16x2_mul(lo_g[w][1], s_g);
                            v.z = bf16x2_mul(hi_g[w][0], s_g);
                            v.w = bf16x2_mul(hi_g[w][1], s_g);
                            *reinterpret_cast<uint4*>(a_stage + row * 128 + ((chunk ^ g) << 4)) = v;
                            v.x = bf16x2_mul(lo_g8[w][0], s_g8);
                            v.y = bf16x2_mul(lo_g8[w][1], s_g8);
                            v.z = bf16x2_mul(hi_g8[w][0], s_g8);
                            v.w = bf16x2_mul(hi_g8[w][1], s_g8);
                            *reinterpret_cast<uint4*>(a_stage + (row + 8) * 128 + ((chunk ^ g) << 4)) = v;
                        }
                    }
                    fence_proxy_async_smem();                 // generic-proxy stores -> visible to the MMA
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars->w_full[s]));
                }
            }
        } else if (warp >= 12) {
            // ================= epilogue: TMEM -> bf16 -> y ===================================================
            const int quarter = warp - 12;                    // this warp may touch TMEM lanes 32*quarter .. +31
            uint32_t tile_it = 0;
            for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++tile_it) {
                const int n_tile = tile / m_tiles, m_tile = tile - n_tile * m_tiles;
                const int buf = tile_it & 1;
                if (!mbar_wait(smem_u32(&bars->acc_full[buf]), (tile_it >> 1) & 1, abort_flag, 0x600 + buf)) break;
                tc_fence_after();
                const int n = n_tile * kBN + 32 * quarter + lane;
                const uint32_t taddr = tmem_base + (uint32_t(32 * quarter) << 16) + buf * BT;
#pragma unroll 1
                for (int c = 0; c < BT / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld_32x32b_x32(taddr + 32 * c, v);
                    tmem_ld_wait();
                    const int tok0 = m_tile * BT + 32 * c;
                    if (n < N) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (tok0 + j < M) y[(size_t)(tok0 + j) * N + n] = __float2bfloat16_rn(__uint_as_float(v[j]));
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty[buf]));
            }
        }
    }

    // ---------------- teardown --------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) {
        if (!header_ok) {
            if (blockIdx.x == 0) { status->code = TF_ERR_BLOB; status->detail = 1; }
        } else if (bars->abort_flag != 0) {
            status->code = TF_ERR_TIMEOUT;
            status->detail = bars->abort_flag;
            const long long t_begin = clock64();              // let copies / MMAs in flight land before freeing
            while (clock64() - t_begin < 2000000ll) {}
        }
    }
    __syncthreads();
    if (warp == 2) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------------------------
size_t gemm_workspace_bytes(int M, int K, int N) {
    (void)M; (void)K; (void)N;
    return 4096;                                              // status word (+ room for split-K bookkeeping)
}

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is fetched through the runtime so the library never links against libcuda.
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

template <int BITS, int BT>
cudaError_t launch_bt(const void* blob, const void* a, void* y, int M, int K, int N, void* workspace, int sm_count,
                      cudaStream_t stream) {
    EncodeTiledFn encode = encode_tiled_fn();
    if (encode == nullptr) return cudaErrorNotSupported;
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)BT};
    const cuuint32_t estr[2] = {1, 1};
    if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(a), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;

    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemm_kernel<BITS, BT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             gemm_smem_bytes(BITS, BT));
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int n_tiles = (N + kBN - 1) / kBN, m_tiles = (M + BT - 1) / BT;
    const int total = n_tiles * m_tiles;
    const int grid = total < sm_count ? total : sm_count;
    gemm_kernel<BITS, BT><<<grid, kGemmThreads, gemm_smem_bytes(BITS, BT), stream>>>(
        map, static_cast<const uint8_t*>(blob), static_cast<__nv_bfloat16*>(y), M, K, N, K / kTileK, n_tiles, m_tiles,
        static_cast<uint8_t*>(workspace));
    return cudaGetLastError();
}

template <int BITS>
cudaError_t launch_bits(const void* blob, const void* a, void* y, int M, int K, int N, void* workspace, int sm_count,
                        cudaStream_t stream) {
    if (M > 128) return launch_bt<BITS, 256>(blob, a, y, M, K, N, workspace, sm_count, stream);
    if (M > 64) return launch_bt<BITS, 128>(blob, a, y, M, K, N, workspace, sm_count, stream);
    if (M > 32) return launch_bt<BITS, 64>(blob, a, y, M, K, N, workspace, sm_count, stream);
    return launch_bt<BITS, 32>(blob, a, y, M, K, N, workspace, sm_count, stream);
}

}  // namespace

cudaError_t launch_gemm(int bits, const void* blob, const void* a, void* y, int M, int K, int N, void* workspace,
                        size_t workspace_bytes, int sm_count, cudaStream_t stream) {
    (void)workspace_bytes;
    return bits == 4 ? launch_bits<4>(blob, a, y, M, K, N, workspace, sm_count, stream)
                     : launch_bits<8>(blob, a, y, M, K, N, workspace, sm_count, stream);
}

}  // namespace tf
