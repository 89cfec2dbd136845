// Decode-phase fused GEMV, M = 1..16 tokens (Sections 4.3 "GEMV microkernel" and 4.4).
//
// Persistent streaming kernel.  The packed blob is one long sequence of tiles (128 k x 64 n, each a
// contiguous payload carrying its scales and zeros, strip after strip).  That sequence is cut into
// equal contiguous ranges, one per CTA, so every CTA streams one contiguous byte range of HBM:
//
//   producer warp : one thread issues a bulk (TMA) copy per tile into a deep shared-memory ring,
//                   completion on mbarriers; bytes in flight are bounded by the ring, not by registers.
//   consumer warps: take tiles round-robin; 128-bit shared loads, codes -> exact small-integer bf16
//                   (q - z), contraction with the activations on the warp-level tensor-core MMA
//                   (weights = the 16x16 operand, up to 8 tokens = the 16x8 operand: the per-weight
//                   cost does not grow with M), fp16 scale applied in fp32 once per group.
//
// A range may cut a strip (64 output columns) in two.  A CTA that holds a whole strip stores y
// directly.  Otherwise it writes its fp32 partial to the workspace and bumps the strip's counter; the
// CTA that arrives last adds the partials in CTA order (not arrival order) and stores y, so results
// are deterministic and no CTA ever waits for another.  This keeps the paper's rule that partial sums
// do not travel between workers for everything but the (at most two) cut strips of a CTA.
#include "async.cuh"
#include "common.cuh"
#include "kernels.h"

namespace tf {

namespace {

__device__ __forceinline__ void consumer_bar_sync(int nthreads) {
    asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
}

__device__ __forceinline__ int range_start(int cta, int total, int grid) {
    return static_cast<int>((static_cast<long long>(cta) * total) / grid);
}
__device__ __forceinline__ int range_owner(int tile, int total, int grid) {
    return static_cast<int>(((static_cast<long long>(tile) + 1) * grid - 1) / total);
}

}  // namespace

template <int BITS, int MT>
__global__ void __launch_bounds__(kGemvMaxThreads, 1)
gemv_stream_kernel(const uint8_t* __restrict__ blob, const __nv_bfloat16* __restrict__ a,
                   __nv_bfloat16* __restrict__ y, int M, int K, int N, int ktiles, int total_tiles,
                   uint8_t* __restrict__ workspace) {
    constexpr int kTileBytes = BITS == 4 ? kW4TileBytes : kW8TileBytes;
    constexpr int kWeightBytes = BITS == 4 ? kW4WeightBytes : kW8WeightBytes;
    constexpr int kR = gemv_chunk_tiles(BITS);            // tiles per bulk copy / ring stage
    constexpr int kStageBytes = gemv_stage_bytes(BITS);
    constexpr int nstages = gemv_stages(BITS, MT);
    constexpr int kTok = 8 * MT;
    constexpr int kVecPerKb = BITS == 4 ? 1 : 2;

    extern __shared__ __align__(128) uint8_t smem[];
    // layout: [full barriers | empty barriers | flags] (1 KB) | red (consumers x kTok x 64 fp32) | ring
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + 2 * kGemvMaxStages * 8);
    volatile uint32_t* last_flag = abort_flag + 1;     // [2]: one per cut strip of this CTA
    int* contrib_off = reinterpret_cast<int*>(smem + 1024);   // [2][kGemvMaxContrib] partial-sum offsets
    const int nconsumers = (blockDim.x >> 5) - 1;
    float* red = reinterpret_cast<float*>(smem + kGemvBarrierBytes);
    uint8_t* ring = smem + kGemvBarrierBytes + nconsumers * kTok * kTileN * 4;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grid = gridDim.x, cta = blockIdx.x;
    const int t0 = range_start(cta, total_tiles, grid);
    const int ntiles = range_start(cta + 1, total_tiles, grid) - t0;

    DeviceStatus* status = reinterpret_cast<DeviceStatus*>(workspace);
    uint32_t* counters = reinterpret_cast<uint32_t*>(workspace + kGemvCounterOffset);
    float* partials = reinterpret_cast<float*>(workspace + kGemvPartialOffset);

    const bool header_ok = header_matches(blob, BITS, (uint32_t)K, (uint32_t)N);

    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kGemvMaxStages);
    if (threadIdx.x == 0) {
        for (int s = 0; s < nstages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, kR);       // every tile of a chunk is released by its consumer warp
        }
        *abort_flag = 0;
        mbar_init_fence();
    }
    __syncthreads();

    if (warp == 0) {
        // ---------------- producer: stream this CTA's contiguous tile range through the ring --------------
        // lanes 0..3 each issue every fourth chunk: one bulk copy of up to kR contiguous tiles
        if (lane < kGemvProducerLanes && header_ok) {
            const uint8_t* src = blob + kHeaderBytes + (size_t)t0 * kTileBytes;
            const int nchunks = (ntiles + kR - 1) / kR;
            for (int c = lane; c < nchunks; c += kGemvProducerLanes) {
                const int s = c % nstages, use = c / nstages;
                if (use >= 1 && !mbar_wait(empty0 + 8 * s, (use - 1) & 1, abort_flag, 0x100 + s)) break;
                const int tiles_here = min(kR, ntiles - c * kR);
                const uint32_t bytes = (uint32_t)tiles_here * kTileBytes;
                mbar_arrive_expect_tx(full0 + 8 * s, bytes);
                bulk_copy_g2s(smem_u32(ring + (size_t)s * kStageBytes), src + (size_t)c * kR * kTileBytes, bytes,
                              full0 + 8 * s);
            }
        }
    } else if (header_ok) {
        // ---------------- consumers ---------------------------------------------------------------------------
        const int cw = warp - 1, ctid = threadIdx.x - 32, cthreads = nconsumers * 32;
        const int g = lane >> 2, t = lane & 3;
        bool aborted = false;
        int cut0 = -1, cut1 = -1;                      // strips this CTA holds only a part of (head, tail)

        int i = 0;
        while (i < ntiles && !aborted) {
            const int tile0 = t0 + i;
            const int strip = tile0 / ktiles, T0 = tile0 - strip * ktiles;
            const int seg_len = min(ntiles - i, ktiles - T0);

            float acc[4][MT][4];
#pragma unroll
            for (int w = 0; w < 4; ++w)
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[w][mt][e] = 0.f;

            // first local tile index >= i handled by this warp
            int j = i + ((cw - (i % nconsumers)) + nconsumers) % nconsumers;
            for (; j < i + seg_len; j += nconsumers) {
                const int T = T0 + (j - i);
                // activations of this k-tile: lane (g, t) holds token g (+8), k = 16kb + 4t .. +3 per k-block
                uint2 av[MT][8];
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    const int m = g + 8 * mt;
                    const uint2* ap = reinterpret_cast<const uint2*>(a + (size_t)(m < M ? m : 0) * K + T * kTileK + 4 * t);
#pragma unroll
                    for (int kb = 0; kb < 8; ++kb) av[mt][kb] = m < M ? __ldg(ap + 4 * kb) : make_uint2(0u, 0u);
                }
                const int chunk = j / kR;
                const int s = chunk % nstages;
                if (!mbar_wait(full0 + 8 * s, (chunk / nstages) & 1, abort_flag, 0x200 + s)) { aborted = true; break; }
                const uint8_t* tile = ring + (size_t)s * kStageBytes + (size_t)(j - chunk * kR) * kTileBytes;

                const uint4 sc = *(reinterpret_cast<const uint4*>(tile + kWeightBytes) + g);
                uint32_t zg[4], zg8[4];
                if (BITS == 4) {
                    const uint32_t zword = *(reinterpret_cast<const uint32_t*>(tile + kWeightBytes + kScaleBytes) + g);
                    w4_zero_regs(zword, zg, zg8);
                }
                float gacc[4][MT][4];
#pragma unroll
                for (int w = 0; w < 4; ++w)
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                        for (int e = 0; e < 4; ++e) gacc[w][mt][e] = 0.f;

#pragma unroll
                for (int kb = 0; kb < 8; ++kb) {
                    uint32_t b0[MT], b1[MT];
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        b0[mt] = av[mt][kb].x;
                        b1[mt] = av[mt][kb].y;
                    }
                    uint4 wv[kVecPerKb];
#pragma unroll
                    for (int h = 0; h < kVecPerKb; ++h)
                        wv[h] = *reinterpret_cast<const uint4*>(tile + ((size_t)(kb * kVecPerKb + h) * 32 + lane) * 16);
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        uint32_t r0, r1, r2, r3;
                        if (BITS == 4) {
                            const uint4 v = wv[0];
                            const uint32_t x = w == 0 ? v.x : w == 1 ? v.y : w == 2 ? v.z : v.w;
                            r0 = bf16x2_sub(w4_reg_biased(x, 0), zg[w]);
                            r1 = bf16x2_sub(w4_reg_biased(x, 1), zg8[w]);
                            r2 = bf16x2_sub(w4_reg_biased(x, 2), zg[w]);
                            r3 = bf16x2_sub(w4_reg_biased(x, 3), zg8[w]);
                        } else {
                            const uint4 v = wv[(w >> 1) % kVecPerKb];
                            w8_word_to_regs((w & 1) ? v.z : v.x, r0, r1);
                            w8_word_to_regs((w & 1) ? v.w : v.y, r2, r3);
                        }
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) mma_bf16_16816(gacc[w][mt], r0, r1, r2, r3, b0[mt], b1[mt]);
                    }
                }
                // all shared-memory reads of this stage are done: hand it back to the producer
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8 * s);

                // the group's scales, in fp32 (Eq. 1 / Eq. 2 factored per group)
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

            // ---- reduce the segment over the consumer warps (fixed order) -------------------------------------
            float* mine = red + (size_t)cw * kTok * kTileN;
#pragma unroll
            for (int w = 0; w < 4; ++w)
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    const int tok = 8 * mt + 2 * t;
                    mine[tok * kTileN + 16 * w + g] = acc[w][mt][0];
                    mine[(tok + 1) * kTileN + 16 * w + g] = acc[w][mt][1];
                    mine[tok * kTileN + 16 * w + g + 8] = acc[w][mt][2];
                    mine[(tok + 1) * kTileN + 16 * w + g + 8] = acc[w][mt][3];
                }
            consumer_bar_sync(cthreads);
            if (*abort_flag != 0) { aborted = true; break; }

            const bool whole_strip = seg_len == ktiles;
            const int slot = (i == 0) ? 0 : 1;
            float* my_partial = partials + ((size_t)cta * 2 + slot) * (kGemvMaxM * kTileN);
            for (int e = ctid; e < M * kTileN; e += cthreads) {
                float sum = red[e];
                for (int w = 1; w < nconsumers; ++w) sum += red[(size_t)w * kTok * kTileN + e];
                if (whole_strip) {
                    const int m = e / kTileN, n = strip * kTileN + (e % kTileN);
                    if (n < N) y[(size_t)m * N + n] = __float2bfloat16_rn(sum);
                } else {
                    __stcg(my_partial + e, sum);               // published at the end of the kernel
                }
            }
            if (!whole_strip) { if (slot == 0) cut0 = strip; else cut1 = strip; }
            consumer_bar_sync(cthreads);                        // red is reused by the next segment
            i += seg_len;
        }

        // ---- publish the partial sums of the cut strips; the last CTA to arrive for a strip adds the
        //      partials in CTA order and stores y.  One thread per cut strip counts for the whole CTA with a
        //      release/acquire atomic (the barrier before it orders the other threads' stores ahead of it).
        if (!aborted && (cut0 >= 0 || cut1 >= 0)) {
            if (ctid < 2) {
                const int strip = ctid == 0 ? cut0 : cut1;
                uint32_t is_last = 0;
                if (strip >= 0) {
                    const int c_first = range_owner(strip * ktiles, total_tiles, grid);
                    const int c_last = range_owner(strip * ktiles + ktiles - 1, total_tiles, grid);
                    uint32_t prev;
                    asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(prev) : "l"(counters + strip) : "memory");
                    is_last = (prev == (uint32_t)(c_last - c_first)) ? 1u : 0u;
                }
                last_flag[ctid] = is_last;
            }
            consumer_bar_sync(cthreads);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int strip = q == 0 ? cut0 : cut1;
                if (strip < 0 || last_flag[q] == 0) continue;
                const int c_first = range_owner(strip * ktiles, total_tiles, grid);
                const int ncontrib = range_owner(strip * ktiles + ktiles - 1, total_tiles, grid) - c_first + 1;
                // contributor c's slot: 0 if its range starts inside this strip (head), else 1 (tail)
                for (int c = ctid; c < ncontrib; c += cthreads) {
                    const int cslot = range_start(c_first + c, total_tiles, grid) >= strip * ktiles ? 0 : 1;
                    contrib_off[q * kGemvMaxContrib + c] = ((c_first + c) * 2 + cslot) * (kGemvMaxM * kTileN);
                }
                consumer_bar_sync(cthreads);
                for (int e = ctid; e < M * kTileN; e += cthreads) {
                    float sum = 0.f;
#pragma unroll 4
                    for (int c = 0; c < ncontrib; ++c) sum += __ldcg(partials + contrib_off[q * kGemvMaxContrib + c] + e);
                    const int m = e / kTileN, n = strip * kTileN + (e % kTileN);
                    if (n < N) y[(size_t)m * N + n] = __float2bfloat16_rn(sum);
                }
                if (ctid == 0) counters[strip] = 0;            // leave the workspace ready for the next call
            }
        }
    }

    // ---------------- teardown: report, and never leave with copies in flight ------------------------------
    __syncthreads();
    if (threadIdx.x == 0) {
        if (!header_ok) {
            if (cta == 0) { status->code = TF_ERR_BLOB; status->detail = 1; }
        } else if (*abort_flag != 0) {
            status->code = TF_ERR_TIMEOUT;
            status->detail = *abort_flag;
            // copies still in flight land within microseconds; give them a bounded moment before the
            // shared memory of this CTA is released
            const long long t_begin = clock64();
            while (clock64() - t_begin < 2000000ll) {}
        }
    }
}

// Launch geometry: one persistent CTA per SM (fewer when there are fewer tiles than SMs).
GemvPlan plan_gemv(int bits, int M, int K, int N, int sm_count) {
    GemvPlan p;
    p.strips = (N + kTileN - 1) / kTileN;
    p.ktiles = K / kTileK;
    p.total_tiles = p.strips * p.ktiles;
    p.grid = p.total_tiles < sm_count ? p.total_tiles : sm_count;
    p.consumers = kGemvMaxConsumers;
    const int tiles_per_cta = (p.total_tiles + p.grid - 1) / p.grid;
    if (tiles_per_cta < p.consumers) p.consumers = tiles_per_cta < 4 ? 4 : tiles_per_cta;
    p.threads = 32 * (p.consumers + 1);
    const int mt = M <= 8 ? 1 : 2;
    p.stages = gemv_stages(bits, mt);
    p.smem_bytes = kGemvBarrierBytes + kGemvMaxConsumers * 8 * mt * kTileN * 4 + p.stages * gemv_stage_bytes(bits);
    return p;
}

template <int BITS, int MT>
static cudaError_t launch_one(const GemvPlan& p, const void* blob, const void* a, void* y, int M, int K,
                              int N, void* workspace, cudaStream_t stream) {
    static bool configured = false;       // the attribute is per kernel; setting it twice is harmless
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemv_stream_kernel<BITS, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kGemvSmemBudget);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    gemv_stream_kernel<BITS, MT><<<p.grid, p.threads, p.smem_bytes, stream>>>(
        static_cast<const uint8_t*>(blob), static_cast<const __nv_bfloat16*>(a), static_cast<__nv_bfloat16*>(y), M, K,
        N, p.ktiles, p.total_tiles, static_cast<uint8_t*>(workspace));
    return cudaGetLastError();
}

cudaError_t launch_gemv(int bits, const GemvPlan& p, const void* blob, const void* a, void* y, int M, int K,
                        int N, void* workspace, cudaStream_t stream) {
    if (bits == 4) {
        return M <= 8 ? launch_one<4, 1>(p, blob, a, y, M, K, N, workspace, stream)
                      : launch_one<4, 2>(p, blob, a, y, M, K, N, workspace, stream);
    }
    return M <= 8 ? launch_one<8, 1>(p, blob, a, y, M, K, N, workspace, stream)
                  : launch_one<8, 2>(p, blob, a, y, M, K, N, workspace, stream);
}

}  // namespace tf
