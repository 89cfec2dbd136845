// Prefill-phase fused GEMM (Section 4.3 "GEMM microkernel"), 1 <= M <= 4096 tokens.
//
// Output tile of one CTA: 128 weight columns (n) x BT tokens, computed "swapped": the dequantized
// weights are the 128-row operand of the tensor-core instruction, the activations the BT-column one,
//     D[n, token] = sum_k W[n, k] * A[token, k]          (tcgen05.mma, bf16 x bf16 -> fp32 in TMEM)
// so that each packed weight is unpacked and dequantized exactly once per CTA tile and then reused by
// all BT token rows (the dequantize-once rule of Section 4.1).
//
// The dequantized weights never touch shared memory: the dequant warps write them with tcgen05.st
// straight into tensor memory, from where tcgen05.mma reads its 128-row operand.  Shared memory then
// carries only the packed 4/8-bit tiles and the activations, which is what keeps the tensor pipe fed:
// with the bf16 weights staged in shared memory the kernel was bound by shared-memory bandwidth.
// Tensor memory (512 columns): accumulator [0, BT), weight-operand ring [256, 256 + 4 x 32).
//
// Persistent, warp-specialised CTA (512 threads):
//   warp 0      producer A: tiled TMA loads of the activation tile (128B swizzle), one per 64-wide k-step.
//   warp 3      producer W: bulk (TMA) copies of packed weight tiles (payload = weights + their scales
//               and zeros, Section 4.2).
//   warp 1      one thread issues tcgen05.mma (4 per k-step) and tcgen05.commit.
//   warp 2      allocates / frees tensor memory.
//   warps 4-11  dequantize: packed words -> (q - z) exact in bf16 -> times the scale, one rounding (split_scale) -> tcgen05.st.  The
//               packed words are stored in the register order of the 16x256b store, so a word goes from
//               shared memory to the tensor-memory operand without any shuffle.
//   warps 12-15 epilogue: tcgen05.ld accumulator -> bf16 -> y.
// Work split (stream-K): the sequence of (output tile, k-tile) units is cut into equal contiguous ranges, one
// per CTA, so all SMs finish together whatever the tile count.  A CTA that computes only part of a tile's K
// range writes its fp32 partial accumulator to the workspace and bumps the tile's counter; the CTA that arrives
// last adds the partials in CTA order (deterministic, nobody waits) and stores y.
// Every mbarrier wait is bounded; on a timeout all roles leave, TMEM is freed, the status word is set.
#include <cuda.h>

#include <atomic>
#include <cstddef>

#include "async.cuh"
#include "common.cuh"
#include "kernels.h"
#include "tensormap.h"

namespace tf {

namespace {

constexpr int kGemmThreads = 512;
constexpr int kBN = 128;                  // weight columns per CTA tile (two packed strips)
constexpr int kBK = 64;                   // k per pipeline step (one 128-byte swizzled activation row)
constexpr int kMaxDepth = 3;              // pipeline stages (128 k each): activations in shared memory, weight operand in
                                          // tensor memory (64 columns per stage)
constexpr int kTmemAccCols = 256;
constexpr int kTmemCols = 512;
constexpr int kMaxActStages = 12;
constexpr int kWpStages = 3;              // packed-weight ring (one stage = the two strip tiles of one k-tile)
static_assert(kWpStages <= kMaxDepth, "the barrier set-up gives one thread to each of kMaxDepth stages");

// one packed tile of the ring, rounded up to a multiple of 128 bytes (G = groups per tile: 4256, 4416 or 4736 bytes of tile)
__host__ __device__ constexpr int wp_strip_bytes(int bits, int G = 1) { return bits == 4 ? (G == 1 ? 4352 : G == 2 ? 4480 : 4736) : 8320; }
__host__ __device__ constexpr int act_stage_bytes(int bt) { return bt * kBK * 2; }
// activation ring depth: as deep as fits beside the packed ring, at most kMaxActStages
constexpr int kGemmSmemMax = 227 * 1024;  // dynamic shared memory one CTA may ask for
constexpr int kGemmSmemFixed = 1024 /*alignment slack*/ + 4 * 1024 /*epilogue warps*/ + 8 * 512 /*drain duty*/ + 512 /*barriers*/;
__host__ __device__ constexpr int act_stages(int bits, int bt, int G = 1) {
    return (kGemmSmemMax - kGemmSmemFixed - kWpStages * 2 * wp_strip_bytes(bits, G)) / act_stage_bytes(bt) > kMaxActStages
               ? kMaxActStages
               : (kGemmSmemMax - kGemmSmemFixed - kWpStages * 2 * wp_strip_bytes(bits, G)) / act_stage_bytes(bt);
}
// A pipeline stage is 128 k: two 64-k activation sub-tiles and 64 operand columns, one barrier that fills (activations
// landed + operand stored) and one that drains (MMAs done).  The thread that issues the MMAs pays a fixed price per
// stage (barrier waits, commits, loop arithmetic on a scheduler it shares with dequant warps): with 64-k stages and
// separate barriers for the two operands its loop took about 780 cycles per 64 k where the four MMAs of a 256-token
// tile execute in about 520, and it -- not the tensor core -- set the pace.
constexpr int kEpiWarpBytes = 1024;       // per epilogue warp: 16 tokens x 32 columns of bf16, for the transpose
constexpr int kDrainWarpBytes = 512;      // per dequant warp: 8 tokens x 32 columns, for its share of an accumulator drain
__host__ __device__ constexpr int gemm_smem_bytes(int bits, int bt, int G = 1) {
    return 1024 /*alignment slack*/ + act_stages(bits, bt, G) * act_stage_bytes(bt) +
           kWpStages * 2 * wp_strip_bytes(bits, G) + 4 * kEpiWarpBytes + 8 * kDrainWarpBytes + 512;
}
static_assert(kGemmSmemFixed == 1024 + 4 * kEpiWarpBytes + 8 * kDrainWarpBytes + 512, "act_stages budgets for exactly these");
static_assert(gemm_smem_bytes(4, 256, 1) <= kGemmSmemMax && gemm_smem_bytes(4, 128, 2) <= kGemmSmemMax &&
              gemm_smem_bytes(4, 128, 4) <= kGemmSmemMax && gemm_smem_bytes(8, 128, 1) <= kGemmSmemMax, "shared memory budget");

// workspace: [0,16) status | [kGemmCounterOffset, +4 * tiles) arrival counters | (the GEMV's partial-sum slots, not
// touched here) | partial accumulators, two slots of 128 x BT fp32 per CTA (head and tail of its range)
constexpr int kGemmCounterOffset = 4096;       // behind the GEMV's counters: the two kernels may share a workspace
constexpr int kGemmMaxTiles = 4096;            // (32768 / 128) n-tiles x (4096 / 256) token tiles
constexpr size_t kGemmPartialOffset = kWorkspaceZeroBytes;      // behind the GEMV's partial-sum slots, which must stay zero
static_assert(kGemmCounterOffset + 4 * kGemmMaxTiles == kWorkspaceHeadBytes && kGemmCounterOffset >= kGemvStatusBytes,
              "workspace layout shared with the GEMV");
constexpr int kGemmMaxGrid = 160;

// 32-bit arithmetic: at most 256 x 16 x 256 units (N, K <= 32768, M <= 4096) times at most 161 CTAs stays below 2^28,
// and these divisions sit between the start of a CTA and its first copy.
__device__ __forceinline__ int unit_start(int cta, int total, int grid) {
    return static_cast<int>((static_cast<uint32_t>(cta) * static_cast<uint32_t>(total)) / static_cast<uint32_t>(grid));
}
__device__ __forceinline__ int unit_owner(int unit, int total, int grid) {
    return static_cast<int>(((static_cast<uint32_t>(unit) + 1u) * static_cast<uint32_t>(grid) - 1u) / static_cast<uint32_t>(total));
}

// The CTA's unit range [u_begin, u_end) as segments of one output tile each, in processing order: the cut tile at
// the head of the range, the cut tile at its tail, then the whole tiles.  Cut tiles go first so that the fix-up of
// a tile shared with a neighbour runs under the main loop of a whole tile instead of at the end of the kernel.
struct Segments {
    int ktiles, head_tile, head_kt0, head_len, tail_tile, tail_len, first_whole, count, ncut;
    __device__ Segments(int u_begin, int u_end, int ktiles_) : ktiles(ktiles_) {
        head_tile = u_begin / ktiles;
        head_kt0 = u_begin - head_tile * ktiles;
        head_len = min(u_end - u_begin, ktiles - head_kt0);
        if (head_len == ktiles) head_len = 0;                    // the range starts with a whole tile
        const int u1 = u_begin + head_len;
        const int nwhole = (u_end - u1) / ktiles;
        first_whole = u1 / ktiles;                                // u1 is a tile boundary whenever anything follows
        tail_tile = first_whole + nwhole;
        tail_len = (u_end - u1) - nwhole * ktiles;
        ncut = (head_len > 0) + (tail_len > 0);
        count = ncut + nwhole;
    }
    // slot: 0 head, 1 tail, -1 whole
    __device__ void get(int i, int& tile, int& kt0, int& len, int& slot) const {
        if (i == 0 && head_len > 0) { tile = head_tile; kt0 = head_kt0; len = head_len; slot = 0; }
        else if (i < ncut) { tile = tail_tile; kt0 = 0; len = tail_len; slot = 1; }
        else { tile = first_whole + (i - ncut); kt0 = 0; len = ktiles; slot = -1; }
    }
};

struct GemmBarriers {
    uint64_t stage_full[kMaxDepth];       // activations landed (producer's expect_tx) and operand stored (8 dequant warps)
    uint64_t stage_done[kMaxDepth];       // tcgen05.commit: the MMAs that read the stage have run
    uint64_t wp_full[kWpStages];
    uint64_t wp_empty[kWpStages];
    uint64_t acc_full;
    uint64_t acc_empty;
    uint32_t tmem_base;
    uint32_t abort_flag;        // [0] which wait gave up (0 = none) ...
    uint32_t wait_kcycles;      // ... [1] limit of a wait in units of 1024 cycles (read by mbar_wait through the flag's address)
    uint32_t last_flag;
    uint32_t deferred_tile;     // 1 + the cut tile this CTA finishes with all its warps after the role loops (0 = none)
};

static_assert(offsetof(GemmBarriers, wait_kcycles) == offsetof(GemmBarriers, abort_flag) + 4, "mbar_wait reads the limit behind the flag");

// One warp's share of the drain of a whole 128 x BT accumulator: the 8-token chunks `part`, `part + 3`, ... of its
// lane quarter.  TMEM -> bf16 -> transposed through a 512-byte buffer -> one 16-byte store per lane (8 weight
// columns of one token).  Three warps per quarter (one epilogue warp, two dequant warps) share a tile.
template <int BT>
__device__ __forceinline__ void drain_share(uint32_t tmem_base, __nv_bfloat16* tbuf8, __nv_bfloat16* y, int M, int N, int n_tile,
                                            int m_tile, int quarter, int part, int lane) {
    const uint32_t taddr = tmem_base + (uint32_t(32 * quarter) << 16);
    const int n8 = n_tile * 128 + 32 * quarter + 8 * (lane & 3);
    const int tl = lane >> 2;
#pragma unroll 1
    for (int c = part; c < BT / 8; c += 3) {
        uint32_t r[8];
        tmem_ld_32x32b_x8(taddr + 8 * c, r);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 8; ++j) tbuf8[j * 32 + lane] = __float2bfloat16_rn(__uint_as_float(r[j]));
        __syncwarp();
        const int tok = m_tile * BT + 8 * c + tl;
        const uint4 d = *reinterpret_cast<const uint4*>(tbuf8 + tl * 32 + 8 * (lane & 3));
        if (tok < M && n8 < N) *reinterpret_cast<uint4*>(y + (size_t)tok * N + n8) = d;
        __syncwarp();
    }
}

// An fp16 scale has 11 significant bits, a bf16 number 8.  Rounding the scale to bf16 would put the same relative
// error (up to 2^-8) on every weight of a group -- an error that does not average out over k.  So the scale is split
// into its upper 8 bits and the (at most 3) bits below, both exact in bf16, and a weight is
// fma(d, hi, d * lo): for 4-bit codes |d| <= 15 and d * lo is exact, so the result is bf16((q - z) * s) with a single
// rounding; for 8-bit codes d * lo is rounded at 2^-9 of a term that is 2^-8 of the weight, which changes nothing.
__device__ __forceinline__ void split_scale(float s, uint32_t& hi2, uint32_t& lo2) {
    const uint32_t bits = __float_as_uint(s);
    const uint32_t hi = bits & 0xFFFF0000u;                          // truncated to bf16
    const uint32_t lo = __float_as_uint(s - __uint_as_float(hi));    // exact, at most 3 significant bits
    hi2 = (hi >> 16) | hi;
    lo2 = (lo >> 16) | (lo & 0xFFFF0000u);
}
__device__ __forceinline__ uint32_t times_scale(uint32_t d, uint32_t hi2, uint32_t lo2) {
    uint32_t t, w;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(t) : "r"(d), "r"(lo2));
    asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(w) : "r"(d), "r"(hi2), "r"(t));
    return w;
}

__device__ __forceinline__ uint32_t bf16_dup(float v) {
    const uint32_t b = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v));
    return b | (b << 16);
}

}  // namespace

// G = groups per tile: 1 for group sizes that are multiples of 128, 2 / 4 for the 4-bit group sizes 64 / 32.
template <int BITS, int BT, int G = 1>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap act_map, const uint8_t* __restrict__ blob,
            __nv_bfloat16* __restrict__ y, int M, int K, int N, int ktiles, int n_tiles, int m_tiles, int aligned,
            uint8_t* __restrict__ workspace, uint32_t debug) {
    static_assert(G == 1 || BITS == 4, "several groups per tile: the 4-bit format only");
    constexpr int kTileBytes = tile_bytes(BITS, G);
    constexpr int kWeightBytes = BITS == 4 ? kW4WeightBytes : kW8WeightBytes;
    constexpr int kActStage = act_stage_bytes(BT);
    constexpr int kSub = 2;                                           // 64-k sub-steps per pipeline stage
    constexpr int kStages = act_stages(BITS, BT, G) / kSub < kMaxDepth ? act_stages(BITS, BT, G) / kSub : kMaxDepth;
    constexpr int kUStage = kSub * kActStage;
    static_assert(kStages >= 2, "the pipeline needs two stages");
    constexpr int kWpStripBytes = wp_strip_bytes(BITS, G);
    constexpr int kWpStageBytes = 2 * kWpStripBytes;
    constexpr uint32_t kIdesc = umma_idesc_bf16(kBN, BT);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* act_ring = smem;                                        // kStages x kActStage   (1024-aligned)
    uint8_t* wp_ring = act_ring + act_stages(BITS, BT, G) * kActStage;  // kWpStages x packed tiles
    uint8_t* epi_buf = wp_ring + kWpStages * kWpStageBytes;          // 4 x kEpiWarpBytes
    uint8_t* drain_buf = epi_buf + 4 * kEpiWarpBytes;                // 8 x kDrainWarpBytes
    GemmBarriers* bars = reinterpret_cast<GemmBarriers*>(drain_buf + 8 * kDrainWarpBytes);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_units = n_tiles * m_tiles * ktiles;   // unit = (output tile, k-tile of 128)
    // aligned: whole tiles only (no tile is shared between CTAs); otherwise the units are split evenly
    const int total_tiles = n_tiles * m_tiles;
    const int u_begin = aligned ? unit_start(blockIdx.x, total_tiles, gridDim.x) * ktiles : unit_start(blockIdx.x, total_units, gridDim.x);
    const int u_end = aligned ? unit_start(blockIdx.x + 1, total_tiles, gridDim.x) * ktiles : unit_start(blockIdx.x + 1, total_units, gridDim.x);
    const Segments segs(u_begin, u_end, ktiles);
    const int strips = (N + kTileN - 1) / kTileN;
    const bool header_ok = header_matches(blob, BITS, (uint32_t)K, (uint32_t)N) && group_size_fits(blob, G);
    DeviceStatus* status = reinterpret_cast<DeviceStatus*>(workspace);

    // (one thread per pipeline stage and one for the rest: the set-up sits between the start of a CTA and its first copy)
    if (threadIdx.x < kMaxDepth) {
        const int s = threadIdx.x;
        if (s < kStages) {
            mbar_init(smem_u32(&bars->stage_full[s]), 9);    // eight dequant warps + the activation producer (with the bytes)
            mbar_init(smem_u32(&bars->stage_done[s]), 1);    // tcgen05.commit
        }
        if (s < kWpStages) {
            mbar_init(smem_u32(&bars->wp_full[s]), 1);
            mbar_init(smem_u32(&bars->wp_empty[s]), 8);      // all eight dequant warps
        }
        mbar_init_fence();
    } else if (threadIdx.x == 32) {
        mbar_init(smem_u32(&bars->acc_full), 1);
        mbar_init(smem_u32(&bars->acc_empty), 12);           // four epilogue warps + eight dequant warps (drain duty)
        bars->abort_flag = 0;
        bars->wait_kcycles = wait_limit_kcycles(debug);
        bars->deferred_tile = 0;
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
    const uint32_t tmem_a = tmem_base + kTmemAccCols;        // weight-operand ring

    // Programmatic dependent launch: this kernel may have been started while the previous kernel of the stream was
    // still running.  Only the packed weights (constants) are read before grid_dependency_wait(); activations, y and
    // the workspace are touched after it.  The packed-weight producer is the one role that does not wait here.
    if (!(warp == 3)) grid_dependency_wait();

    if (header_ok) {
        if (warp == 0 && lane == 0) {
            // ================= producer A: activation tile, one TMA load per k-step ==========================
            prefetch_tensormap(&act_map);
            uint32_t it = 0;
            bool ok = true;
            for (int i = 0; i < segs.count && ok; ++i) {
                int tile, kt0, len, slot;
                segs.get(i, tile, kt0, len, slot);
                const int n_tile = tile / m_tiles, m_tile = tile - n_tile * m_tiles;
                for (int ks = 2 * kt0; ks < 2 * (kt0 + len); ks += kSub, ++it) {
                    const int s = it % kStages;
                    ok = mbar_wait(smem_u32(&bars->stage_done[s]), ((it / kStages) & 1) ^ 1, abort_flag, 0x310 + s);
                    if (!ok) break;
                    mbar_arrive_expect_tx(smem_u32(&bars->stage_full[s]), kUStage);
#pragma unroll
                    for (int sub = 0; sub < kSub; ++sub)
                        tma_load_2d(smem_u32(act_ring + s * kUStage + sub * kActStage), &act_map, (ks + sub) * kBK, m_tile * BT,
                                    smem_u32(&bars->stage_full[s]));
                }
            }
        } else if (warp == 3 && lane == 0) {
            // ================= producer W: packed weight tiles (weights + scales + zeros in one payload) =====
            uint32_t wit = 0;
            bool ok = true;
            for (int i = 0; i < segs.count && ok; ++i) {
                int tile, kt0, len, slot;
                segs.get(i, tile, kt0, len, slot);
                const int n_tile = tile / m_tiles;
                const int strip0 = 2 * n_tile;
                const int nstrips = (strip0 + 1 < strips) ? 2 : 1;
                for (int T = kt0; T < kt0 + len; ++T, ++wit) {
                    const int ws = wit % kWpStages;
                    ok = mbar_wait(smem_u32(&bars->wp_empty[ws]), ((wit / kWpStages) & 1) ^ 1, abort_flag, 0x300 + ws);
                    if (!ok) break;
                    if (debug & kDebugDropWeights) continue;      // failure-path test: nothing ever arrives on wp_full
                    mbar_arrive_expect_tx(smem_u32(&bars->wp_full[ws]), nstrips * kTileBytes);
                    for (int q = 0; q < nstrips; ++q)
                        bulk_copy_g2s(smem_u32(wp_ring + ws * kWpStageBytes + q * kWpStripBytes),
                                      blob + kHeaderBytes + ((size_t)(strip0 + q) * ktiles + T) * kTileBytes, kTileBytes,
                                      smem_u32(&bars->wp_full[ws]));
                }
            }
        } else if (warp == 1 && lane == 0) {
            // ================= MMA issuer ==================================================================
            uint32_t it = 0, tile_it = 0;
            bool ok = true;
            for (; tile_it < (uint32_t)segs.count && ok; ++tile_it) {
                int tile, kt0, len, slot;
                segs.get((int)tile_it, tile, kt0, len, slot);
                ok = mbar_wait(smem_u32(&bars->acc_empty), (tile_it & 1) ^ 1, abort_flag, 0x400);
                if (!ok) break;
                tc_fence_after();
                for (int ks = 0; ks < 2 * len; ks += kSub, ++it) {
                    const int s = it % kStages;
                    ok = mbar_wait(smem_u32(&bars->stage_full[s]), (it / kStages) & 1, abort_flag, 0x410 + s);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int sub = 0; sub < kSub; ++sub) {
                        const uint64_t b_desc = umma_desc_k_sw128(smem_u32(act_ring + s * kUStage + sub * kActStage));
#pragma unroll
                        for (int j = 0; j < kBK / 16; ++j)   // 16 k per instruction: 8 TMEM columns / 32 smem bytes
                            tc_mma_f16_tmem_a(tmem_base, tmem_a + 32 * (kSub * s + sub) + 8 * j, b_desc + 2 * j, kIdesc,
                                              (ks | sub | j) != 0 ? 1u : 0u);
                    }
                    tc_commit(smem_u32(&bars->stage_done[s]));
                }
                if (!ok) break;
                tc_commit(smem_u32(&bars->acc_full));
            }
        } else if (warp >= 4 && warp < 12) {
            // ================= dequantize: packed tile -> bf16 operand in tensor memory ========================
            // warp -> (TMEM lane quarter q = 32 weight columns, k-half of the tile).  Quarter q covers strip q>>1,
            // 16-column blocks w0 = 2(q&1) and w0+1.  Thread (g, t) owns rows g, g+8 of both blocks and, per
            // k-block, the four consecutive k its packed word holds.
            const int q = warp & 3, half = (warp - 4) >> 2;
            const int strip_sel = q >> 1, w0 = 2 * (q & 1);
            const int g = lane >> 2;
            uint32_t wit = 0;
            bool ok = true;
            // Drain duty: every segment's accumulator is released by twelve arrivals, the four epilogue warps and
            // these eight.  For a whole tile a dequant warp first drains its third of its lane quarter.  The duty
            // for segment s is done just before this warp's job number kStages after the end of s: the first job whose
            // operand stage can only be freed by an MMA of segment s + 1, which in turn waits for that release.
            int duty = 0;
            __nv_bfloat16* tbuf8 = reinterpret_cast<__nv_bfloat16*>(drain_buf + (warp - 4) * kDrainWarpBytes);
            auto do_duty = [&](int sidx) -> bool {
                int dtile, dkt0, dlen, dslot;
                segs.get(sidx, dtile, dkt0, dlen, dslot);
                if (!mbar_wait(smem_u32(&bars->acc_full), sidx & 1, abort_flag, 0x520)) return false;
                tc_fence_after();
                if (dslot < 0) {
                    const int dn = dtile / m_tiles, dm = dtile - dn * m_tiles;
                    drain_share<BT>(tmem_base, tbuf8, y, M, N, dn, dm, q, 1 + half, lane);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty));
                return true;
            };
            for (int i = 0; i < segs.count && ok; ++i) {
                int tile, kt0, len, slot;
                segs.get(i, tile, kt0, len, slot);
                const int n_tile = tile / m_tiles;
                const bool strip_exists = 2 * n_tile + strip_sel < strips;
                for (int T = kt0; T < kt0 + len; ++T, ++wit) {
                    while (ok && (duty < i - 1 || (duty < i && T - kt0 >= kStages))) ok = do_duty(duty++);
                    if (!ok) break;
                    const int ws = wit % kWpStages;
                    ok = mbar_wait(smem_u32(&bars->wp_full[ws]), (wit / kWpStages) & 1, abort_flag, 0x500 + ws);
                    if (!ok) break;
                    const uint8_t* tile_smem = wp_ring + ws * kWpStageBytes + strip_sel * kWpStripBytes;
                    uint32_t op[2][16];                        // [block][register of the 16x256b.x4 store]
                    // scales of rows (w0,g), (w0,g+8), (w0+1,g), (w0+1,g+8), split into two exact bf16 parts
                    uint32_t s_g[2], s_g8[2], l_g[2], l_g8[2];
                    auto load_scales = [&](int gr) {
                        const uint2 sc = *(reinterpret_cast<const uint2*>(tile_smem + kWeightBytes + gr * kScaleBytes + g * 16) + (q & 1));
                        const uint32_t sw[2] = {sc.x, sc.y};
#pragma unroll
                        for (int b = 0; b < 2; ++b) {
                            split_scale(fp16_bits_to_float((uint16_t)(sw[b] & 0xFFFFu)), s_g[b], l_g[b]);
                            split_scale(fp16_bits_to_float((uint16_t)(sw[b] >> 16)), s_g8[b], l_g8[b]);
                        }
                    };
                    if (BITS == 4) {
                        // This warp's 64 k of the tile lie in one group (group sizes >= 64: group `half` of two, or the
                        // tile's only one) or in two (group size 32: k-steps 0, 1 and 2, 3).
                        constexpr int kSubGroups = G == 4 ? 2 : 1;
#pragma unroll
                        for (int sub = 0; sub < kSubGroups; ++sub) {
                            const int gr = G == 1 ? 0 : G == 2 ? half : 2 * half + sub;
                            load_scales(gr);
                            const uint32_t zword = *(reinterpret_cast<const uint32_t*>(tile_smem + w4_zero_offset(G, gr)) + g);
                            uint32_t zg[2], zg8[2];
#pragma unroll
                            for (int b = 0; b < 2; ++b) {
                                const uint32_t pair = w4_reg_biased(zword, w0 + b);   // (128 + z[row g], 128 + z[row g+8])
                                zg[b] = __byte_perm(pair, 0, 0x1010);
                                zg8[b] = __byte_perm(pair, 0, 0x3232);
                            }
#pragma unroll
                            for (int i = sub * (4 / kSubGroups); i < (sub + 1) * (4 / kSubGroups); ++i) {   // k-block 4*half + i = MMA k-step i of this operand stage
                                const uint2 x = *(reinterpret_cast<const uint2*>(tile_smem + ((4 * half + i) * 32 + lane) * 16) + (q & 1));
                                const uint32_t xs[2] = {x.x, x.y};
#pragma unroll
                                for (int b = 0; b < 2; ++b) {
                                    op[b][4 * i + 0] = times_scale(bf16x2_sub(w4_reg_biased(xs[b], 0), zg[b]), s_g[b], l_g[b]);    // row g,   k 0,1
                                    op[b][4 * i + 1] = times_scale(bf16x2_sub(w4_reg_biased(xs[b], 2), zg[b]), s_g[b], l_g[b]);    // row g,   k 2,3
                                    op[b][4 * i + 2] = times_scale(bf16x2_sub(w4_reg_biased(xs[b], 1), zg8[b]), s_g8[b], l_g8[b]);  // row g+8, k 0,1
                                    op[b][4 * i + 3] = times_scale(bf16x2_sub(w4_reg_biased(xs[b], 3), zg8[b]), s_g8[b], l_g8[b]);  // row g+8, k 2,3
                                }
                            }
                        }
                    } else {
                        load_scales(0);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint4 x = *reinterpret_cast<const uint4*>(tile_smem + (((4 * half + i) * 2 + (q & 1)) * 32 + lane) * 16);
                            const uint32_t xs[2][2] = {{x.x, x.y}, {x.z, x.w}};
#pragma unroll
                            for (int b = 0; b < 2; ++b) {
                                uint32_t r0, r1, r2, r3;
                                w8_word_to_regs(xs[b][0], r0, r1);                     // (row g; k 0,1), (row g+8; k 0,1)
                                w8_word_to_regs(xs[b][1], r2, r3);                     // (row g; k 2,3), (row g+8; k 2,3)
                                op[b][4 * i + 0] = times_scale(r0, s_g[b], l_g[b]);
                                op[b][4 * i + 1] = times_scale(r2, s_g[b], l_g[b]);
                                op[b][4 * i + 2] = times_scale(r1, s_g8[b], l_g8[b]);
                                op[b][4 * i + 3] = times_scale(r3, s_g8[b], l_g8[b]);
                            }
                        }
                    }
                    // the packed stage has been read
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars->wp_empty[ws]));

                    // wait until the MMAs that read this operand stage (kStages stages ago) are done
                    const uint32_t it = wit;                                     // pipeline stage = k-tile
                    const int sa = it % kStages;
                    ok = mbar_wait(smem_u32(&bars->stage_done[sa]), ((it / kStages) & 1) ^ 1, abort_flag, 0x510 + sa);
                    if (!ok) break;
                    tc_fence_after();
                    if (strip_exists) {
                        const uint32_t taddr = tmem_a + 32 * (kSub * sa + half) + (uint32_t(32 * q) << 16);
                        tmem_st_16x256b_x4(taddr, op[0]);
                        tmem_st_16x256b_x4(taddr + (16u << 16), op[1]);
                        tmem_st_wait();
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars->stage_full[sa]));
                }
            }
            while (ok && duty < segs.count) ok = do_duty(duty++);
        } else if (warp >= 12) {
            // ================= epilogue: TMEM -> bf16 -> y, or -> fp32 partial for a tile cut between CTAs ==========
            const int quarter = warp & 3;                     // this warp may touch TMEM lanes 32*quarter .. +31
            const int row = 32 * quarter + lane;              // this thread's weight column inside the tile
            const uint32_t taddr = tmem_base + (uint32_t(32 * quarter) << 16);
            __nv_bfloat16* tbuf = reinterpret_cast<__nv_bfloat16*>(epi_buf + quarter * kEpiWarpBytes);   // [16][32]
            uint32_t* counters = reinterpret_cast<uint32_t*>(workspace + kGemmCounterOffset);
            float* partials = reinterpret_cast<float*>(workspace + kGemmPartialOffset);
            // 16 tokens of this thread's column -> the warp transposes them through its 1 KB buffer so that each
            // thread stores 8 consecutive columns (16 bytes) of one token
            auto store_chunk = [&](const float (&v)[16], int n_tile, int m_tile, int c) {
                const int n8 = n_tile * kBN + 32 * quarter + 8 * (lane & 3);
#pragma unroll
                for (int j = 0; j < 16; ++j) tbuf[j * 32 + lane] = __float2bfloat16_rn(v[j]);
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int tl = 8 * i + (lane >> 2);
                    const int tok = m_tile * BT + 16 * c + tl;
                    const uint4 d = *reinterpret_cast<const uint4*>(tbuf + tl * 32 + 8 * (lane & 3));
                    if (tok < M && n8 < N) *reinterpret_cast<uint4*>(y + (size_t)tok * N + n8) = d;
                }
                __syncwarp();
            };
            uint32_t seg_it = 0;
            for (; seg_it < (uint32_t)segs.count; ++seg_it) {
                int tile, kt0, len, slot;
                segs.get((int)seg_it, tile, kt0, len, slot);
                const int n_tile = tile / m_tiles, m_tile = tile - n_tile * m_tiles;
                if (!mbar_wait(smem_u32(&bars->acc_full), seg_it & 1, abort_flag, 0x600)) break;
                tc_fence_after();
                if (slot < 0) {
                    // ---- the whole K range of the tile was computed here: round and store this warp's third ---------
                    drain_share<BT>(tmem_base, tbuf, y, M, N, n_tile, m_tile, quarter, 0, lane);
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty));
                } else {
                    // ---- part of the K range: publish the fp32 partial, last arriver finishes the tile ----------
                    // slot layout: float4 index (4 c + j) * 128 + row, so that a warp's accesses are contiguous
                    constexpr size_t kSlotVec = (size_t)kBN * BT / 4;
                    uint4* mine = reinterpret_cast<uint4*>(partials) + (size_t)(blockIdx.x * 2 + slot) * kSlotVec + row;
#pragma unroll 1
                    for (int c = 0; c < BT / 16; ++c) {
                        uint32_t r[16];
                        tmem_ld_32x32b_x16(taddr + 16 * c, r);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            __stcg(mine + (4 * c + j) * kBN, make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]));
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty));      // the accumulator is free again
                    const int c_first = unit_owner(tile * ktiles, total_units, gridDim.x);
                    const int ncontrib = unit_owner(tile * ktiles + ktiles - 1, total_units, gridDim.x) - c_first + 1;
                    asm volatile("bar.sync 2, 128;" ::: "memory");               // all four epilogue warps have stored
                    if (warp == 12 && lane == 0) {
                        uint32_t prev;
                        asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(prev) : "l"(counters + tile) : "memory");
                        bars->last_flag = (prev == (uint32_t)(ncontrib - 1)) ? 1u : 0u;
                    }
                    asm volatile("bar.sync 2, 128;" ::: "memory");
                    if (*reinterpret_cast<volatile uint32_t*>(&bars->last_flag) != 0 && seg_it + 1 == (uint32_t)segs.count) {
                        // nothing left to hide the fix-up behind: every warp of the CTA takes a share of it after the
                        // role loops (four warps alone are bound by the latency of their few loads in flight)
                        if (warp == 12 && lane == 0) bars->deferred_tile = (uint32_t)tile + 1u;
                    } else if (*reinterpret_cast<volatile uint32_t*>(&bars->last_flag) != 0) {
                        // sum in CTA order whoever arrived last; only the first contributor can hold a tail slot
                        const float4* first = reinterpret_cast<const float4*>(partials) +
                            (size_t)(c_first * 2 + (unit_start(c_first, total_units, gridDim.x) >= tile * ktiles ? 0 : 1)) * kSlotVec + row;
                        const float4* rest = reinterpret_cast<const float4*>(partials) + (size_t)((c_first + 1) * 2) * kSlotVec + row;
#pragma unroll 1
                        for (int c = 0; c < BT / 16; ++c) {
                            float4 p[4], q4[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) p[j] = __ldcg(first + (4 * c + j) * kBN);
#pragma unroll
                            for (int j = 0; j < 4; ++j) q4[j] = __ldcg(rest + (4 * c + j) * kBN);
                            float v[16];
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                v[4 * j] = p[j].x + q4[j].x; v[4 * j + 1] = p[j].y + q4[j].y;
                                v[4 * j + 2] = p[j].z + q4[j].z; v[4 * j + 3] = p[j].w + q4[j].w;
                            }
                            for (int cc = 2; cc < ncontrib; ++cc) {
                                const float4* src = rest + (size_t)(cc - 1) * 2 * kSlotVec;
#pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    const float4 t4 = __ldcg(src + (4 * c + j) * kBN);
                                    v[4 * j] += t4.x; v[4 * j + 1] += t4.y; v[4 * j + 2] += t4.z; v[4 * j + 3] += t4.w;
                                }
                            }
                            store_chunk(v, n_tile, m_tile, c);
                        }
                        if (warp == 12 && lane == 0) counters[tile] = 0;         // leave the workspace ready for the next call
                    }
                    asm volatile("bar.sync 2, 128;" ::: "memory");               // last_flag is reused by the next cut tile
                }
            }
        }
    }

    // ---------------- deferred fix-up of the CTA's last cut tile, by all 16 warps --------------------------------
    if (warp == 3) grid_dependency_wait();
    tc_fence_before();
    __syncthreads();
    if (header_ok && bars->deferred_tile != 0 && bars->abort_flag == 0) {
        // all MMAs of this CTA have completed, so the activation ring is free: one 1 KB transpose buffer per warp
        const int tile = (int)bars->deferred_tile - 1;
        const int n_tile = tile / m_tiles, m_tile = tile - n_tile * m_tiles;
        const int quarter = warp & 3, part = warp >> 2;               // rows 32 quarter .. +31, chunks part, part + 4, ..
        const int row = 32 * quarter + lane;
        __nv_bfloat16* tbuf = reinterpret_cast<__nv_bfloat16*>(act_ring + warp * kEpiWarpBytes);
        constexpr size_t kSlotVec = (size_t)kBN * BT / 4;
        const float4* partials4 = reinterpret_cast<const float4*>(workspace + kGemmPartialOffset);
        const int c_first = unit_owner(tile * ktiles, total_units, gridDim.x);
        const int ncontrib = unit_owner(tile * ktiles + ktiles - 1, total_units, gridDim.x) - c_first + 1;
        const float4* first = partials4 +
            (size_t)(c_first * 2 + (unit_start(c_first, total_units, gridDim.x) >= tile * ktiles ? 0 : 1)) * kSlotVec + row;
        const float4* rest = partials4 + (size_t)((c_first + 1) * 2) * kSlotVec + row;     // later contributors: head slots
        const int n8 = n_tile * kBN + 32 * quarter + 8 * (lane & 3);
#pragma unroll 1
        for (int c = part; c < BT / 16; c += 4) {
            float4 acc4[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) acc4[j] = __ldcg(first + (4 * c + j) * kBN);
            for (int cc = 1; cc < ncontrib; cc += 2) {                 // CTA order; two contributors' loads in flight
                float4 x[4], z[4];
                const float4* s0 = rest + (size_t)(cc - 1) * 2 * kSlotVec;
                const bool two = cc + 1 < ncontrib;
#pragma unroll
                for (int j = 0; j < 4; ++j) x[j] = __ldcg(s0 + (4 * c + j) * kBN);
#pragma unroll
                for (int j = 0; j < 4; ++j) z[j] = two ? __ldcg(s0 + 2 * kSlotVec + (4 * c + j) * kBN) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc4[j].x += x[j].x; acc4[j].y += x[j].y; acc4[j].z += x[j].z; acc4[j].w += x[j].w;
                    if (two) { acc4[j].x += z[j].x; acc4[j].y += z[j].y; acc4[j].z += z[j].z; acc4[j].w += z[j].w; }
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                tbuf[(4 * j + 0) * 32 + lane] = __float2bfloat16_rn(acc4[j].x);
                tbuf[(4 * j + 1) * 32 + lane] = __float2bfloat16_rn(acc4[j].y);
                tbuf[(4 * j + 2) * 32 + lane] = __float2bfloat16_rn(acc4[j].z);
                tbuf[(4 * j + 3) * 32 + lane] = __float2bfloat16_rn(acc4[j].w);
            }
            __syncwarp();
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int tl = 8 * i + (lane >> 2);
                const int tok = m_tile * BT + 16 * c + tl;
                const uint4 d = *reinterpret_cast<const uint4*>(tbuf + tl * 32 + 8 * (lane & 3));
                if (tok < M && n8 < N) *reinterpret_cast<uint4*>(y + (size_t)tok * N + n8) = d;
            }
            __syncwarp();
        }
        if (threadIdx.x == 0) reinterpret_cast<uint32_t*>(workspace + kGemmCounterOffset)[tile] = 0;   // ready for the next call
    }

    // ---------------- teardown --------------------------------------------------------------------------------
    __syncthreads();
    // this CTA's results are out: the next kernel of the stream may start (a whole-SM kernel releases its dependents
    // late, see the GEMV)
    if (threadIdx.x == 0) grid_launch_dependents();
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
static int gemm_token_tile(int M) { return M > 128 ? 256 : M > 64 ? 128 : M > 32 ? 64 : 32; }

size_t gemm_workspace_bytes(int M, int K, int N) {
    (void)K; (void)N;
    return (size_t)kGemmPartialOffset + (size_t)kGemmMaxGrid * 2 * kBN * gemm_token_tile(M) * 4;
}

namespace {

template <int BITS, int BT, int G = 1>
cudaError_t launch_bt(const void* blob, const void* a, void* y, int M, int K, int N, void* workspace, int sm_count,
                      cudaStream_t stream) {
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)BT};
    cudaError_t me = encode_bf16_map(&map, a, 2, dims, strides, box);
    if (me != cudaSuccess) return me;

    // function attributes belong to one device: set them once per device and kernel (twice is harmless)
    constexpr int kMaxDevices = 64;
    // (an atomic flag: two host threads may both find it unset and both set the attribute, which is harmless)
    static std::atomic<bool> configured_on[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
    const bool seen = dev >= 0 && dev < kMaxDevices;
    if (!seen || !configured_on[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(gemm_kernel<BITS, BT, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             gemm_smem_bytes(BITS, BT, G));
        if (e != cudaSuccess) return e;
        if (seen) configured_on[dev].store(true, std::memory_order_release);
    }
    const int n_tiles = (N + kBN - 1) / kBN, m_tiles = (M + BT - 1) / BT;
    const long long units = (long long)n_tiles * m_tiles * (K / kTileK);
    if (sm_count > kGemmMaxGrid) sm_count = kGemmMaxGrid;
    // Two ways to spread the work.  Even split of the (tile, k-tile) units: no SM idles, but a CTA whose range
    // holds no whole tile finishes with the fix-up of a cut tile in the open (about 10 k-tile times for a
    // 256-token tile, measured; less for narrower tiles).  Whole tiles only: no fix-up, but the last wave of
    // tiles may leave SMs idle.  Take the cheaper one, in k-tile times of the longest CTA.
    const int ktiles = K / kTileK, tiles = n_tiles * m_tiles;
    int grid = units < sm_count ? (int)units : sm_count;
    const long long split_len = (units + grid - 1) / grid;
    const long long split_cost = split_len + (split_len < 2 * ktiles ? 10 * BT / 256 : 0);
    const int tile_grid = tiles < sm_count ? tiles : sm_count;
    const long long tile_cost = (long long)((tiles + tile_grid - 1) / tile_grid) * ktiles;
    const int aligned = tile_cost <= split_cost ? 1 : 0;
    if (aligned) grid = tile_grid;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(kGemmThreads, 1, 1);
    cfg.dynamicSmemBytes = gemm_smem_bytes(BITS, BT, G);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // see grid_dependency_wait() in the kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    note_whole_sm_launch(stream);
    return cudaLaunchKernelEx(&cfg, gemm_kernel<BITS, BT, G>, map, static_cast<const uint8_t*>(blob), static_cast<__nv_bfloat16*>(y), M, K,
                              N, ktiles, n_tiles, m_tiles, aligned, static_cast<uint8_t*>(workspace), debug_word());
}

template <int BITS, int G = 1>
cudaError_t launch_bits(const void* blob, const void* a, void* y, int M, int K, int N, void* workspace, int sm_count,
                        cudaStream_t stream) {
    if (M > 128) return launch_bt<BITS, 256, G>(blob, a, y, M, K, N, workspace, sm_count, stream);
    if (M > 64) return launch_bt<BITS, 128, G>(blob, a, y, M, K, N, workspace, sm_count, stream);
    if (M > 32) return launch_bt<BITS, 64, G>(blob, a, y, M, K, N, workspace, sm_count, stream);
    return launch_bt<BITS, 32, G>(blob, a, y, M, K, N, workspace, sm_count, stream);
}

}  // namespace

cudaError_t launch_gemm(int bits, const void* blob, const void* a, void* y, int M, int K, int N, void* workspace,
                        size_t workspace_bytes, int sm_count, cudaStream_t stream, int groups) {
    (void)workspace_bytes;
    if (groups == 2 && bits == 4) return launch_bits<4, 2>(blob, a, y, M, K, N, workspace, sm_count, stream);
    if (groups == 4 && bits == 4) return launch_bits<4, 4>(blob, a, y, M, K, N, workspace, sm_count, stream);
    if (groups != 1) return cudaErrorInvalidValue;
    return bits == 4 ? launch_bits<4>(blob, a, y, M, K, N, workspace, sm_count, stream)
                     : launch_bits<8>(blob, a, y, M, K, N, workspace, sm_count, stream);
}

}  // namespace tf
