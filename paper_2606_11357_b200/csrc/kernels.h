// Internal launch interface between the C-ABI layer and the kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace tf {

// Tuning knobs of the integer path (overridable at compile time for measurements).
#ifndef TF_I8_FULL_BYTES_W4
#define TF_I8_FULL_BYTES_W4 (288 * 1024)
#endif
#ifndef TF_I8_FULL_BYTES_W8
#define TF_I8_FULL_BYTES_W8 (160 * 1024)
#endif

// ---- GEMV (persistent streaming kernel) ----------------------------------------------------------
// Configurations, chosen by plan_gemv:
//   integer path (1 and 2 tokens), short ranges: 8 consumer warps and half an SM per CTA, so the next GEMV's CTAs
//     fit beside this one's and have their rings full of weights when this kernel completes.
//   integer path, long ranges: the whole SM, a ring of eight stages, and as many consumer warps as hold about
//     66 KB of tiles (16 on 4-bit tiles, 8 on int8 tiles).
//   Either form, 4-bit tiles: where a range passes over its k-tiles more than once and K is a multiple of 128 x
//     consumer warps, a warp keeps the activation pieces of the k-tiles it has visited (piece table) instead of
//     preparing them per tile.
//   floating-point path up to 8 tokens: the whole SM and 12 consumer warps; on 4-bit tiles a ring of five stages
//     (three in the warps' hands, two in flight; deeper was measured slower), on int8 tiles the deepest that fits.
//     A consumer warp of the floating-point path is bound by instruction issue (about 20 issue cycles per packed
//     word of 8 weights, measured on registers alone), and since a GEMV may not read its activations before the
//     kernel ahead of it has completed, only one kernel's consumers work on an SM at a time: three warps per
//     scheduler beat two warps plus a waiting neighbour (decode step of the benchmark: 133 against 140 us).
//   9..16 tokens: twice the MMA and activation work per tile and the whole SM, but 8 consumer warps: every tile a
//     warp is working on is a tile that is not in flight (measured on the four layer shapes with the ring holding
//     weights only: 8 warps 7.9 / 4.1 / 14.5 / 15.4 us, 10 warps 8.4 / 4.1 / 15.2 / 16.1 us; 12 warps do not fit the
//     register file).
__host__ __device__ constexpr int gemv_max_consumers(int mt, bool full, bool i8 = false) { return mt == 1 ? (full ? (i8 ? 16 : 12) : 8) : 8; }
__host__ __device__ constexpr int gemv_max_threads(int mt, bool full, bool i8 = false) { return 32 * (gemv_max_consumers(mt, full, i8) + 2); }   // + producer + reducer
__host__ __device__ constexpr int gemv_smem_budget(int mt, bool full) { return (mt == 1 && !full ? 110 : 220) * 1024; }
// Shared memory a half-SM CTA asks for when two of its kind must not share an SM: with 228 KB per SM and 1 KB reserved
// per CTA, two of these do not fit (2 x 115 KB), one beside a plain half-SM CTA (at most 110 KB) does.
constexpr int kGemvSoloSmemBytes = 114 * 1024;
// Integer path, piece table: one entry per k-tile: per token 3 piece columns of 36 words (32 used; the padding keeps
// the columns in different banks), then 8 columns x 8 bytes of column metadata; 512 bytes per token.
constexpr int kGemvPieceEntryBytes = 512;
// Packed bytes per CTA from which the integer path uses the whole-SM configuration, and its consumer warps there.
// A half-SM CTA has a ring of four or five 17 KB stages, and every tile a warp works on is a tile that is not in flight: eight
// warps on int8 tiles (8.3 KB) hold nearly the whole ring, on 4-bit tiles half of it.  The whole-SM form has a ring of
// eight stages; with about 66 KB of tiles in the warps' hands (8 warps on int8, 16 on 4-bit tiles) it streams long
// ranges faster than the half-SM form, which wins on short ranges because the next GEMV's CTAs sit beside it with
// their rings full.
constexpr int kGemvFullFromBytesI8W4 = TF_I8_FULL_BYTES_W4;
constexpr int kGemvFullFromBytesI8W8 = TF_I8_FULL_BYTES_W8;
__host__ __device__ constexpr int gemv_i8_full_consumers(int bits) { return bits == 8 ? 8 : 16; }
constexpr int kGemvI8FullMaxStages = 8;
constexpr int kGemvFpW4MaxStages = 5;
constexpr int kGemvMaxDevices = 64;            // devices the per-device caches cover
constexpr int kGemvMaxStages = 48;
constexpr int kGemvBarrierBytes = 4096;       // 2 x 48 mbarriers + flags, then contributor offsets
constexpr int kGemvMaxContrib = 320;          // CTAs that can share one strip (<= K/128 + 1 = 257)
// A ring stage holds one bulk copy of several contiguous tiles (about 16.6 KB either way).
__host__ __device__ constexpr int gemv_chunk_tiles(int bits) { return bits == 4 ? 4 : 2; }
constexpr int kGemvStageBytes = 17408;        // 17 x 1024 >= 4 x 4256 and >= 2 x 8320
constexpr int kGemvMaxM = 16;
// 9..16 tokens: per consumer warp two buffers of 16 token rows x 128 k of activations, rows padded to 288 bytes
constexpr int kGemvActRowBytes = 288;
constexpr int kGemvActBufBytes = 16 * kGemvActRowBytes;
constexpr int kGemvActWarpBytes = 2 * kGemvActBufBytes;
constexpr int kGemvI8MaxM = 2;                // up to this many tokens the GEMV runs on the integer warp MMA (4-bit and int8 weights)
constexpr int kGemvMaxGrid = 256;             // CTAs (one per SM); sizes the partial-sum area
// Workspace layout, shared with the GEMM so that one workspace serves every call of a stream:
//   [0,16) status word | [4096, 20480) GEMM per-tile arrival counters | from 20480: one GEMV partial-sum slot
//   (16 tokens x 64 columns fp32) per persistent CTA | behind them the GEMM's partial tiles (written before they are
//   read, so the GEMM may leave anything there).
// Everything below kWorkspaceZeroBytes is zero between calls: the GEMV's hand-over of a cut strip relies on its slots
// being all +0.0 bits (see gather_partials in gemv.cu), the GEMM on its counters.
constexpr int kWorkspaceHeadBytes = 20480;
constexpr int kGemvStatusBytes = 256;         // what the GEMV itself needs cleared besides its slots
constexpr int kGemvPartialOffset = kWorkspaceHeadBytes;
constexpr int kGemvSlotBytes = kGemvMaxM * 64 * 4;
constexpr size_t kWorkspaceZeroBytes = kGemvPartialOffset + (size_t)kGemvMaxGrid * kGemvSlotBytes;
constexpr size_t kGemvWorkspaceBytes = kWorkspaceZeroBytes;

struct GemvPlan {
    int grid;          // persistent CTAs
    int threads;       // 32 * (consumers + 2): producer warp, reducer warp, consumer warps
    int consumers;     // consumer warps
    int stages;        // ring depth
    bool full;         // whole-SM configuration
    bool i8;           // integer path: codes x activation pieces on the integer warp MMA (1 or 2 tokens)
    int piece_tab;     // integer path: entries of the CTA-wide table of activation pieces (0 = every warp prepares its own tile's)
    int cluster;       // CTAs per cluster (1 = global mode: cut strips go through the workspace)
    int nclusters;     // cluster mode: number of clusters (grid = nclusters * cluster); global mode: CTAs that get tiles
    int xslot_bytes;   // cluster mode: bytes of one partial-sum slot in shared memory
    int stage_bytes;   // bytes of one ring stage
    int smem_bytes;
    int strips, ktiles, total_tiles;
    int nred;          // buffers for the consumer warps' partial sums of a strip segment (1 or 2)
    int groups;        // groups per tile: 1, or 2 / 4 for the 4-bit group sizes 64 / 32
};

GemvPlan plan_gemv(int bits, int M, int K, int N, int sm_count, int groups = 1);
cudaError_t launch_gemv(int bits, const GemvPlan& plan, const void* blob, const void* a, void* y,
                        int M, int K, int N, void* workspace, cudaStream_t stream);

// Do every one-time, per-device step of the GEMV launcher now (function attributes, occupancy queries).
cudaError_t configure_gemv_kernels();

// The `debug` argument every GEMV / GEMM launch passes to its kernel (0 unless tf_debug_inject set it; see async.cuh).
uint32_t debug_word();
void set_debug_word(uint32_t word);

// Tell the GEMV launcher that a whole-SM kernel of this library (the GEMM) was launched on `stream`.
void note_whole_sm_launch(cudaStream_t stream);

cudaError_t launch_unpack_w4(const void* blob, uint8_t* q, uint8_t* z, uint16_t* s, int K, int N,
                             int group_size, cudaStream_t stream);
cudaError_t launch_unpack_w8(const void* blob, int8_t* q, uint16_t* s, int K, int N, int group_size,
                             cudaStream_t stream);

// Ablation baseline: the dequantized matrix written to global memory as bf16 [K][N].
cudaError_t launch_dequant(int bits, const void* blob, void* w_bf16, int K, int N, cudaStream_t stream);

// Fused W4A16 GEMV on the AWQ arrays as they come (no pre-tiling): the second arm of the layout ablation.
struct RawGemvPlan {
    bool mma;            // 9..16 tokens: tensor-core kernel (units are 16-row blocks); up to 8: the fp32 kernel (units are groups)
    int groups;          // units along K
    int col_blocks;      // blocks of 256 (fp32) or 64 (tensor-core) output columns
    int splits;          // CTAs that share a column block (split-K over whole units)
    int groups_per_cta;
};
RawGemvPlan plan_gemv_raw(int M, int K, int N, int group_size, int sm_count);
size_t gemv_raw_workspace_bytes(int M, int N, int sm_count);
cudaError_t launch_gemv_raw(const RawGemvPlan& plan, const uint32_t* qweight, const uint16_t* scales,
                            const uint32_t* qzeros, const void* a, void* y, int M, int K, int N, int group_size,
                            void* workspace, cudaStream_t stream);

// Pre-tiling on the GPU: the AWQ arrays (device) -> the packed blob (device), byte for byte what tf_pack_awq writes.
cudaError_t launch_repack_awq(const uint32_t* qweight, const uint16_t* scales, const uint32_t* qzeros, void* out, int K, int N,
                              int group_size, cudaStream_t stream);

// Prefill GEMM (tcgen05).  `workspace` starts with the DeviceStatus word.
size_t gemm_workspace_bytes(int M, int K, int N);
cudaError_t launch_gemm(int bits, const void* blob, const void* a, void* y, int M, int K, int N,
                        void* workspace, size_t workspace_bytes, int sm_count, cudaStream_t stream, int groups = 1);

}  // namespace tf
