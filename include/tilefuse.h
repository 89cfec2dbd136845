/*
 * tilefuse.h -- C ABI of libtilefuse.so: the fused mixed-precision linear layer
 *
 *     Y[M,N] = A[M,K] . dequant(Wq)[K,N]
 *
 * for NVIDIA B200 (sm_100a).  Weights stay 4-bit / 8-bit in device memory and are
 * unpacked, dequantized and multiplied inside one kernel; no bf16 copy of the weights
 * is ever written to global memory (the fusion property of Section 4.1 of the paper).
 *
 * Conventions for every entry point
 *   - "host" / "device" on a pointer says which memory it must point into.
 *   - The caller owns every buffer.  The library allocates nothing, frees nothing and
 *     keeps no pointer after a call returns.
 *     (It remembers, per process, which kind of kernel it launched last on a stream; that
 *     only steers how consecutive kernels overlap.)
 *   - Device calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*;
 *     NULL = the default stream) and never synchronise, except tf_device_status.
 *   - Errors are return codes.  Nothing is printed, nothing aborts, no exception
 *     crosses the boundary.  On any error the outputs are left untouched.
 *   - Device pointers must be 16-byte aligned (TF_ERR_ALIGN otherwise).
 *   - Outputs must not overlap inputs or the workspace.
 *   - Same inputs give bit-identical outputs (no atomics on results).
 *   - There is no CPU or other-GPU fallback: a device that is not compute capability
 *     10.x gives TF_ERR_ARCH.
 *   - Thread safety: every entry point may be called from several host threads at once.  The
 *     library's only state is per-device caches of immutable facts (device attributes, "this
 *     kernel's attributes are set", occupancy answers) and the per-stream note above, all held
 *     in atomics; a race on first use repeats an idempotent query.  The caller keeps calls that
 *     share a workspace (or the fixed scratch of tf_gemv_w4a16_static) from overlapping on the
 *     GPU, and makes the CUDA device current on the calling thread.
 */
#ifndef TILEFUSE_H
#define TILEFUSE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum tf_status {
    TF_OK = 0,
    TF_ERR_NULL = 1,       /* a required pointer is NULL */
    TF_ERR_SHAPE = 2,      /* M, K, N or group_size outside the legal set (see each call) */
    TF_ERR_ALIGN = 3,      /* a device pointer is not 16-byte aligned */
    TF_ERR_BLOB = 4,       /* packed blob: bad magic / version, or bits, K, N do not match */
    TF_ERR_WORKSPACE = 5,  /* workspace missing or smaller than tf_workspace_size() */
    TF_ERR_ARCH = 6,       /* current device is not compute capability 10.x */
    TF_ERR_CUDA = 7,       /* a CUDA runtime call or a kernel launch failed */
    TF_ERR_TIMEOUT = 8     /* a bounded device-side wait gave up (see tf_device_status) */
} tf_status;

/* Operation selector for tf_workspace_size. */
typedef enum tf_op {
    TF_OP_GEMV_W4A16 = 0,
    TF_OP_GEMV_W8A16 = 1,
    TF_OP_GEMM_W4A16 = 2,
    TF_OP_GEMM_W8A16 = 3
} tf_op;

/* Limits of the problem statement (Section 2.1: C = A x B; Section 4.2: K, N up to 32K). */
#define TF_MAX_DIM      32768   /* K and N */
#define TF_MAX_M_GEMV   16
#define TF_MAX_M_GEMM   4096
#define TF_TILE_K       128     /* k-extent of one packed tile = the AWQ group size */
#define TF_TILE_N       64      /* n-extent of one packed tile (a "strip" of columns) */
#define TF_WORKSPACE_ZERO_BYTES 1069056 /* start of a workspace that must be zero before its first use (or zero all of it) */

/*
 * The packed blob (output of tf_pack_awq / tf_pack_w8).
 *
 * Offline pre-tiling with per-tile metadata (Section 4.2): the weight matrix is cut into
 * tiles of TF_TILE_K rows (k) x TF_TILE_N columns (n); each tile is one contiguous payload
 * that carries its packed weights followed by the scales (and zero points) that dequantize
 * it, so that one stream delivers everything a tile needs.  Tiles of one column strip are
 * consecutive along K (tile-major order: a strip is one long contiguous read).
 *
 *   blob   = header (256 bytes) | tile(strip 0, ktile 0) | tile(0,1) | ... | tile(1,0) | ...
 *   W4 tile (4256 bytes) = 4096 B weights | 64 fp16 scales (128 B) | 64 4-bit zeros (32 B)
 *           (group size 64 / 32: two / four scale blocks, then as many zero blocks: 4416 / 4736 bytes)
 *   W8 tile (8320 bytes) = 8192 B weights | 64 fp16 scales (128 B)
 *
 * Inside a tile the weights are stored in the register order of the tensor-core operand
 * that consumes them; tf_unpack_w4 / tf_unpack_w8 are the authoritative decoders.  N is
 * padded up to a multiple of TF_TILE_N with weights that dequantize to exactly 0
 * (q = z, s = 0), the padding noted in Section 5.2; padded columns are never written to Y.
 * The blob is position independent: copy it to the device with any memcpy.
 */
typedef struct tf_blob_header {
    uint32_t magic;        /* 0x31424654 = "TFB1" */
    uint32_t version;      /* 1 */
    uint32_t bits;         /* 4 or 8 */
    uint32_t K;
    uint32_t N;
    uint32_t group_size;   /* as given to the packer; a multiple of TF_TILE_K, or 64 / 32 (4-bit) */
    uint32_t n_padded;     /* N rounded up to a multiple of TF_TILE_N */
    uint32_t strips;       /* n_padded / TF_TILE_N */
    uint32_t ktiles;       /* K / TF_TILE_K */
    uint32_t tile_bytes;   /* 4256 (W4; 4416 / 4736 for group size 64 / 32) or 8320 (W8) */
    uint64_t tiles_offset; /* 256 */
    uint64_t total_bytes;  /* = tf_packed_size(bits, K, N, group_size) */
    uint8_t  reserved[200];
} tf_blob_header;

/* Bytes of the packed blob, or 0 if the shape is illegal.
 * Legal: bits in {4, 8}; 128 <= K <= TF_MAX_DIM; 8 <= N <= TF_MAX_DIM; N % 8 == 0; K % group_size == 0;
 * group_size % 128 == 0, or, for bits == 4, group_size 64 or 32 (the tile then carries two or four
 * scale and zero-point blocks, group after group along k: 4416 or 4736 bytes per tile). */
size_t tf_packed_size(int bits, int K, int N, int group_size);

/*
 * Offline pre-tiling of AWQ-format W4A16 weights (Section 4.2; format of Section 2.2).
 *   qweight     host, uint32 [K][N/8]: eight 4-bit codes per word along N; bits [4i,4i+4) of
 *               word j hold column 8j + (0,2,4,6,1,3,5,7)[i].
 *   scales_fp16 host, IEEE fp16 bit patterns [K/group_size][N].
 *   qzeros      host, uint32 [K/group_size][N/8], same nibble order as qweight.
 *   out         host, out_bytes >= tf_packed_size(4, K, N, group_size); written completely.
 * Dequantization meaning of the result: w[k][n] = s[k/g][n] * (q[k][n] - z[k/g][n])  (Eq. 2).
 * Pure host code, deterministic, no allocation proportional to the input.
 * Errors: TF_ERR_NULL, TF_ERR_SHAPE (see tf_packed_size), TF_ERR_WORKSPACE (out_bytes too small).
 */
tf_status tf_pack_awq(const uint32_t* qweight, const uint16_t* scales_fp16, const uint32_t* qzeros,
                      int K, int N, int group_size, void* out, size_t out_bytes);

/*
 * Offline pre-tiling of symmetric W8A16 weights (Section 4.2, last paragraph; Eq. 1).
 *   w           host, int8 [K][N] row-major (the full range -128..127 is accepted).
 *   scales_fp16 host, fp16 bit patterns [K/group_size][N]; group_size == K is the
 *               per-channel case of Section 2.2.
 * Meaning: w_hat[k][n] = s[k/g][n] * w[k][n].  Otherwise as tf_pack_awq.
 */
tf_status tf_pack_w8(const int8_t* w, const uint16_t* scales_fp16,
                     int K, int N, int group_size, void* out, size_t out_bytes);

/*
 * Decode a packed blob on the GPU with the same device routines the GEMV / GEMM kernels use
 * (the unpack step of Section 4.3).  Outputs are bit-exact copies of what was packed:
 *   q      device, uint8 [K][N] (W4: 0..15) / int8 [K][N] (W8)
 *   z      device, uint8 [K/group_size][N]            (W4 only)
 *   s_fp16 device, fp16 bit patterns [K/group_size][N]
 * Any of the output pointers may be NULL to skip that output.
 * Errors: TF_ERR_NULL (packed), TF_ERR_SHAPE, TF_ERR_ALIGN (packed), TF_ERR_ARCH, TF_ERR_CUDA.
 * A blob whose header does not match (bits, K, N) leaves the outputs untouched.
 */
tf_status tf_unpack_w4(const void* packed, uint8_t* q, uint8_t* z, uint16_t* s_fp16,
                       int K, int N, int group_size, void* cuda_stream);
tf_status tf_unpack_w8(const void* packed, int8_t* q, uint16_t* s_fp16,
                       int K, int N, int group_size, void* cuda_stream);

/*
 * Concatenation along N at pack time.  Section 4.5: dispatching a kernel is amortized by a large
 * prefill GEMM but costly for the short GEMV operators of token generation.  A decoder layer applies
 * several weight matrices to the same activations; packing them side by side turns their GEMVs/GEMMs
 * into one launch (fused QKV, fused gate + up).
 *   parts    host, `count` pointers to blobs from tf_pack_awq / tf_pack_w8 (or from this call).
 *   out      host, receives the blob of the matrix [W_0 | W_1 | ... ] with N = sum of the parts' N:
 *            byte for byte what the packer gives for the column-concatenated inputs.
 *   out_bytes  capacity of `out`; at least tf_packed_size(bits, K, N, group_size).
 * All parts must have the same bits, K and group_size; every part but the last must have N % 64 == 0
 * (it must end on a strip boundary); the total N must not exceed TF_MAX_DIM.  `out` must not overlap a part.
 * Errors: TF_ERR_NULL, TF_ERR_BLOB (a part is not a valid blob), TF_ERR_SHAPE (count < 1, mismatch,
 *         unaligned part, N too large), TF_ERR_WORKSPACE (out_bytes too small).
 */
tf_status tf_pack_concat(const void* const* parts, int count, void* out, size_t out_bytes);

/*
 * Column-parallel sharding over several GPUs (Section 4.4: every worker owns distinct output columns, the
 * activations are shared, no partial sums travel between workers).
 * tf_shard_columns: the column range [n_begin, n_begin + n_count) of part `part` of `parts` when the N columns are
 *   dealt out in whole strips of TF_TILE_N (the last part takes the ragged end); pure arithmetic.
 * tf_pack_shard: the blob of that column range, cut out of the blob of the whole matrix (host): byte for byte what
 *   the packer gives for the column-sliced inputs.  Each GPU then calls tf_gemv_* / tf_gemm_* with N = n_count on
 *   its shard and the full activations, and writes y[:, n_begin : n_begin + n_count]; the only exchange is an
 *   all-gather of the results (NCCL), done by the caller.
 *   out_bytes at least tf_packed_size(bits, K, n_count, group_size).  `out` must not overlap `packed`.
 * Errors: TF_ERR_NULL, TF_ERR_BLOB (not a valid blob), TF_ERR_SHAPE (part outside 0..parts-1, more parts than
 *         strips), TF_ERR_WORKSPACE (out_bytes too small).
 */
tf_status tf_shard_columns(int N, int part, int parts, int* n_begin, int* n_count);
tf_status tf_pack_shard(const void* packed, int part, int parts, void* out, size_t out_bytes);

/*
 * Ablation baseline (Sections 4.1 and 5.5): dequantize the whole matrix into global memory, to be
 * multiplied by a separate full-precision kernel -- the arrangement the fused kernels replace.
 *   packed   device blob; bits = 4 or 8 must match it.
 *   w_bf16   device, bf16 [K][N] row-major; receives w[k][n] = bf16((q - z) * s) for W4, bf16(q * s) for
 *            W8, rounded to nearest even once ((q - z) * s itself is exact in fp32).
 * Errors: TF_ERR_NULL, TF_ERR_SHAPE, TF_ERR_ALIGN, TF_ERR_ARCH, TF_ERR_CUDA.  A blob whose header does
 * not match (bits, K, N) leaves w_bf16 untouched.
 */
tf_status tf_dequant_bf16(const void* packed, void* w_bf16, int bits, int K, int N, void* cuda_stream);

/*
 * Decode-phase fused GEMV (Sections 4.3 "GEMV microkernel" and 4.4): 1 <= M <= 16 tokens.
 *   packed   device, blob from tf_pack_awq (w4a16) / tf_pack_w8 (w8a16) for this K, N.  Weights are treated
 *            as constants: the kernels start fetching them before the stream's earlier kernels have finished
 *            where those release their dependents early (programmatic dependent launch, as this library's
 *            own kernels do).  Ordinary stream order covers a blob written by a copy or by a kernel that does
 *            not do that.  Activations, results and the workspace are always touched in stream order: every
 *            warp that reads a_bf16, writes y_bf16 or uses the workspace first waits until all earlier work
 *            of the stream has completed, so a call may consume what the call before it wrote.
 *   a_bf16   device, bf16 [M][K] row-major, leading dimension K.
 *   y_bf16   device, bf16 [M][N] row-major, leading dimension N; fully overwritten.
 *   workspace, workspace_bytes   device scratch of at least tf_workspace_size(op, M, K, N)
 *            bytes.  Its first TF_WORKSPACE_ZERO_BYTES bytes must be zero before the first call that
 *            uses it; every call leaves them zero again unless it reports an error there (after an error
 *            status, clear them before the next call).  Bytes [0,16) hold the device status word read by
 *            tf_device_status; the rest holds arrival counters and the fp32 partial sums of the few
 *            column strips that are split between CTAs (a partial sum announces itself: its slot is all
 *            +0.0 until the sums, with +0.0 written as -0.0, arrive; no fence, no counter).  GEMV and
 *            GEMM calls lay the workspace out compatibly: one workspace of the largest size needed may
 *            serve every call of a stream, in any order.  Use one workspace per stream: calls that run
 *            concurrently must not share one.
 * Arithmetic: weights are kept exact ((q - z) as small integers, scale applied in fp32 to
 * per-group partial sums), fp32 accumulation, one round-to-nearest-even to bf16 at the end.
 * With M <= 2 both calls form the products in integers: per token and 128-deep k-tile the
 * activations are rewritten on the tile's own power-of-two scale (exact for values within 2^14
 * of the tile's largest magnitude, rounded at 2^-22 of it below that), multiplied with the codes
 * exactly in 32 bits (4-bit: sum of q times activation minus z times the sum of the activations,
 * both exact integers, so q == z still gives exactly 0), and scaled back in fp32.  An Inf or NaN
 * activation makes every output of its token NaN there (the floating-point paths give Inf or NaN,
 * as IEEE arithmetic does).
 * Each persistent CTA streams one contiguous range of packed tiles; a strip of 64 output
 * columns that is cut between CTAs is summed in a fixed order by the CTA that holds its first tile.
 * The blob must be at least tf_packed_size(bits, K, N, 128) bytes for the K, N passed here.
 * Errors: TF_ERR_NULL, TF_ERR_SHAPE (M outside 1..16, K % 128, N % 8, limits), TF_ERR_ALIGN,
 *         TF_ERR_WORKSPACE, TF_ERR_ARCH, TF_ERR_CUDA.  A blob/argument mismatch is detected on
 *         the device: y is left untouched and the status word becomes TF_ERR_BLOB.
 */
tf_status tf_gemv_w4a16(const void* packed, const void* a_bf16, void* y_bf16,
                        int M, int K, int N, void* workspace, size_t workspace_bytes,
                        void* cuda_stream);
tf_status tf_gemv_w8a16(const void* packed, const void* a_bf16, void* y_bf16,
                        int M, int K, int N, void* workspace, size_t workspace_bytes,
                        void* cuda_stream);

/*
 * Prefill-phase fused GEMM (Section 4.3 "GEMM microkernel"): 1 <= M <= 4096 tokens,
 * K, N <= 32768.  Same arguments as the GEMV.  Each packed weight tile is dequantized once
 * per CTA tile into the tensor-memory operand of the tcgen05 tensor cores as bf16 and reused by
 * every token row of the tile (the dequantize-once rule of Section 4.1); accumulation is fp32 in
 * tensor memory.  The operand is w = bf16((q-z) * s), the exact product rounded to bf16 once (what
 * tf_dequant_bf16 writes); for W8 the fp16 scale is split into its upper 8 bits and the rest and
 * w = bf16(q * hi + bf16(q * lo)), which differs from one rounding by at most 2^-17 of w.
 * Work is split evenly over the persistent CTAs in units of (output tile, 128-deep k-tile): an
 * output tile whose K range is cut between CTAs is summed in fp32 through the workspace, in CTA
 * order, by the last CTA to finish its part, so results do not depend on timing.
 * Workspace: tf_workspace_size() bytes (tens of MB: two fp32 tile slots per CTA).  Its first
 * TF_WORKSPACE_ZERO_BYTES bytes (status word, arrival counters, the GEMV's slots) must be zero before the first
 * call that uses it; every call leaves them zero again unless it reports an error there.  One
 * workspace per stream (it may be the one the GEMV calls of that stream use): calls that run
 * concurrently must not share one.
 * Errors as for the GEMV; M range 1..4096.
 */
tf_status tf_gemm_w4a16(const void* packed, const void* a_bf16, void* y_bf16,
                        int M, int K, int N, void* workspace, size_t workspace_bytes,
                        void* cuda_stream);
tf_status tf_gemm_w8a16(const void* packed, const void* a_bf16, void* y_bf16,
                        int M, int K, int N, void* workspace, size_t workspace_bytes,
                        void* cuda_stream);

/*
 * The same two W4A16 operations for blobs packed with any legal group size (Section 2.2: group-wise
 * quantization; 128 is the paper's and the default, 64 and 32 are the other sizes in common use).  group_size
 * must be the one given to tf_pack_awq; tf_gemv_w4a16 / tf_gemm_w4a16 are these calls with group_size = 128
 * and serve every blob whose group size is a multiple of 128.  With two or four groups per tile the GEMV
 * takes its floating-point path for every token count (scale applied to the fp32 sum of each group), the
 * GEMM reads the scale and zero point of each 64- or 32-deep slice of its dequantization job; everything
 * else, including workspace size and layout, is unchanged.
 * Errors: as tf_gemv_w4a16 / tf_gemm_w4a16; TF_ERR_SHAPE also for an illegal group size; a blob packed with
 * another group size is detected on the device (TF_ERR_BLOB, y untouched).
 */
tf_status tf_gemv_w4a16_grouped(const void* packed, const void* a_bf16, void* y_bf16,
                                int M, int K, int N, int group_size, void* workspace, size_t workspace_bytes,
                                void* cuda_stream);
tf_status tf_gemm_w4a16_grouped(const void* packed, const void* a_bf16, void* y_bf16,
                                int M, int K, int N, int group_size, void* workspace, size_t workspace_bytes,
                                void* cuda_stream);

/*
 * tf_gemv_w4a16 without a caller-provided workspace and without any allocation.  (The paper has no
 * counterpart to this call; it exists for hosts of this library that cannot give it device memory: a
 * plug-in in a process whose memory pool another framework owns, a thread that must stay out of the
 * allocator, code inside a stream capture.)
 *   Scratch (status word, fp32 partial sums of strips cut between CTAs) is a fixed array of 675,840 bytes
 *   inside the library's device image: every GPU that loads the library holds it
 *   until the process exits.  It covers every shape tf_gemv_w4a16 accepts (1 <= M <= 16, K and N up to
 *   32768) on devices with any SM count (at most 160 persistent CTAs are used); shapes beyond those limits
 *   are rejected with TF_ERR_SHAPE.
 *   The call never calls cudaMalloc, cudaFree or an allocating library routine.  The first call on a device
 *   (of either function below) looks up the array's device address and does every other one-time step a
 *   launch of any shape can need (function attributes of all kernel variants, occupancy queries), with that
 *   device current: make that first call before any stream capture.  Each call first clears, on
 *   `cuda_stream`, the part of the array that must start at zero.  All calls share the array: calls that
 *   overlap on the GPU (different streams) race on it, so serialise them.
 *   Arguments, arithmetic and results are those of tf_gemv_w4a16.  What tf_device_status reports for a
 *   workspace (a blob that does not match the arguments, a device-side wait that gave up) is reported for the
 *   last static call of the current device by tf_gemv_w4a16_static_status, which synchronises `cuda_stream`
 *   (and, when it reports an error, clears the whole array so that the next call starts clean).
 * Errors: TF_ERR_NULL, TF_ERR_SHAPE, TF_ERR_ALIGN, TF_ERR_ARCH, TF_ERR_CUDA.
 */
tf_status tf_gemv_w4a16_static(const void* packed, const void* a_bf16, void* y_bf16,
                               int M, int K, int N, void* cuda_stream);
tf_status tf_gemv_w4a16_static_status(void* cuda_stream);

/*
 * Second ablation arm (Section 5.5 separates the gain of fusing from the gain of the offline re-tiling of
 * Section 4.2): the fused W4A16 GEMV computed straight from the AWQ arrays, without tf_pack_awq.
 *   qweight     device, uint32 [K][N/8], eight 4-bit codes per word in nibble order 0,2,4,6,1,3,5,7
 *   scales_fp16 device, fp16 bits [K/group_size][N]
 *   qzeros      device, uint32 [K/group_size][N/8], same nibble order
 *   a_bf16      device, bf16 [M][K];  y_bf16  device, bf16 [M][N], fully overwritten
 *   group_size  32, 64 or 128 (this arm has no tile format to constrain it)
 *   workspace   device scratch of at least tf_gemv_awq_raw_workspace_size(M, K, N, group_size) bytes
 *               (fp32 partial sums of the split over K; no initial contents required, no status word).
 * Arithmetic: (q - z) exact; fp32 multiply-add per group and group sum times the fp16 scale in fp32 (up to 8
 * tokens), or bf16 x bf16 products of exact operands accumulated in fp32 over 16 rows on the warp MMA and
 * scaled in fp32 (9 to 16 tokens); fp32 partial sums added in a fixed order, one rounding to bf16.  Two kernel
 * launches on `cuda_stream`.
 * 1 <= M <= 16; K % group_size == 0; N % 8 == 0; K, N <= TF_MAX_DIM.
 * Errors: TF_ERR_NULL, TF_ERR_SHAPE, TF_ERR_ALIGN (every device pointer 16-byte aligned),
 *         TF_ERR_WORKSPACE, TF_ERR_ARCH, TF_ERR_CUDA.
 */
tf_status tf_gemv_awq_raw(const uint32_t* qweight, const uint16_t* scales_fp16, const uint32_t* qzeros,
                          const void* a_bf16, void* y_bf16, int M, int K, int N, int group_size,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);
/*
 * Pre-tiling on the GPU (Section 4.2's re-tiling done at run time): the AWQ arrays in device memory -> the packed
 * blob in device memory, byte for byte what tf_pack_awq writes (header included).  Arguments as tf_pack_awq, all
 * pointers device, 16-byte aligned; asynchronous on `cuda_stream`.
 * Errors: TF_ERR_NULL, TF_ERR_SHAPE, TF_ERR_WORKSPACE (out_bytes < tf_packed_size), TF_ERR_ALIGN, TF_ERR_ARCH, TF_ERR_CUDA.
 */
tf_status tf_pack_awq_device(const uint32_t* qweight, const uint16_t* scales_fp16, const uint32_t* qzeros,
                             int K, int N, int group_size, void* out, size_t out_bytes, void* cuda_stream);

/*
 * GEMM arm of the layout ablation (Section 5.5): the fused W4A16 GEMM computed from the AWQ arrays as given, with no
 * offline pre-tiling -- the arrays are re-tiled into scratch memory on every call (tf_pack_awq_device) and multiplied
 * by the pre-tiled GEMM.  The difference to tf_gemm_w4a16 on an offline blob is the cost the offline pre-tiling of
 * Section 4.2 removes.  Arguments as tf_gemv_awq_raw, 1 <= M <= 4096, group_size 32, 64 or a multiple of 128;
 *   workspace   device, at least tf_gemm_awq_raw_workspace_size(M, K, N, group_size) bytes (the GEMM's workspace,
 *               then the re-tiled blob); its first TF_WORKSPACE_ZERO_BYTES must be zero before first use and are left
 *               zero; tf_device_status reads its status word.
 * Results are those of tf_gemm_w4a16_grouped on the blob tf_pack_awq would write.  Two kernel launches.
 */
tf_status tf_gemm_awq_raw(const uint32_t* qweight, const uint16_t* scales_fp16, const uint32_t* qzeros,
                          const void* a_bf16, void* y_bf16, int M, int K, int N, int group_size,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);
size_t tf_gemm_awq_raw_workspace_size(int M, int K, int N, int group_size);

/* Scratch bytes tf_gemv_awq_raw needs on the current device (0 if the shape is illegal or the device is
 * not compute capability 10.x). */
size_t tf_gemv_awq_raw_workspace_size(int M, int K, int N, int group_size);

/*
 * Test and tuning hook: the launch geometry tf_gemv_w4a16 / tf_gemv_w8a16 would choose for this shape (Section
 * 4.4 maps work to cores statically; here the mapping depends on the shape, and tests assert which one they hit).
 *   sm_count  SMs to plan for; <= 0 = the current device (then TF_ERR_ARCH / TF_ERR_CUDA as for a compute call).
 *   out       host, 8 ints: persistent CTAs, threads per CTA, consumer warps, ring stages, whole-SM CTA (1) or
 *             half-SM (0), integer path (0 = no, 1 = activation pieces prepared per tile, 2 = kept per k-tile
 *             in a table), CTAs per cluster (1 = cut strips go through the workspace), and the number of clusters
 *             (cluster mode) or of CTAs that get tiles (otherwise).
 * Pure host code apart from the device query; launches nothing.  Errors: TF_ERR_NULL, TF_ERR_SHAPE.
 */
tf_status tf_gemv_plan(int bits, int M, int K, int N, int sm_count, int* out);

/*
 * Test hook for the failure path (the paper has no counterpart: its kernels run under a host runtime that owns
 * error handling).  Every device-side wait of the GEMV and GEMM kernels is bounded; when one runs out, all
 * roles of the CTA leave their loops, copies in flight are given time to land, tensor memory is freed, the
 * kernel returns and the status word of the workspace becomes TF_ERR_TIMEOUT.  This call makes that happen on
 * purpose, without faulting or hanging anything, for every tf_gemv_* / tf_gemm_* launch of this process that
 * follows it:
 *   wait_limit_kcycles   limit of a device-side wait in units of 1024 SM cycles (0 = the default, about 1 s);
 *                        must be below 2^24.
 *   drop_weight_copies   non-zero: the packed-weight producer issues no copies, so every wait for weights
 *                        runs out after the limit (y is then left untouched).
 * tf_debug_inject(0, 0) restores normal operation.  Process-wide, not for production use.
 * Errors: TF_ERR_SHAPE (limit out of range).
 */
tf_status tf_debug_inject(unsigned wait_limit_kcycles, int drop_weight_copies);

/* Scratch bytes the given operation needs for this shape (0 if none; 0 also if the shape
 * is illegal -- the compute call then reports TF_ERR_SHAPE). */
size_t tf_workspace_size(int op, int M, int K, int N);

/* Synchronise `cuda_stream`, read the status word at the start of `workspace` (device) and
 * return it: TF_OK, TF_ERR_BLOB or TF_ERR_TIMEOUT; TF_ERR_CUDA if the stream reports an error.
 * The word is sticky until the caller clears the first 16 bytes of the workspace. */
tf_status tf_device_status(const void* workspace, void* cuda_stream);

/* Static, NUL-terminated description of a status code. */
const char* tf_status_string(tf_status status);

/* Library version: major * 10000 + minor * 100 + patch. */
int tf_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TILEFUSE_H */
