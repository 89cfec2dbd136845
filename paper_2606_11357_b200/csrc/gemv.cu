// Decode-phase fused GEMV, M = 1..16 tokens (Sections 4.3 "GEMV microkernel" and 4.4).
//
// Persistent streaming kernel.  The packed blob is one long sequence of tiles (128 k x 64 n, each a
// contiguous payload carrying its scales and zeros, strip after strip).  That sequence is cut into
// equal contiguous ranges, one per CTA, so every CTA streams one contiguous byte range of HBM:
//
//   producer warp : one lane issues, per ring stage, one bulk (TMA) copy of several consecutive tiles;
//                   completion on mbarriers.  Weight bytes in flight are bounded by the ring, not by
//                   registers.  One lane with a short loop is enough: a lone lane streams 16 KB copies at
//                   the full HBM rate, while several lanes of one warp only take turns, and every
//                   instruction of this warp competes for issue slots with consumer warps that never idle.
//                   It reads nothing but weights, which are constants, so it does not wait for earlier
//                   kernels of the stream.
//   consumer warps: take tiles round-robin.  A warp reads the activations of a tile -- its own MMA
//                   fragment, 8 bytes per lane and 16-k block (integer path: its 4 k of the tile's 128 per
//                   token) -- straight from global memory (they sit in L2), never before the kernels ahead
//                   of this one on the stream have completed (every consumer warp executes the dependency
//                   wait first), and one tile ahead: the registers of a k-block are refilled for the warp's
//                   next tile as soon as that k-block's MMAs have been issued, so the L2 latency runs under
//                   the rest of the tile.  The ring holds nothing but weights (staging activations through
//                   the ring put a TMA load behind the dependency wait of every call, about 1 us, and took
//                   ring space from the weights: half of it for 9..16 tokens).  128-bit shared loads, codes -> exact small-integer bf16
//                   (q - z), contraction with the activations on the warp-level tensor-core MMA
//                   (weights = the 16x16 operand, up to 8 tokens = the 16x8 operand: the per-weight
//                   cost does not grow with M), fp16 scale applied in fp32 once per group.
//
//   reducer warp  : when the consumers finish the tiles of one strip inside this CTA's range they drop
//                   their fp32 partials into shared memory and move on; the reducer adds them up (fixed
//                   order), rounds to bf16 and stores y, so the consumers never wait at a strip boundary.
//
// A range may cut a strip (64 output columns) in two.  A CTA that holds a whole strip stores y
// directly.  Otherwise the reducer writes the fp32 partial to the workspace and bumps the strip's
// counter; the CTA that arrives last adds the partials in CTA order (not arrival order) and stores y, so
// results are deterministic and no CTA ever waits for another.  The head cut of a range is published as
// soon as it is complete (early in the kernel).  For the tail cut the reducer looks ahead: if every other
// contributor has already published, it fetches their partials while the consumers still work, and the
// end of the kernel is just one more add.  This keeps the paper's rule that partial sums do not travel
// between workers for everything but the (at most two) cut strips of a CTA.
#include <atomic>

#include "async.cuh"
#include "common.cuh"
#include "kernels.h"

namespace tf {

namespace {

// Integer warp MMA: D(16x8, s32) += A(16x32, s8) . B(32x8, s8).  Thread (g, t): a0 = row g, k 4t..4t+3; a1 = row g+8;
// a2, a3 = the same rows, k + 16; b0 = column g, k 4t..4t+3; b1 = k + 16; d = rows g, g+8 x columns 2t, 2t+1.
__device__ __forceinline__ void mma_s8_16832(int d[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// The same with D = A . B + c in every element (no accumulator to set first).
__device__ __forceinline__ void mma_s8_16832_first(int d[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1, int c) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(c));
}

// The same shapes with unsigned bytes in the 16-row operand (4-bit codes 0..15 as they come out of a packed word).
__device__ __forceinline__ void mma_u8s8_16832(int d[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_u8s8_16832_first(int d[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1, int c) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(c));
}

// int -> float for |v| < 2^22 without the conversion unit: the bits of the integer 0x4B400000 + v are the float
// 1.5 * 2^23 + v, exactly.  The integer MMAs start their accumulators at kIntAsFloatBias, so a tile's sums come out of
// the tensor pipe already in that form, and (f - 1.5 * 2^23) * c is one fused multiply-add with -1.5 * 2^23 * c.
constexpr int kIntAsFloatBias = 0x4B400000;
constexpr float kIntAsFloatBiasValue = 12582912.0f;

// Even split of `total` tiles over `grid` CTAs.  The products fit 32 bits (at most 256 x 512 tiles, K and N <= 32768,
// times at most 257 CTAs), and a 32-bit division is a fraction of the instructions of a 64-bit one.  These sit between
// the start of a CTA and its first weight copy, in the reducer's bookkeeping and in the cluster-mode finish; k32 chooses
// the width per kernel instantiation, by measurement: the 9..16-token kernels gained 1.1 us over the four layer shapes
// with 32 bits, the others lost 0.3 to 0.4 us (the same kernels, differently scheduled by the compiler).
template <bool k32>
__device__ __forceinline__ int range_start(int cta, int total, int grid) {
    if constexpr (k32) return static_cast<int>((static_cast<uint32_t>(cta) * static_cast<uint32_t>(total)) / static_cast<uint32_t>(grid));
    else return static_cast<int>((static_cast<long long>(cta) * total) / grid);
}
template <bool k32>
__device__ __forceinline__ int range_owner(int tile, int total, int grid) {
    if constexpr (k32) return static_cast<int>(((static_cast<uint32_t>(tile) + 1u) * static_cast<uint32_t>(grid) - 1u) / static_cast<uint32_t>(total));
    else return static_cast<int>(((static_cast<long long>(tile) + 1) * grid - 1) / total);
}

// The chunks of a tile range [t0, t0 + ntiles): up to kR consecutive tiles of one strip each.  Tiles are stored
// strip after strip, so the source pointer only ever advances.
struct ChunkWalk {
    int left, seg_left, T, ktiles, tile_bytes;
    const uint8_t* src;
    __device__ ChunkWalk(int t0, int ntiles, int ktiles_, const uint8_t* tiles, int tile_bytes_)
        : left(ntiles), ktiles(ktiles_), tile_bytes(tile_bytes_) {
        const int strip = t0 / ktiles;
        T = t0 - strip * ktiles;
        seg_left = min(ntiles, ktiles - T);
        src = tiles + (size_t)t0 * tile_bytes;
    }
    __device__ bool done() const { return left == 0; }
    __device__ void next(int kR, int& tiles_here, int& T_first, const uint8_t*& src_first) {
        tiles_here = min(kR, seg_left);
        T_first = T;
        src_first = src;
        src += (size_t)tiles_here * tile_bytes;
        T += tiles_here;
        seg_left -= tiles_here;
        left -= tiles_here;
        if (seg_left == 0) { T = 0; seg_left = min(left, ktiles); }
    }
};

// fp32 [token][64 n] tile held as float4 per lane (element 4 (lane + 32 e)) -> bf16 -> y; rows >= M and columns >= N
// are not written (N % 8 == 0: a group of 4 columns is in or out)
template <int kVec>
__device__ __forceinline__ void store_strip(__nv_bfloat16* y, const float4 (&tot)[kVec], int strip, int M, int N, int lane) {
#pragma unroll
    for (int e = 0; e < kVec; ++e) {
        const int idx = 4 * (lane + 32 * e);
        const int m = idx / kTileN, n = strip * kTileN + (idx % kTileN);
        if (m < M && n < N) {
            uint2 o;
            o.x = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(tot[e].x)) |
                  ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(tot[e].y)) << 16);
            o.y = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(tot[e].z)) |
                  ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(tot[e].w)) << 16);
            *reinterpret_cast<uint2*>(y + (size_t)m * N + n) = o;
        }
    }
}

// Hand-over of a cut strip without a fence or a counter.  The partial-sum slots of a workspace are all +0.0 bits
// between calls.  A contributor stores its sums with every +0.0 replaced by -0.0 (the same number), so a word that is
// not +0.0 has arrived, whatever the order in which the memory system delivers the words.  The finisher reads a slot
// until all of its words have arrived, adds it, and puts +0.0 back for the next call.  It waits for stores that were
// issued at about the time it starts to look (every wait is bounded), and the critical path of a cut strip is one
// trip to the L2 instead of three (stores acknowledged -> arrival counter returned -> partial sums loaded).
__device__ __forceinline__ float4 never_plus_zero(float4 v) {
    const uint32_t x = __float_as_uint(v.x), y = __float_as_uint(v.y), z = __float_as_uint(v.z), w = __float_as_uint(v.w);
    return make_float4(__uint_as_float(x == 0u ? 0x80000000u : x), __uint_as_float(y == 0u ? 0x80000000u : y),
                       __uint_as_float(z == 0u ? 0x80000000u : z), __uint_as_float(w == 0u ? 0x80000000u : w));
}
// `slot` already points at this lane's first float4 of the partial of the first of `count` (<= kBatch) consecutive
// CTAs; rows of tokens >= M are neither written nor read.  The loads of all `count` partials are issued together (one
// trip to the L2 per turn), then the partials are added to `acc` in CTA order and their slots cleared.  Returns false
// if the wait ran out.  Kept out of line so that the polling loop does not take part in the register allocation of the
// streaming kernel around it.
template <int kVec, int kBatch>
__device__ __noinline__ bool gather_partials(float4* slot, int count, int M, float4 (&acc)[kVec], volatile uint32_t* abort_flag, uint32_t site) {
    constexpr int kSlotVec = kGemvSlotBytes / 16;
    float4 v[kBatch][kVec];
    const long long t_begin = clock64();
    for (;;) {
        bool here = true;
#pragma unroll
        for (int b = 0; b < kBatch; ++b)
#pragma unroll
            for (int e = 0; e < kVec; ++e) {
                v[b][e] = make_float4(-0.f, -0.f, -0.f, -0.f);
                if (b < count && 2 * e < M)                       // a real load on every turn of the loop, from the L2
                    asm volatile("ld.relaxed.gpu.global.v4.f32 {%0, %1, %2, %3}, [%4];"
                                 : "=f"(v[b][e].x), "=f"(v[b][e].y), "=f"(v[b][e].z), "=f"(v[b][e].w)
                                 : "l"(slot + b * kSlotVec + 32 * e) : "memory");
            }
#pragma unroll
        for (int b = 0; b < kBatch; ++b)
#pragma unroll
            for (int e = 0; e < kVec; ++e)
                here = here && __float_as_uint(v[b][e].x) != 0u && __float_as_uint(v[b][e].y) != 0u &&
                       __float_as_uint(v[b][e].z) != 0u && __float_as_uint(v[b][e].w) != 0u;
        if (__all_sync(0xFFFFFFFFu, here)) break;
        if (*abort_flag != 0) return false;
        if (wait_expired(t_begin, abort_flag)) { *abort_flag = site; return false; }
    }
#pragma unroll
    for (int b = 0; b < kBatch; ++b)
#pragma unroll
        for (int e = 0; e < kVec; ++e) {
            acc[e].x += v[b][e].x; acc[e].y += v[b][e].y; acc[e].z += v[b][e].z; acc[e].w += v[b][e].w;
            if (b < count && 2 * e < M) __stcg(slot + b * kSlotVec + 32 * e, make_float4(0.f, 0.f, 0.f, 0.f));
        }
    return true;
}

// The same hand-over taken row pair by row pair: for float4 index e (token rows 2e, 2e + 1) the words of up to four
// consecutive CTAs' partials are requested together, so a strip shared by many CTAs and few tokens costs one trip per
// row pair instead of one per contributor, in 16 registers.  `slot` as above; adds to acc[e] in CTA order.
template <int kVec>
__device__ __noinline__ bool gather_rows(float4* slot, int count, int M, float4 (&acc)[kVec], volatile uint32_t* abort_flag, uint32_t site) {
    constexpr int kSlotVec = kGemvSlotBytes / 16;
    const long long t_begin = clock64();
    for (int e = 0; e < kVec && 2 * e < M; ++e) {
        float4 v[4];
        for (;;) {
            bool here = true;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                v[b] = make_float4(-0.f, -0.f, -0.f, -0.f);
                if (b < count)
                    asm volatile("ld.relaxed.gpu.global.v4.f32 {%0, %1, %2, %3}, [%4];"
                                 : "=f"(v[b].x), "=f"(v[b].y), "=f"(v[b].z), "=f"(v[b].w) : "l"(slot + b * kSlotVec + 32 * e) : "memory");
            }
#pragma unroll
            for (int b = 0; b < 4; ++b)
                here = here && __float_as_uint(v[b].x) != 0u && __float_as_uint(v[b].y) != 0u && __float_as_uint(v[b].z) != 0u &&
                       __float_as_uint(v[b].w) != 0u;
            if (__all_sync(0xFFFFFFFFu, here)) break;
            if (*abort_flag != 0) return false;
            if (wait_expired(t_begin, abort_flag)) { *abort_flag = site; return false; }
        }
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            a.x += v[b].x; a.y += v[b].y; a.z += v[b].z; a.w += v[b].w;
            if (b < count) __stcg(slot + b * kSlotVec + 32 * e, make_float4(0.f, 0.f, 0.f, 0.f));
        }
#pragma unroll
        for (int k = 0; k < kVec; ++k)
            if (k == e) { acc[k].x += a.x; acc[k].y += a.y; acc[k].z += a.z; acc[k].w += a.w; }
    }
    return true;
}

}  // namespace

// Integer path: the activation pieces of one k-tile (up to two tokens), from the raw bf16 of lane L (k = 4L .. 4L+3).
// dst: [column][kGemvPieceColWords] piece words, the word of lane L at (L & 3) * 8 + (L >> 2), so that a thread of the
// MMA phase finds the eight k-blocks of its column and k quarter in two 16-byte loads (columns 36 words apart fall
// into different banks); meta: [column] {2^(emax-148) 256^j, sum of the piece over the tile} in 8-byte entries, a
// thread's two columns = one 16-byte load (with 4-byte entries and an 8-byte load the same kernel ran 12 % slower:
// measured, cause not established).
constexpr int kGemvPieceColWords = 36;
template <int BITS>
__device__ __forceinline__ void make_pieces(const uint2 (&raws)[2], uint32_t* dst, uint2* meta, int M, int lane) {
    constexpr int kColWords = kGemvPieceColWords;
#pragma unroll
    for (int m = 0; m < 2; ++m) {
        if (m < M) {
            const uint2 raw = raws[m];
            const uint32_t x0 = raw.x, x1 = raw.y;
            uint32_t e = max(max((x0 << 17) >> 24, (x0 << 1) >> 24), max((x1 << 17) >> 24, (x1 << 1) >> 24));
            e = __reduce_max_sync(0xFFFFFFFFu, e);
            e = max(e, 22u);                                  // keeps both powers of two normal numbers
            const float mult = __uint_as_float((275u - e) << 23);          // 2^(148 - emax)
            // v + 0x808080 has the bytes p0 + 128, p1 + 128, p2 + 128 of the balanced split
            uint32_t v[4];
            v[0] = (uint32_t)__float2int_rn(__uint_as_float(x0 << 16) * mult) + 0x808080u;
            v[1] = (uint32_t)__float2int_rn(__uint_as_float(x0 & 0xFFFF0000u) * mult) + 0x808080u;
            v[2] = (uint32_t)__float2int_rn(__uint_as_float(x1 << 16) * mult) + 0x808080u;
            v[3] = (uint32_t)__float2int_rn(__uint_as_float(x1 & 0xFFFF0000u) * mult) + 0x808080u;
            // 4 x 3 byte transpose: one word per piece, bytes in the k order of the weight operand's bytes
            // (int8: k, k+1, k+2, k+3; 4-bit: k, k+2, k+1, k+3, the order of a packed word's nibble pairs)
            const uint32_t ab01 = __byte_perm(v[0], v[1], 0x5140), ab2 = __byte_perm(v[0], v[1], 0x0062);
            const uint32_t cd01 = __byte_perm(v[2], v[3], 0x5140), cd2 = __byte_perm(v[2], v[3], 0x0062);
            uint32_t word[3];
            word[0] = __byte_perm(ab01, cd01, BITS == 8 ? 0x5410 : 0x5140) ^ 0x80808080u;
            word[1] = __byte_perm(ab01, cd01, BITS == 8 ? 0x7632 : 0x7362) ^ 0x80808080u;
            word[2] = __byte_perm(ab2, cd2, BITS == 8 ? 0x5410 : 0x5140) ^ 0x80808080u;
            // 2^(emax - 148); an Inf or NaN among the 128 activations makes this token's outputs NaN
            const float se = e == 255u ? __uint_as_float(0x7FC00000u) : __uint_as_float((e - 21u) << 23);
#pragma unroll
            for (int j = 0; j < 3; ++j) {
                const int c = 3 * m + j;
                dst[c * kColWords + (lane & 3) * 8 + (lane >> 2)] = word[j];
                int psum = 0;                           // 4-bit: sum of the piece over the tile's 128 k, for the zero point
                if constexpr (BITS == 4) psum = __reduce_add_sync(0xFFFFFFFFu, __dp4a((int)word[j], 0x01010101, 0));
                if (lane == 0) meta[c] = make_uint2(__float_as_uint(se * (j == 0 ? 1.f : j == 1 ? 256.f : 65536.f)), (uint32_t)psum);
            }
        }
    }
    if (lane == 0) {                                    // columns without a token contribute nothing
#pragma unroll
        for (int c = 3; c < 8; ++c)
            if (c >= 3 * M) meta[c] = make_uint2(0u, 0u);
    }
}
// The same as a call: where pieces are prepared on the first visit of a k-tile only, the code stays out of the tile
// loop's register allocation.
template <int BITS>
__device__ __noinline__ void make_pieces_call(const uint2 (&raws)[2], uint32_t* dst, uint2* meta, int M, int lane) {
    make_pieces<BITS>(raws, dst, meta, M, lane);
}

// G = groups per tile: 1 for group sizes that are multiples of 128, 2 / 4 for the 4-bit group sizes 64 / 32.
// I8 = 0: floating-point path; 1: integer path, a consumer warp prepares the activation pieces of every tile it works
// on; 2: integer path for ranges that pass over the same k-tiles more than once, with K a multiple of 128 times the
// number of consumer warps: a warp then meets the same k-tiles on every pass, prepares the pieces of a k-tile on its
// first visit and keeps them (piece table, one entry per k-tile, each entry written and read by one warp only).
template <int BITS, int MT, bool FULL, bool CL, int I8, int G = 1>
__global__ void __launch_bounds__(gemv_max_threads(MT, FULL, I8 != 0), FULL ? 1 : 2)
gemv_stream_kernel(const uint8_t* __restrict__ blob, const __nv_bfloat16* __restrict__ a_glob, __nv_bfloat16* __restrict__ y, int M, int K, int N, int ktiles, int total_tiles,
                   int nstages, int stage_bytes, int csize, int nclusters, int xslot_bytes, int nred, int piece_tab,
                   uint8_t* __restrict__ workspace, uint32_t debug) {
    static_assert(G == 1 || (BITS == 4 && !I8 && !CL && FULL), "several groups per tile: 4-bit, floating-point path, whole SM");
    constexpr int kTileBytes = tile_bytes(BITS, G);
    constexpr int kWeightBytes = BITS == 4 ? kW4WeightBytes : kW8WeightBytes;
    constexpr int kR = gemv_chunk_tiles(BITS);            // tiles per bulk copy / ring stage
    constexpr int kTok = 8 * MT;
    constexpr int kVecPerKb = BITS == 4 ? 1 : 2;
    constexpr int kRedWarp = (I8 ? 2 : kTok) * kTileN;    // floats one consumer warp drops per strip segment (integer path: two token rows)

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    // layout: barriers + flags (kGemvBarrierBytes) | red [consumers][kTok][64] fp32 | ring (1024-aligned stages)
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + (2 * kGemvMaxStages + 4) * 8);
    // stage_tag[s] = index of the chunk whose copies were last issued into ring stage s.  A consumer warp does
    // not touch every use of a stage, so the parity of the stage's mbarrier alone could alias (a warp two uses
    // ahead would see "parity differs" and run on old data); it first waits for its own chunk's tag.
    volatile uint32_t* stage_tag = reinterpret_cast<volatile uint32_t*>(smem + 1024);
    const int nconsumers = (blockDim.x >> 5) - 2;
    float* red = reinterpret_cast<float*>(smem + kGemvBarrierBytes);
    // xred [csize][xslot]: in cluster mode, the partials other CTAs of the cluster send to the finisher of a strip
    uint8_t* xred = smem + kGemvBarrierBytes + nred * nconsumers * kRedWarp * 4;
    // pscr: integer path.  [consumers][1 KB], a warp's activation pieces of the tile it works on; or
    // [piece_tab][kGemvPieceEntryBytes per token], the pieces of every k-tile of the CTA's range
    uint32_t* pscr = reinterpret_cast<uint32_t*>(xred + ((CL && csize > 1 ? csize * xslot_bytes : 0) + 1023) / 1024 * 1024);
    // abuf [consumers][2][16 rows of kActRowBytes]: 9..16 tokens, a warp's activations of the tile it works on and of its next one
    uint8_t* abuf = reinterpret_cast<uint8_t*>(pscr) + (I8 == 2 ? (piece_tab * kGemvPieceEntryBytes * M + 1023) / 1024 * 1024 : I8 == 1 ? nconsumers * 1024 : 0);
    uint8_t* ring = abuf + (MT == 2 ? nconsumers * kGemvActWarpBytes : 0);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x;
    // "Contributor space": the CTAs that split one pool of tiles evenly among themselves.  Global mode: all CTAs
    // of the grid over all tiles.  Cluster mode: the CTAs of one cluster over the whole strips that cluster owns,
    // so that a strip is only ever shared inside a cluster and can be summed through distributed shared memory.
    // In global mode `nclusters` carries the number of CTAs that take part (the first ones of the grid); the rest
    // of the grid has no tiles and only keeps one CTA of this kernel on every SM (see plan_gemv).
    int cn = nclusters, crank = cta, cbase = 0, ctiles = total_tiles;
    if (CL && csize > 1) {
        const int q = cta / csize, strips = total_tiles / ktiles;
        const int s0 = range_start<MT == 2>(q, strips, nclusters), s1 = range_start<MT == 2>(q + 1, strips, nclusters);
        cn = csize; crank = cta - q * csize; cbase = s0 * ktiles; ctiles = (s1 - s0) * ktiles;
    }
    const bool idle = crank >= cn;
    const int t0 = idle ? 0 : cbase + range_start<MT == 2>(crank, ctiles, cn);
    const int ntiles = idle ? 0 : cbase + range_start<MT == 2>(crank + 1, ctiles, cn) - t0;
    int fin_strip = -1, fin_first = 0;          // cluster mode: the strip this CTA finishes after the cluster barrier

    DeviceStatus* status = reinterpret_cast<DeviceStatus*>(workspace);
    float* partials = reinterpret_cast<float*>(workspace + kGemvPartialOffset);

    const bool header_ok = header_matches(blob, BITS, (uint32_t)K, (uint32_t)N) && group_size_fits(blob, G);

    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kGemvMaxStages);
    const uint32_t seg_full0 = smem_u32(bars + 2 * kGemvMaxStages), seg_free0 = seg_full0 + 16;
    // One thread per ring stage, one more for the rest: the set-up sits between the start of a CTA and its first
    // weight copy (one thread doing all of it in turn cost the decode step 1.7 us).
    if (threadIdx.x < (unsigned)nstages) {
        const int s = threadIdx.x;
        mbar_init(full0 + 8 * s, 1);
        mbar_init(empty0 + 8 * s, kR);           // every tile of a chunk is released by its consumer warp
        stage_tag[s] = 0xFFFFFFFFu;
        mbar_init_fence();
    } else if (threadIdx.x == 64) {
        for (int b = 0; b < 2; ++b) {                   // one pair per partial-sum buffer (nred = 1 or 2)
            mbar_init(seg_full0 + 8 * b, nconsumers);   // every consumer warp has dropped its partial
            mbar_init(seg_free0 + 8 * b, 1);            // the reducer has read them
        }
        abort_flag[0] = 0;
        abort_flag[1] = wait_limit_kcycles(debug);
        mbar_init_fence();
    }
    __syncthreads();
    // Programmatic dependent launch: the next kernel on the stream may start as SMs free up.  In this kernel
    // only the packed weights (constants) are read before grid_dependency_wait(): the producer lane never waits,
    // every consumer warp waits before its first activation load, the reducer warp before it touches y or the
    // workspace, thread 0 before it writes the status word.  (What keeps two half-SM CTAs of one GEMV off the same
    // SM when they come in behind a whole-SM kernel is decided at launch: see launch_one.)
    grid_launch_dependents();

    if (warp == 0) {
        // ---------------- producer: stream this CTA's contiguous tile range through the ring --------------
        // One lane issues, per chunk, one bulk copy of up to kR contiguous tiles of one strip.  Chunks never straddle
        // a strip boundary.  The loop is kept to a few dozen instructions per chunk: this warp shares its scheduler
        // with consumer warps that never idle.  It reads nothing but the packed weights, which are constants, so it
        // does not wait for the kernels before this one: the first ring fill is on its way while they finish.
        if (lane == 0 && header_ok && (debug & kDebugDropWeights) == 0) {
            ChunkWalk walk(t0, ntiles, ktiles, blob + kHeaderBytes, kTileBytes);
            // first ring fill, weights only: they are constants, so they may be fetched before the dependency wait
            int cg = 0;
            for (; cg < nstages && !walk.done(); ++cg) {
                int tiles_here, T;
                const uint8_t* src;
                walk.next(kR, tiles_here, T, src);
                stage_tag[cg] = (uint32_t)cg;
                mbar_arrive_expect_tx(full0 + 8 * cg, (uint32_t)tiles_here * kTileBytes);
                bulk_copy_g2s(smem_u32(ring + (size_t)cg * stage_bytes), src, (uint32_t)tiles_here * kTileBytes, full0 + 8 * cg);
            }
            // everything else in ring order
            int s = 0;
            uint32_t parity = 0;
            for (; !walk.done(); ++cg) {
                if (!mbar_wait(empty0 + 8 * s, parity, abort_flag, 0x100 + s)) break;
                int tiles_here, T;
                const uint8_t* src;
                walk.next(kR, tiles_here, T, src);
                const uint32_t dst = smem_u32(ring + (size_t)s * stage_bytes);
                stage_tag[s] = (uint32_t)cg;                 // the stage's previous use is fully consumed by now
                mbar_arrive_expect_tx(full0 + 8 * s, (uint32_t)tiles_here * kTileBytes);
                bulk_copy_g2s(dst, src, (uint32_t)tiles_here * kTileBytes, full0 + 8 * s);
                if (++s == nstages) { s = 0; parity ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ---------------- reducer: one strip segment at a time, behind the consumers ------------------------
        // Lane l owns output elements 4(l + 32e) .. +3 of the [token][64 n] tile (e < kVec), as float4.
        if (header_ok) {
            constexpr int kVec = kTok * kTileN / 128;  // float4 per lane
            int sidx = 0, i = 0;
            bool ok = true;
            grid_dependency_wait();                    // y and the partial sums belong to earlier kernels until now
            while (i < ntiles && ok) {
                const int tile0 = t0 + i;
                const int strip = tile0 / ktiles, T0 = tile0 - strip * ktiles;
                const int seg_len = min(ntiles - i, ktiles - T0);
                const bool whole = seg_len == ktiles;
                const int c_first = range_owner<MT == 2>(strip * ktiles - cbase, ctiles, cn);
                const int c_last = range_owner<MT == 2>(strip * ktiles + ktiles - 1 - cbase, ctiles, cn);
                // Global mode, cut strip: the CTA that holds the strip's first tile finishes it.  Its part of the strip
                // is the tail of its range; for every other contributor the strip is the head of the range, done early.
                const bool finisher = (!CL || csize == 1) && !whole && c_first == crank;

                // While the consumers still work on this segment, collect what the other contributors have dropped
                // (in CTA order; a partial has arrived when none of its words is +0.0, see gather_partials).
                float4 others[kVec];
#pragma unroll
                for (int e = 0; e < kVec; ++e) others[e] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (finisher) {
                    // one partial per trip: with four at once the finisher of a strip shared by four CTAs would wait one
                    // trip instead of three, but the gathering code then needs 64 registers more and the whole step was
                    // slower (measured: 125.7 against 122.6 us), 2 MB shapes gained 0.3 us, 9 MB shapes lost 1 us
                    constexpr int kBatch = 1;
                    const int nothers = c_last - c_first;
                    if (nothers > 1 && nothers <= 4 && (M + 1) / 2 < nothers) {
                        // more contributors than pairs of token rows: row pair by row pair, all contributors at once
                        float4* slot = reinterpret_cast<float4*>(partials + (size_t)(c_first + 1) * (kGemvMaxM * kTileN)) + lane;
                        ok = gather_rows<kVec>(slot, nothers, M, others, abort_flag, 0x450);
                    } else {
                        for (int c = c_first + 1; c <= c_last && ok; c += kBatch) {
                            float4* slot = reinterpret_cast<float4*>(partials + (size_t)c * (kGemvMaxM * kTileN)) + lane;
                            ok = gather_partials<kVec, kBatch>(slot, min(kBatch, c_last - c + 1), M, others, abort_flag, 0x440);
                        }
                    }
                    if (!ok) break;
                }

                // segment sidx goes through buffer sidx % nred, in that buffer's use number sidx / nred
                const int rb = nred == 2 ? (sidx & 1) : 0, ru = nred == 2 ? (sidx >> 1) : sidx;
                ok = mbar_wait(seg_full0 + 8 * rb, ru & 1, abort_flag, 0x400);
                if (!ok) break;
                // sum = partial of warp 0 + warp 1 + ... (fixed order); rows of tokens >= M hold zeros
                float4 sum[kVec];
#pragma unroll
                for (int e = 0; e < kVec; ++e) sum[e] = make_float4(0.f, 0.f, 0.f, 0.f);
                // (the integer path has at most two tokens, one row pair: a quarter of the loads and additions of this
                // loop, which for the last segment of a range is the tail of the kernel; a run-time bound on the row
                // pairs for the other paths made them slower: 36.7 against 35.7 us over the four shapes at 4 tokens)
                // Four warps' loads in flight at a time: this loop is the tail of every CTA (the last segment's sum sits
                // between the last consumer warp and the store), and rolled up it cost the decode step 1.8 us (115.7 ->
                // 113.9; unrolled by 2: 115.3, by 8: 114.7).
                constexpr int kVecUsed = I8 ? 1 : kVec;
#pragma unroll 4
                for (int w = 0; w < nconsumers; ++w) {
                    const float4* src = reinterpret_cast<const float4*>(red + (size_t)(rb * nconsumers + w) * kRedWarp) + lane;
#pragma unroll
                    for (int e = 0; e < kVecUsed; ++e) {
                        const float4 v = src[32 * e];
                        sum[e].x += v.x; sum[e].y += v.y; sum[e].z += v.z; sum[e].w += v.w;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(seg_free0 + 8 * rb);         // consumers may reuse the buffer

                if (whole || finisher) {
                    // fixed order: the other contributors in CTA order, then this CTA
#pragma unroll
                    for (int e = 0; e < kVec; ++e) {
                        sum[e].x += others[e].x; sum[e].y += others[e].y; sum[e].z += others[e].z; sum[e].w += others[e].w;
                    }
                    store_strip<kVec>(y, sum, strip, M, N, lane);
                } else if (CL && csize > 1) {
                    // cluster mode: hand the partial to the CTA that holds the strip's last tile (maybe this one);
                    // it adds the slots up in rank order after the cluster barrier at the end of the kernel
                    const uint32_t remote = map_to_cta(smem_u32(xred + (size_t)crank * xslot_bytes), (uint32_t)c_last);
#pragma unroll
                    for (int e = 0; e < kVec; ++e)
                        if (2 * e < M)
                            asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(remote + (lane + 32 * e) * 16),
                                         "f"(sum[e].x), "f"(sum[e].y), "f"(sum[e].z), "f"(sum[e].w) : "memory");
                    if (c_last == crank) { fin_strip = strip; fin_first = c_first; }
                } else {
                    // Drop this CTA's partial for the finisher and go on: no fence, no counter.  The data says by itself
                    // that it has arrived: the slot is all +0.0 between calls and no word stored here is +0.0.
                    float4* mine = reinterpret_cast<float4*>(partials + (size_t)crank * (kGemvMaxM * kTileN)) + lane;
#pragma unroll
                    for (int e = 0; e < kVec; ++e)
                        if (2 * e < M) __stcg(mine + 32 * e, never_plus_zero(sum[e]));
                }
                i += seg_len;
                ++sidx;
            }
        }
    } else if (header_ok) {
        // ---------------- consumers ---------------------------------------------------------------------------
        const int cw = warp - 2;
        const int g = lane >> 2, t = lane & 3;
        bool aborted = false;

        int i = 0, sidx = 0, chunk_base = 0;
        int cg_cur = 0, s_cur = 0, use_cur = 0;         // this warp's position in the ring (chunks only move forward)
        // This warp's tiles are the local indices cw, cw + nconsumers, ... of the CTA's range, whatever strip they
        // fall into.  The activations of a tile are this lane's own MMA fragments (integer path: its 4 k per token),
        // read straight from global memory.  They are written by earlier kernels of the stream, so nothing is read
        // before the dependency wait; up to 8 tokens the fragments of the NEXT tile are then requested as soon as a
        // k-block of the current tile has used its registers, so their L2 latency runs under the rest of the tile.
        uint2 araw[2];                                  // integer path: token m, k = 128 T + 4 lane .. +3
        constexpr bool kRegActs = !I8 && MT == 1;       // floating-point path up to 8 tokens: fragments in registers
        uint2 ag[1][kRegActs ? 8 : 1];                  // token g: k = 128 T + 16 kb + 4t .. +3
        int T_act = (t0 + cw) % ktiles;                 // k-tile index of this warp's current tile (one division per kernel)
        auto load_araw = [&](const __nv_bfloat16* base) {
#pragma unroll
            for (int m = 0; m < 2; ++m) {
                araw[m] = make_uint2(0u, 0u);
                if (m < M) araw[m] = __ldcg(reinterpret_cast<const uint2*>(base + (size_t)m * K + 4 * lane));
            }
        };
        auto load_ag_kb = [&](const __nv_bfloat16* base, int kb) {
            if (g < M) ag[0][kRegActs ? kb : 0] = __ldcg(reinterpret_cast<const uint2*>(base + (size_t)g * K + 4 * t + 16 * kb));
        };
        constexpr int kColWords = kGemvPieceColWords;
        // Piece table (I8 == 2): local tile j of the range finds its pieces in entry j mod piece_n, piece_n =
        // min(ntiles, ktiles); j < piece_n is the first visit of that k-tile.  ktiles is a multiple of the number of
        // consumer warps, so tiles j and j + ktiles belong to the same warp: no warp reads another warp's entry.
        const int piece_entry_words = (kGemvPieceEntryBytes / 4) * M;
        const int piece_n = min(ntiles, ktiles);
        const int T_first = t0 % ktiles;                // k-tile index of the range's first tile
        int piece_e = cw;                               // entry of this warp's next tile (cw < piece_n whenever it has one)
        if constexpr (kRegActs) {
#pragma unroll
            for (int kb = 0; kb < 8; ++kb) ag[0][kb] = make_uint2(0u, 0u);
        }
        // Up to 8 tokens the fragments are held in registers, one tile ahead.  With 9..16 tokens they would be 32
        // registers live across the whole tile (measured slower), and a tile that asks for them when it begins waits a
        // whole trip to the L2 for its first MMA; there the warp copies the 16 x 128 activations of its NEXT tile into
        // its own shared-memory buffer with cp.async (no registers, from the L2) while it works on the current one, and
        // takes each fragment from there with one 8-byte load.  Rows are 288 bytes apart, so the eight token rows of a
        // fragment load fall into different banks (two wavefronts for 256 bytes, the minimum).
        constexpr bool kAhead = MT == 1;
        constexpr bool kStaged = MT == 2;
        uint8_t* my_abuf = abuf + (size_t)cw * kGemvActWarpBytes;
        auto stage_acts = [&](const __nv_bfloat16* base, int buf) {     // one k-tile of activations, rows < M only
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int chunk = lane + 32 * c, row = chunk >> 4, col = chunk & 15;
                if (row < M) cp_async_16(smem_u32(my_abuf + buf * kGemvActBufBytes + row * kGemvActRowBytes + col * 16), base + (size_t)row * K + col * 8);
            }
            cp_async_commit();
        };
        if constexpr (kStaged) {
            // rows of tokens >= M stay zero in both buffers for the whole kernel
            for (int idx = lane; idx < 2 * 16 * (kGemvActRowBytes / 16); idx += 32) {
                const int row = (idx / (kGemvActRowBytes / 16)) & 15;
                if (row >= M) reinterpret_cast<uint4*>(my_abuf)[idx] = make_uint4(0u, 0u, 0u, 0u);
            }
            __syncwarp();
        }
        // Everything above touches registers and this CTA's shared memory only; from here on the warp reads activations.
        grid_dependency_wait();                         // the activations belong to earlier kernels until now
        if constexpr (kStaged) {
            if (cw < ntiles) stage_acts(a_glob + (size_t)T_act * kTileK, 0);
        }
        int abuf_cur = 0;
        if (kAhead && cw < ntiles) {
            const __nv_bfloat16* base = a_glob + (size_t)T_act * kTileK;
            if constexpr (I8 != 0) load_araw(base);
            else {
#pragma unroll
                for (int kb = 0; kb < 8; ++kb) load_ag_kb(base, kb);
            }
        }
        int T0 = T_first;                               // k-tile index at which the current segment starts (0 after the first)
        int j = cw;                                     // this warp's next tile, as a local index of the CTA's range
        while (i < ntiles && !aborted) {
            const int seg_len = min(ntiles - i, ktiles - T0);
            T0 = 0;

            float acc[4][MT][4];
#pragma unroll
            for (int w = 0; w < 4; ++w)
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[w][mt][e] = 0.f;

            // the warp's tiles come every nconsumers-th tile of the range, whatever segment they fall into
            // Find a tile of this segment in the ring, wait until it has landed and fetch the metadata of its first
            // group.  Called once per tile, in order (the ring position only moves forward).  (Calling it for the next
            // tile already before the current tile's scales are applied, so that the wait would run under the tail of
            // the current tile, was measured slower: 36.9 against 35.8 us over the four shapes at 4 tokens, 53.4 against
            // 52.3 at 16.)
            const uint8_t* nx_tile = nullptr;
            int nx_s = 0, nx_slot = 0, nx_cl = 0;
            uint4 nx_sc = make_uint4(0u, 0u, 0u, 0u);
            uint32_t nx_zw = 0u;
            auto locate_and_wait = [&](int jj) -> bool {
                const int lj = jj - i, cl = lj / kR, slot = lj - cl * kR;
                const int cg = chunk_base + cl;
                s_cur += cg - cg_cur;
                cg_cur = cg;
                while (s_cur >= nstages) { s_cur -= nstages; ++use_cur; }
                const int s = s_cur;
                if (stage_tag[s] != (uint32_t)cg) {            // the producer has not reached this chunk yet
                    const long long t_begin = clock64();
                    while (stage_tag[s] != (uint32_t)cg) {
                        if (*abort_flag != 0) return false;
                        if (wait_expired(t_begin, abort_flag)) { *abort_flag = 0x280 + s; return false; }
                    }
                }
                if (!mbar_wait(full0 + 8 * s, use_cur & 1, abort_flag, 0x200 + s)) return false;
                nx_tile = ring + (size_t)s * stage_bytes + (size_t)slot * kTileBytes;
                nx_s = s; nx_slot = slot; nx_cl = cl;
                if constexpr (!I8) {
                    nx_sc = *(reinterpret_cast<const uint4*>(nx_tile + kWeightBytes) + g);
                    if (BITS == 4) nx_zw = *(reinterpret_cast<const uint32_t*>(nx_tile + w4_zero_offset(G, 0)) + g);
                }
                return true;
            };
            for (; j < i + seg_len; j += nconsumers) {
                if (!locate_and_wait(j)) { aborted = true; break; }
                const uint8_t* tile = nx_tile;
                const int s = nx_s, slot = nx_slot, cl = nx_cl;
                const uint4 sc_first = nx_sc;
                const uint32_t zw_first = nx_zw;
                const bool has_next = kAhead && j + nconsumers < ntiles;
                int T_nx = T_act + nconsumers;                  // the warp's next tile is nconsumers tiles further along K
                while (T_nx >= ktiles) T_nx -= ktiles;
                T_act = T_nx;
                const __nv_bfloat16* next_base = a_glob + (size_t)T_nx * kTileK;
                const uint8_t* acts = my_abuf + abuf_cur * kGemvActBufBytes;       // 9..16 tokens: this tile's activations
                if constexpr (kStaged) {
                    if (j + nconsumers < ntiles) {
                        stage_acts(next_base, abuf_cur ^ 1);     // the next tile's, into the other buffer
                        cp_async_wait<1>();                      // everything but that last group has landed
                    } else {
                        cp_async_wait<0>();
                    }
                    __syncwarp();                                // every lane's copies are visible to the warp
                    abuf_cur ^= 1;
                }

                if constexpr (I8) {
                    const uint4 sc = *(reinterpret_cast<const uint4*>(tile + kWeightBytes) + g);
                    // ---- integer path (1 or 2 tokens): codes x activation pieces on the integer warp MMA ----
                    // The 128 activations of a (token, k-tile) are scaled by 2^(148 - emax) (emax = largest biased
                    // exponent among them), rounded to integers |v| < 2^22 and split into signed bytes
                    // v = p0 + 256 p1 + 65536 p2: values within 2^14 of the largest are exact, smaller ones are rounded
                    // at 2^-22 of it.  Piece j of token m is column 3m + j of the MMA's 8-column operand; the codes are
                    // the other operand as they are (int8), or after two ANDs per packed word (4-bit: the low nibbles of a
                    // word are this lane's row g, the high nibbles, left in place as 16 q, its row g + 8, as unsigned bytes),
                    // so no weight is ever converted to floating point:
                    //     D[n][3m+j] = sum_k q[k][n] p_j[m][k]            (exact, 32-bit integers)
                    //     4-bit: D[n][3m+j] -= z[n] sum_k p_j[m][k]       (the zero point of Eq. 2, still exact)
                    //     y[m][n] += s[n] 2^(emax-148) sum_j 256^j D[n][3m+j]
                    static_assert(!I8 || MT == 1, "the integer path is built for up to 2 tokens");
                    const uint32_t* scr;                                // this tile's piece words and column metadata
                    const uint2* col_meta;
                    if constexpr (I8 == 2) {
                        uint32_t* ent = pscr + piece_e * piece_entry_words;
                        uint2* ent_meta = reinterpret_cast<uint2*>(ent + 3 * kColWords * M);
                        piece_e += nconsumers;                          // the warp's next tile is nconsumers k-tiles further
                        while (piece_e >= piece_n) piece_e -= piece_n;
                        if (j < piece_n) {                              // first visit of this k-tile
                            // (as a call in the whole-SM form with its 96 registers: inlined it spilled inside the tile loop,
                            // 17.8 against 17.1 us on 1x4096x32768; inlined in the half-SM form, where the call was the
                            // slower one, 12.0 against 10.9 us on 1x4096x14336)
                            if constexpr (FULL) make_pieces_call<BITS>(araw, ent, ent_meta, M, lane);
                            else make_pieces<BITS>(araw, ent, ent_meta, M, lane);
                            if (j + nconsumers < piece_n) load_araw(next_base);    // later visits need no activations
                            __syncwarp();
                        }
                        scr = ent;
                        col_meta = ent_meta;
                    } else {
                        uint32_t* mine_scr = pscr + cw * 256;
                        make_pieces<BITS>(araw, mine_scr, reinterpret_cast<uint2*>(mine_scr + 216), M, lane);
                        scr = mine_scr;
                        col_meta = reinterpret_cast<const uint2*>(mine_scr + 216);
                        if (has_next) load_araw(next_base);             // the next tile's activations, under this tile's MMAs
                        __syncwarp();
                    }
                    const uint4 cm = *reinterpret_cast<const uint4*>(col_meta + 2 * t);
                    const float2 col_scale = make_float2(__uint_as_float(cm.x), __uint_as_float(cm.z));
                    uint32_t bw[8];                                     // column g: the words of k-blocks 0..7 for this t
#pragma unroll
                    for (int i = 0; i < 8; ++i) bw[i] = 0u;
                    if (g < 3 * M) {
                        const uint4 lo = *reinterpret_cast<const uint4*>(scr + g * kColWords + t * 8);
                        const uint4 hi = *reinterpret_cast<const uint4*>(scr + g * kColWords + t * 8 + 4);
                        bw[0] = lo.x; bw[1] = lo.y; bw[2] = lo.z; bw[3] = lo.w;
                        bw[4] = hi.x; bw[5] = hi.y; bw[6] = hi.z; bw[7] = hi.w;
                    }
                    if constexpr (I8 == 1) __syncwarp();                // the scratch is rewritten for the next tile
                    int d[4][4];
                    if constexpr (BITS == 4) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {                   // 32 k per MMA: k-blocks 2i and 2i+1, one packed word each
                            const uint4 v0 = *reinterpret_cast<const uint4*>(tile + ((size_t)(2 * i) * 32 + lane) * 16);
                            const uint4 v1 = *reinterpret_cast<const uint4*>(tile + ((size_t)(2 * i + 1) * 32 + lane) * 16);
#pragma unroll
                            for (int w = 0; w < 4; ++w) {
                                const uint32_t x0 = w == 0 ? v0.x : w == 1 ? v0.y : w == 2 ? v0.z : v0.w;
                                const uint32_t x1 = w == 0 ? v1.x : w == 1 ? v1.y : w == 2 ? v1.z : v1.w;
                                // Row g: the low nibbles.  Row g + 8: the high nibbles stay where they are, so the row carries
                                // 16 q (at most 240, still an unsigned byte), its sums come out 16 times too large and its scale
                                // is taken 16 times smaller below (all exact; |16 (q - z) p| summed over 128 k stays below 2^22).
                                // One AND per operand register instead of a shift and an AND: 32 instructions less per tile.
                                const uint32_t a0 = x0 & 0x0F0F0F0Fu, a1 = x0 & 0xF0F0F0F0u;            // k-block 2i
                                const uint32_t a2 = x1 & 0x0F0F0F0Fu, a3 = x1 & 0xF0F0F0F0u;            // k-block 2i + 1
                                if (i == 0) mma_u8s8_16832_first(d[w], a0, a1, a2, a3, bw[0], bw[1], kIntAsFloatBias);
                                else mma_u8s8_16832(d[w], a0, a1, a2, a3, bw[2 * i], bw[2 * i + 1]);
                            }
                        }
                    } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {                       // 32 k per MMA: k-blocks 2i and 2i+1
                        uint4 wv[2][2];
#pragma unroll
                        for (int hb = 0; hb < 2; ++hb)
#pragma unroll
                            for (int h = 0; h < 2; ++h)
                                wv[hb][h] = *reinterpret_cast<const uint4*>(tile + ((size_t)((2 * i + hb) * 2 + h) * 32 + lane) * 16);
#pragma unroll
                        for (int w = 0; w < 4; ++w) {
                            uint32_t a[4];
#pragma unroll
                            for (int hb = 0; hb < 2; ++hb) {
                                const uint4 v = wv[hb][w >> 1];
                                const uint32_t w0 = (w & 1) ? v.z : v.x, w1 = (w & 1) ? v.w : v.y;
                                a[2 * hb] = __byte_perm(w0, w1, 0x5410);         // row g,   k 0..3 of this thread
                                a[2 * hb + 1] = __byte_perm(w0, w1, 0x7632);     // row g+8
                            }
                            if (i == 0) mma_s8_16832_first(d[w], a[0], a[1], a[2], a[3], bw[0], bw[1], kIntAsFloatBias);
                            else mma_s8_16832(d[w], a[0], a[1], a[2], a[3], bw[2 * i], bw[2 * i + 1]);
                        }
                    }
                    }
                    if constexpr (BITS == 4) {
                        // zero point: every code of row n stands for q - z[n], so the row's sum loses z[n] times the column's piece sum
                        const uint32_t zword = *(reinterpret_cast<const uint32_t*>(tile + kWeightBytes + kScaleBytes) + g);
                        const int p0 = (int)cm.y, p1 = (int)cm.w;
#pragma unroll
                        for (int w = 0; w < 4; ++w) {
                            const int zr = (int)((zword >> (4 * w)) & 15u), zr8 = (int)((zword >> (4 * w + 12)) & 0xF0u);     // z, 16 z
                            d[w][0] -= zr * p0; d[w][1] -= zr * p1;
                            d[w][2] -= zr8 * p0; d[w][3] -= zr8 * p1;
                        }
                    }
                    __syncwarp();
                    if (lane == 0) {
                        const int tiles_here = min(kR, seg_len - cl * kR);
                        mbar_arrive_n(empty0 + 8 * s, slot == tiles_here - 1 ? (uint32_t)(kR - tiles_here + 1) : 1u);
                    }
                    const uint32_t sw[4] = {sc.x, sc.y, sc.z, sc.w};
                    // d holds the bits of 1.5 * 2^23 + D: (that - 1.5 * 2^23) * column scale is one exact fused multiply-add
                    const float off_x = -kIntAsFloatBiasValue * col_scale.x, off_y = -kIntAsFloatBiasValue * col_scale.y;
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        const float s_g = fp16_bits_to_float((uint16_t)(sw[w] & 0xFFFFu));
                        const float s_g8 = fp16_bits_to_float((uint16_t)(sw[w] >> 16)) * (BITS == 4 ? 0.0625f : 1.f);     // 4-bit: row g + 8 holds 16 (q - z)
                        acc[w][0][0] = fmaf(fmaf(__int_as_float(d[w][0]), col_scale.x, off_x), s_g, acc[w][0][0]);
                        acc[w][0][1] = fmaf(fmaf(__int_as_float(d[w][1]), col_scale.y, off_y), s_g, acc[w][0][1]);
                        acc[w][0][2] = fmaf(fmaf(__int_as_float(d[w][2]), col_scale.x, off_x), s_g8, acc[w][0][2]);
                        acc[w][0][3] = fmaf(fmaf(__int_as_float(d[w][3]), col_scale.y, off_y), s_g8, acc[w][0][3]);
                    }
                } else {
                // ---- floating-point path: group after group (one group per tile unless the group size is 64 or 32) ----
#pragma unroll
                for (int gr = 0; gr < G; ++gr) {
                    uint4 sc = sc_first;
                    uint32_t zword = zw_first;
                    if (gr > 0) {
                        sc = *(reinterpret_cast<const uint4*>(tile + kWeightBytes + gr * kScaleBytes) + g);
                        if (BITS == 4) zword = *(reinterpret_cast<const uint32_t*>(tile + w4_zero_offset(G, gr)) + g);
                    }
                    uint32_t zg[4], zg8[4];
                    if (BITS == 4) w4_zero_regs(zword, zg, zg8);
                    float gacc[4][MT][4];
#pragma unroll
                    for (int w = 0; w < 4; ++w)
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                            for (int e = 0; e < 4; ++e) gacc[w][mt][e] = 0.f;

#pragma unroll
                    for (int kb = gr * (8 / G); kb < (gr + 1) * (8 / G); ++kb) {
                        uint2 av[MT];                              // token g (+8): k = 16kb + 4t .. +3
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) {
                            if constexpr (kStaged) av[mt] = *reinterpret_cast<const uint2*>(acts + (g + 8 * mt) * kGemvActRowBytes + kb * 32 + t * 8);
                            else av[mt] = ag[0][kRegActs ? kb : 0];
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
                            for (int mt = 0; mt < MT; ++mt)
                                mma_bf16_16816(gacc[w][mt], r0, r1, r2, r3, av[mt].x, av[mt].y);
                        }
                        if (has_next) load_ag_kb(next_base, kb);    // this k-block's registers are free: ask for the next tile's
                    }
                    if (gr == G - 1) {
                        // all shared-memory reads of this tile are done: hand its share of the stage back to the
                        // producer (the last tile of a short chunk also returns the shares of the missing tiles)
                        __syncwarp();
                        if (lane == 0) {
                            const int tiles_here = min(kR, seg_len - cl * kR);
                            mbar_arrive_n(empty0 + 8 * s, slot == tiles_here - 1 ? (uint32_t)(kR - tiles_here + 1) : 1u);
                        }

                    }

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
                if (aborted) break;
                }
            }
            if (aborted) break;

            // ---- drop this warp's partial of the segment for the reducer and move on ---------------------------
            // With two buffers a warp that is a segment ahead of the slowest warp does not wait for it: a segment's
            // partials go to buffer sidx % nred, which the reducer must have read nred segments ago.
            const int rb = nred == 2 ? (sidx & 1) : 0, ru = nred == 2 ? (sidx >> 1) : sidx;
            if (!mbar_wait(seg_free0 + 8 * rb, (ru & 1) ^ 1, abort_flag, 0x300)) { aborted = true; break; }
            float* mine = red + (size_t)(rb * nconsumers + cw) * kRedWarp;      // [token][n]
            if constexpr (I8) {
                // columns 3m .. 3m+2 are the pieces of token m, already on a common scale: add them up across the four
                // threads of a row (fixed order) and leave tokens 0, 1 where the bf16 path has them (t = 0)
#pragma unroll
                for (int w = 0; w < 4; ++w)
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        const float c0 = acc[w][0][2 * r], c1 = acc[w][0][2 * r + 1];
                        float tok0 = t == 0 ? c0 + c1 : t == 1 ? c0 : 0.f;
                        float tok1 = t == 1 ? c1 : t == 2 ? c0 + c1 : 0.f;
                        tok0 += __shfl_xor_sync(0xFFFFFFFFu, tok0, 1);
                        tok1 += __shfl_xor_sync(0xFFFFFFFFu, tok1, 1);
                        tok0 += __shfl_xor_sync(0xFFFFFFFFu, tok0, 2);
                        tok1 += __shfl_xor_sync(0xFFFFFFFFu, tok1, 2);
                        acc[w][0][2 * r] = t == 0 ? tok0 : 0.f;
                        acc[w][0][2 * r + 1] = t == 0 ? tok1 : 0.f;
                    }
            }
#pragma unroll
            for (int w = 0; w < 4; ++w)
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    const int tok = 8 * mt + 2 * t;
                    if (I8 && t != 0) continue;                 // integer path: tokens 0 and 1 sit in the t = 0 threads, the buffer has two rows
                    mine[tok * kTileN + 16 * w + g] = acc[w][mt][0];
                    mine[(tok + 1) * kTileN + 16 * w + g] = acc[w][mt][1];
                    mine[tok * kTileN + 16 * w + g + 8] = acc[w][mt][2];
                    mine[(tok + 1) * kTileN + 16 * w + g + 8] = acc[w][mt][3];
                }
            __syncwarp();
            if (lane == 0) mbar_arrive(seg_full0 + 8 * rb);
            chunk_base += (seg_len + kR - 1) / kR;
            i += seg_len;
            ++sidx;
        }
    }

    // ---------------- cluster mode: finish the strip whose last tile this CTA holds -----------------------------
    __syncthreads();
    if (CL && csize > 1) {
        // Every CTA of the cluster gets here (all waits above are bounded).  After the barrier the partials the
        // other CTAs stored into this CTA's slots are visible, and nobody touches another CTA's memory again.
        cluster_sync_all();
        if (warp == 1 && fin_strip >= 0 && header_ok && *abort_flag == 0) {
            constexpr int kVec = kTok * kTileN / 128;
            float4 tot[kVec];
#pragma unroll
            for (int e = 0; e < kVec; ++e) tot[e] = make_float4(0.f, 0.f, 0.f, 0.f);
            // (a range can be empty only where the cluster has fewer tiles than CTAs: the divisions of
            // range_start stay out of this loop, which is the tail of the kernel, in every other case)
            const bool some_empty = ctiles < cn;
#pragma unroll 2
            for (int c = fin_first; c <= crank; ++c) {                     // rank order, as in global mode
                if (some_empty && range_start<MT == 2>(c + 1, ctiles, cn) == range_start<MT == 2>(c, ctiles, cn)) continue;   // empty range: no partial
                const float4* src = reinterpret_cast<const float4*>(xred + (size_t)c * xslot_bytes) + lane;
#pragma unroll
                for (int e = 0; e < kVec; ++e)
                    if (2 * e < M) {
                        const float4 v = src[32 * e];
                        tot[e].x += v.x; tot[e].y += v.y; tot[e].z += v.z; tot[e].w += v.w;
                    }
            }
            store_strip<kVec>(y, tot, fin_strip, M, N, lane);
        }
    }

    // A CTA without tiles leaves about a microsecond after the dependency is met, not at once.  Measured: when the
    // surplus CTAs of a short GEMV all exit in the instant the previous kernel completes, the kernels behind it
    // on the stream are placed unevenly and a pass over four layer shapes takes 46 us instead of 37; any delay
    // between 1 and 4 us gives the 37 (the CTAs with tiles need 3 us or more from that instant anyway).
    if (idle && threadIdx.x == 0) {
        const long long t_begin = clock64();
        while (clock64() - t_begin < 2000ll) {}
    }

    // ---------------- teardown: report, and never leave with copies in flight ------------------------------
    if (threadIdx.x == 0 && (!header_ok || *abort_flag != 0)) {
        grid_dependency_wait();
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

// How many clusters of `csize` CTAs the device can hold at once, for half-SM CTAs (two per SM) or whole-SM ones
// (asked once per device).  0 if the question fails: cluster mode is then not used.
static int max_resident_clusters(int csize, bool full) {
    static std::atomic<int> cached[kGemvMaxDevices][2][4];   // [device][full][log2 csize], 0 = not asked yet, -1 = failed
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kGemvMaxDevices) return 0;
    const int slot = csize == 2 ? 1 : csize == 4 ? 2 : 3;
    int entry = cached[dev][full ? 1 : 0][slot].load(std::memory_order_relaxed);
    if (entry == 0) {                           // two host threads may both ask: same answer, harmless
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(csize * 64, 1, 1);
        cfg.blockDim = dim3(gemv_max_threads(1, full), 1, 1);
        cfg.dynamicSmemBytes = gemv_smem_budget(1, full);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = csize; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e;
        if (full) {
            e = cudaFuncSetAttribute(gemv_stream_kernel<4, 1, true, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     gemv_smem_budget(1, true));
            if (e == cudaSuccess) e = cudaOccupancyMaxActiveClusters(&n, gemv_stream_kernel<4, 1, true, true, false>, &cfg);
        } else {
            e = cudaFuncSetAttribute(gemv_stream_kernel<4, 1, false, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     gemv_smem_budget(1, false));
            if (e == cudaSuccess) e = cudaOccupancyMaxActiveClusters(&n, gemv_stream_kernel<4, 1, false, true, false>, &cfg);
        }
        if (e != cudaSuccess) { cudaGetLastError(); n = 0; }
        entry = n > 0 ? n : -1;
        cached[dev][full ? 1 : 0][slot].store(entry, std::memory_order_relaxed);
    }
    return entry > 0 ? entry : 0;
}

// Launch geometry.  Global mode: one persistent CTA per SM (fewer when there are fewer tiles than SMs), all tiles
// cut into equal ranges; a strip cut between CTAs is summed through the workspace.  Cluster mode: clusters of 2, 4
// or 8 CTAs, each cluster owning whole strips and cutting its tiles into equal ranges among its CTAs; a cut strip
// is summed through distributed shared memory, which is several microseconds shorter than the workspace hand-over
// (partial to L2, atomic, loads by the last arriver).  A kernel that contains cluster instructions starts about
// 0.7 us later than one that does not, even when launched without clusters, and a cluster launch overlaps less
// with its neighbours on the stream, so cluster mode has instantiations of its own and is taken only for short
// ranges, where the hand-over dominates the call.
GemvPlan plan_gemv(int bits, int M, int K, int N, int sm_count, int groups) {
    GemvPlan p;
    p.groups = groups;
    p.strips = (N + kTileN - 1) / kTileN;
    p.ktiles = K / kTileK;
    p.total_tiles = p.strips * p.ktiles;
    p.grid = p.total_tiles < sm_count ? p.total_tiles : sm_count;
    const int mt = M <= 8 ? 1 : 2;
    int tiles_per_cta = (p.total_tiles + p.grid - 1) / p.grid;
    // CTAs that get tiles.  The grid of a half-SM launch stays at one CTA per SM even when fewer take part: the
    // block scheduler puts the next GEMV's CTAs wherever a half SM is free, and an SM without a CTA of this
    // kernel would get two of them, which then share one SM for their whole range (measured: 2.5 us per call).
    int active = p.grid;
    // Short ranges (at most two rounds of a half-SM CTA's consumer warps): the hand-over of cut strips is most of the
    // call, so pick ranges that line up with the strips.  (a) Few tiles: no more CTAs than give every consumer warp
    // one tile; the call lasts one tile-time either way, and a strip is shared by fewer CTAs.  (b) Otherwise a
    // range length that divides a strip (or is a multiple of it) and needs no more rounds: every CTA then has one
    // cut instead of two.
    if (mt == 1) {
        const int nc = gemv_max_consumers(1, false);
        int want = 0;
        if (tiles_per_cta < nc) {
            want = nc;
        } else if (tiles_per_cta <= 2 * nc) {
            const int rounds = (tiles_per_cta + nc - 1) / nc;
            for (int t = tiles_per_cta; t <= rounds * nc; ++t)
                if ((p.ktiles % t == 0 || t % p.ktiles == 0) && p.total_tiles % t == 0) { want = t; break; }
        }
        if (want > 0) {
            int g = (p.total_tiles + want - 1) / want;
            if (g >= 1 && g < p.grid) { active = g; tiles_per_cta = (p.total_tiles + active - 1) / active; }
        }
    }
    p.cluster = 1;
    p.nclusters = 0;
    int best_t = 0;
    for (int c = 2; c <= 8; c *= 2) {
        // one CTA per SM even where two half-SM ones would fit: the other half is where the next GEMV's CTAs
        // wait with their rings full (measured: filling both halves shortens the call and lengthens the step)
        int maxc = max_resident_clusters(c, mt == 2);
        if (maxc > sm_count / c) maxc = sm_count / c;
        if (maxc < 1) continue;
        const int j = (p.strips + maxc - 1) / maxc;                 // whole strips per cluster, at most
        const int ncl = (p.strips + j - 1) / j;
        const int t = (j * p.ktiles + c - 1) / c;                   // longest range of a CTA
        if (p.cluster == 1 || t < best_t) { p.cluster = c; p.nclusters = ncl; best_t = t; }
    }
    // Worth it for short ranges only (there the hand-over dominates the call), only if the longest range stays
    // within one round of the consumer warps or close to the evenly split one, and only for the whole-SM
    // configuration of 9..16 tokens: a half-SM GEMV overlaps its start with the previous kernel's end, a cluster
    // launch next to a plain one does not (about 2.7 us per transition, measured), and in a pass over layers of
    // different sizes that loss is larger than what the short hand-over wins for up to 8 tokens.
    const int one_round = gemv_max_consumers(mt, mt == 2);
    const bool cluster_ok = mt == 2 && groups == 1;
    if (p.cluster > 1 && cluster_ok && tiles_per_cta <= 16 && (best_t <= one_round || best_t * 10 <= tiles_per_cta * 11 + 20)) {
        p.grid = p.nclusters * p.cluster;
        tiles_per_cta = best_t;
    } else {
        p.cluster = 1;
        p.nclusters = active;
        if (mt == 1 && p.grid < sm_count) p.grid = sm_count;
    }
    // The floating-point path is bound by instruction issue in its consumer warps: it takes the whole SM (12 consumer
    // warps, deeper ring).  The integer path of 1 and 2 tokens needs a fraction of the instructions; its short ranges
    // gain more from the next GEMV's CTAs sitting beside this one's with their rings already full, long ones
    // amortise the start of the kernel and take the whole SM too.
    const bool i8_path = M <= kGemvI8MaxM && groups == 1;     // several groups per tile: floating-point path only
    p.full = mt == 2 || !i8_path || tiles_per_cta * tile_bytes(bits, groups) >= (bits == 8 ? kGemvFullFromBytesI8W8 : kGemvFullFromBytesI8W4);
    p.i8 = i8_path && p.cluster == 1;
    // whole-SM integer path: about 66 KB of tiles in the consumer warps' hands (16 warps on 4-bit tiles, 8 on int8 tiles)
    // and the rest of the ring in flight.  Measured alone, one token: 4096x32768 4-bit 20.7 us half SM, 20.7 / 18.8 /
    // 18.1 whole SM with 8 / 12 / 16 warps; 4096x14336 int8 15.8 us half SM, 12.7 / 13.3 / 14.6 whole SM with 8 / 12 / 16.
    p.consumers = p.i8 && p.full ? gemv_i8_full_consumers(bits) : gemv_max_consumers(mt, p.full);
    if (tiles_per_cta < p.consumers) p.consumers = tiles_per_cta < 4 ? 4 : tiles_per_cta;
    p.threads = 32 * (p.consumers + 2);          // + producer warp + reducer warp
    const int kr = gemv_chunk_tiles(bits);
    // a stage: one bulk copy of kR packed tiles, padded to a multiple of 1 KB
    p.stage_bytes = groups == 1 ? kGemvStageBytes : (kr * tile_bytes(bits, groups) + 1023) / 1024 * 1024;
    // cluster mode: one slot per CTA of the cluster for the rows of real tokens (two token rows = 512 bytes)
    p.xslot_bytes = p.cluster > 1 ? ((M + 1) / 2) * 512 : 0;
    // two buffers for the consumer warps' partial sums where the whole SM is taken (a boundary between strips then
    // costs a fast warp nothing; measured below), one in the half-SM form, where the second would cost a ring stage
    p.nred = p.full ? 2 : 1;
    const int base = 1024 /*alignment slack*/ + kGemvBarrierBytes + p.nred * p.consumers * (p.i8 ? 2 : 8 * mt) * kTileN * 4 +
                     (p.cluster * p.xslot_bytes + 1023) / 1024 * 1024 + (mt == 2 ? p.consumers * kGemvActWarpBytes : 0);
    int fixed = base + (p.i8 ? p.consumers * 1024 : 0);
    int stages = (gemv_smem_budget(mt, p.full) - fixed) / p.stage_bytes;
    if (stages > kGemvMaxStages) stages = kGemvMaxStages;
    // no more stages than the range has chunks
    const int chunks = (tiles_per_cta + kr - 1) / kr + 2;
    if (stages > chunks) stages = chunks;
    // whole-SM integer path: a ring deeper than eight stages was slower (1x4096x32768 4-bit: 17.0 / 16.9 / 17.5 us with
    // 6 / 8 / 10 stages; int8 1x4096x14336: 12.8 / 12.5 / 12.7 us with 6 / 8 / 11)
    if (p.i8 && p.full && stages > kGemvI8FullMaxStages) stages = kGemvI8FullMaxStages;
    // floating-point path up to 8 tokens on 4-bit tiles: five stages (three in the hands of the 12 consumer warps, two in
    // flight).  Measured at 4 tokens with 4 / 5 / 6 / 7 / 9 stages: 4096x14336 12.2 / 11.6 / 11.7 / 11.9 / 12.3 us,
    // 4096x32768 20.9 / 19.8 / 19.9 / 20.1 / 20.5 us; int8 tiles (six stages in the warps' hands) want the deep ring:
    // 4096x14336 19.6 / 18.4 / 17.4 / 16.6 / 16.0 us.  (Why a deeper ring is slower on 4-bit tiles was not established;
    // the consumers, not HBM, set the pace of this path.)
    if (!p.i8 && mt == 1 && bits == 4 && stages > kGemvFpW4MaxStages) stages = kGemvFpW4MaxStages;
    // Integer path: where a range passes over the same k-tiles more than once and K is a multiple of 128 x consumer
    // warps, every warp meets the same k-tiles on each pass and keeps the activation pieces it has prepared (one table
    // entry per k-tile instead of one scratch entry per warp), if that costs the ring no stage.
    p.piece_tab = 0;
    // (4-bit weights only: on int8 tiles, whole SM, the table was the slower form, 13.1 against 12.5 us on 1x4096x14336)
    if (p.i8 && bits == 4 && tiles_per_cta >= p.ktiles + p.consumers && p.ktiles % p.consumers == 0) {
        const int table = (p.ktiles * kGemvPieceEntryBytes * M + 1023) / 1024 * 1024;
        int with = (gemv_smem_budget(mt, p.full) - (base + table)) / p.stage_bytes;
        if (with > kGemvMaxStages) with = kGemvMaxStages;
        if (with > chunks) with = chunks;
        if (with >= stages) {
            p.piece_tab = p.ktiles;
            fixed = base + table;
        }
    }
    p.stages = stages;
    p.smem_bytes = fixed + p.stages * p.stage_bytes;
    return p;
}

// What this library launched last on a stream: whole-SM kernel or half-SM GEMV.  A scheduling hint only (see
// launch_one): a stale, missing or raced entry costs overlap between kernels, never correctness.
namespace {
constexpr int kLaunchNotes = 8;
std::atomic<uintptr_t> g_note_stream[kLaunchNotes];
std::atomic<int> g_note_whole_sm[kLaunchNotes];
std::atomic<unsigned> g_note_next{0};

bool last_launch_was_half_sm(cudaStream_t stream) {
    const uintptr_t key = reinterpret_cast<uintptr_t>(stream) + 1;          // 0 = empty slot
    for (int i = 0; i < kLaunchNotes; ++i)
        if (g_note_stream[i].load(std::memory_order_relaxed) == key) return g_note_whole_sm[i].load(std::memory_order_relaxed) == 0;
    return false;
}
void note_launch(cudaStream_t stream, bool whole_sm) {
    const uintptr_t key = reinterpret_cast<uintptr_t>(stream) + 1;
    for (int i = 0; i < kLaunchNotes; ++i)
        if (g_note_stream[i].load(std::memory_order_relaxed) == key) {
            g_note_whole_sm[i].store(whole_sm ? 1 : 0, std::memory_order_relaxed);
            return;
        }
    const int slot = (int)(g_note_next.fetch_add(1, std::memory_order_relaxed) % kLaunchNotes);
    g_note_whole_sm[slot].store(whole_sm ? 1 : 0, std::memory_order_relaxed);
    g_note_stream[slot].store(key, std::memory_order_relaxed);
}
}  // namespace

void note_whole_sm_launch(cudaStream_t stream) { note_launch(stream, true); }


// Function attributes belong to one device: set once per device and kernel instantiation.  The flag is atomic: two
// host threads may both find it unset and both set the attributes, which is harmless.
template <int BITS, int MT, bool FULL, bool CL, int I8, int G = 1>
static cudaError_t configure_one() {
    static std::atomic<bool> configured_on[kGemvMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
    const bool seen = dev >= 0 && dev < kGemvMaxDevices;
    if (seen && configured_on[dev].load(std::memory_order_acquire)) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(gemv_stream_kernel<BITS, MT, FULL, CL, I8, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         FULL ? gemv_smem_budget(MT, FULL) : kGemvSoloSmemBytes);
    if (e != cudaSuccess) return e;
    // Always the largest shared-memory carve-out: a GEMV whose ring happens to be a little smaller would
    // otherwise ask for a smaller split of the SM's memory, and an SM changes its split only when idle, so
    // consecutive GEMVs of different shapes could not share an SM.
    e = cudaFuncSetAttribute(gemv_stream_kernel<BITS, MT, FULL, CL, I8, G>, cudaFuncAttributePreferredSharedMemoryCarveout,
                             cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    if (seen) configured_on[dev].store(true, std::memory_order_release);
    return cudaSuccess;
}

template <int BITS>
static cudaError_t configure_bits() {
    cudaError_t e = cudaSuccess;
    auto all = [&](cudaError_t r) { if (e == cudaSuccess) e = r; };
    all(configure_one<BITS, 1, false, false, 0>()); all(configure_one<BITS, 1, true, false, 0>());
    all(configure_one<BITS, 1, false, false, 1>());  all(configure_one<BITS, 1, true, false, 1>());
    all(configure_one<BITS, 1, false, false, 2>());  all(configure_one<BITS, 1, true, false, 2>());
    all(configure_one<BITS, 2, true, false, 0>());
    all(configure_one<BITS, 1, false, true, 0>());  all(configure_one<BITS, 1, true, true, 0>());
    all(configure_one<BITS, 2, true, true, 0>());
    if constexpr (BITS == 4) {
        all(configure_one<4, 1, true, false, 0, 2>()); all(configure_one<4, 2, true, false, 0, 2>());
        all(configure_one<4, 1, true, false, 0, 4>()); all(configure_one<4, 2, true, false, 0, 4>());
    }
    return e;
}

// Every one-time step a later launch on the current device could need (function attributes of every instantiation,
// the cluster-occupancy answers), for callers that must not meet them inside a stream capture.
cudaError_t configure_gemv_kernels() {
    cudaError_t e = configure_bits<4>();
    if (e == cudaSuccess) e = configure_bits<8>();
    for (int c = 2; c <= 8; c *= 2) { max_resident_clusters(c, false); max_resident_clusters(c, true); }
    return e;
}

template <int BITS, int MT, bool FULL, bool CL, int I8, int G = 1>
static cudaError_t launch_one(const GemvPlan& p, const void* blob, const void* a, void* y, int M, int K,
                              int N, void* workspace, cudaStream_t stream) {
    cudaError_t ce = configure_one<BITS, MT, FULL, CL, I8, G>();
    if (ce != cudaSuccess) return ce;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.grid, 1, 1);
    cfg.blockDim = dim3(p.threads, 1, 1);
    cfg.dynamicSmemBytes = p.smem_bytes;
    cfg.stream = stream;
    // A whole-SM kernel lets its dependents start as its CTAs leave, one by one.  Every SM freed that way is empty and
    // takes two half-SM CTAs of the next GEMV while other SMs get none: that kernel then runs on half of the SMs, and
    // so does every half-SM GEMV behind it, each on the half the one before left free (measured with %smid: 74 SMs
    // with two CTAs each, 11 us lost per transition, until the next whole-SM kernel).  So a half-SM GEMV that does not
    // follow another half-SM GEMV of this library on its stream asks for a little more than half of an SM's shared
    // memory: two of its CTAs no longer fit on one SM, a CTA of the next (plain) half-SM GEMV still fits beside it.
    if (!FULL && !last_launch_was_half_sm(stream) && cfg.dynamicSmemBytes < (size_t)kGemvSoloSmemBytes)
        cfg.dynamicSmemBytes = kGemvSoloSmemBytes;
    note_launch(stream, FULL);
    // Programmatic dependent launch: a CTA uses less than half of an SM (shared memory, registers), so the
    // CTAs of the next GEMV on the stream become resident while this one still runs, fill their rings with
    // weights and then wait for this kernel to finish before they touch activations, y or the workspace.
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (p.cluster > 1) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = p.cluster; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    return cudaLaunchKernelEx(&cfg, gemv_stream_kernel<BITS, MT, FULL, CL, I8, G>, static_cast<const uint8_t*>(blob),
                              static_cast<const __nv_bfloat16*>(a), static_cast<__nv_bfloat16*>(y), M, K, N, p.ktiles, p.total_tiles, p.stages, p.stage_bytes,
                              p.cluster, p.nclusters, p.xslot_bytes, p.nred, p.piece_tab, static_cast<uint8_t*>(workspace), debug_word());
}

template <int BITS>
static cudaError_t launch_bits(const GemvPlan& p, const void* blob, const void* a, void* y, int M, int K, int N,
                               void* workspace, cudaStream_t stream) {
    if constexpr (BITS == 4) {
        // group sizes 64 and 32: the whole-SM floating-point kernel with two or four groups per tile
        if (p.groups == 2)
            return M > 8 ? launch_one<4, 2, true, false, 0, 2>(p, blob, a, y, M, K, N, workspace, stream)
                         : launch_one<4, 1, true, false, 0, 2>(p, blob, a, y, M, K, N, workspace, stream);
        if (p.groups == 4)
            return M > 8 ? launch_one<4, 2, true, false, 0, 4>(p, blob, a, y, M, K, N, workspace, stream)
                         : launch_one<4, 1, true, false, 0, 4>(p, blob, a, y, M, K, N, workspace, stream);
    }
    if (p.groups != 1) return cudaErrorInvalidValue;
    // the cluster instructions are compiled only into the instantiations that are launched as clusters
    if (p.cluster > 1) {
        if (M > 8) return launch_one<BITS, 2, true, true, 0>(p, blob, a, y, M, K, N, workspace, stream);
        return p.full ? launch_one<BITS, 1, true, true, 0>(p, blob, a, y, M, K, N, workspace, stream)
                      : launch_one<BITS, 1, false, true, 0>(p, blob, a, y, M, K, N, workspace, stream);
    }
    if (M > 8) return launch_one<BITS, 2, true, false, 0>(p, blob, a, y, M, K, N, workspace, stream);
    if (p.i8 && p.piece_tab > 0)
        return p.full ? launch_one<BITS, 1, true, false, 2>(p, blob, a, y, M, K, N, workspace, stream)
                      : launch_one<BITS, 1, false, false, 2>(p, blob, a, y, M, K, N, workspace, stream);
    if (p.i8)
        return p.full ? launch_one<BITS, 1, true, false, 1>(p, blob, a, y, M, K, N, workspace, stream)
                      : launch_one<BITS, 1, false, false, 1>(p, blob, a, y, M, K, N, workspace, stream);
    return p.full ? launch_one<BITS, 1, true, false, 0>(p, blob, a, y, M, K, N, workspace, stream)
                  : launch_one<BITS, 1, false, false, 0>(p, blob, a, y, M, K, N, workspace, stream);
}

cudaError_t launch_gemv(int bits, const GemvPlan& p, const void* blob, const void* a, void* y, int M, int K,
                        int N, void* workspace, cudaStream_t stream) {
    return bits == 4 ? launch_bits<4>(p, blob, a, y, M, K, N, workspace, stream)
                     : launch_bits<8>(p, blob, a, y, M, K, N, workspace, stream);
}

}  // namespace tf
