// Tile layout of the packed blob, shared by the host packer and the device kernels.
//
// A tile covers TF_TILE_K = 128 rows (k) x TF_TILE_N = 64 columns (n).  Its weights are stored
// in the register order of the warp-level tensor-core operand "A" of shape 16 (n) x 16 (k):
// lane L = (g << 2) | t  (g = 0..7, t = 0..3) owns, per 16x16 block, four bf16x2 registers
//     r0 = (row g,   k 4t, 4t+1)      r1 = (row g+8, k 4t, 4t+1)
//     r2 = (row g,   k 4t+2, 4t+3)    r3 = (row g+8, k 4t+2, 4t+3)
// A tile has 8 k-blocks (kb, 16 k each) x 4 n-blocks (w, 16 n each):
//     k = k0 + 16*kb + 4*t + {0,1 (r0/r1 lo,hi), 2,3 (r2/r3 lo,hi)}
//     n = n0 + 16*w + g + 8*(register is r1 or r3)
// (The warp-level MMA numbers its k-slots 2t,2t+1,2t+8,2t+9; the contraction index may be permuted
// freely as long as weights and activations agree, and this choice gives every lane four consecutive
// k -- one 8-byte activation load -- and is also the register order of the 16x256b tensor-memory
// store, so the GEMM can move a word straight into the TMEM operand of tcgen05.mma.)
//
// W4: one uint32 per (kb, lane, w) at word index (kb*32 + lane)*4 + w; nibble p holds register
//     (p & 3), element (p >> 2)  -- so  (x >> 4*i) & 0x000F000F  is register i as two integers.
// W8: two uint32 per (kb, lane, w): 16-byte vector (kb*2 + (w>>1))*32 + lane, words 2*(w&1)+r;
//     byte b of word r holds register 2r + (b>>1), element (b & 1).
// Scales: fp16 [g][2w+h] for column n0 + 16w + g + 8h  (one 16-byte vector per g).
// Zeros (W4): uint32 [g]; nibble i (0..3) = column n0 + 16i + g, nibble i+4 = column n0+16i+g+8.
// Group sizes below the tile's k-extent (W4 only: 64 or 32) put G = 128 / group_size groups into a tile: the
// tile then carries G scale blocks followed by G zero blocks, group after group along k, and is 160 (G - 1) bytes
// longer (4416 bytes for group size 64, 4736 for 32).
#pragma once
#include <stdint.h>

namespace tf {

constexpr int kTileK = 128;
constexpr int kTileN = 64;
constexpr int kHeaderBytes = 256;
constexpr uint32_t kMagic = 0x31424654u;   // "TFB1"
constexpr uint32_t kBlobVersion = 1;

constexpr int kW4WeightBytes = 4096;
constexpr int kW8WeightBytes = 8192;
constexpr int kScaleBytes = 128;
constexpr int kZeroBytes = 32;
constexpr int kW4TileBytes = kW4WeightBytes + kScaleBytes + kZeroBytes;   // 4256
constexpr int kW8TileBytes = kW8WeightBytes + kScaleBytes;                // 8320

// Groups per tile for a legal group size (a multiple of 128 that divides K: one; 64: two; 32: four).
#ifdef __CUDACC__
#define TF_HD __host__ __device__
#else
#define TF_HD
#endif
TF_HD constexpr int groups_per_tile(int group_size) { return group_size >= kTileK ? 1 : kTileK / group_size; }
// W4 tile with G groups: weights | G scale blocks | G zero blocks.
TF_HD constexpr int w4_tile_bytes(int G) { return kW4WeightBytes + G * (kScaleBytes + kZeroBytes); }
TF_HD constexpr int w4_scale_offset(int gr) { return kW4WeightBytes + gr * kScaleBytes; }
TF_HD constexpr int w4_zero_offset(int G, int gr) { return kW4WeightBytes + G * kScaleBytes + gr * kZeroBytes; }
TF_HD constexpr int tile_bytes(int bits, int G) { return bits == 4 ? w4_tile_bytes(G) : kW8TileBytes; }

}  // namespace tf
