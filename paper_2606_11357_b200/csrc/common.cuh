// Device helpers shared by the kernels: unpack (Section 4.3 "unpacking"), exact de-bias,
// warp-level MMA, header check.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "../../include/tilefuse.h"
#include "layout.h"

namespace tf {

// Device status word layout at the start of a workspace.
struct DeviceStatus {
    uint32_t code;      // tf_status
    uint32_t detail;    // where a bounded wait gave up / which header field mismatched
    uint32_t pad[2];
};

// ---- 4-bit codes -> bf16 --------------------------------------------------------------
// bf16 0x4300 is 128.0 with a unit in the last place of 1, so OR-ing a 4-bit code into the
// mantissa gives exactly 128 + q.  Register i of a packed word sits in nibbles i and i+4.
// Written as one three-input logic op (a & b) | c with mask and magic held in registers; left to
// the compiler it becomes two two-input ops because each may carry only one immediate.
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t w4_reg_biased(uint32_t word, int i) {
    uint32_t mask, magic;
    asm("mov.b32 %0, 0x000F000F;" : "=r"(mask));      // opaque to constant folding on purpose
    asm("mov.b32 %0, 0x43004300;" : "=r"(magic));
    return and_or(word >> (4 * i), mask, magic);
}

__device__ __forceinline__ uint32_t bf16x2_sub(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t bf16x2_mul(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// The 8 zero points of a lane: pair i = (128 + z[16i+g], 128 + z[16i+g+8]) as bf16x2, then
// each half duplicated so it can be subtracted from a (k, k+1) register of that row.
__device__ __forceinline__ void w4_zero_regs(uint32_t zword, uint32_t zrow_g[4], uint32_t zrow_g8[4]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t pair = w4_reg_biased(zword, i);
        zrow_g[i] = __byte_perm(pair, 0, 0x1010);
        zrow_g8[i] = __byte_perm(pair, 0, 0x3232);
    }
}

// ---- int8 -> bf16 ---------------------------------------------------------------------
// Four int8 in a word -> two bf16x2 registers (bytes 0,1 and bytes 2,3), exactly:
// offset-binary byte placed in the mantissa of 2^23, minus (2^23 + 128); the upper halves of
// the fp32 results are the bf16 values (|q| <= 128 needs 8 significant bits).
__device__ __forceinline__ void w8_word_to_regs(uint32_t word, uint32_t& lo, uint32_t& hi) {
    const uint32_t u = word ^ 0x80808080u;
    const float bias = 8388736.0f;   // 2^23 + 128
    float f0 = __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7440)) - bias;
    float f1 = __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7441)) - bias;
    float f2 = __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7442)) - bias;
    float f3 = __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7443)) - bias;
    lo = __byte_perm(__float_as_uint(f0), __float_as_uint(f1), 0x7632);
    hi = __byte_perm(__float_as_uint(f2), __float_as_uint(f3), 0x7632);
}

// ---- warp MMA: D(16x8, fp32) += A(16x16, bf16) . B(16x8, bf16) ---------------------------
__device__ __forceinline__ void mma_bf16_16816(float d[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Header fields every kernel compares with its arguments (first 24 bytes of the blob).
__device__ __forceinline__ bool header_matches(const void* blob, uint32_t bits, uint32_t K, uint32_t N) {
    const uint4 h = __ldg(reinterpret_cast<const uint4*>(blob));            // magic, version, bits, K
    const uint2 h2 = __ldg(reinterpret_cast<const uint2*>(blob) + 2);       // N, group_size
    return h.x == kMagic && h.y == kBlobVersion && h.z == bits && h.w == K && h2.x == N;
}

// The group size recorded in the header, and whether it fits a kernel built for G groups per tile (G = 1: any
// multiple of the tile's k-extent; G = 2, 4: exactly 128 / G).
__device__ __forceinline__ uint32_t header_group_size(const void* blob) {
    return __ldg(reinterpret_cast<const uint32_t*>(blob) + 5);
}
__device__ __forceinline__ bool group_size_fits(const void* blob, int G) {
    const uint32_t gs = header_group_size(blob);
    return G == 1 ? (gs >= (uint32_t)kTileK && gs % kTileK == 0) : gs == (uint32_t)(kTileK / G);
}

__device__ __forceinline__ float fp16_bits_to_float(uint16_t h) {
    return __half2float(__ushort_as_half(h));
}

}  // namespace tf
