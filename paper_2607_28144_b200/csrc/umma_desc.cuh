// Encoders for the two descriptors a tcgen05.mma (kind::f16) takes.
#pragma once
#include <stdint.h>

namespace regenvc {

// 32-bit instruction descriptor, dense kind::f16:
//   [4,6)  accumulator format (1 = fp32)      [7,10)  A format (0 = fp16, 1 = bf16)
//   [10,13) B format                           [15]/[16] A/B major (0 = K-major)
//   [17,23) N >> 3                             [24,29) M >> 4
__host__ __device__ constexpr uint32_t umma_idesc_f16_f32acc(int m, int n) {
    return (1u << 4) | (0u << 7) | (0u << 10) | (0u << 15) | (0u << 16) |
           (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}

// The same with both operands bf16 (format code 1 in the A and B fields).
__host__ __device__ constexpr uint32_t umma_idesc_bf16_f32acc(int m, int n) {
    return umma_idesc_f16_f32acc(m, n) | (1u << 7) | (1u << 10);
}

// 64-bit shared-memory matrix descriptor for a K-major operand stored as
// rows of 128 bytes (64 16-bit elements) with the 128-byte swizzle, eight
// rows per 1024-byte group (the layout a TMA box of {64, rows} with
// SWIZZLE_128B produces; the tile base must be 1024-byte aligned):
//   [0,14)  start address >> 4     [16,30) leading-dim byte offset >> 4 (unused here: K extent
//   [32,46) stride-dim byte offset >> 4 (1024 B between 8-row groups)    of one MMA stays in a row)
//   [46,49) constant 0b001         [61,64) swizzle mode (2 = 128 B)
// Advancing K by 16 elements inside the 128-byte row = +32 bytes on the start address.
__host__ __device__ constexpr uint64_t umma_smem_desc_k_sw128(uint32_t smem_byte_addr) {
    return static_cast<uint64_t>((smem_byte_addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(1) << 16) |
           (static_cast<uint64_t>(1024 >> 4) << 32) | (static_cast<uint64_t>(1) << 46) |
           (static_cast<uint64_t>(2) << 61);
}

// Byte offset of 16-byte chunk `chunk16` (0..7) of row `row` inside one
// [rows][64 x 16-bit] swizzled block: the chunk index is XORed with row % 8.
__host__ __device__ constexpr uint32_t sw128_offset(int row, int chunk16) {
    return static_cast<uint32_t>(row) * 128u + (static_cast<uint32_t>(chunk16 ^ (row & 7)) << 4);
}

}  // namespace regenvc
