// Query-tile staging shared by the attention kernels.
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include "rope.cuh"
#include "umma_desc.cuh"

namespace regenvc {

constexpr uint32_t kTileBytes = kTile * kHeadDim * 2;  // 32 KB: one 128 x 128 16-bit tile
constexpr uint32_t kBlockBytes = kTileBytes / 2;       // 16 KB: one [128][64] swizzled block

// Loads a 128-row query tile, applies the rotary embedding and writes it to
// shared memory as two swizzled K-major blocks (d 0..63, d 64..127).
// Rows >= n_q are zero.  `nthreads` threads cooperate (multiple of 16).
__device__ __forceinline__ void load_rotate_q_tile(const AttnParams& p, int head, int q0, uint8_t* sQ, int tid,
                                                   int nthreads) {
    const int chunk = tid & 15;
    for (int row = tid >> 4; row < kTile; row += nthreads >> 4) {
        const int n = q0 + row;
        uint4 packed = make_uint4(0, 0, 0, 0);
        if (n < p.n_q) {
            const uint4 raw = __ldg(reinterpret_cast<const uint4*>(p.q + ((size_t)n * p.h + head) * kHeadDim) + chunk);
            float x[8];
            bf16x8_to_float(raw, x);
            if (p.rope) rope_rotate8(x, p.grid, token_pos(n, p.grid), chunk);
            packed.x = pack_f16x2(x[0], x[1]);
            packed.y = pack_f16x2(x[2], x[3]);
            packed.z = pack_f16x2(x[4], x[5]);
            packed.w = pack_f16x2(x[6], x[7]);
        }
        *reinterpret_cast<uint4*>(sQ + (chunk >> 3) * kBlockBytes + sw128_offset(row, chunk & 7)) = packed;
    }
}


}  // namespace regenvc
