// Query-tile staging shared by the attention kernels.
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include "rope.cuh"
#include "umma_desc.cuh"

namespace regenvc {

constexpr uint32_t kTileBytes = kTile * kHeadDim * 2;  // 32 KB: one 128 x 128 16-bit tile
constexpr uint32_t kBlockBytes = kTileBytes / 2;       // 16 KB: one [128][64] swizzled block

// Loads kTilesQ consecutive 128-row query tiles (rows q0 ..), applies the rotary embedding and writes each to
// shared memory (sQ + tile * 32 KB) as two swizzled K-major fp16 blocks (d 0..63, d 64..127).  Rows >= n_q are
// zero.  kThreadsN threads cooperate; every thread first issues all of its 16-byte global loads, then rotates
// and stores, so that the loads overlap.
template <int kThreadsN, int kTilesQ>
__device__ __forceinline__ void load_rotate_q_tiles(const AttnParams& p, int head, int q0, uint8_t* sQ, int tid) {
    static_assert(kThreadsN % 16 == 0 && (kTile * 16) % kThreadsN == 0, "thread count must tile the rows");
    constexpr int kRowsPerPass = kThreadsN / 16;
    constexpr int kPasses = kTile / kRowsPerPass;
    const int chunk = tid & 15;
    const RopeChunk rc = rope_chunk(p.grid, chunk);
    uint4 raw[kTilesQ][kPasses];
#pragma unroll
    for (int t = 0; t < kTilesQ; ++t)
#pragma unroll
        for (int it = 0; it < kPasses; ++it) {
            const int n = q0 + t * kTile + it * kRowsPerPass + (tid >> 4);
            raw[t][it] = make_uint4(0, 0, 0, 0);
            if (n < p.n_q)
                raw[t][it] = __ldg(reinterpret_cast<const uint4*>(p.q + ((size_t)n * p.h + head) * kHeadDim) + chunk);
        }
    // Grid position of this thread's first row by division, of its later rows (kRowsPerPass tokens further each) by
    // stepping: the two integer divisions per row were the largest part of this routine's instructions.
    TokenPos pos = {0, 0, 0};
    if (p.rope) pos = token_pos(q0 + (tid >> 4) + p.q_pos_offset, p.grid);
#pragma unroll
    for (int t = 0; t < kTilesQ; ++t)
#pragma unroll
        for (int it = 0; it < kPasses; ++it) {
            const int row = it * kRowsPerPass + (tid >> 4);
            const int n = q0 + t * kTile + row;
            float x[8];
            bf16x8_to_float(raw[t][it], x);
            if (p.rope) {
                if (n < p.n_q) rope_rotate8(x, p.grid, pos, rc);
                pos.x += kRowsPerPass;   // the next row of this thread
                while (pos.x >= p.grid.W) {
                    pos.x -= p.grid.W;
                    if (++pos.y == p.grid.H) {
                        pos.y = 0;
                        ++pos.t;
                    }
                }
            }
            uint4 packed;
            packed.x = pack_f16x2(x[0], x[1]);
            packed.y = pack_f16x2(x[2], x[3]);
            packed.z = pack_f16x2(x[4], x[5]);
            packed.w = pack_f16x2(x[6], x[7]);
            *reinterpret_cast<uint4*>(sQ + t * kTileBytes + (chunk >> 3) * kBlockBytes + sw128_offset(row, chunk & 7)) = packed;
        }
}

// The same for ONE tile by a few threads with few registers (two warps that prepare the next work item's query tile
// while the others work on the current one): the rows of a thread are taken in batches of kBatch, every batch's loads
// issued together.
template <int kThreadsN, int kBatch>
__device__ __forceinline__ void load_rotate_q_tile_batched(const AttnParams& p, int head, int q0, uint8_t* sQ, int tid) {
    static_assert(kThreadsN % 16 == 0 && (kTile * 16) % kThreadsN == 0, "thread count must tile the rows");
    constexpr int kRowsPerPass = kThreadsN / 16;
    constexpr int kPasses = kTile / kRowsPerPass;
    static_assert(kPasses % kBatch == 0, "batches must tile the passes");
    const int chunk = tid & 15;
    const RopeChunk rc = rope_chunk(p.grid, chunk);
    TokenPos pos = {0, 0, 0};
    if (p.rope) pos = token_pos(q0 + (tid >> 4) + p.q_pos_offset, p.grid);
#pragma unroll 1
    for (int it0 = 0; it0 < kPasses; it0 += kBatch) {
        uint4 raw[kBatch];
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            const int n = q0 + (it0 + b) * kRowsPerPass + (tid >> 4);
            raw[b] = make_uint4(0, 0, 0, 0);
            if (n < p.n_q)
                raw[b] = __ldg(reinterpret_cast<const uint4*>(p.q + ((size_t)n * p.h + head) * kHeadDim) + chunk);
        }
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            const int row = (it0 + b) * kRowsPerPass + (tid >> 4);
            float x[8];
            bf16x8_to_float(raw[b], x);
            if (p.rope) {
                if (q0 + row < p.n_q) rope_rotate8(x, p.grid, pos, rc);
                pos.x += kRowsPerPass;
                while (pos.x >= p.grid.W) {
                    pos.x -= p.grid.W;
                    if (++pos.y == p.grid.H) {
                        pos.y = 0;
                        ++pos.t;
                    }
                }
            }
            uint4 packed;
            packed.x = pack_f16x2(x[0], x[1]);
            packed.y = pack_f16x2(x[2], x[3]);
            packed.z = pack_f16x2(x[4], x[5]);
            packed.w = pack_f16x2(x[6], x[7]);
            *reinterpret_cast<uint4*>(sQ + (chunk >> 3) * kBlockBytes + sw128_offset(row, chunk & 7)) = packed;
        }
    }
}

}  // namespace regenvc
