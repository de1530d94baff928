// Device-side lookup of the rotary angle table and the pair rotation.
#pragma once
#include "common.cuh"

namespace regenvc {

struct TokenPos {
    int t, y, x;
};

__device__ __forceinline__ TokenPos token_pos(int n, const RopeGrid& g) {
    TokenPos p;
    int hw = g.H * g.W;
    p.t = n / hw;
    int rem = n - p.t * hw;
    p.y = rem / g.W;
    p.x = rem - p.y * g.W;
    return p;
}

// Where the (cos, sin) entries of the four rotary pairs of one 16-byte chunk (pairs 4 * chunk ..) sit in the
// table: entry = position on axis `axis` * mult + off.  Depends on the chunk only, so a thread that keeps its
// chunk computes it once.
struct RopeChunk {
    int axis[4], mult[4], off[4];
};
__device__ __forceinline__ RopeChunk rope_chunk(const RopeGrid& g, int chunk) {
    RopeChunk rc;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int j = chunk * 4 + i;
        if (j < kPairsT) {
            rc.axis[i] = 0, rc.mult[i] = kPairsT, rc.off[i] = j;
        } else if (j < kPairsT + kPairsY) {
            rc.axis[i] = 1, rc.mult[i] = kPairsY, rc.off[i] = g.T * kPairsT + (j - kPairsT);
        } else {
            rc.axis[i] = 2, rc.mult[i] = kPairsX, rc.off[i] = g.T * kPairsT + g.H * kPairsY + (j - kPairsT - kPairsY);
        }
    }
    return rc;
}

// Rotates the 4 adjacent pairs held in 8 floats (elements 8*chunk .. 8*chunk+7 of the head vector).
__device__ __forceinline__ void rope_rotate8(float* x, const RopeGrid& g, const TokenPos& p, const RopeChunk& rc) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int pos = rc.axis[i] == 0 ? p.t : (rc.axis[i] == 1 ? p.y : p.x);
        const float2 cs = __ldg(g.tab + pos * rc.mult[i] + rc.off[i]);
        float a = x[2 * i], b = x[2 * i + 1];
        x[2 * i] = a * cs.x - b * cs.y;
        x[2 * i + 1] = a * cs.y + b * cs.x;
    }
}

__device__ __forceinline__ void bf16x8_to_float(const uint4& raw, float* x) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

}  // namespace regenvc
