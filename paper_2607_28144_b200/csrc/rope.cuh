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

// (cos, sin) of pair j (0..63) for a token at position p.
__device__ __forceinline__ float2 rope_cs(const RopeGrid& g, const TokenPos& p, int j) {
    int idx;
    if (j < kPairsT) {
        idx = p.t * kPairsT + j;
    } else if (j < kPairsT + kPairsY) {
        idx = g.T * kPairsT + p.y * kPairsY + (j - kPairsT);
    } else {
        idx = g.T * kPairsT + g.H * kPairsY + p.x * kPairsX + (j - kPairsT - kPairsY);
    }
    return __ldg(g.tab + idx);
}

// Rotates the 4 adjacent pairs held in 8 floats (elements 8*chunk .. 8*chunk+7 of the head vector).
__device__ __forceinline__ void rope_rotate8(float* x, const RopeGrid& g, const TokenPos& p, int chunk) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 cs = rope_cs(g, p, chunk * 4 + i);
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
