// Key/value preparation pass: one read of K and V, one write of the two
// tensor-core operand tensors the attention kernel streams through TMA.
//   K' [h][n_kv_pad][128] fp16 : keys, rotated by the 3D rotary embedding
//                                (self-attention) or just converted (cross)
//   V't [h][128][n_kv_pad] fp16: values transposed so that keys are the
//                                contiguous (K-major) dimension of P.V
// Rotating K here, once per key, replaces rotating every K tile again in each
// of the ~N/128 query-tile CTAs that stream it.  HBM-bound: 2 x 256 B read and
// 2 x 256 B written per (token, head).
#include "common.cuh"
#include "rope.cuh"

namespace regenvc {

constexpr int kPrepThreads = 256;
constexpr int kVtStride = 65;  // words per d-row of the transpose tile (64 token pairs + 1 pad)

__global__ void __launch_bounds__(kPrepThreads) prep_kv_kernel(PrepParams p) {
    const int tid = threadIdx.x;
    const int tile0 = blockIdx.x * kTile;
    const int head = blockIdx.y;

    if (blockIdx.z == 0) {
        // ---- K: 16 threads per row (16 B = 8 elements = 4 rotary pairs each)
        const int chunk = tid & 15;
        bool out_of_range = false;
#pragma unroll 2
        for (int it = 0; it < kTile / 16; ++it) {
            const int n = tile0 + it * 16 + (tid >> 4);
            uint4 packed = make_uint4(0, 0, 0, 0);
            if (n < p.n_kv) {
                const uint4 raw =
                    __ldg(reinterpret_cast<const uint4*>(p.k + ((size_t)n * p.h + head) * kHeadDim) + chunk);
                float x[8];
                bf16x8_to_float(raw, x);
                if (p.rope) rope_rotate8(x, p.grid, token_pos(n, p.grid), chunk);
                __half2 h0 = __floats2half2_rn(x[0], x[1]);
                __half2 h1 = __floats2half2_rn(x[2], x[3]);
                __half2 h2 = __floats2half2_rn(x[4], x[5]);
                __half2 h3 = __floats2half2_rn(x[6], x[7]);
#pragma unroll
                for (int i = 0; i < 8; ++i) out_of_range |= !(fabsf(x[i]) <= 65504.0f);
                packed.x = *reinterpret_cast<uint32_t*>(&h0);
                packed.y = *reinterpret_cast<uint32_t*>(&h1);
                packed.z = *reinterpret_cast<uint32_t*>(&h2);
                packed.w = *reinterpret_cast<uint32_t*>(&h3);
            }
            reinterpret_cast<uint4*>(p.kp + ((size_t)head * p.n_kv_pad + n) * kHeadDim)[chunk] = packed;
        }
        if (out_of_range) atomicCAS(p.status, 0, kStatusRange);
    } else {
        // ---- V: transpose a [128 tokens][128 d] tile through shared memory.
        // tile[d][tp] holds the fp16 pair (token 2*tp, token 2*tp+1) of column d.
        __shared__ uint32_t tile[kHeadDim * kVtStride];
        const int warp = tid >> 5, lane = tid & 31;
        bool out_of_range = false;
        for (int it = 0; it < 8; ++it) {
            const int tp = warp * 8 + it;
            const int n0 = tile0 + 2 * tp;
#pragma unroll
            for (int half_row = 0; half_row < 2; ++half_row) {
                const int d = half_row * 64 + 2 * lane;
                uint32_t a = 0, b = 0;  // (v[n0][d], v[n0][d+1]) and the same for n0+1, as bf16 pairs
                if (n0 < p.n_kv)
                    a = __ldg(reinterpret_cast<const uint32_t*>(p.v + ((size_t)n0 * p.h + head) * kHeadDim + d));
                if (n0 + 1 < p.n_kv)
                    b = __ldg(reinterpret_cast<const uint32_t*>(p.v + ((size_t)(n0 + 1) * p.h + head) * kHeadDim + d));
                const float a0 = __uint_as_float(a << 16), a1 = __uint_as_float(a & 0xffff0000u);
                const float b0 = __uint_as_float(b << 16), b1 = __uint_as_float(b & 0xffff0000u);
                out_of_range |= !(fabsf(a0) <= 65504.0f) | !(fabsf(a1) <= 65504.0f) | !(fabsf(b0) <= 65504.0f) |
                                !(fabsf(b1) <= 65504.0f);
                __half2 c0 = __floats2half2_rn(a0, b0);  // column d:   tokens n0, n0+1
                __half2 c1 = __floats2half2_rn(a1, b1);  // column d+1
                tile[d * kVtStride + tp] = *reinterpret_cast<uint32_t*>(&c0);
                tile[(d + 1) * kVtStride + tp] = *reinterpret_cast<uint32_t*>(&c1);
            }
        }
        if (out_of_range) atomicCAS(p.status, 0, kStatusRange);
        __syncthreads();
        uint32_t* dst = reinterpret_cast<uint32_t*>(p.vt + (size_t)head * kHeadDim * p.n_kv_pad + tile0);
        const size_t row_words = (size_t)p.n_kv_pad / 2;
        for (int it = 0; it < kHeadDim / 8; ++it) {
            const int d = it * 8 + warp;
            dst[d * row_words + lane] = tile[d * kVtStride + lane];
            dst[d * row_words + 32 + lane] = tile[d * kVtStride + 32 + lane];
        }
    }
}

cudaError_t launch_prep_kv(const PrepParams& p, cudaStream_t stream) {
    dim3 grid(p.n_kv_pad / kTile, p.h, 2);
    prep_kv_kernel<<<grid, kPrepThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace regenvc
