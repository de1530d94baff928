// Key/value preparation pass: one read of K and V, one write of the two
// tensor-core operand tensors the attention kernel streams through TMA.
//   K' [h][n_kv_pad][128] fp16 : keys, rotated by the 3D rotary embedding
//                                (self-attention) or just converted (cross);
//                                with k_bf16 set the bf16 bits are kept as they are
//   V't [h][128][n_kv_pad] fp16: values transposed so that keys are the
//                                contiguous (K-major) dimension of P.V
// Rotating K here, once per key, replaces rotating every K tile again in each
// of the ~N/128 query-tile CTAs that stream it.  HBM-bound: 2 x 256 B read and
// 2 x 256 B written per (token, head).
#include "common.cuh"
#include "ptx.cuh"
#include "rope.cuh"

namespace regenvc {

constexpr int kPrepThreads = 256;

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

__global__ void __launch_bounds__(kPrepThreads, 4) prep_kv_kernel(PrepParams p) {
    const int tid = threadIdx.x;
    const int tile0 = blockIdx.x * kTile;
    const int head = blockIdx.y;

    if (blockIdx.z == 0) {
        // ---- K: 16 threads per row (16 B = 8 elements = 4 rotary pairs each); all loads first
        const int chunk = tid & 15;
        float amax = 0.f;  // largest magnitude this thread writes (for the fp16 range check)
        __shared__ TokenPos s_pos[kTile];  // grid position of every row of the tile: one division pair per row
        uint4 raw[kTile / 16];
#pragma unroll
        for (int it = 0; it < kTile / 16; ++it) {
            const int n = tile0 + it * 16 + (tid >> 4);
            raw[it] = make_uint4(0, 0, 0, 0);
            if (n < p.n_kv)
                raw[it] = __ldg(reinterpret_cast<const uint4*>(p.k + ((size_t)n * p.h + head) * kHeadDim) + chunk);
        }
        RopeChunk rc;
        if (p.rope) {  // uniform over the grid
            rc = rope_chunk(p.grid, chunk);
            if (tid < kTile) s_pos[tid] = token_pos(tile0 + tid + p.pos_offset, p.grid);
            __syncthreads();
        }
#pragma unroll
        for (int it = 0; it < kTile / 16; ++it) {
            const int row = it * 16 + (tid >> 4);
            const int n = tile0 + row;
            if (p.k_bf16) {  // uniform over the grid: the keys stay bf16 (cross-attention with bf16 queries)
                reinterpret_cast<uint4*>(p.kp + ((size_t)head * p.n_kv_pad + n) * kHeadDim)[chunk] = raw[it];
                continue;
            }
            float x[8];
            bf16x8_to_float(raw[it], x);
            if (p.rope && n < p.n_kv) rope_rotate8(x, p.grid, s_pos[row], rc);
#pragma unroll
            for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(x[i]));
            uint4 packed;
            packed.x = pack_f16x2(x[0], x[1]);
            packed.y = pack_f16x2(x[2], x[3]);
            packed.z = pack_f16x2(x[4], x[5]);
            packed.w = pack_f16x2(x[6], x[7]);
            reinterpret_cast<uint4*>(p.kp + ((size_t)head * p.n_kv_pad + n) * kHeadDim)[chunk] = packed;
        }
        if (!(amax <= 65504.0f)) atomicCAS(p.status, 0, kStatusRange);
    } else {
        // ---- V: transpose a [128 tokens][128 d] tile through shared memory.
        // tile[d][tp ^ swz(d)] holds the fp16 pair (token 2*tp, token 2*tp+1) of column d; swz(d) = (d / 4) % 32
        // makes both the column-wise writes below and the row-wise reads conflict-free.
        __shared__ uint32_t tile[kHeadDim * 64];
        const int warp = tid >> 5, lane = tid & 31;
        const int tb = lane >> 4, c = lane & 15;  // token of the pair, 8-column chunk
        // |v| <= 65504 on the bf16 bit patterns: the largest bf16 not above 65504 is 0x477F (65280), so a 15-bit
        // magnitude above it (Inf and NaN included) is out of range; checked two values per word with a running maximum
        uint32_t mag_max = 0;
        uint4 raw[8];
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int n = tile0 + 2 * (warp * 8 + it) + tb;
            raw[it] = make_uint4(0, 0, 0, 0);
            if (n < p.n_kv)
                raw[it] = __ldg(reinterpret_cast<const uint4*>(p.v + ((size_t)n * p.h + head) * kHeadDim) + c);
        }
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int tp = warp * 8 + it;
            float x[8];
            bf16x8_to_float(raw[it], x);
            mag_max = __vmaxu2(mag_max, __vmaxu2(__vmaxu2(raw[it].x & 0x7fff7fffu, raw[it].y & 0x7fff7fffu),
                                                 __vmaxu2(raw[it].z & 0x7fff7fffu, raw[it].w & 0x7fff7fffu)));
            const uint32_t h0 = pack_f16x2(x[0], x[1]), h1 = pack_f16x2(x[2], x[3]);
            const uint32_t h2 = pack_f16x2(x[4], x[5]), h3 = pack_f16x2(x[6], x[7]);
            // the lane of token 0 keeps columns 0..3 of the chunk, the lane of token 1 columns 4..7
            const uint32_t recv_a = __shfl_xor_sync(0xffffffffu, tb ? h0 : h2, 16);
            const uint32_t recv_b = __shfl_xor_sync(0xffffffffu, tb ? h1 : h3, 16);
            const uint32_t mine_a = tb ? h2 : h0, mine_b = tb ? h3 : h1;
            const uint32_t lo_a = tb ? recv_a : mine_a, hi_a = tb ? mine_a : recv_a;  // token 0 / token 1
            const uint32_t lo_b = tb ? recv_b : mine_b, hi_b = tb ? mine_b : recv_b;
            const int d0 = 8 * c + 4 * tb;
            const int col = tp ^ ((d0 >> 2) & 31);
            tile[(d0 + 0) * 64 + col] = prmt(lo_a, hi_a, 0x5410);
            tile[(d0 + 1) * 64 + col] = prmt(lo_a, hi_a, 0x7632);
            tile[(d0 + 2) * 64 + col] = prmt(lo_b, hi_b, 0x5410);
            tile[(d0 + 3) * 64 + col] = prmt(lo_b, hi_b, 0x7632);
        }
        if ((mag_max & 0xffffu) > 0x477fu || (mag_max >> 16) > 0x477fu) atomicCAS(p.status, 0, kStatusRange);
        __syncthreads();
        uint32_t* dst = reinterpret_cast<uint32_t*>(p.vt + (size_t)head * kHeadDim * p.n_kv_pad + tile0);
        const size_t row_words = (size_t)p.n_kv_pad / 2;
#pragma unroll 4
        for (int r = 0; r < kHeadDim / 8; ++r) {
            const int d = warp * (kHeadDim / 8) + r;
            const int swz = (d >> 2) & 31;
            dst[d * row_words + lane] = tile[d * 64 + (lane ^ swz)];
            dst[d * row_words + 32 + lane] = tile[d * 64 + 32 + (lane ^ swz)];
        }
    }
}

cudaError_t launch_prep_kv(const PrepParams& p, cudaStream_t stream) {
    dim3 grid(p.n_kv_pad / kTile, p.h, 2);
    prep_kv_kernel<<<grid, kPrepThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace regenvc
