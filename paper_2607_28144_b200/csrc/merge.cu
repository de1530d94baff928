// Merge of split-key partial results: the last, incomplete wave of work items of the attention kernel is cut
// along the key axis so that its pieces fill the GPU; each piece leaves, per query row, an unnormalised
// accumulator o_i = sum_m 2^(s_m - m_i) v_m, its reference m_i (log2 units) and its row sum l_i.  The exact
// result is sum_i w_i o_i / sum_i w_i l_i with w_i = 2^(m_i - max_i m_i) -- the same online-softmax merge a
// ring of key/value blocks uses (Sec. 3.5).
#include "common.cuh"

namespace regenvc {

constexpr int kMergeThreads = 256;  // one warp per query row, 4 output columns per lane

__global__ void __launch_bounds__(kMergeThreads) merge_partials_kernel(MergeParams p) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row_global = blockIdx.x * (kMergeThreads / 32) + warp;  // over n_split_items * 256 rows
    const int split_item = row_global / (2 * kTile), r = row_global % (2 * kTile);
    if (split_item >= p.n_split_items) return;
    const int item = p.n_full_items + split_item;
    const int head = item / p.pairs_per_head;
    const int n = (item % p.pairs_per_head) * 2 * kTile + r;
    if (n >= p.n_q) return;
    float m_max = -INFINITY;
    for (int i = 0; i < p.split_k; ++i)
        m_max = fmaxf(m_max, p.part_ml[((size_t)split_item * p.split_k + i) * 2 * kTile + r].x);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
    for (int i = 0; i < p.split_k; ++i) {
        const size_t slot = ((size_t)split_item * p.split_k + i) * 2 * kTile + r;
        const float2 ml = p.part_ml[slot];
        const float w = exp2f(ml.x - m_max);
        const float4 o = reinterpret_cast<const float4*>(p.part_o + slot * kHeadDim)[lane];
        acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
        l += w * ml.y;
    }
    const float inv = 1.0f / l;
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
    __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t*>(&lo);
    packed.y = *reinterpret_cast<uint32_t*>(&hi);
    reinterpret_cast<uint2*>(p.out + ((size_t)n * p.h + head) * kHeadDim)[lane] = packed;
}

// The same merge for block-wise attention: part i holds, for every (query row, head), the unnormalised result
// of that row against key/value block i (token-major fp32 [n_q, h, 128] and (m, l) [n_q, h]).  One warp per row.
__global__ void __launch_bounds__(kMergeThreads) merge_token_partials_kernel(TokenMergeParams p) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long r = (long long)blockIdx.x * (kMergeThreads / 32) + warp;  // row = n * h + head
    if (r >= p.n_rows) return;
    float m_max = -INFINITY;
    for (int i = 0; i < p.n_parts; ++i) m_max = fmaxf(m_max, p.ml[i][r].x);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
    for (int i = 0; i < p.n_parts; ++i) {
        const float2 ml = p.ml[i][r];
        const float w = exp2f(ml.x - m_max);
        const float4 o = reinterpret_cast<const float4*>(p.o[i] + r * kHeadDim)[lane];
        acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
        l += w * ml.y;
    }
    const float inv = 1.0f / l;
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
    __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t*>(&lo);
    packed.y = *reinterpret_cast<uint32_t*>(&hi);
    reinterpret_cast<uint2*>(p.out + r * kHeadDim)[lane] = packed;
}

cudaError_t launch_merge_token_partials(const TokenMergeParams& p, cudaStream_t stream) {
    const long long blocks = (p.n_rows + kMergeThreads / 32 - 1) / (kMergeThreads / 32);
    merge_token_partials_kernel<<<(unsigned)blocks, kMergeThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_merge_partials(const MergeParams& p, cudaStream_t stream) {
    const int rows = p.n_split_items * 2 * kTile;
    merge_partials_kernel<<<(rows + kMergeThreads / 32 - 1) / (kMergeThreads / 32), kMergeThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace regenvc
