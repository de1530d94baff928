// Merge of split-key partial results: the last, incomplete wave of work items of the attention kernel is cut
// along the key axis so that its pieces fill the GPU; each piece leaves, per query row, an unnormalised
// accumulator o_i = sum_m 2^(s_m - m_i) v_m, its reference m_i (log2 units) and its row sum l_i.  The exact
// result is sum_i w_i o_i / sum_i w_i l_i with w_i = 2^(m_i - max_i m_i) -- the same online-softmax merge a
// ring of key/value blocks uses (Sec. 3.5).
#include "common.cuh"

namespace regenvc {

constexpr int kMergeThreads = 256;  // one warp per query row, 4 output columns per lane

// Combines up to kMaxMergeParts partial rows.  All loads (references, row sums, accumulator parts) are issued
// before anything is used, so that a row costs one memory round trip instead of one per dependent step.
template <typename MlAt, typename OAt>
__device__ __forceinline__ uint2 merge_row(int n_parts, MlAt ml_at, OAt o_at) {
    float2 ml[kMaxMergeParts];
    float4 o[kMaxMergeParts];
#pragma unroll
    for (int i = 0; i < kMaxMergeParts; ++i) {
        ml[i] = make_float2(-INFINITY, 0.f);
        o[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < n_parts) {
            ml[i] = ml_at(i);
            o[i] = o_at(i);
        }
    }
    float m_max = -INFINITY;
#pragma unroll
    for (int i = 0; i < kMaxMergeParts; ++i) m_max = fmaxf(m_max, ml[i].x);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
#pragma unroll
    for (int i = 0; i < kMaxMergeParts; ++i) {
        if (i < n_parts) {
            const float w = exp2f(ml[i].x - m_max);
            acc.x += w * o[i].x; acc.y += w * o[i].y; acc.z += w * o[i].z; acc.w += w * o[i].w;
            l += w * ml[i].y;
        }
    }
    const float inv = 1.0f / l;
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
    __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t*>(&lo);
    packed.y = *reinterpret_cast<uint32_t*>(&hi);
    return packed;
}

__global__ void __launch_bounds__(kMergeThreads) merge_partials_kernel(MergeParams p) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row_global = blockIdx.x * (kMergeThreads / 32) + warp;  // over n_split_items * 256 rows
    const int split_item = row_global / (2 * kTile), r = row_global % (2 * kTile);
    if (split_item >= p.n_split_items) return;
    const int item = p.n_full_items + split_item;
    const int head = item / p.pairs_per_head;
    const int n = (item % p.pairs_per_head) * 2 * kTile + r;
    if (n >= p.n_q) return;
    const size_t slot0 = (size_t)split_item * p.split_k * 2 * kTile + r;  // piece i of this row: + i * 256 rows
    const uint2 packed = merge_row(
        p.split_k, [&](int i) { return p.part_ml[slot0 + (size_t)i * 2 * kTile]; },
        [&](int i) { return reinterpret_cast<const float4*>(p.part_o + (slot0 + (size_t)i * 2 * kTile) * kHeadDim)[lane]; });
    reinterpret_cast<uint2*>(p.out + ((size_t)n * p.h + head) * kHeadDim)[lane] = packed;
}

// The same merge for block-wise attention: part i holds, for every (query row, head), the unnormalised result
// of that row against key/value block i (token-major fp32 [n_q, h, 128] and (m, l) [n_q, h]).  One warp per row.
__global__ void __launch_bounds__(kMergeThreads) merge_token_partials_kernel(TokenMergeParams p) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long r = (long long)blockIdx.x * (kMergeThreads / 32) + warp;  // row = n * h + head
    if (r >= p.n_rows) return;
    const uint2 packed = merge_row(
        p.n_parts, [&](int i) { return p.ml[i][r]; },
        [&](int i) { return reinterpret_cast<const float4*>(p.o[i] + r * kHeadDim)[lane]; });
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
