// Head <-> sequence resharding kernels (Ulysses, Sec. 3.5): the data movement of the all-to-all that turns a
// sequence-sharded tensor [tokens of this GPU][all heads][128] into a head-sharded one
// [all tokens of the group][heads of one GPU][128] and back.  Each destination may be a buffer of this GPU (a
// send buffer handed to a collective afterwards) or peer memory of another GPU mapped into this process, in which
// case the stores travel over NVLink and the kernel is the exchange itself.  Plain 16-byte loads and stores only.
// HBM-bound: every byte is read once and written once.
#include "common.cuh"

namespace regenvc {

namespace {

constexpr int kReshardThreads = 256;
constexpr int kVecPerRow = kHeadDim * 2 / 16;  // uint4 per (token, head) vector

// blockIdx.y = destination.  The elements of one destination are walked with a grid-stride loop, four
// independent 16-byte copies per thread and step.
template <bool kScatter>
__global__ void __launch_bounds__(kReshardThreads) reshard_kernel(ReshardParams p) {
    const int r = blockIdx.y;
    const int heads = kScatter ? p.h_dst : p.h_src;  // heads moved per row for this destination
    const size_t n_vec = (size_t)p.rows[r] * heads * kVecPerRow;
    const size_t stride = (size_t)gridDim.x * kReshardThreads;
    uint4* __restrict__ dst = p.dst[r];
    const uint4* __restrict__ src = p.src;
    for (size_t i0 = (size_t)blockIdx.x * kReshardThreads + threadIdx.x; i0 < n_vec; i0 += 4 * stride) {
        uint4 val[4];
        size_t at[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const size_t i = i0 + u * stride;
            if (i < n_vec) {
                const size_t row = i / ((size_t)heads * kVecPerRow);   // row of this destination's range
                const size_t in_row = i - row * heads * kVecPerRow;    // (head, 16-byte piece) inside the row
                size_t from;
                if (kScatter) {
                    from = (row * p.h_src + (size_t)r * p.h_dst) * kVecPerRow + in_row;
                    at[u] = ((size_t)(p.dst_row0 + row) * p.h_dst) * kVecPerRow + in_row;
                } else {
                    from = ((size_t)p.row0[r] + row) * p.h_src * kVecPerRow + in_row;
                    at[u] = (row * p.h_dst + p.dst_head0) * kVecPerRow + in_row;
                }
                val[u] = __ldg(src + from);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (i0 + u * stride < n_vec) dst[at[u]] = val[u];
    }
}

template <bool kScatter>
cudaError_t launch(const ReshardParams& p, int sm_count, cudaStream_t stream) {
    size_t most = 0;
    for (int r = 0; r < p.world; ++r) {
        const size_t n_vec = (size_t)p.rows[r] * (kScatter ? p.h_dst : p.h_src) * kVecPerRow;
        if (n_vec > most) most = n_vec;
    }
    if (most == 0) return cudaSuccess;
    // enough CTAs to fill the GPU a few times over, but no more than the data needs
    size_t want = (most + 4 * kReshardThreads - 1) / (4 * kReshardThreads);
    const size_t cap = (size_t)(sm_count > 0 ? sm_count : 148) * 8 / p.world + 1;
    if (want > cap) want = cap;
    dim3 grid((unsigned)want, p.world);
    reshard_kernel<kScatter><<<grid, kReshardThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_scatter_heads(const ReshardParams& p, int sm_count, cudaStream_t stream) {
    return launch<true>(p, sm_count, stream);
}
cudaError_t launch_gather_heads(const ReshardParams& p, int sm_count, cudaStream_t stream) {
    return launch<false>(p, sm_count, stream);
}

}  // namespace regenvc
