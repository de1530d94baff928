// Producer of the attention operands: the QKV projection of one transformer block with everything that stands
// between it and the attention kernel fused into its epilogue (the backbone the paper takes by reference,
// Sec. 3.2 / 3.4: three linear maps, an RMS norm over all features of a token on q and k, the head split and
// the 3D rotary embedding).  One pass over x and W_qkv writes
//   Q'  fp16 [N, h, 128]          normalised, rotated queries
//   K'  fp16 [h][n_pad][128]      normalised, rotated keys      } the operand layout the attention kernel streams,
//   V't fp16 [h][128][n_pad]      values, keys contiguous       } so no separate preparation pass is needed
// and nothing of q, k, v is ever rounded to bf16 or written in token-major form.
//
// One CTA computes 128 tokens x 256 output features (two heads) of one of q, k, v:
//   warp 0      TMA producer: x tile [128 tokens][64] and W tile [256 features][64] per stage (bf16, 128B swizzle)
//   warp 1      tcgen05.mma issuer (bf16 x bf16 -> fp32 in 256 tensor-memory columns) and TMEM owner
//   warps 2-9   epilogue, two threads per accumulator row (one per head)
// q and k: D[token][feature] = x W^T (A = x tile, B = W tile, N = 256).  v: D[feature][token] = W x^T (A = W rows of
// one head, B = x tile), which is V't directly -- no transpose anywhere.
// The RMS norm needs the sum of squares over ALL features of a token, which are spread over the h/2 CTAs that
// share the token tile: those CTAs form a thread-block cluster and read each other's partial row sums through
// distributed shared memory.  96 KB of shared memory and 256 tensor-memory columns per CTA: two CTAs share an SM,
// so one's epilogue overlaps the other's main loop.
#include "common.cuh"
#include "ptx.cuh"
#include "rope.cuh"
#include "umma_desc.cuh"

namespace regenvc {

namespace {

constexpr int kBK = 64;                                  // K elements per stage: one 128-byte swizzled row
constexpr int kProjStages = 2;
constexpr int kFeat = kProjHeadsPerCta * kHeadDim;       // 256 output features per CTA
constexpr uint32_t kXBytes = kTile * kBK * 2;            // 16 KB
constexpr uint32_t kWBytes = kFeat * kBK * 2;            // 32 KB
constexpr uint32_t kStageBytes = kXBytes + kWBytes;      // 48 KB
constexpr int kEpiThreads = 256;
constexpr int kProjThreads = 64 + kEpiThreads;
constexpr uint32_t kOutTileBytes = kTile * kHeadDim * 2; // 32 KB: one head's [128][128] fp16 tile, staged for TMA
constexpr uint32_t kOutBlockBytes = kOutTileBytes / 2;
static_assert(kProjHeadsPerCta * kOutTileBytes <= kProjStages * kStageBytes, "output staging reuses the stage buffers");
constexpr uint32_t kProjSmem = kProjStages * kStageBytes + 1024 /*align*/ + 128 /*barriers*/ +
                               2 * kFeat * 4 /*bias, gain*/ + 3 * kTile * 4 /*row sums*/;
constexpr uint64_t kProjWaitNs = 500000000ull;
constexpr uint32_t kIdescQK = umma_idesc_bf16_f32acc(128, kFeat);
constexpr uint32_t kIdescV = umma_idesc_bf16_f32acc(128, 128);

struct ProjBarriers {
    uint64_t full[kProjStages];
    uint64_t empty[kProjStages];
    uint64_t acc_full;
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(ProjBarriers) <= 128, "barrier block too large");

__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_size() {
    uint32_t n;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(n));
    return n;
}
// Reads a float at the same shared-memory offset in CTA `rank` of this cluster.
__device__ __forceinline__ float ld_cluster_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

}  // namespace

__global__ void __launch_bounds__(kProjThreads, 2)
qkv_project_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                   const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                   const __grid_constant__ CUtensorMap tmap_v, const ProjParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* stages = base;
    ProjBarriers* bar = reinterpret_cast<ProjBarriers*>(base + kProjStages * kStageBytes);
    float* bias_s = reinterpret_cast<float*>(base + kProjStages * kStageBytes + 128);
    float* gain_s = bias_s + kFeat;
    float* part_s = gain_s + kFeat;          // [2][128] partial sums of squares of the two column halves
    float* rowsum_s = part_s + 2 * kTile;    // [128]    this CTA's sum of squares per token, read by the cluster

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int pair = blockIdx.x;             // which two heads (= rank in the cluster)
    const int n0 = blockIdx.y * kTile;       // first token of the tile
    const int part = blockIdx.z;             // 0 q, 1 k, 2 v
    const int f0 = part * p.C + pair * kFeat;  // first row of W_qkv (output feature) of this CTA
    const int n_kb = p.C / kBK;
    const WaitCtl ctl{&bar->abort_flag, p.status, kStatusTimeout, kProjWaitNs};
    uint32_t tmem_base = 0;

    if (tid == 0) {
        for (int s = 0; s < kProjStages; ++s) {
            mbar_init(smem_u32(&bar->full[s]), 1);
            mbar_init(smem_u32(&bar->empty[s]), 1);
        }
        mbar_init(smem_u32(&bar->acc_full), 1);
        bar->abort_flag = (*reinterpret_cast<volatile int*>(p.status) != 0) ? 1 : 0;
        fence_mbar_init();
    }
    __syncwarp();
    if (warp == 1) {
        tmem_alloc(smem_u32(&bar->tmem_base), kFeat);
        tmem_relinquish();
    }
    if (warp >= 2) {
        // this CTA's slice of the bias and of the norm gains, once
        const int t = tid - 64;
        bias_s[t] = p.bias ? __ldg(p.bias + f0 + t) : 0.0f;
        const float* g = part == 0 ? p.g_q : p.g_k;
        gain_s[t] = (part < 2 && g) ? __ldg(g + pair * kFeat + t) : 1.0f;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    tmem_base = bar->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            tma_prefetch_desc(&tmap_x);
            tma_prefetch_desc(&tmap_w);
            for (int kb = 0; kb < n_kb; ++kb) {
                const int s = kb % kProjStages, round = kb / kProjStages;
                if (round > 0 && !mbar_wait(smem_u32(&bar->empty[s]), (round - 1) & 1, ctl)) break;
                const uint32_t full = smem_u32(&bar->full[s]);
                const uint32_t dst = smem_u32(stages + s * kStageBytes);
                mbar_expect_tx(full, kStageBytes);
                tma_load_2d(dst, &tmap_x, kb * kBK, n0, full);             // rows past the last token arrive as zeros
                tma_load_2d(dst + kXBytes, &tmap_w, kb * kBK, f0, full);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            bool ok = true;
            for (int kb = 0; kb < n_kb && ok; ++kb) {
                const int s = kb % kProjStages;
                ok = mbar_wait(smem_u32(&bar->full[s]), (kb / kProjStages) & 1, ctl);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sx = smem_u32(stages + s * kStageBytes), sw = sx + kXBytes;
                const uint64_t dx = umma_smem_desc_k_sw128(sx), dw = umma_smem_desc_k_sw128(sw);
#pragma unroll
                for (int kk = 0; kk < kBK / 16; ++kk) {
                    const uint32_t acc = (kb > 0 || kk > 0) ? 1u : 0u;
                    if (part < 2) {
                        umma_ss(tmem_base, dx + 2 * kk, dw + 2 * kk, kIdescQK, acc);
                    } else {
#pragma unroll
                        for (int i = 0; i < kProjHeadsPerCta; ++i)
                            umma_ss(tmem_base + i * 128, dw + i * ((kTile * kBK * 2) >> 4) + 2 * kk, dx + 2 * kk, kIdescV, acc);
                    }
                }
                umma_commit(smem_u32(&bar->empty[s]));
            }
            if (ok) umma_commit(smem_u32(&bar->acc_full));
        }
    }
    __syncwarp();

    const bool normed = part < 2;                      // uniform over the cluster
    const int half = warp >= 2 ? (warp - 2) >> 2 : 0;  // which head of the CTA's two this thread works on
    const int row = (warp & 3) * 32 + lane;            // accumulator row = TMEM lane
    const uint32_t t_acc = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16) + half * 128;
    bool ok = true;
    float inv_rms = 1.0f;
    if (warp >= 2) {
        ok = mbar_wait(smem_u32(&bar->acc_full), 0, ctl);
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();
        if (normed) {
            // pass 1: this thread's share of the sum of squares of its token's features
            float ss = 0.f;
            if (ok) {
#pragma unroll 1
                for (int cb = 0; cb < 4; ++cb) {
                    uint32_t a[32];
                    tmem_ld32(t_acc + cb * 32, a);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        const float y = __uint_as_float(a[c]) + bias_s[half * 128 + cb * 32 + c];
                        ss = fmaf(y, y, ss);
                    }
                }
            }
            part_s[half * kTile + row] = ss;
            epi_barrier();
            if (half == 0) rowsum_s[row] = part_s[row] + part_s[kTile + row];
        }
    }
    if (normed) {
        // every thread of every CTA of the cluster meets here: the partial sums are visible cluster-wide afterwards
        __syncwarp();
        cluster_sync_all();
        if (warp >= 2) {
            float total = 0.f;
            const uint32_t n_rank = cluster_size();
            for (uint32_t r = 0; r < n_rank; ++r) total += ld_cluster_f32(smem_u32(rowsum_s + row), r);
            inv_rms = rsqrtf(total / static_cast<float>(p.C) + p.eps);
        }
    }

    if (warp >= 2) {
        bool out_of_range = false;
        uint8_t* stage_out = stages + half * kOutTileBytes;  // the stage buffers are idle: all MMAs have completed
        if (normed) {
            const int n = n0 + row;
            const bool live = n < p.n_tokens;
            const TokenPos pos = token_pos(live ? n : 0, p.grid);
#pragma unroll 1
            for (int cb = 0; cb < 4; ++cb) {
                uint32_t a[32];
                if (ok) {
                    tmem_ld32(t_acc + cb * 32, a);
                    tmem_wait_ld();
                }
#pragma unroll
                for (int c8 = 0; c8 < 4; ++c8) {
                    float x[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int col = half * 128 + cb * 32 + c8 * 8 + i;
                        x[i] = (__uint_as_float(a[c8 * 8 + i]) + bias_s[col]) * inv_rms * gain_s[col];
                    }
                    const int chunk = cb * 4 + c8;  // 16-byte chunk of the head vector: pairs 4 * chunk ..
                    rope_rotate8(x, p.grid, pos, rope_chunk(p.grid, chunk));
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        out_of_range |= !(fabsf(x[i]) <= 65504.0f);
                        if (!live || !ok) x[i] = 0.f;   // padding rows of K' are zero
                    }
                    uint4 w;
                    w.x = pack_f16x2(x[0], x[1]);
                    w.y = pack_f16x2(x[2], x[3]);
                    w.z = pack_f16x2(x[4], x[5]);
                    w.w = pack_f16x2(x[6], x[7]);
                    const int col = cb * 32 + c8 * 8;
                    *reinterpret_cast<uint4*>(stage_out + (col >> 6) * kOutBlockBytes + sw128_offset(row, (col >> 3) & 7)) = w;
                }
            }
            if (out_of_range && live && ok) atomicCAS(p.status, 0, kStatusRange);
        } else {
            // v: row = feature of head `half`, columns = the tile's tokens
            const float b = bias_s[half * 128 + row];
#pragma unroll 1
            for (int cb = 0; cb < 4; ++cb) {
                uint32_t a[32];
                if (ok) {
                    tmem_ld32(t_acc + cb * 32, a);
                    tmem_wait_ld();
                }
#pragma unroll
                for (int c8 = 0; c8 < 4; ++c8) {
                    float x[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int n = n0 + cb * 32 + c8 * 8 + i;
                        x[i] = (ok && n < p.n_tokens) ? __uint_as_float(a[c8 * 8 + i]) + b : 0.f;  // padding columns zero
                        out_of_range |= !(fabsf(x[i]) <= 65504.0f);
                    }
                    uint4 w;
                    w.x = pack_f16x2(x[0], x[1]);
                    w.y = pack_f16x2(x[2], x[3]);
                    w.z = pack_f16x2(x[4], x[5]);
                    w.w = pack_f16x2(x[6], x[7]);
                    const int col = cb * 32 + c8 * 8;
                    *reinterpret_cast<uint4*>(stage_out + (col >> 6) * kOutBlockBytes + sw128_offset(row, (col >> 3) & 7)) = w;
                }
            }
            if (out_of_range) atomicCAS(p.status, 0, kStatusRange);
        }
        fence_proxy_async_smem();
        epi_barrier();
        if (tid == 64 && ok) {
#pragma unroll
            for (int i = 0; i < kProjHeadsPerCta; ++i) {
                const int head = pair * kProjHeadsPerCta + i;
                const uint32_t src = smem_u32(stages + i * kOutTileBytes);
                if (part == 0) {
                    tma_store_2d(&tmap_q, head * kHeadDim, n0, src);
                    tma_store_2d(&tmap_q, head * kHeadDim + 64, n0, src + kOutBlockBytes);
                } else if (part == 1) {
                    tma_store_2d(&tmap_k, 0, head * p.n_pad + n0, src);
                    tma_store_2d(&tmap_k, 64, head * p.n_pad + n0, src + kOutBlockBytes);
                } else {
                    tma_store_2d(&tmap_v, n0, head * kHeadDim, src);
                    tma_store_2d(&tmap_v, n0 + 64, head * kHeadDim, src + kOutBlockBytes);
                }
            }
            tma_store_commit();
            tma_store_wait_read();
        }
        __syncwarp();
    }

    // ---------------------------------------------------------------- tear-down
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        if (bar->abort_flag) {
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
        __syncwarp();
        tmem_dealloc(tmem_base, kFeat);
    }
    // no CTA of the cluster may exit while another can still read its row sums
    if (normed) {
        __syncwarp();
        cluster_sync_all();
    }
}

cudaError_t configure_qkv_project() {
    return cudaFuncSetAttribute(qkv_project_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kProjSmem);
}

cudaError_t launch_qkv_project(const CUtensorMap& tmap_x, const CUtensorMap& tmap_w, const CUtensorMap& tmap_q,
                               const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, const ProjParams& p,
                               cudaStream_t stream) {
    const unsigned cluster = p.h / kProjHeadsPerCta;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cluster, (p.n_tokens + kTile - 1) / kTile, 3);
    cfg.blockDim = dim3(kProjThreads);
    cfg.dynamicSmemBytes = kProjSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, qkv_project_kernel, tmap_x, tmap_w, tmap_q, tmap_k, tmap_v, p);
}

}  // namespace regenvc
