// Pipelined, warp-specialised tcgen05 attention kernel for sm_100a.
//
// One CTA owns one head and two 128-row query tiles (256 query rows):
//   warps 0-3  softmax group 0 (query tile 0): one thread per query row
//   warps 4-7  softmax group 1 (query tile 1)
//   warp  8    UMMA issuer (one elected lane) and TMEM owner
//   warp  9    TMA producer (one elected lane): streams K' and V't tiles
// The two query tiles ping-pong: while a softmax group turns S_t into P_t the
// tensor core runs the other tile's P.V and next Q.K^T.
//
// Tensor memory (512 columns x 128 lanes, fp32 cells):
//   [0,128) S0  [128,256) S1  [256,384) O0  [384,512) O1 ; P_t (fp16) aliases the first 64 columns of S_t.
// Shared memory: Q0, Q1 (32 KB each, rotated, fp16, 128B-swizzled K-major
// blocks), then a ring of kStages 32 KB slots holding K'_0, V't_0, K'_1, ...
//
// Softmax keeps a running reference m (log2 domain) and row sum l per thread.
// m is only raised when the tile maximum exceeds it by more than kRescaleGap
// (probabilities then stay <= 2^kRescaleGap, well inside fp16/fp32 range), so
// the rescale of the O accumulator in TMEM is rare after the first tiles.
#include "common.cuh"
#include "ptx.cuh"
#include "q_tile.cuh"
#include "rope.cuh"
#include "umma_desc.cuh"

namespace regenvc {

namespace {

constexpr int kStages = 4;                       // K/V ring slots (32 KB each)
constexpr int kSoftmaxThreads = 256;
constexpr int kThreads = kSoftmaxThreads + 64;   // + UMMA warp + TMA warp
constexpr int kMmaWarp = 8, kTmaWarp = 9;
constexpr float kRescaleGap = 8.0f;
constexpr uint32_t kIdesc = umma_idesc_f16_f32acc(128, 128);
constexpr uint32_t kSmemBytes = (2 + kStages) * kTileBytes + 1024 /*align*/ + 256 /*barriers*/;
constexpr uint64_t kWaitLimitNs = 2000000000ull;

struct Barriers {
    uint64_t kv_full[kStages];
    uint64_t kv_empty[kStages];
    uint64_t q_full[2];
    uint64_t s_full[2];
    uint64_t p_full[2];
    uint64_t o_full[2];
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Barriers) <= 256, "barrier block too large");

__device__ __forceinline__ void issue_qk(uint32_t d_tmem, uint32_t sQ, uint32_t sK) {
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
        const uint32_t off = (kk >> 2) * kBlockBytes + (kk & 3) * 32;
        umma_ss(d_tmem, umma_smem_desc_k_sw128(sQ + off), umma_smem_desc_k_sw128(sK + off), kIdesc, kk > 0);
    }
}
__device__ __forceinline__ void issue_pv(uint32_t d_tmem, uint32_t p_tmem, uint32_t sV, bool accumulate) {
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
        const uint32_t off = (kk >> 2) * kBlockBytes + (kk & 3) * 32;
        umma_ts(d_tmem, p_tmem + kk * 8, umma_smem_desc_k_sw128(sV + off), kIdesc, accumulate || kk > 0);
    }
}

}  // namespace

__global__ void __launch_bounds__(kThreads, 1)
attn_pipelined_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                      const AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = base;                       // 2 tiles
    uint8_t* sKV = base + 2 * kTileBytes;     // ring
    Barriers* bar = reinterpret_cast<Barriers*>(base + (2 + kStages) * kTileBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int head = blockIdx.y;
    const int q0 = blockIdx.x * 2 * kTile;
    const bool tile1_active = q0 + kTile < p.n_q;
    const int n_tiles = p.n_kv_pad / kTile;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&bar->kv_full[s]), 1);
            mbar_init(smem_u32(&bar->kv_empty[s]), 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_u32(&bar->q_full[t]), kSoftmaxThreads / 2);
            mbar_init(smem_u32(&bar->s_full[t]), 1);
            mbar_init(smem_u32(&bar->p_full[t]), kSoftmaxThreads / 2);
            mbar_init(smem_u32(&bar->o_full[t]), 1);
        }
        bar->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(&bar->tmem_base), 512);
        tmem_relinquish();
    }
    if (warp == kTmaWarp && lane == 0) {
        tma_prefetch_desc(&tmap_k);
        tma_prefetch_desc(&tmap_v);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const uint32_t tmem_base = bar->tmem_base;
    const WaitCtl ctl{&bar->abort_flag, p.status, kStatusTimeout, kWaitLimitNs};

    if (warp == kTmaWarp) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const int total = 2 * n_tiles;
            for (int i = 0; i < total; ++i) {
                const int slot = i % kStages, round = i / kStages;
                if (round > 0 && !mbar_wait(smem_u32(&bar->kv_empty[slot]), (round - 1) & 1, ctl)) break;
                const uint32_t full = smem_u32(&bar->kv_full[slot]);
                const uint32_t dst = smem_u32(sKV + slot * kTileBytes);
                const int kv0 = (i >> 1) * kTile;
                mbar_expect_tx(full, kTileBytes);
                if ((i & 1) == 0) {
                    tma_load_2d(dst, &tmap_k, 0, head * p.n_kv_pad + kv0, full);
                    tma_load_2d(dst + kBlockBytes, &tmap_k, 64, head * p.n_kv_pad + kv0, full);
                } else {
                    tma_load_2d(dst, &tmap_v, kv0, head * kHeadDim, full);
                    tma_load_2d(dst + kBlockBytes, &tmap_v, kv0 + 64, head * kHeadDim, full);
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------ UMMA issuer
        if (lane == 0) {
            const uint32_t sQ0 = smem_u32(sQ), sQ1 = smem_u32(sQ) + kTileBytes;
            const int n_active = tile1_active ? 2 : 1;
            bool ok = mbar_wait(smem_u32(&bar->q_full[0]), 0, ctl);
            if (ok && tile1_active) ok = mbar_wait(smem_u32(&bar->q_full[1]), 0, ctl);
            if (ok) ok = mbar_wait(smem_u32(&bar->kv_full[0]), 0, ctl);
            if (ok) {
                tc_fence_after();
                for (int t = 0; t < n_active; ++t) {
                    issue_qk(tmem_base + t * 128, t ? sQ1 : sQ0, smem_u32(sKV));
                    umma_commit(smem_u32(&bar->s_full[t]));
                }
                umma_commit(smem_u32(&bar->kv_empty[0]));
            }
            for (int j = 0; ok && j < n_tiles; ++j) {
                const int iv = 2 * j + 1, ik = 2 * j + 2;
                const int slot_v = iv % kStages, slot_k = ik % kStages;
                const bool more = j + 1 < n_tiles;
                ok = mbar_wait(smem_u32(&bar->kv_full[slot_v]), (iv / kStages) & 1, ctl);
                if (ok && more) ok = mbar_wait(smem_u32(&bar->kv_full[slot_k]), (ik / kStages) & 1, ctl);
                for (int t = 0; ok && t < n_active; ++t) {
                    ok = mbar_wait(smem_u32(&bar->p_full[t]), j & 1, ctl);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(tmem_base + 256 + t * 128, tmem_base + t * 128, smem_u32(sKV + slot_v * kTileBytes), j > 0);
                    umma_commit(smem_u32(&bar->o_full[t]));
                    if (more) {
                        issue_qk(tmem_base + t * 128, t ? sQ1 : sQ0, smem_u32(sKV + slot_k * kTileBytes));
                        umma_commit(smem_u32(&bar->s_full[t]));
                    }
                }
                if (ok) {
                    umma_commit(smem_u32(&bar->kv_empty[slot_v]));
                    if (more) umma_commit(smem_u32(&bar->kv_empty[slot_k]));
                }
            }
        }
    } else {
        // ------------------------------------------------------------ softmax groups
        const int t = warp >> 2;                 // query tile of this group
        const int row = tid & 127;               // row in the tile == TMEM lane
        const int qt0 = q0 + t * kTile;
        if (t == 0 || tile1_active) {
            load_rotate_q_tile(p, head, qt0, sQ + t * kTileBytes, row, kSoftmaxThreads / 2);
            fence_proxy_async_smem();
            mbar_arrive(smem_u32(&bar->q_full[t]));

            const uint32_t lane_base = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
            const uint32_t t_S = lane_base + t * 128, t_O = lane_base + 256 + t * 128;
            const uint32_t s_full = smem_u32(&bar->s_full[t]), p_full = smem_u32(&bar->p_full[t]),
                           o_full = smem_u32(&bar->o_full[t]);
            const float scale = p.scale_log2;
            float m_ref = 0.f, l_run = 0.f;
            bool ok = true;

            for (int j = 0; j < n_tiles; ++j) {
                ok = mbar_wait(s_full, j & 1, ctl);
                if (!ok) break;
                tc_fence_after();
                uint32_t sr[128];
                tmem_ld32(t_S + 0, sr + 0);
                tmem_ld32(t_S + 32, sr + 32);
                tmem_ld32(t_S + 64, sr + 64);
                tmem_ld32(t_S + 96, sr + 96);
                tmem_wait_ld();
                if (j == n_tiles - 1) {
                    const int valid = p.n_kv - j * kTile;  // columns >= valid are padding
#pragma unroll
                    for (int c = 0; c < 128; ++c)
                        if (c >= valid) sr[c] = 0xff800000u;  // -inf
                }
                float mx = -INFINITY;
#pragma unroll
                for (int c = 0; c < 128; ++c) mx = fmaxf(mx, __uint_as_float(sr[c]));
                const float m_tile = mx * scale;
                bool raise = (j == 0) || (m_tile > m_ref + kRescaleGap);
                if (j > 0 && __any_sync(0xffffffffu, raise)) {
                    // some row of this warp moves its reference: rescale this warp's O rows and row sums
                    ok = mbar_wait(o_full, (j - 1) & 1, ctl);
                    if (!ok) break;
                    tc_fence_after();
                    const float alpha = raise ? ex2_approx(m_ref - m_tile) : 1.0f;
                    l_run *= alpha;
#pragma unroll 1
                    for (int cb = 0; cb < 4; ++cb) {
                        uint32_t o[32];
                        tmem_ld32(t_O + cb * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                        tmem_st32(t_O + cb * 32, o);
                    }
                }
                if (raise) m_ref = m_tile;
                float rowsum = 0.f;
#pragma unroll
                for (int cb = 0; cb < 4; ++cb) {
                    uint32_t pr[16];
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        const float p0 = ex2_approx(fmaf(__uint_as_float(sr[cb * 32 + 2 * c]), scale, -m_ref));
                        const float p1 = ex2_approx(fmaf(__uint_as_float(sr[cb * 32 + 2 * c + 1]), scale, -m_ref));
                        rowsum += p0 + p1;
                        pr[c] = pack_f16x2(p0, p1);
                    }
                    tmem_st16(t_S + cb * 16, pr);
                }
                l_run += rowsum;
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(p_full);
            }

            // epilogue: O / l -> bf16 -> out
            if (ok) ok = mbar_wait(o_full, (n_tiles - 1) & 1, ctl);
            if (ok) {
                tc_fence_after();
                const int n = qt0 + row;
                const float inv_l = 1.0f / l_run;
#pragma unroll 1
                for (int cb = 0; cb < 4; ++cb) {
                    uint32_t o[32];
                    tmem_ld32(t_O + cb * 32, o);
                    tmem_wait_ld();
                    if (n < p.n_q) {
                        uint4* dst = reinterpret_cast<uint4*>(p.out + ((size_t)n * p.h + head) * kHeadDim + cb * 32);
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint4 w;
                            w.x = pack_bf16x2(__uint_as_float(o[8 * c + 0]) * inv_l, __uint_as_float(o[8 * c + 1]) * inv_l);
                            w.y = pack_bf16x2(__uint_as_float(o[8 * c + 2]) * inv_l, __uint_as_float(o[8 * c + 3]) * inv_l);
                            w.z = pack_bf16x2(__uint_as_float(o[8 * c + 4]) * inv_l, __uint_as_float(o[8 * c + 5]) * inv_l);
                            w.w = pack_bf16x2(__uint_as_float(o[8 * c + 6]) * inv_l, __uint_as_float(o[8 * c + 7]) * inv_l);
                            dst[c] = w;
                        }
                    }
                }
            }
        }
    }

    // ---------------------------------------------------------------- tear-down
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        if (bar->abort_flag) {
            // a wait expired: give copies and MMAs that may still be in flight time to land before TMEM is released
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
        tmem_dealloc(tmem_base, 512);
    }
}

cudaError_t configure_attn_pipelined() {
    return cudaFuncSetAttribute(attn_pipelined_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
}

cudaError_t launch_attn_pipelined(const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, const AttnParams& p,
                                  cudaStream_t stream) {
    dim3 grid((p.n_q + 2 * kTile - 1) / (2 * kTile), p.h);
    attn_pipelined_kernel<<<grid, kThreads, kSmemBytes, stream>>>(tmap_k, tmap_v, p);
    return cudaGetLastError();
}

}  // namespace regenvc
