// Serial (un-pipelined) tcgen05 attention kernel: one CTA of 128 threads per
// (head, 128-row query tile); TMA load, QK^T, softmax, P.V run one after the
// other for every 128-key tile.  It is the bring-up / cross-check variant of
// the pipelined kernel (same operand layouts, descriptors and TMEM usage) and
// is selected with REGENVC_KERNEL=serial.
//
// TMEM (256 columns): S fp32 [0,128) with P fp16 aliased on [0,64); O fp32 [128,256).
// Thread i of the CTA owns query row i (TMEM lane i).
#include "common.cuh"
#include "ptx.cuh"
#include "rope.cuh"
#include "umma_desc.cuh"
#include "q_tile.cuh"

namespace regenvc {

namespace {

constexpr int kSerialThreads = 128;
constexpr uint32_t kSerialSmem = 3 * kTileBytes + 1024 /*align*/ + 128 /*barriers*/;
constexpr uint32_t kIdesc = umma_idesc_f16_f32acc(128, 128);

}  // namespace

__global__ void __launch_bounds__(kSerialThreads, 1)
attn_serial_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                   const AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = base;
    uint8_t* sK = base + kTileBytes;
    uint8_t* sV = base + 2 * kTileBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + 3 * kTileBytes);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 5);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int head = blockIdx.y;
    const int q0 = blockIdx.x * kTile;
    const uint32_t bar_kv = smem_u32(&bars[0]), bar_s = smem_u32(&bars[1]), bar_o = smem_u32(&bars[2]);

    if (tid == 0) {
        mbar_init(bar_kv, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        fence_mbar_init();
        *abort_flag = 0;
        tma_prefetch_desc(&tmap_k);
        tma_prefetch_desc(&tmap_v);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(tmem_slot), 256);
        tmem_relinquish();
    }
    load_rotate_q_tiles<kSerialThreads, 1>(p, head, q0, sQ, tid);
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const uint32_t tmem_base = *tmem_slot;
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
    const uint32_t t_S = t_lane, t_O = t_lane + 128;
    const WaitCtl ctl{abort_flag, p.status, kStatusTimeout, 2000000000ull};

    const int n_tiles = p.n_kv_pad / kTile;
    float m_run = -INFINITY, l_run = 0.f;

    for (int j = 0; j < n_tiles; ++j) {
        const uint32_t ph = j & 1;
        const int kv0 = j * kTile;
        if (tid == 0 && !*abort_flag) {
            mbar_expect_tx(bar_kv, 2 * kTileBytes);
            tma_load_2d(smem_u32(sK), &tmap_k, 0, head * p.n_kv_pad + kv0, bar_kv);
            tma_load_2d(smem_u32(sK) + kBlockBytes, &tmap_k, 64, head * p.n_kv_pad + kv0, bar_kv);
            tma_load_2d(smem_u32(sV), &tmap_v, kv0, head * kHeadDim, bar_kv);
            tma_load_2d(smem_u32(sV) + kBlockBytes, &tmap_v, kv0 + 64, head * kHeadDim, bar_kv);
        }
        mbar_wait(bar_kv, ph, ctl);
        if (tid == 0 && !*abort_flag) {
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t off = (kk >> 2) * kBlockBytes + (kk & 3) * 32;
                umma_ss(tmem_base, umma_smem_desc_k_sw128(smem_u32(sQ) + off),
                        umma_smem_desc_k_sw128(smem_u32(sK) + off), kIdesc, kk > 0);
            }
            umma_commit(bar_s);
        }
        mbar_wait(bar_s, ph, ctl);
        __syncwarp();
        tc_fence_after();

        // ---- softmax on this thread's row
        uint32_t sr[128];
        tmem_ld32(t_S + 0, sr + 0);
        tmem_ld32(t_S + 32, sr + 32);
        tmem_ld32(t_S + 64, sr + 64);
        tmem_ld32(t_S + 96, sr + 96);
        tmem_wait_ld();
        const int valid = p.n_kv - kv0;  // columns >= valid are padding
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < 128; ++c) {
            float s = __uint_as_float(sr[c]);
            if (c >= valid) s = -INFINITY;
            sr[c] = __float_as_uint(s);
            mx = fmaxf(mx, s);
        }
        const float m_new = fmaxf(m_run, mx * p.scale_log2);
        const float alpha = ex2_approx(m_run - m_new);
        float rowsum = 0.f;
        uint32_t pr[64];
#pragma unroll
        for (int c = 0; c < 64; ++c) {
            const float p0 = ex2_approx(fmaf(__uint_as_float(sr[2 * c]), p.scale_log2, -m_new));
            const float p1 = ex2_approx(fmaf(__uint_as_float(sr[2 * c + 1]), p.scale_log2, -m_new));
            rowsum += p0 + p1;
            pr[c] = pack_f16x2(p0, p1);
        }
        l_run = l_run * alpha + rowsum;
        m_run = m_new;
        tmem_st32(t_S + 0, pr + 0);
        tmem_st32(t_S + 32, pr + 32);
        if (j > 0) {
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
        tmem_wait_st();
        tc_fence_before();
        __syncthreads();

        if (tid == 0 && !*abort_flag) {
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t off = (kk >> 2) * kBlockBytes + (kk & 3) * 32;
                umma_ts(tmem_base + 128, tmem_base + kk * 8, umma_smem_desc_k_sw128(smem_u32(sV) + off), kIdesc,
                        (j > 0) || (kk > 0));
            }
            umma_commit(bar_o);
        }
        mbar_wait(bar_o, ph, ctl);
        __syncwarp();
        tc_fence_after();
    }

    // ---- epilogue: O / l -> bf16 -> out
    const int n = q0 + tid;
    const float inv_l = 1.0f / l_run;
#pragma unroll 1
    for (int cb = 0; cb < 4; ++cb) {
        uint32_t o[32];
        tmem_ld32(t_O + cb * 32, o);
        tmem_wait_ld();
        if (n < p.n_q && !*abort_flag) {
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
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, 256);
    }
}

cudaError_t configure_attn_serial() {
    return cudaFuncSetAttribute(attn_serial_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSerialSmem);
}

cudaError_t launch_attn_serial(const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, const AttnParams& p,
                               cudaStream_t stream) {
    dim3 grid((p.n_q + kTile - 1) / kTile, p.h);
    attn_serial_kernel<<<grid, kSerialThreads, kSerialSmem, stream>>>(tmap_k, tmap_v, p);
    return cudaGetLastError();
}

}  // namespace regenvc
