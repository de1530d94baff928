// Producer of the attention operands: the QKV projection of one transformer block with everything that stands
// between it and the attention kernel fused into its epilogue (the backbone the paper takes by reference,
// Sec. 3.2 / 3.4: three linear maps, an RMS norm over all features of a token on q and k, the head split and
// the 3D rotary embedding).  One pass over x and W_qkv writes
//   Q'  fp16 [N, h, 128]          normalised, rotated queries
//   K'  fp16 [h][n_pad][128]      normalised, rotated keys      } the operand layout the attention kernel streams,
//   V't fp16 [h][128][n_pad]      values, keys contiguous       } so no separate preparation pass is needed
// and nothing of q, k, v is ever rounded to bf16 or written in token-major form.
//
// A work unit is (128-token tile, one of q / k / v), cut into h/2 slices of 256 output features (two heads).  The
// grid is persistent, one CTA per SM: CTA c takes slices c, c + gridDim.x, ... of the unit-major list, so the
// slices of a unit run on neighbouring CTAs at about the same time.
//   warp 0      TMA producer: x tile [128 tokens][64] and W tile [256 features][64] per stage (bf16, 128B swizzle),
//               a 3-stage ring that runs on into the next unit
//   warp 1      tcgen05.mma issuer (bf16 x bf16 -> fp32) and TMEM owner; two accumulators of 256 columns, used in
//               turn, so that the main loop of one unit runs while the epilogue warps empty the other accumulator
//   warps 2-9   epilogue, two threads per accumulator row (one per head)
// q and k: D[token][feature] = x W^T (A = x tile, B = W tile, N = 256).  v: D[feature][token] = W x^T (A = W rows of
// one head, B = x tile), which is V't directly -- no transpose anywhere.
// The RMS norm needs the sum of squares over ALL features of a token, which are spread over the h/2 CTAs that hold
// the slices of the unit: each writes its partial row sums to a scratch array in global memory and counts itself in
// on the unit's counter; the epilogue warps (only they -- the producer and the MMA warp run ahead) wait until the
// counter shows all slices and add the partial sums in slice order, so the result does not depend on timing.  The
// wait is bounded like every other; it cannot deadlock because every CTA works through its slices in increasing
// order and the whole grid is resident (grid <= number of SMs, one CTA per SM, cooperative launch).  (A first form
// exchanged the sums through distributed shared memory inside clusters of h/2 CTAs; clusters of 6 left 16 of this
// part's 148 SMs idle and capped the head count at 16.)
#include <cstddef>

#include "common.cuh"
#include "ptx.cuh"
#include "rope.cuh"
#include "umma_desc.cuh"

namespace regenvc {

namespace {

constexpr int kBK = 64;                                  // K elements per stage: one 128-byte swizzled row
constexpr int kProjStages = 3;
constexpr int kFeat = kProjHeadsPerCta * kHeadDim;       // 256 output features per CTA
constexpr uint32_t kXBytes = kTile * kBK * 2;            // 16 KB
constexpr uint32_t kWBytes = kFeat * kBK * 2;            // 32 KB
constexpr uint32_t kStageBytes = kXBytes + kWBytes;      // 48 KB
constexpr int kEpiThreads = 256;
constexpr int kProjThreads = 64 + kEpiThreads;
constexpr uint32_t kOutTileBytes = kTile * kHeadDim * 2; // 32 KB: one head's [128][128] fp16 tile, staged for TMA
constexpr uint32_t kOutBlockBytes = kOutTileBytes / 2;
constexpr uint64_t kProjWaitNs = 500000000ull;
constexpr uint32_t kIdescQK = umma_idesc_bf16_f32acc(128, kFeat);
constexpr uint32_t kIdescV = umma_idesc_bf16_f32acc(128, 128);

struct ProjShared {
    uint64_t full[kProjStages];
    uint64_t empty[kProjStages];
    uint64_t acc_full[2];      // accumulator b holds a finished unit
    uint64_t acc_empty[2];     // the epilogue has read accumulator b out
    uint32_t tmem_base;
    int abort_flag;
    float bias[kFeat];         // this unit's slice of the bias
    float gain[kFeat];         //             ... and of the norm gains
    float part[2][kTile];      // partial sums of squares of the two heads of this CTA
};
constexpr uint32_t kProjSmem = kProjStages * kStageBytes + kProjHeadsPerCta * kOutTileBytes + 1024 /*align*/ +
                               sizeof(ProjShared);
static_assert(kProjSmem <= 232448, "shared memory of one SM");

__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }
// Value of a counter in global memory as other CTAs have left it (acquire at device scope).
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Unit index -> (token tile, part: 0 q, 1 k, 2 v), part-major: all token tiles of q, then of k, then of v, so that
// only one third of W_qkv is live at a time.  (With the three parts of a token tile next to each other the whole of
// W_qkv is re-read every few token tiles; for 40 heads that is 157 MB, more than the L2 holds, and the kernel ran at
// 0.94-0.99 PFLOP/s instead of 1.22.  x is read three times instead, from L2 or at a third of the weights' size.)
struct Unit {
    int tile, part;
};
__device__ __forceinline__ Unit decode_unit(int unit, int n_tiles) { return Unit{unit % n_tiles, unit / n_tiles}; }

}  // namespace

__global__ void __launch_bounds__(kProjThreads, 1)
qkv_project_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                   const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                   const __grid_constant__ CUtensorMap tmap_v, const ProjParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* stages = base;
    uint8_t* stage_out = base + kProjStages * kStageBytes;   // two [128][128] fp16 tiles for the tiled stores
    ProjShared* sh = reinterpret_cast<ProjShared*>(stage_out + kProjHeadsPerCta * kOutTileBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_rank = p.h / kProjHeadsPerCta;               // slices per unit
    const int n_tiles = (p.n_tokens + kTile - 1) / kTile;
    const int n_slices = 3 * n_tiles * n_rank;               // slice s: unit s / n_rank (token tile and part: decode_unit),
    const int slice0 = blockIdx.x, slice_step = gridDim.x;   // heads 2 (s % n_rank) and 2 (s % n_rank) + 1
    const int n_kb = p.C / kBK;
    const WaitCtl ctl{&sh->abort_flag, p.status, kStatusTimeout, kProjWaitNs};
    uint32_t tmem_base = 0;

    if (tid == 0) {
        for (int s = 0; s < kProjStages; ++s) {
            mbar_init(smem_u32(&sh->full[s]), 1);
            mbar_init(smem_u32(&sh->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sh->acc_full[b]), 1);
            mbar_init(smem_u32(&sh->acc_empty[b]), kEpiThreads);
        }
        sh->abort_flag = (*reinterpret_cast<volatile int*>(p.status) != 0) ? 1 : 0;
        fence_mbar_init();
    }
    __syncwarp();
    if (warp == 1) {
        tmem_alloc(smem_u32(&sh->tmem_base), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    tmem_base = sh->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            tma_prefetch_desc(&tmap_x);
            tma_prefetch_desc(&tmap_w);
            int fill = 0;  // stages filled so far over all units
            bool ok = true;
            for (int slice = slice0; ok && slice < n_slices; slice += slice_step) {
                const int unit = slice / n_rank, pair = slice % n_rank;
                const Unit u = decode_unit(unit, n_tiles);
                const int n0 = u.tile * kTile;
                const int f0 = u.part * p.C + pair * kFeat;   // first row of W_qkv (output feature) of this slice
                for (int kb = 0; kb < n_kb; ++kb, ++fill) {
                    const int s = fill % kProjStages, round = fill / kProjStages;
                    if (round > 0) ok = mbar_wait(smem_u32(&sh->empty[s]), (round - 1) & 1, ctl);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&sh->full[s]);
                    const uint32_t dst = smem_u32(stages + s * kStageBytes);
                    mbar_expect_tx(full, kStageBytes);
                    tma_load_2d(dst, &tmap_x, kb * kBK, n0, full);   // rows past the last token arrive as zeros
                    tma_load_2d(dst + kXBytes, &tmap_w, kb * kBK, f0, full);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            int fill = 0, it = 0;
            bool ok = true;
            for (int slice = slice0; ok && slice < n_slices; slice += slice_step, ++it) {
                const int part = decode_unit(slice / n_rank, n_tiles).part, b = it & 1;
                const uint32_t acc_tmem = tmem_base + b * kFeat;
                // the accumulator must have been read out by the epilogue of the unit before last
                if (it >= 2) ok = mbar_wait(smem_u32(&sh->acc_empty[b]), ((it >> 1) - 1) & 1, ctl);
                if (!ok) break;
                tc_fence_after();
                for (int kb = 0; kb < n_kb; ++kb, ++fill) {
                    const int s = fill % kProjStages;
                    ok = mbar_wait(smem_u32(&sh->full[s]), (fill / kProjStages) & 1, ctl);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sx = smem_u32(stages + s * kStageBytes), sw = sx + kXBytes;
                    const uint64_t dx = umma_smem_desc_k_sw128(sx), dw = umma_smem_desc_k_sw128(sw);
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk) {
                        const uint32_t acc = (kb > 0 || kk > 0) ? 1u : 0u;
                        if (part < 2) {
                            umma_ss(acc_tmem, dx + 2 * kk, dw + 2 * kk, kIdescQK, acc);
                        } else {
#pragma unroll
                            for (int i = 0; i < kProjHeadsPerCta; ++i)
                                umma_ss(acc_tmem + i * 128, dw + i * ((kTile * kBK * 2) >> 4) + 2 * kk, dx + 2 * kk,
                                        kIdescV, acc);
                        }
                    }
                    umma_commit(smem_u32(&sh->empty[s]));
                }
                if (ok) umma_commit(smem_u32(&sh->acc_full[b]));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int half = (warp - 2) >> 2;             // which head of the CTA's two this thread works on
        const int row = (warp & 3) * 32 + lane;       // accumulator row = TMEM lane
        const int et = tid - 64;                      // 0 .. 255
        uint8_t* my_stage = stage_out + half * kOutTileBytes;
        bool ok = true;
        int it = 0;
        for (int slice = slice0; slice < n_slices; slice += slice_step, ++it) {
            const int unit = slice / n_rank, pair = slice % n_rank;
            const Unit u = decode_unit(unit, n_tiles);
            const int part = u.part, n0 = u.tile * kTile, b = it & 1;
            const bool normed = part < 2;
            const uint32_t t_acc = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16) + b * kFeat + half * 128;
            // this unit's slice of the bias and of the norm gains (the previous unit's readers are past the barrier
            // that closed its epilogue)
            {
                const int f0 = part * p.C + pair * kFeat;
                sh->bias[et] = p.bias ? __ldg(p.bias + f0 + et) : 0.0f;
                const float* g = part == 0 ? p.g_q : p.g_k;
                sh->gain[et] = (normed && g) ? __ldg(g + pair * kFeat + et) : 1.0f;
            }
            epi_barrier();
            if (ok) ok = mbar_wait(smem_u32(&sh->acc_full[b]), (it >> 1) & 1, ctl);
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();

            float inv_rms = 1.0f;
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
                            const float y = __uint_as_float(a[c]) + sh->bias[half * 128 + cb * 32 + c];
                            ss = fmaf(y, y, ss);
                        }
                    }
                }
                sh->part[half][row] = ss;
                epi_barrier();
                // publish this slice's partial sum of every token, then count the slice in
                if (half == 0)
                    __stcg(p.unit_sums + ((size_t)unit * n_rank + pair) * kTile + row, sh->part[0][row] + sh->part[1][row]);
                __threadfence();
                epi_barrier();
                if (et == 0) {
                    atomicAdd(p.unit_count + unit, 1);
                    uint64_t t0 = 0;
                    uint32_t spins = 0;
                    while (ok && ld_acquire_gpu(p.unit_count + unit) < n_rank) {   // all slices of the unit are in?
                        __nanosleep(64);
                        if ((++spins & 63u) == 0) {
                            if (sh->abort_flag) ok = false;
                            const uint64_t now = global_timer_ns();
                            if (t0 == 0) t0 = now;
                            else if (now - t0 > kProjWaitNs) {
                                sh->abort_flag = 1;
                                atomicCAS(p.status, 0, kStatusTimeout);
                                ok = false;
                            }
                        }
                    }
                }
                epi_barrier();
                if (sh->abort_flag) ok = false;
                ok = __all_sync(0xffffffffu, ok);
                float total = 0.f;
                for (int r = 0; r < n_rank; ++r)   // slice order: the same sum whatever the timing
                    total += __ldcg(p.unit_sums + ((size_t)unit * n_rank + r) * kTile + row);
                inv_rms = rsqrtf(total / static_cast<float>(p.C) + p.eps);
            }

            // the staging tiles are free once the previous unit's stores have read them (thread 64 issued them)
            if (tid == 64) tma_store_wait_read();
            epi_barrier();
            if (normed) {
                const int n = n0 + row;
                const bool live = n < p.n_tokens;
                const TokenPos pos = token_pos(live ? n : 0, p.grid);
                float amax = 0.f;  // largest magnitude of this row, for the fp16 range check
                // Fully unrolled so that the place of every pair in the rotary table is a compile-time constant.  The 16
                // (cos, sin) entries of a 32-column chunk are requested one chunk ahead, so that their latency (with
                // two warps per scheduler nothing else hides it) falls on the arithmetic of the chunk before.
                float2 cs_next[16];
                auto fetch_cs = [&](int cbn, float2* dst) {
#pragma unroll
                    for (int c8 = 0; c8 < 4; ++c8) {
                        const RopeChunk rc = rope_chunk(p.grid, cbn * 4 + c8);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int at = rc.axis[i] == 0 ? pos.t : (rc.axis[i] == 1 ? pos.y : pos.x);
                            dst[c8 * 4 + i] = __ldg(p.grid.tab + at * rc.mult[i] + rc.off[i]);
                        }
                    }
                };
                fetch_cs(0, cs_next);
#pragma unroll
                for (int cb = 0; cb < 4; ++cb) {
                    float2 cs[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) cs[i] = cs_next[i];
                    if (cb + 1 < 4) fetch_cs(cb + 1, cs_next);
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
                            x[i] = (__uint_as_float(a[c8 * 8 + i]) + sh->bias[col]) * inv_rms * sh->gain[col];
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i) {  // pair (2i, 2i + 1) of this 8-column piece turns by its angle
                            const float2 w2 = cs[c8 * 4 + i];
                            const float xa = x[2 * i], xb2 = x[2 * i + 1];
                            x[2 * i] = xa * w2.x - xb2 * w2.y;
                            x[2 * i + 1] = xa * w2.y + xb2 * w2.x;
                        }
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            amax = fmaxf(amax, fabsf(x[i]));
                            if (!live || !ok) x[i] = 0.f;   // padding rows of K' are zero
                        }
                        uint4 w;
                        w.x = pack_f16x2(x[0], x[1]);
                        w.y = pack_f16x2(x[2], x[3]);
                        w.z = pack_f16x2(x[4], x[5]);
                        w.w = pack_f16x2(x[6], x[7]);
                        const int col = cb * 32 + c8 * 8;
                        *reinterpret_cast<uint4*>(my_stage + (col >> 6) * kOutBlockBytes + sw128_offset(row, (col >> 3) & 7)) = w;
                    }
                }
                if (!(amax <= 65504.0f) && live && ok) atomicCAS(p.status, 0, kStatusRange);
            } else {
                // v: row = feature of head `half`, columns = the tile's tokens
                const float bv = sh->bias[half * 128 + row];
                float vmax = 0.f;
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
                            x[i] = (ok && n < p.n_tokens) ? __uint_as_float(a[c8 * 8 + i]) + bv : 0.f;  // padding columns zero
                            vmax = fmaxf(vmax, fabsf(x[i]));
                        }
                        uint4 w;
                        w.x = pack_f16x2(x[0], x[1]);
                        w.y = pack_f16x2(x[2], x[3]);
                        w.z = pack_f16x2(x[4], x[5]);
                        w.w = pack_f16x2(x[6], x[7]);
                        const int col = cb * 32 + c8 * 8;
                        *reinterpret_cast<uint4*>(my_stage + (col >> 6) * kOutBlockBytes + sw128_offset(row, (col >> 3) & 7)) = w;
                    }
                }
                if (!(vmax <= 65504.0f)) atomicCAS(p.status, 0, kStatusRange);
            }
            // the accumulator may be overwritten by the unit after next
            tc_fence_before();
            mbar_arrive(smem_u32(&sh->acc_empty[b]));
            fence_proxy_async_smem();
            epi_barrier();
            if (tid == 64 && ok) {
#pragma unroll
                for (int i = 0; i < kProjHeadsPerCta; ++i) {
                    const int head = pair * kProjHeadsPerCta + i;
                    const uint32_t src = smem_u32(stage_out + i * kOutTileBytes);
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
            }
        }
        if (tid == 64) tma_store_wait_read();
        __syncwarp();
    }

    // ---------------------------------------------------------------- tear-down
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        if (sh->abort_flag) {
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

cudaError_t configure_qkv_project() {
    cudaError_t e = cudaFuncSetAttribute(qkv_project_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kProjSmem);
    return e;
}

cudaError_t launch_qkv_project(const CUtensorMap& tmap_x, const CUtensorMap& tmap_w, const CUtensorMap& tmap_q,
                               const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, const ProjParams& p,
                               int sm_count, cudaStream_t stream) {
    const int n_units = 3 * ((p.n_tokens + kTile - 1) / kTile);
    const int n_slices = n_units * (p.h / kProjHeadsPerCta);
    // the counters of the units start at zero; the partial sums need no clearing (every slot is written before read)
    cudaError_t e = cudaMemsetAsync(p.unit_count, 0, (size_t)n_units * sizeof(int), stream);
    if (e != cudaSuccess) return e;
    // One CTA per SM and never more CTAs than SMs, launched cooperatively: the waits between slices rely on the whole
    // grid being resident at once, and a cooperative launch either guarantees that or fails (on a GPU whose SMs are
    // partly taken it is refused instead of running into the bounded waits).
    const int grid = n_slices < sm_count ? n_slices : sm_count;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kProjThreads);
    cfg.dynamicSmemBytes = kProjSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, qkv_project_kernel, tmap_x, tmap_w, tmap_q, tmap_k, tmap_v, p);
}

}  // namespace regenvc
