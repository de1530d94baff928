// Producer of the attention operands on pairs of CTAs: the QKV projection of one transformer block with everything
// that stands between it and the attention kernel fused into its epilogue (the backbone the paper takes by reference,
// Sec. 3.2 / 3.4: three linear maps, an RMS norm over all features of a token on q and k, the head split and the 3D
// rotary embedding).  One pass over x and W_qkv writes
//   Q'  fp16 [N, h, 128]          normalised, rotated queries
//   K'  fp16 [h][n_pad][128]      normalised, rotated keys      } the operand layout the attention kernel streams,
//   V't fp16 [h][128][n_pad]      values, keys contiguous       } so no separate preparation pass is needed
// and nothing of q, k, v is ever rounded to bf16 or written in token-major form.
//
// A slice is (pair of 128-token tiles, one of q / k / v, 256 output features = two heads), computed by a cluster of
// two CTAs with tcgen05 cta_group::2 MMAs (M = 256 over the pair, N = 256): every CTA stages its own 128-token x tile
// and HALF of the slice's 256 weight rows, 8 KB read and 8 KB written per CTA and MMA -- what a shared memory
// delivers; with one CTA per tile it is 12 + 12 KB and the main loop runs at 0.7 of the tensor rate.  The grid is
// persistent: cluster c takes slices c, c + n_clusters, ... of the list (part-major: all token tiles of q, then k,
// then v, so that one third of W_qkv is live at a time).
//   warp 0      TMA producer of THIS CTA's operand halves (4-stage ring); all bytes of a stage count on the leader's
//               barrier.  Every load reads this GPU's own memory and every CTA fetches its own tiles.
//   warp 1      leader CTA: issues the pair MMAs and commits to the barriers of both CTAs
//   warps 2-9   epilogue of this CTA's half of the accumulator, two threads per row
// q and k: D[token][feature] = x W^T (A = x tiles, B = W halves): a CTA ends up with ITS 128 tokens x 256 features.
// v: D[feature][token] = W x^T (A = W halves, B = x tiles), which is V't directly: a CTA ends up with ONE head's 128
// features x the 256 tokens of both tiles.
// The RMS norm needs the sum of squares over ALL features of a token, which are spread over the h/2 clusters that
// hold the slices of the token tile: each CTA writes its partial row sums to a scratch array in global memory and
// counts itself in on the (token tile, part) counter; the epilogue warps (only they) wait until the counter shows all
// slices and add the partial sums in slice order, so the result does not depend on timing.  The wait is bounded like
// every other; it cannot deadlock because every cluster works through its slices in increasing order and the whole
// grid is resident (never more pairs than the device holds at once, one CTA per SM).
// An accumulator is handed back to the leader's MMA thread by ONE epilogue thread per CTA (cluster-scope arrive on the
// leader's barrier) -- not by the MMA-issuing thread itself, whose release-arrive would wait for its queued MMAs.
#include <cstddef>

#include "common.cuh"
#include "cta_pair.cuh"
#include "ptx.cuh"
#include "rope.cuh"
#include "umma_desc.cuh"

namespace regenvc {

namespace {

constexpr int kBK = 64;                                  // K elements per stage: one 128-byte swizzled row
constexpr int kProjStages = 4;
constexpr int kFeat = kProjHeadsPerCta * kHeadDim;       // 256 output features per slice
constexpr uint32_t kXBytes = kTile * kBK * 2;            // 16 KB: this CTA's token tile
constexpr uint32_t kWBytes = (kFeat / 2) * kBK * 2;      // 16 KB: this CTA's half of the slice's W rows
constexpr uint32_t kStageBytes = kXBytes + kWBytes;      // 32 KB per CTA and stage
constexpr int kEpiThreads = 256;
constexpr int kProjThreads = 64 + kEpiThreads;
constexpr uint32_t kOutTileBytes = kTile * kHeadDim * 2; // 32 KB: one head's [128][128] fp16 tile, staged for TMA
constexpr uint32_t kOutBlockBytes = kOutTileBytes / 2;
constexpr uint64_t kProjWaitNs = 500000000ull;
constexpr uint32_t kIdescPair = umma_idesc_bf16_f32acc(256, 256);   // M = 256 over the two CTAs, N = 256

struct ProjShared {
    uint64_t full[kProjStages];
    uint64_t empty[kProjStages];
    uint64_t acc_full[2];      // accumulator b holds a finished slice
    uint64_t acc_empty[2];     // the epilogue warps of BOTH CTAs have read accumulator b out (the leader's barrier
                               // counts; one arrival per CTA)
    uint32_t tmem_base;
    int abort_flag;
    alignas(16) float bias[kFeat];   // this slice's part of the bias
    alignas(16) float gain[kFeat];   //             ... of the norm gains g
    alignas(16) float gb[kFeat];     //             ... and g * bias
    float part[2][kTile];      // partial sums of squares of the two heads of this CTA
};
constexpr uint32_t kProjSmem = kProjStages * kStageBytes + kProjHeadsPerCta * kOutTileBytes + 1024 /*align*/ +
                               sizeof(ProjShared);
static_assert(kProjSmem <= 232448, "shared memory of one SM");

__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }
// A word in global memory as other CTAs have left it (read at L2, never from this SM's L1).
__device__ __forceinline__ uint32_t ld_relaxed_gpu(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

}  // namespace

__global__ void __launch_bounds__(kProjThreads, 1)
qkv_project_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                   const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                   const __grid_constant__ CUtensorMap tmap_v, const ProjParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* stages = base;
    uint8_t* stage_out = base + kProjStages * kStageBytes;   // two [128][128] fp16 tiles for the tiled stores
    ProjShared* sh = reinterpret_cast<ProjShared*>(stage_out + kProjHeadsPerCta * kOutTileBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rank = static_cast<int>(cluster_rank());       // 0: leader of the pair (issues the MMAs), 1: the other CTA
    const int n_rank = p.h / kProjHeadsPerCta;               // slices per pair of token tiles and part
    const int n_tiles = (p.n_tokens + kTile - 1) / kTile;
    const int n_tile_pairs = (n_tiles + 1) / 2;
    // slice s: part s / n_rank / n_tile_pairs (0 q, 1 k, 2 v), token tiles 2 (s / n_rank % n_tile_pairs) + {0, 1},
    // heads 2 (s % n_rank) and 2 (s % n_rank) + 1
    const int n_slices = 3 * n_tile_pairs * n_rank;
    const int slice0 = static_cast<int>(cluster_id_x()), slice_step = static_cast<int>(n_clusters_x());
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
            mbar_init(smem_u32(&sh->acc_empty[b]), 2);
        }
        sh->abort_flag = (*reinterpret_cast<volatile int*>(p.status) != 0) ? 1 : 0;
        fence_mbar_init();
    }
    __syncwarp();
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(&sh->tmem_base), 512);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    // neither CTA may count bytes on, or commit to, a barrier of the other before that one has initialised it
    cluster_sync_all();
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
                const int pair = slice % n_rank, tp = (slice / n_rank) % n_tile_pairs, part = slice / n_rank / n_tile_pairs;
                const int n0 = (2 * tp + rank) * kTile;   // this CTA's token tile (may lie past the last token)
                const int f0 = part * p.C + pair * kFeat + rank * (kFeat / 2);   // this CTA's half of the W rows
                for (int kb = 0; kb < n_kb; ++kb, ++fill) {
                    const int s = fill % kProjStages, round = fill / kProjStages;
                    if (round > 0) ok = mbar_wait(smem_u32(&sh->empty[s]), (round - 1) & 1, ctl);
                    if (!ok) break;
                    // the leader announces the bytes of both CTAs on its barrier; both CTAs' loads count there
                    if (rank == 0) mbar_expect_tx(smem_u32(&sh->full[s]), 2 * kStageBytes);
                    const uint32_t full = map_to_rank(smem_u32(&sh->full[s]), 0);
                    const uint32_t dst = smem_u32(stages + s * kStageBytes);
                    tma_load_2d_pair(dst, &tmap_x, kb * kBK, n0, full);   // rows past the last token arrive as zeros
                    tma_load_2d_pair(dst + kXBytes, &tmap_w, kb * kBK, f0, full);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (the leader CTA only)
        if (rank == 0 && elect_one()) {
            int fill = 0, it = 0;
            bool ok = true;
            for (int slice = slice0; ok && slice < n_slices; slice += slice_step, ++it) {
                const int part = slice / n_rank / n_tile_pairs, b = it & 1;
                const uint32_t acc_tmem = tmem_base + b * kFeat;
                // the accumulator must have been read out by both CTAs' epilogues of the slice before last
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
                        if (part < 2) umma_ss_pair(acc_tmem, dx + 2 * kk, dw + 2 * kk, kIdescPair, acc);   // tokens x features
                        else umma_ss_pair(acc_tmem, dw + 2 * kk, dx + 2 * kk, kIdescPair, acc);             // features x tokens
                    }
                    // the stage is free in both CTAs once these MMAs have read it
                    umma_commit_pair(smem_u32(&sh->empty[s]));
                    umma_commit_pair(map_to_rank(smem_u32(&sh->empty[s]), 1));
                }
                if (ok) {
                    umma_commit_pair(smem_u32(&sh->acc_full[b]));
                    umma_commit_pair(map_to_rank(smem_u32(&sh->acc_full[b]), 1));
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        // q, k: row = token of this CTA's tile, half = which of the slice's two heads
        // v   : row = feature of this CTA's head 2 pair + rank, half = which of the pair's two token tiles
        const int half = (warp - 2) >> 2;
        const int row = (warp & 3) * 32 + lane;       // accumulator row = TMEM lane
        const int et = tid - 64;                      // 0 .. 255
        uint8_t* my_stage = stage_out + half * kOutTileBytes;
        bool ok = true;
        int it = 0;
        // this thread's bias value and norm gain of a slice, requested one slice ahead
        float bias_next = 0.f, gain_next = 1.f;
        auto fetch_bias_gain = [&](int sl) {
            const int pr = sl % n_rank, pt = sl / n_rank / n_tile_pairs;
            bias_next = p.bias ? __ldg(p.bias + pt * p.C + pr * kFeat + et) : 0.0f;
            const float* g = pt == 0 ? p.g_q : p.g_k;
            gain_next = (pt < 2 && g) ? __ldg(g + pr * kFeat + et) : 1.0f;
        };
        if (slice0 < n_slices) fetch_bias_gain(slice0);
        for (int slice = slice0; slice < n_slices; slice += slice_step, ++it) {
            const int pair = slice % n_rank, tp = (slice / n_rank) % n_tile_pairs, part = slice / n_rank / n_tile_pairs;
            const int b = it & 1;
            const int tile = 2 * tp + rank, n0 = tile * kTile;   // q, k: this CTA's own token tile
            const bool normed = part < 2 && tile < n_tiles;      // an odd tile count leaves the last pair's second CTA
            const int unit = part * n_tiles + tile;              // without one; (token tile, part): the norm's exchange
            const uint32_t t_acc = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16) + b * kFeat + half * 128;
            // this unit's slice of the bias and of the norm gains (the previous unit's readers are past the barrier
            // that closed its epilogue)
            sh->bias[et] = bias_next;
            sh->gain[et] = gain_next;
            sh->gb[et] = gain_next * bias_next;
            epi_barrier();
            if (slice + slice_step < n_slices) fetch_bias_gain(slice + slice_step);
            if (ok) ok = mbar_wait(smem_u32(&sh->acc_full[b]), (it >> 1) & 1, ctl);
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();

            float inv_rms = 1.0f;
            if (normed) {
                // pass 1: this thread's share of the sum of squares of its token's features
                float ss = 0.f, ss2 = 0.f;
                if (ok) {
#pragma unroll 1
                    for (int cb = 0; cb < 4; ++cb) {
                        uint32_t a[32];
                        tmem_ld32(t_acc + cb * 32, a);
                        tmem_wait_ld();
                        const float4* b4 = reinterpret_cast<const float4*>(sh->bias + half * 128 + cb * 32);
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const float4 bb = b4[c];
                            const float y0 = __uint_as_float(a[4 * c]) + bb.x, y1 = __uint_as_float(a[4 * c + 1]) + bb.y;
                            const float y2 = __uint_as_float(a[4 * c + 2]) + bb.z, y3 = __uint_as_float(a[4 * c + 3]) + bb.w;
                            ss = fmaf(y0, y0, ss);
                            ss2 = fmaf(y1, y1, ss2);
                            ss = fmaf(y2, y2, ss);
                            ss2 = fmaf(y3, y3, ss2);
                        }
                    }
                }
                sh->part[half][row] = ss + ss2;
                epi_barrier();
                // Publish this slice's partial sum of every token.  The scratch array starts out as all-ones bit
                // patterns (set by the launcher); a slot that holds anything else has been written, so the value is its
                // own flag: no counter, no fence, one trip to L2 for the writer and one for each reader.
                if (half == 0) {
                    uint32_t bits = __float_as_uint(sh->part[0][row] + sh->part[1][row]);
                    if (bits == 0xffffffffu) bits = 0x7fffffffu;   // keep the "unwritten" pattern out of the data
                    __stcg(reinterpret_cast<uint32_t*>(p.unit_sums) + ((size_t)unit * n_rank + pair) * kTile + row, bits);
                }
                // wait until all slices of the unit are in, then add them in slice order (the same sum whatever the
                // timing)
                float total = 0.f;
                {
                    const uint32_t* src = reinterpret_cast<const uint32_t*>(p.unit_sums) + (size_t)unit * n_rank * kTile + row;
                    uint64_t t0 = 0;
                    uint32_t spins = 0;
                    while (ok) {
                        bool all = true;
                        total = 0.f;
                        for (int r = 0; r < n_rank; ++r) {
                            const uint32_t v = ld_relaxed_gpu(src + (size_t)r * kTile);
                            all = all && v != 0xffffffffu;
                            total += __uint_as_float(v);
                        }
                        if (all) break;
                        __nanosleep(32);
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
                ok = __all_sync(0xffffffffu, ok);
                inv_rms = rsqrtf(total / static_cast<float>(p.C) + p.eps);
            }

            // the staging tiles are free once the previous unit's stores have read them (thread 64 issued them)
            if (tid == 64) tma_store_wait_read();
            epi_barrier();
            if (normed) {
                const int n = n0 + row;
                const bool live = n < p.n_tokens;
                const TokenPos pos = token_pos(live ? n : 0, p.grid);
                // Everything that multiplies a whole row goes into the (cos, sin) pair: 1 / rms, and zero for rows past
                // the last token (the padding rows of K' are zero).  With u = acc * g + g * bias (one FMA per element)
                // the rotated, normalised pair is (ua c' - ub s', ua s' + ub c'), c' = c / rms, s' = s / rms.
                const float row_scale = (live && ok) ? inv_rms : 0.f;
                const uint64_t scale2 = pack2(row_scale, row_scale);
                uint32_t hmax = 0;  // largest fp16 magnitude bits of this row (per 16-bit half), for the range check
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
                    for (int i = 0; i < 16; ++i) {
                        float c, sn;
                        unpack2(fma2(pack2(cs_next[i].x, cs_next[i].y), scale2, 0ull), c, sn);
                        cs[i] = make_float2(c, sn);
                    }
                    if (cb + 1 < 4) fetch_cs(cb + 1, cs_next);
                    uint32_t a[32];
                    if (ok) {
                        tmem_ld32(t_acc + cb * 32, a);
                        tmem_wait_ld();
                    }
                    const float4* g4 = reinterpret_cast<const float4*>(sh->gain + half * 128 + cb * 32);
                    const float4* gb4 = reinterpret_cast<const float4*>(sh->gb + half * 128 + cb * 32);
#pragma unroll
                    for (int c8 = 0; c8 < 4; ++c8) {
                        const float4 g0 = g4[2 * c8], g1 = g4[2 * c8 + 1], b0 = gb4[2 * c8], b1 = gb4[2 * c8 + 1];
                        const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
                        const float gb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
                        uint32_t wv[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {  // pair (2i, 2i + 1) of this 8-column piece turns by its angle
                            const float ua = fmaf(__uint_as_float(a[c8 * 8 + 2 * i]), g[2 * i], gb[2 * i]);
                            const float ub = fmaf(__uint_as_float(a[c8 * 8 + 2 * i + 1]), g[2 * i + 1], gb[2 * i + 1]);
                            const float2 w2 = cs[c8 * 4 + i];
                            wv[i] = pack_f16x2(ua * w2.x - ub * w2.y, ua * w2.y + ub * w2.x);
                            hmax = __vmaxu2(hmax, wv[i] & 0x7fff7fffu);
                        }
                        const int col = cb * 32 + c8 * 8;
                        *reinterpret_cast<uint4*>(my_stage + (col >> 6) * kOutBlockBytes + sw128_offset(row, (col >> 3) & 7)) =
                            make_uint4(wv[0], wv[1], wv[2], wv[3]);
                    }
                }
                // a result that rounds to infinity (or is not a number) is beyond the fp16 range
                if (((hmax & 0xffffu) > 0x7bffu || (hmax >> 16) > 0x7bffu) && live && ok) atomicCAS(p.status, 0, kStatusRange);
            } else if (part == 2) {
                // v: row = feature of this CTA's head, columns = the tokens of tile 2 tp + half
                const float bv = sh->bias[rank * 128 + row];
                const int nv0 = (2 * tp + half) * kTile;
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
                            const int n = nv0 + cb * 32 + c8 * 8 + i;
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
            tc_fence_before();
            fence_proxy_async_smem();
            epi_barrier();
            // every epilogue thread of this CTA is done with the accumulator: it may be overwritten by the slice after
            // next once the other CTA has said the same
            if (tid == 64) mbar_arrive_cluster(map_to_rank(smem_u32(&sh->acc_empty[b]), 0));
            if (tid == 64 && ok) {
#pragma unroll
                for (int i = 0; i < kProjHeadsPerCta; ++i) {
                    const uint32_t src = smem_u32(stage_out + i * kOutTileBytes);
                    if (part < 2) {
                        if (tile >= n_tiles) continue;
                        const int head = pair * kProjHeadsPerCta + i;   // staging tile i = head i of the slice
                        if (part == 0) {
                            tma_store_2d(&tmap_q, head * kHeadDim, n0, src);
                            tma_store_2d(&tmap_q, head * kHeadDim + 64, n0, src + kOutBlockBytes);
                        } else {
                            tma_store_2d(&tmap_k, 0, head * p.n_pad + n0, src);
                            tma_store_2d(&tmap_k, 64, head * p.n_pad + n0, src + kOutBlockBytes);
                        }
                    } else {
                        if (2 * tp + i >= n_tiles) continue;
                        const int head = pair * kProjHeadsPerCta + rank;   // staging tile i = token tile 2 tp + i
                        tma_store_2d(&tmap_v, (2 * tp + i) * kTile, head * kHeadDim, src);
                        tma_store_2d(&tmap_v, (2 * tp + i) * kTile + 64, head * kHeadDim, src + kOutBlockBytes);
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
    // both CTAs are done with each other's barriers and tensor memory before either releases it or exits
    cluster_sync_all();
    if (warp == 1) {
        __syncwarp();
        if (sh->abort_flag) {
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
        __syncwarp();
        tmem_dealloc_pair(tmem_base, 512);
    }
}

cudaError_t configure_qkv_project_pair() {
    return cudaFuncSetAttribute(qkv_project_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kProjSmem);
}

cudaError_t launch_qkv_project_pair(const CUtensorMap& tmap_x, const CUtensorMap& tmap_w, const CUtensorMap& tmap_q,
                                    const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, const ProjParams& p,
                                    int sm_count, cudaStream_t stream) {
    const int n_tiles = (p.n_tokens + kTile - 1) / kTile;
    const int n_slices = 3 * ((n_tiles + 1) / 2) * (p.h / kProjHeadsPerCta);   // work of one pair of CTAs each
    // every slot of the partial sums starts as the "unwritten" pattern
    cudaError_t e = cudaMemsetAsync(p.unit_sums, 0xff, (size_t)3 * n_tiles * (p.h / kProjHeadsPerCta) * kTile * sizeof(float),
                                    stream);
    if (e != cudaSuccess) return e;
    // Pairs of CTAs, one CTA per SM, and never more pairs than the device holds at once: the waits between slices rely
    // on the whole grid being resident.  (The cooperative launch attribute, which would have the driver guarantee
    // that, was tried: with it this kernel fails to launch under the profiler.  On a device shared with other work
    // part of the grid may stay out; the waits then run out and the sticky status reports it.)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (unsigned)(sm_count / 2));
    cfg.blockDim = dim3(kProjThreads);
    cfg.dynamicSmemBytes = kProjSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // how many pairs the device can hold at once (fewer than SMs / 2 where a GPC has an odd number of free SMs)
    int resident = 0;
    e = cudaOccupancyMaxActiveClusters(&resident, qkv_project_pair_kernel, &cfg);
    if (e != cudaSuccess) return e;
    const int pairs = n_slices < resident ? n_slices : resident;
    if (pairs < 1) return cudaErrorInvalidConfiguration;
    cfg.gridDim = dim3(2 * (unsigned)pairs);
    return cudaLaunchKernelEx(&cfg, qkv_project_pair_kernel, tmap_x, tmap_w, tmap_q, tmap_k, tmap_v, p);
}

}  // namespace regenvc
