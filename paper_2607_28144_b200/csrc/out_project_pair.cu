// Output projection of the block, y = o W_o^T + b_o (bf16 in, fp32 accumulation, bf16 out), on pairs of CTAs
// (clusters of two, tcgen05 cta_group::2): the step behind the attention in the backbone the paper takes by reference
// (Sec. 3.2 / 3.4).  o is the attention output exactly as the attention kernels write it: [N, C] with the heads of a
// token side by side.
//
// Why pairs.  With one CTA per tile a 128 x 256 x 16 MMA reads 12 KB of operands from shared memory in its 128
// cycles while TMA writes the next 12 KB: 192 B/clk against the 128 B/clk a shared memory delivers, and the main loop
// runs at about 0.7 of the tensor rate (the QKV projection kernel, whose long epilogue hides behind that, lives with
// it).  A pair computes a 256 x 256 tile with every CTA holding its own 128 token rows (A) and HALF of the 256
// weight rows (B): 8 KB read and 8 KB written per CTA and MMA, exactly what the shared memory can do.
//
// A slice is (pair of 128-token tiles, 256 output features); the grid is persistent, cluster c takes slices c,
// c + n_clusters, ...
//   warp 0      TMA producer of THIS CTA's operand halves; all bytes of a stage are counted on the leader's barrier
//   warp 1      leader CTA: issues the pair MMAs (M = 256 over both CTAs, N = 256) and commits to the barriers of
//               both CTAs
//   warps 2-9   epilogue of this CTA's 128 x 256 accumulator half: + bias, bf16, swizzled staging tile, tiled store;
//               one of its threads tells the leader's barrier that this CTA has read accumulator b out
// Two accumulators of 256 columns per CTA, used in turn.  (The hand-back of an accumulator first went through each
// CTA's warp 1; a release-arrive at cluster scope from the thread that issues the MMAs waits for its earlier commits,
// i.e. for the queued MMAs to finish, and left the tensor core idle for about 2 k cycles per slice.)  Every TMA load
// here reads this GPU's own memory and every CTA fetches its own tiles.
#include <cstddef>

#include "common.cuh"
#include "cta_pair.cuh"
#include "ptx.cuh"
#include "umma_desc.cuh"

namespace regenvc {

namespace {

constexpr int kBK = 64;                                  // K elements per stage: one 128-byte swizzled row
constexpr int kStages = 5;                               // (4 stages: 1-4 % slower)
constexpr int kFeat = kProjHeadsPerCta * kHeadDim;       // 256 output features per slice
constexpr uint32_t kABytes = kTile * kBK * 2;            // 16 KB: this CTA's token tile
constexpr uint32_t kBBytes = (kFeat / 2) * kBK * 2;      // 16 KB: this CTA's half of the slice's weight rows
constexpr uint32_t kStageBytes = kABytes + kBBytes;      // 32 KB per CTA and stage
constexpr int kEpiThreads = 256;
constexpr int kThreadsPair = 64 + kEpiThreads;
constexpr uint32_t kOutTileBytes = kTile * 128 * 2;      // 32 KB: [128 tokens][128 features] bf16, staged for TMA
constexpr uint32_t kOutBlockBytes = kOutTileBytes / 2;
constexpr uint64_t kWaitNs = 500000000ull;
constexpr uint32_t kIdescPair = umma_idesc_bf16_f32acc(256, 256);   // M = 256 over the two CTAs, N = 256

struct PairShared {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t acc_full[2];      // accumulator b holds a finished slice
    uint64_t acc_empty[2];     // the epilogue warps of BOTH CTAs have read accumulator b out (the leader's barrier
                               // counts; one arrival per CTA)
    uint32_t tmem_base;
    int abort_flag;
    alignas(16) float bias[kFeat];
};
constexpr uint32_t kPairSmem = kStages * kStageBytes + 2 * kOutTileBytes + 1024 /*align*/ + sizeof(PairShared);
static_assert(kPairSmem <= 232448, "shared memory of one SM");

__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }
}  // namespace

__global__ void __launch_bounds__(kThreadsPair, 1)
out_project_pair_kernel(const __grid_constant__ CUtensorMap tmap_o, const __grid_constant__ CUtensorMap tmap_w,
                        const __grid_constant__ CUtensorMap tmap_y, const ProjParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* stages = base;
    uint8_t* stage_out = base + kStages * kStageBytes;       // two [128][128] bf16 tiles for the tiled stores
    PairShared* sh = reinterpret_cast<PairShared*>(stage_out + 2 * kOutTileBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rank = static_cast<int>(cluster_rank());       // 0: leader of the pair (issues the MMAs), 1: the other CTA
    const int n_rank = p.h / kProjHeadsPerCta;               // 256-feature slices per token tile
    const int n_tiles = (p.n_tokens + kTile - 1) / kTile;
    const int n_slices = ((n_tiles + 1) / 2) * n_rank;       // slice s: token tiles 2 (s / n_rank) + {0, 1}, features
    const int slice0 = static_cast<int>(cluster_id_x());     // 256 (s % n_rank) ...
    const int slice_step = static_cast<int>(n_clusters_x());
    const int n_kb = p.C / kBK;
    const WaitCtl ctl{&sh->abort_flag, p.status, kStatusTimeout, kWaitNs};
    uint32_t tmem_base = 0;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
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
            tma_prefetch_desc(&tmap_o);
            tma_prefetch_desc(&tmap_w);
            int fill = 0;  // stages filled so far over all slices
            bool ok = true;
            for (int slice = slice0; ok && slice < n_slices; slice += slice_step) {
                const int n0 = (2 * (slice / n_rank) + rank) * kTile;            // this CTA's token tile (may lie past the end)
                const int f0 = (slice % n_rank) * kFeat + rank * (kFeat / 2);    // this CTA's half of the weight rows
                for (int kb = 0; kb < n_kb; ++kb, ++fill) {
                    const int s = fill % kStages, round = fill / kStages;
                    if (round > 0) ok = mbar_wait(smem_u32(&sh->empty[s]), (round - 1) & 1, ctl);
                    if (!ok) break;
                    // the leader announces the bytes of both CTAs on its barrier; both CTAs' loads count there
                    if (rank == 0) mbar_expect_tx(smem_u32(&sh->full[s]), 2 * kStageBytes);
                    const uint32_t full = map_to_rank(smem_u32(&sh->full[s]), 0);
                    const uint32_t dst = smem_u32(stages + s * kStageBytes);
                    tma_load_2d_pair(dst, &tmap_o, kb * kBK, n0, full);   // rows past the last token arrive as zeros
                    tma_load_2d_pair(dst + kABytes, &tmap_w, kb * kBK, f0, full);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (MMAs from the leader CTA only)
        if (elect_one()) {
            int fill = 0, it = 0;
            bool ok = true;
            for (int slice = slice0; ok && slice < n_slices; slice += slice_step, ++it) {
                const int b = it & 1;
                const uint32_t acc_tmem = tmem_base + b * kFeat;
                if (rank != 0) break;      // only the leader issues MMAs
                if (it >= 2) {
                    // accumulator b was last used two slices ago: both CTAs' epilogue warps must have read it out
                    ok = mbar_wait(smem_u32(&sh->acc_empty[b]), ((it >> 1) - 1) & 1, ctl);
                    if (!ok) break;
                    tc_fence_after();
                }
                for (int kb = 0; kb < n_kb; ++kb, ++fill) {
                    const int s = fill % kStages;
                    ok = mbar_wait(smem_u32(&sh->full[s]), (fill / kStages) & 1, ctl);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sa = smem_u32(stages + s * kStageBytes), sb = sa + kABytes;
                    const uint64_t da = umma_smem_desc_k_sw128(sa), db = umma_smem_desc_k_sw128(sb);
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk)
                        umma_ss_pair(acc_tmem, da + 2 * kk, db + 2 * kk, kIdescPair, (kb > 0 || kk > 0) ? 1u : 0u);
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
        // two threads per accumulator row (= token of this CTA's tile): thread (row, half) owns 128 of the 256 columns
        const int half = (warp - 2) >> 2;
        const int row = (warp & 3) * 32 + lane;       // accumulator row = TMEM lane
        const int et = tid - 64;                      // 0 .. 255
        uint8_t* my_stage = stage_out + half * kOutTileBytes;
        bool ok = true;
        int it = 0;
        for (int slice = slice0; slice < n_slices; slice += slice_step, ++it) {
            const int fslice = slice % n_rank, b = it & 1;
            const int tile = 2 * (slice / n_rank) + rank;
            const bool tile_live = tile < n_tiles;    // an odd tile count leaves the last pair's second CTA without one
            const uint32_t t_acc = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16) + b * kFeat + half * 128;
            // this slice's bias values (the previous slice's readers are past the barrier that closed its epilogue),
            // and the staging tiles, free once the previous slice's stores have read them (thread 64 issued them)
            sh->bias[et] = p.bias ? __ldg(p.bias + fslice * kFeat + et) : 0.0f;
            if (tid == 64) tma_store_wait_read();
            epi_barrier();
            if (ok) ok = mbar_wait(smem_u32(&sh->acc_full[b]), (it >> 1) & 1, ctl);
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();
#pragma unroll 1
            for (int cb = 0; cb < 4; ++cb) {
                uint32_t a[32];
                if (ok) {
                    tmem_ld32(t_acc + cb * 32, a);
                    tmem_wait_ld();
                }
                const float4* b4 = reinterpret_cast<const float4*>(sh->bias + half * 128 + cb * 32);
#pragma unroll
                for (int c8 = 0; c8 < 4; ++c8) {
                    const float4 b0 = b4[2 * c8], b1 = b4[2 * c8 + 1];
                    uint4 w;
                    w.x = pack_bf16x2(__uint_as_float(a[c8 * 8 + 0]) + b0.x, __uint_as_float(a[c8 * 8 + 1]) + b0.y);
                    w.y = pack_bf16x2(__uint_as_float(a[c8 * 8 + 2]) + b0.z, __uint_as_float(a[c8 * 8 + 3]) + b0.w);
                    w.z = pack_bf16x2(__uint_as_float(a[c8 * 8 + 4]) + b1.x, __uint_as_float(a[c8 * 8 + 5]) + b1.y);
                    w.w = pack_bf16x2(__uint_as_float(a[c8 * 8 + 6]) + b1.z, __uint_as_float(a[c8 * 8 + 7]) + b1.w);
                    const int col = cb * 32 + c8 * 8;
                    if (ok)
                        *reinterpret_cast<uint4*>(my_stage + (col >> 6) * kOutBlockBytes + sw128_offset(row, (col >> 3) & 7)) = w;
                }
            }
            tc_fence_before();
            fence_proxy_async_smem();
            epi_barrier();
            // every epilogue thread of this CTA has its accumulator values: tell the leader
            if (tid == 64) mbar_arrive_cluster(map_to_rank(smem_u32(&sh->acc_empty[b]), 0));
            if (tid == 64 && ok && tile_live) {
                // rows past the last token fall outside the tensor map and are dropped by the store
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const uint32_t src = smem_u32(stage_out + i * kOutTileBytes);
                    const int col = fslice * kFeat + i * 128;
                    tma_store_2d(&tmap_y, col, tile * kTile, src);
                    tma_store_2d(&tmap_y, col + 64, tile * kTile, src + kOutBlockBytes);
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

cudaError_t configure_out_project() {
    return cudaFuncSetAttribute(out_project_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmem);
}

cudaError_t launch_out_project(const CUtensorMap& tmap_o, const CUtensorMap& tmap_w, const CUtensorMap& tmap_y,
                               const ProjParams& p, int sm_count, cudaStream_t stream) {
    const int n_tiles = (p.n_tokens + kTile - 1) / kTile;
    const int n_slices = ((n_tiles + 1) / 2) * (p.h / kProjHeadsPerCta);   // work of one pair of CTAs each
    const int pairs = n_slices < sm_count / 2 ? n_slices : sm_count / 2;
    if (pairs < 1) return cudaErrorInvalidConfiguration;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (unsigned)pairs);
    cfg.blockDim = dim3(kThreadsPair);
    cfg.dynamicSmemBytes = kPairSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, out_project_pair_kernel, tmap_o, tmap_w, tmap_y, p);
}

}  // namespace regenvc
