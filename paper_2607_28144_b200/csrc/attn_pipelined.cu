// Pipelined, warp-specialised tcgen05 attention kernel for sm_100a.
//
// One CTA owns one head, two 128-row query tiles (256 query rows) and a range of key tiles:
//   warps 0-15 softmax (kSplit = 4): warp w works on TMEM lanes (query rows) 32*(w%4).. and on key columns
//              32*(w/4)..+31 of every score tile, so four threads share a score row; all sixteen warps take
//              the score tiles of the two query tiles in turn (S0(j), S1(j), S0(j+1), ...)
//   warp  16   UMMA issuer (one elect.sync-elected lane) and TMEM owner
//   warp  17   TMA producer (one elected lane): streams K' and V't tiles into a 4-slot ring
//   warps 18-19 idle (they complete the control warpgroup, which hands registers to the softmax warps)
// (kSplit = 2 builds the same kernel with eight softmax warps and two threads per row.)
// While the softmax warps turn S_t into P_t the tensor core runs the other tile's P.V and next Q.K^T.
//
// Tensor memory (512 columns x 128 lanes, fp32 cells):
//   [0,128) S0  [128,256) S1  [256,384) O0  [384,512) O1.  P_t (fp16, two keys per cell) aliases S_t: the
//   probabilities of keys [c, c + 32) go to the first 16 of the score columns [c, c + 32), i.e. each thread
//   writes its probabilities over score columns it has already read itself.
// Shared memory: Q0, Q1 (32 KB each, rotated, fp16, 128B-swizzled K-major blocks; reused as the staging buffer
// of the finished output tile), then a ring of kStages 32 KB slots holding K'_0, V't_0, K'_1, ...
//
// Softmax keeps, per row, a reference m (log2 domain) and a row sum l.  m is set from the first tile's row
// maximum (plus kRefMargin of headroom) and afterwards only raised when a probability would leave the fp16 range
// (p = 2^(s - m) > 65504), so the probabilities of a tile are formed directly against the reference of the earlier tiles as soon as
// the scores arrive.  A saturated probability shows in the fp32 sum of its thread's part of the row.
// The CTA first runs its key tiles OPTIMISTICALLY: every thread only remembers whether any of its sums
// saturated, nothing is exchanged per tile (the per-tile agreement of the four warps that share 32 rows cost
// 3.6 % of the kernel although it practically never fires), and at the end of the item one OR-reduction over
// the softmax warps says whether the pass was clean.  If it was not, the result of the pass is discarded and
// the whole item is run again CAREFULLY: one named barrier with an OR-reduction per tile lets the warps of a
// row group agree on a saturation at once, the row maximum is taken, the reference raised, O rescaled and the
// tile redone.  The control warps learn the verdict through an mbarrier and stream the tiles a second time.
#include "common.cuh"
#include "attn_core.cuh"
#include "rope.cuh"

#include <type_traits>

namespace regenvc {


namespace {

constexpr int kStages = 4;                       // K/V ring slots (32 KB each)
constexpr uint32_t kSmemBytes = (2 + kStages) * kTileBytes + 1024 /*align*/ + 256 /*barriers*/ + 8192 /*row exchange*/;

struct Barriers {
    uint64_t kv_full[kStages];
    uint64_t kv_empty[kStages];
    uint64_t q_full[2];
    uint64_t s_full[2];
    uint64_t p_full[2];
    uint64_t o_full[2];
    uint64_t verdict;        // the softmax warps have judged the optimistic pass (second_pass is valid)
    uint32_t tmem_base;
    int abort_flag;
    int second_pass;         // 1: a probability saturated in the optimistic pass, the item is run again
};
static_assert(sizeof(Barriers) <= 256, "barrier block too large");

}  // namespace

// kQTma = false: the softmax warps fetch the bf16 query rows, rotate them and write the fp16 tiles themselves.
// kQTma = true : the query tiles are already in operand form in global memory (16-bit, same type as K', token-major)
//                and the TMA warp copies them; the softmax warps go straight to the first score tile.
template <bool kQTma>
__global__ void __launch_bounds__(kThreads, 1)
attn_pipelined_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                      const __grid_constant__ CUtensorMap tmap_out, const __grid_constant__ CUtensorMap tmap_q,
                      const AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = base;                       // 2 tiles
    uint8_t* sKV = base + 2 * kTileBytes;     // ring
    Barriers* bar = reinterpret_cast<Barriers*>(base + (2 + kStages) * kTileBytes);
    RowExchange* xch = reinterpret_cast<RowExchange*>(base + (2 + kStages) * kTileBytes + 256);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint32_t tmem_base = 0;
    const WaitCtl ctl{&bar->abort_flag, p.status, kStatusTimeout, kWaitLimitNs};
    // work item and key-tile range of this CTA
    const int n_tiles_total = p.n_kv_pad / kTile;
    int item = blockIdx.x, kv_tile0 = 0, n_tiles = n_tiles_total;
    const bool piece = static_cast<int>(blockIdx.x) >= p.n_full_items;  // one of several key-range pieces of an item
    const bool partial = piece || p.tok_o != nullptr;                     // leaves an unnormalised result
    const int piece_cta = static_cast<int>(blockIdx.x) - p.n_full_items;
    if (piece) {
        item = p.n_full_items + piece_cta / p.split_k;
        kv_tile0 = (piece_cta % p.split_k) * p.tiles_per_piece;
        n_tiles = min(p.tiles_per_piece, n_tiles_total - kv_tile0);
    }
    const int head = item / p.pairs_per_head;
    const int q0 = (item % p.pairs_per_head) * 2 * kTile;
    const bool tile1_active = q0 + kTile < p.n_q;

    // Set-up is the control warpgroup's: barriers, tensor memory, descriptor prefetch.  The softmax warps do not
    // wait for it: they fetch and rotate their query tiles first and meet the control warps at barrier 7 afterwards.
    if (warp >= kMmaWarp) {
      setmaxnreg_dec<kControlRegs>();
      if (tid == kMmaWarp * 32) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&bar->kv_full[s]), 1);
            mbar_init(smem_u32(&bar->kv_empty[s]), 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_u32(&bar->q_full[t]), kQTma ? 1 : kSoftmaxThreads);
            mbar_init(smem_u32(&bar->s_full[t]), 1);
            mbar_init(smem_u32(&bar->p_full[t]), kSoftmaxThreads);
            mbar_init(smem_u32(&bar->o_full[t]), 1);
        }
        mbar_init(smem_u32(&bar->verdict), 1);
        // a sticky error from an earlier kernel makes this CTA skip its work (every bounded wait falls through)
        bar->abort_flag = (*reinterpret_cast<volatile int*>(p.status) != 0) ? 1 : 0;
        fence_mbar_init();
      }
      __syncwarp();
      if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(&bar->tmem_base), 512);
        tmem_relinquish();
      }
      if (warp == kTmaWarp && elect_one()) {
        tma_prefetch_desc(&tmap_k);
        tma_prefetch_desc(&tmap_v);
        tma_prefetch_desc(&tmap_out);
        if (kQTma) tma_prefetch_desc(&tmap_q);
      }
      __syncwarp();
      tc_fence_before();
      control_barrier();                 // the four control warps: set-up is complete
      tc_fence_after();
      setup_done_arrive();               // ... and the softmax warps may rely on it (they wait at barrier 7)
      tmem_base = bar->tmem_base;
      if (warp == kTmaWarp) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            if (kQTma) {
                // rows past n_q lie outside the tensor map and arrive as zeros
                for (int t = 0; t < (tile1_active ? 2 : 1); ++t) {
                    const uint32_t full = smem_u32(&bar->q_full[t]);
                    const uint32_t dst = smem_u32(sQ + t * kTileBytes);
                    mbar_expect_tx(full, kTileBytes);
                    tma_load_2d(dst, &tmap_q, head * kHeadDim, q0 + t * kTile, full);
                    tma_load_2d(dst + kBlockBytes, &tmap_q, head * kHeadDim + 64, q0 + t * kTile, full);
                }
            }
            const int total = 2 * n_tiles;
            bool ok = true;
            for (int pass = 0; ok && pass < 2; ++pass) {   // the ring index runs on through the second pass
                for (int i = 0; ok && i < total; ++i) {
                    const int g = pass * total + i;
                    const int slot = g % kStages, round = g / kStages;
                    if (round > 0) ok = mbar_wait(smem_u32(&bar->kv_empty[slot]), (round - 1) & 1, ctl);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&bar->kv_full[slot]);
                    const uint32_t dst = smem_u32(sKV + slot * kTileBytes);
                    const int kv0 = (kv_tile0 + (i >> 1)) * kTile;
                    mbar_expect_tx(full, kTileBytes);
                    if ((i & 1) == 0) {
                        tma_load_2d(dst, &tmap_k, 0, head * p.n_kv_pad + kv0, full);
                        tma_load_2d(dst + kBlockBytes, &tmap_k, 64, head * p.n_kv_pad + kv0, full);
                    } else {
                        tma_load_2d(dst, &tmap_v, kv0, head * kHeadDim, full);
                        tma_load_2d(dst + kBlockBytes, &tmap_v, kv0 + 64, head * kHeadDim, full);
                    }
                }
                if (pass == 0 && ok) {
                    ok = mbar_wait(smem_u32(&bar->verdict), 0, ctl);
                    if (!ok || !*reinterpret_cast<volatile int*>(&bar->second_pass)) break;
                }
            }
        }
      } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------ UMMA issuer
        if (elect_one()) {
            const uint32_t sQ0 = smem_u32(sQ), sQ1 = smem_u32(sQ) + kTileBytes;
            const int n_active = tile1_active ? 2 : 1;
            const uint32_t idesc_qk = p.qk_bf16 ? kIdescBf16 : kIdesc;
            bool ok = mbar_wait(smem_u32(&bar->q_full[0]), 0, ctl);
            if (ok && tile1_active) ok = mbar_wait(smem_u32(&bar->q_full[1]), 0, ctl);
            // pass 0: the optimistic run; pass 1 (only after a saturation): the same tiles again.  Ring index and
            // visit count (the phases of s_full / p_full / o_full) run on through the second pass.
            for (int pass = 0; ok && pass < 2; ++pass) {
                const int g0 = pass * 2 * n_tiles, v0 = pass * n_tiles;
                ok = mbar_wait(smem_u32(&bar->kv_full[g0 % kStages]), (g0 / kStages) & 1, ctl);
                if (!ok) break;
                tc_fence_after();
                // (on the second pass the score columns are free: the last P.V of the first pass, issued earlier by
                // this thread, reads them before these MMAs run)
                for (int t = 0; t < n_active; ++t) {
                    issue_qk(tmem_base + t * 128, t ? sQ1 : sQ0, smem_u32(sKV + (g0 % kStages) * kTileBytes), idesc_qk);
                    umma_commit(smem_u32(&bar->s_full[t]));
                }
                umma_commit(smem_u32(&bar->kv_empty[g0 % kStages]));
                for (int j = 0; ok && j < n_tiles; ++j) {
                    const int iv = g0 + 2 * j + 1, ik = g0 + 2 * j + 2;
                    const int slot_v = iv % kStages, slot_k = ik % kStages;
                    const bool more = j + 1 < n_tiles;
                    ok = mbar_wait(smem_u32(&bar->kv_full[slot_v]), (iv / kStages) & 1, ctl);
                    if (ok && more) ok = mbar_wait(smem_u32(&bar->kv_full[slot_k]), (ik / kStages) & 1, ctl);
                    for (int t = 0; ok && t < n_active; ++t) {
                        ok = mbar_wait(smem_u32(&bar->p_full[t]), (v0 + j) & 1, ctl);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(tmem_base + 256 + t * 128, tmem_base + t * 128, smem_u32(sKV + slot_v * kTileBytes), j > 0);
                        umma_commit(smem_u32(&bar->o_full[t]));
                        if (more) {
                            issue_qk(tmem_base + t * 128, t ? sQ1 : sQ0, smem_u32(sKV + slot_k * kTileBytes), idesc_qk);
                            umma_commit(smem_u32(&bar->s_full[t]));
                        }
                    }
                    if (ok) {
                        umma_commit(smem_u32(&bar->kv_empty[slot_v]));
                        if (more) umma_commit(smem_u32(&bar->kv_empty[slot_k]));
                    }
                }
                if (pass == 0 && ok) {
                    ok = mbar_wait(smem_u32(&bar->verdict), 0, ctl);
                    if (!ok || !*reinterpret_cast<volatile int*>(&bar->second_pass)) break;
                }
            }
        }
      }
    } else {
        // ------------------------------------------------------------ softmax groups
        setmaxnreg_inc<kSoftmaxRegs>();
        const int part = warp >> 2;                      // which kColsPerThread key columns of a score row
        const int row = (warp & 3) * 32 + lane;          // row in the tile == TMEM lane
        const int n_active = tile1_active ? 2 : 1;
        if (!kQTma) {
            if (tile1_active) load_rotate_q_tiles<kSoftmaxThreads, 2>(p, head, q0, sQ, tid);
            else load_rotate_q_tiles<kSoftmaxThreads, 1>(p, head, q0, sQ, tid);
            fence_proxy_async_smem();
        }
        setup_done_wait();   // barriers and tensor memory exist from here on
        tc_fence_after();
        tmem_base = bar->tmem_base;
        if (!kQTma)
            for (int t = 0; t < n_active; ++t) mbar_arrive(smem_u32(&bar->q_full[t]));
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const float scale = p.scale_log2;
        const uint64_t scale2 = pack2(scale, scale);
        const uint32_t opaque_zero = static_cast<uint32_t>(p.n_kv) >> 31;  // 0, but not to the compiler
        float m_ref[2], l_run[2];
        bool ok = true;  // false once a wait expired: keep the loop structure (named barriers) but skip the work
        bool sat = false;  // optimistic pass: one of this thread's partial row sums saturated
        // the one key tile of the sequence that is partly padding (if this CTA has it), and how many of this
        // thread's columns of that tile are real keys
        const int j_ragged = (p.n_kv % kTile != 0 && kv_tile0 + n_tiles == n_tiles_total) ? n_tiles - 1 : -1;
        const int valid_last = p.n_kv - (n_tiles_total - 1) * kTile - part * kColsPerThread;

        // One pass over the CTA's key tiles.  kCareful = false: optimistic (see the header), saturation is only
        // recorded in `sat`; true: the warps of a row group agree per tile and redo a saturated tile against a higher
        // reference.  v0: visits done before this pass (the phases of s_full / p_full / o_full run on).
        auto run_pass = [&](auto careful_tag, const int v0) {
          constexpr bool kCareful = decltype(careful_tag)::value;
          m_ref[0] = m_ref[1] = -INFINITY;
          l_run[0] = l_run[1] = 0.f;
          for (int j = 0; j < n_tiles; ++j) {
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                if (t >= n_active) continue;
                const uint32_t t_S = lane_base + t * 128 + part * kColsPerThread;
                const uint32_t t_O = lane_base + 256 + t * 128 + part * kColsPerThread;
                if (ok) ok = mbar_wait(smem_u32(&bar->s_full[t]), (v0 + j) & 1, ctl);
                ok = __all_sync(0xffffffffu, ok);  // keep the warp-wide TMEM instructions below convergent
                tc_fence_after();
                // From the second tile on, the probabilities of each 32-column chunk are formed as soon as it
                // arrives, against the reference m_ref of the earlier tiles; no maximum is taken.  Probabilities
                // saturate at 65504 when rounded to fp16, and a saturated one makes the fp32 sum of its part reach
                // 65504.  Optimistic pass: the thread remembers it.  Careful pass: the threads of the row group agree
                // on it; only then (and on the first tile of either pass) the row maximum is taken, the reference
                // raised, O rescaled and the tile redone.
                uint32_t sr[kColsPerThread];
                uint64_t negm2 = pack2(-m_ref[t], -m_ref[t]);
                uint64_t sum_a = 0, sum_b = 0;  // packed partial row sums
                const bool stream = j > 0;
                if (ok) {
                    tmem_ld32(t_S, sr);
#pragma unroll
                    for (int cb = 0; cb < kChunks; ++cb) {
                        tmem_wait_ld();
                        if (cb + 1 < kChunks) tmem_ld32(t_S + 32 * (cb + 1), sr + 32 * (cb + 1));
                        if (j == j_ragged) {  // the sequence's last, partly padded key tile
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (cb * 32 + c >= valid_last) sr[cb * 32 + c] = 0xff800000u;  // -inf
                        }
                        if (stream) {
                            uint32_t pr[16];
                            exp_chunk<kPolyMask>(sr + cb * 32, scale2, negm2, pr, sum_a, sum_b, opaque_zero);
                            tmem_st16(t_S + cb * 16, pr);
                        }
                    }
                }
                float part_sum;
                {
                    float s0, s1;
                    unpack2(add2(sum_a, sum_b), s0, s1);
                    part_sum = s0 + s1;
                }
                // Careful pass: one barrier with an OR-reduction tells the threads sharing these 32 rows whether any
                // part of any row saturated (or this is the first tile); only then do they exchange anything.
                bool any_redo;
                if (kCareful) {
                    any_redo = row_group_any(warp & 3, !stream || !(part_sum < 65504.0f));
                } else {
                    any_redo = !stream;                               // uniform over the CTA
                    if (stream) sat |= !(part_sum < 65504.0f);
                }
                if (any_redo) {
                    // Rare after the first tile.  All threads of the row group take this branch together: row
                    // maximum, a higher reference for the rows whose maximum exceeds theirs, rescale of this
                    // thread's part of the O row and of its row sum, then the probabilities against the reference.
                    float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                    for (int c = 0; c < kColsPerThread; c += 8) {
                        mx0 = max3(mx0, __uint_as_float(sr[c + 0]), __uint_as_float(sr[c + 1]));
                        mx1 = max3(mx1, __uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3]));
                        mx2 = max3(mx2, __uint_as_float(sr[c + 4]), __uint_as_float(sr[c + 5]));
                        mx3 = max3(mx3, __uint_as_float(sr[c + 6]), __uint_as_float(sr[c + 7]));
                    }
                    const float mx_part = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                    xch->m[t][row][part] = mx_part;
                    row_group_barrier(warp & 3);
                    float mx_row = mx_part;
#pragma unroll
                    for (int o = 1; o < kSplit; ++o) mx_row = fmaxf(mx_row, xch->m[t][row][(part + o) % kSplit]);
                    row_group_barrier(warp & 3);  // everyone has read xch->m before a later redo overwrites it
                    const float m_tile = mx_row * scale + kRefMargin;
                    const bool raise = m_tile > m_ref[t];  // always on the first tile (reference starts at -inf)
                    if (j > 0) {
                        if (ok) ok = mbar_wait(smem_u32(&bar->o_full[t]), (v0 + j - 1) & 1, ctl);
                        ok = __all_sync(0xffffffffu, ok);
                        tc_fence_after();
                        const float alpha = raise ? ex2_approx(m_ref[t] - m_tile) : 1.0f;
                        l_run[t] *= alpha;
                        if (ok) {
#pragma unroll 1
                            for (int cb = 0; cb < kChunks; ++cb) {
                                uint32_t o[32];
                                tmem_ld32(t_O + cb * 32, o);
                                tmem_wait_ld();
#pragma unroll
                                for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                                tmem_st32(t_O + cb * 32, o);
                            }
                        }
                    }
                    if (raise) m_ref[t] = m_tile;
                    negm2 = pack2(-m_ref[t], -m_ref[t]);
                    sum_a = 0;
                    sum_b = 0;
                    if (ok) {
#pragma unroll
                        for (int cb = 0; cb < kChunks; ++cb) {
                            uint32_t pr[16];
                            exp_chunk<kPolyMask>(sr + cb * 32, scale2, negm2, pr, sum_a, sum_b, opaque_zero);
                            tmem_st16(t_S + cb * 16, pr);
                        }
                    }
                }
                float s0, s1;
                unpack2(add2(sum_a, sum_b), s0, s1);
                l_run[t] += s0 + s1;
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&bar->p_full[t]));
            }
          }
        };
        run_pass(std::false_type{}, 0);
        // verdict on the optimistic pass, for these warps and (through the mbarrier) for the control warps
        const bool again = softmax_any(sat);
        if (tid == 0) {
            bar->second_pass = again ? 1 : 0;
            mbar_arrive(smem_u32(&bar->verdict));
        }
        if (again) run_pass(std::true_type{}, n_tiles);
        const int v_last = (again ? 2 : 1) * n_tiles - 1;   // the visit whose P.V the epilogue waits for

        // epilogue: O / l -> bf16 -> out; each thread owns kColsPerThread of the 128 output columns of its row
        for (int t = 0; t < n_active; ++t) {
            xch->l[t][row][part] = l_run[t];
            softmax_barrier();
            float l_row = 0.f;
#pragma unroll
            for (int o = 0; o < kSplit; ++o) l_row += xch->l[t][row][o];
            const float inv_l = 1.0f / l_row;
            if (ok) ok = mbar_wait(smem_u32(&bar->o_full[t]), v_last & 1, ctl);
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();
            const uint32_t t_O = lane_base + 256 + t * 128 + part * kColsPerThread;
            const int n_row = q0 + t * kTile + row;  // query row of this thread
            if (partial && part == 0) {
                if (piece) p.part_ml[(size_t)piece_cta * 2 * kTile + t * kTile + row] = make_float2(m_ref[t], l_row);
                else if (n_row < p.n_q) p.tok_ml[(size_t)n_row * p.h + head] = make_float2(m_ref[t], l_row);
            }
#pragma unroll 1
            for (int cb = 0; cb < kChunks; ++cb) {
                uint32_t o[32];
                if (ok) {
                    tmem_ld32(t_O + cb * 32, o);
                    tmem_wait_ld();
                }
                if (ok && partial) {
                    // unnormalised fp32 row part for a merge kernel: piece scratch, or the caller's token-major buffer
                    float* row_o = piece ? p.part_o + ((size_t)piece_cta * 2 * kTile + t * kTile + row) * kHeadDim
                                         : p.tok_o + ((size_t)n_row * p.h + head) * kHeadDim;
                    uint4* dst = reinterpret_cast<uint4*>(row_o + part * kColsPerThread + cb * 32);
                    if (piece || n_row < p.n_q) {
#pragma unroll
                        for (int c = 0; c < 8; ++c) dst[c] = make_uint4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]);
                    }
                } else if (ok) {
                    // normalised bf16 row part into the (now idle) query tile buffer, in the swizzled layout of a
                    // TMA box {64 columns, 128 rows}; one tiled store per 64-column block writes the tile out
                    uint8_t* stage = sQ + t * kTileBytes;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(o[8 * c + 0]) * inv_l, __uint_as_float(o[8 * c + 1]) * inv_l);
                        w.y = pack_bf16x2(__uint_as_float(o[8 * c + 2]) * inv_l, __uint_as_float(o[8 * c + 3]) * inv_l);
                        w.z = pack_bf16x2(__uint_as_float(o[8 * c + 4]) * inv_l, __uint_as_float(o[8 * c + 5]) * inv_l);
                        w.w = pack_bf16x2(__uint_as_float(o[8 * c + 6]) * inv_l, __uint_as_float(o[8 * c + 7]) * inv_l);
                        const int col = part * kColsPerThread + cb * 32 + c * 8;  // first of 8 output columns
                        *reinterpret_cast<uint4*>(stage + (col >> 6) * kBlockBytes + sw128_offset(row, (col >> 3) & 7)) = w;
                    }
                }
            }
            if (!partial) {
                fence_proxy_async_smem();
                softmax_barrier();
                if (tid == 0 && ok) {
                    const uint32_t src = smem_u32(sQ + t * kTileBytes);
                    tma_store_2d(&tmap_out, head * kHeadDim, q0 + t * kTile, src);
                    tma_store_2d(&tmap_out, head * kHeadDim + 64, q0 + t * kTile, src + kBlockBytes);
                    tma_store_commit();
                }
            }
        }
        // the tiled stores read shared memory asynchronously: they must be done before the CTA may exit
        if (tid == 0 && !partial) tma_store_wait_read();
        __syncwarp();
    }

    // ---------------------------------------------------------------- tear-down
    __syncwarp();  // lanes that left a single-lane role loop rejoin before the warp-wide instructions below
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        __syncwarp();
        if (bar->abort_flag) {
            // a wait expired: give copies and MMAs that may still be in flight time to land before TMEM is released
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}


namespace {
template <bool kQTma>
cudaError_t configure_one() {
    cudaFuncAttributes attr;
    cudaError_t e = cudaFuncGetAttributes(&attr, attn_pipelined_kernel<kQTma>);
    if (e != cudaSuccess) return e;
    // the register hand-over above assumes the kernel was compiled to exactly kLaunchRegs registers per thread
    if (attr.numRegs != kLaunchRegs) return cudaErrorInvalidConfiguration;
    return cudaFuncSetAttribute(attn_pipelined_kernel<kQTma>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)kSmemBytes);
}
}  // namespace

cudaError_t configure_attn_pipelined() {
    cudaError_t e = configure_one<false>();
    return e != cudaSuccess ? e : configure_one<true>();
}

cudaError_t launch_attn_pipelined(const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, const CUtensorMap& tmap_out,
                                  const CUtensorMap* tmap_q, const AttnParams& p, cudaStream_t stream) {
    const int n_items = p.pairs_per_head * p.h;
    dim3 grid(p.n_full_items + (n_items - p.n_full_items) * p.split_k);
    if (tmap_q)
        attn_pipelined_kernel<true><<<grid, kThreads, kSmemBytes, stream>>>(tmap_k, tmap_v, tmap_out, *tmap_q, p);
    else
        attn_pipelined_kernel<false><<<grid, kThreads, kSmemBytes, stream>>>(tmap_k, tmap_v, tmap_out, tmap_out, p);
    return cudaGetLastError();
}

}  // namespace regenvc
