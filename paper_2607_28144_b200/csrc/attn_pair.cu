// Streaming, warp-specialised tcgen05 attention kernel for sm_100a on PAIRS of CTAs (clusters of two, cta_group::2).
//
// A pair owns one head, 256 query rows and a range of key tiles; CTA r of the pair owns the query rows 128 r ..
// 128 r + 127 (its Q tile, its score / probability / output columns in ITS tensor memory, its softmax warps) and
// HALF of every K' tile (keys 64 r .. 64 r + 63) and of every V't tile (head-dim rows 64 r .. 64 r + 63).  The MMAs
// are issued by the leader (rank 0) for both CTAs: M = 256 over the pair, N = 128, each CTA supplying its 128 rows
// of A and 64 rows of B.  Per MMA a CTA then reads 6 KB (Q.K^T) or 2 KB (P.V) of shared memory instead of 8 / 4 KB,
// and TMA writes half as much: with one query tile per CTA and whole K'/V't tiles the shared memory's 128 B/clk
// bound the loop (measured 1560 clk per key tile against 1120 clk of tensor work).
//   warps 0-15 softmax (kSplit = 4): warp w works on TMEM lanes (query rows) 32*(w%4).. and on key columns
//              32*(w/4)..+31 of every score tile, so four threads share a score row
//   warp  16   leader: UMMA issuer (one elect.sync-elected lane); both CTAs: tensor-memory owner
//   warp  17   TMA producer of THIS CTA's halves (one elected lane); the bytes count on the leader's barrier
//   warps 18-19 idle (they complete the control warpgroup, which hands registers to the softmax warps)
//
// Tensor memory of each CTA (512 columns x 128 lanes, fp32 cells):
//   [0,128) S_0  [128,256) S_1  [256,384) S_2  [384,512) O
// The scores of key tile j go to S_(j%3); its probabilities (fp16, two keys per cell) overwrite them in place, every
// thread writing over score columns it has read itself.  Issue order of the tensor core: Q.K^T(0), Q.K^T(1), then,
// whenever the probabilities of tile j have been handed over: Q.K^T(j+2), P.V(j).  Scores first, so that the scores a
// softmax visit needs are complete long before it starts and the only chain left between the softmax warps and the
// tensor core is P(j) -> P.V(j).  Three buffers make that order safe without anybody waiting for it: S_((j+2)%3)
// last held the probabilities of tile j - 1, whose P.V was issued one hand-over earlier, and the MMAs complete in the
// order they are issued.  (With two score buffers and the probabilities in columns of their own the same order let
// a visit overwrite probabilities that P.V(j-2) was still reading: about one wrong tile in ten thousand calls.)
// Shared memory of each CTA: Q (32 KB, rotated, fp16, 128B-swizzled K-major blocks; reused as the staging buffer of
// the finished output tile), then a ring of kPairStages 16 KB slots (one half tile each) filled in the order the
// tensor core consumes them: K'_0, K'_1, V't_0, K'_2, V't_1, K'_3, ...
// Who tells whom: both CTAs' loads count on the leader's kv_full / q_full; every softmax warp of both CTAs arrives
// on the leader's p_full once its probabilities are in tensor memory; the leader commits s_full, o_full and
// kv_empty to both CTAs.  Every load reads this GPU's own memory, every CTA fetches its own halves.
//
// Softmax keeps, per row, a reference m (log2 domain) and a row sum l.  m is set from the first tile's row
// maximum and afterwards only raised when a probability would leave the fp16 range (p = 2^(s - m) > 65504).  As in
// attn_pipelined.cu the pair first runs its key tiles optimistically (a thread only remembers a saturated partial
// sum); the verdict is taken over both CTAs behind one cluster barrier, and after a saturation in either the pair
// runs the tiles again carefully (per-tile agreement of a row group, row maximum, rescale of O, redo of the tile).
#include "common.cuh"
#include "attn_core.cuh"
#include "cta_pair.cuh"
#include "rope.cuh"

#include <type_traits>

namespace regenvc {


namespace {

constexpr int kPairStages = 12;                  // ring slots of one half tile (16 KB) each
constexpr uint32_t kHalfBytes = kTileBytes / 2;  // this CTA's half of a K' or V't tile: two [64 rows][64] blocks
constexpr uint32_t kHalfBlockBytes = kHalfBytes / 2;
constexpr uint32_t kPairXchBytes = kTile * kSplit * 4;   // one [128 rows][kSplit] float array for every row exchange
// no alignment slack: the dynamic shared memory of a kernel without static shared memory starts on a 1024-byte
// boundary (checked at run time)
constexpr uint32_t kPairAttnSmem = kTileBytes + kPairStages * kHalfBytes + 320 /*barriers*/ + kPairXchBytes;
static_assert(kPairAttnSmem <= 232448, "shared memory of one SM");
constexpr uint32_t kPColS = 0, kPColO = 384;   // tensor-memory columns: three score buffers, then the accumulator

struct PairBarriers {
    uint64_t kv_full[kPairStages];
    uint64_t kv_empty[kPairStages];
    uint64_t q_full;
    uint64_t s_full[3];      // scores of key tile j complete: barrier j % 3, phase j / 3
    uint64_t p_full[3];      // probabilities of key tile j in tensor memory (every softmax warp of the pair): same
    uint64_t o_full[2];      // P.V(j) complete: barrier j % 2, phase j / 2
    uint32_t tmem_base;
    int abort_flag;
    int sat_flag[2];         // CTA r of the pair saw a saturated probability in the optimistic pass (read by both CTAs
                             // behind the cluster barrier that ends the pass)
};
static_assert(sizeof(PairBarriers) <= 320, "barrier block too large");
// Phase parity of a barrier that is indexed by j % kMod (s_full and p_full: 3, o_full: 2): visit j of pass `pass`
// is phase (visits with the same remainder in the first pass, if this is the second) + j / kMod.
template <int kMod>
__device__ __forceinline__ uint32_t parity_of(int pass, int j, int n_tiles) {
    const int r = j % kMod;
    const int before = pass ? (n_tiles - r + kMod - 1) / kMod : 0;   // n_tiles > r whenever visit j exists
    return static_cast<uint32_t>(before + j / kMod) & 1u;
}

constexpr uint32_t kIdescPairF16 = umma_idesc_f16_f32acc(256, 128);     // M = 256 over the two CTAs, N = 128
constexpr uint32_t kIdescPairBf16 = umma_idesc_bf16_f32acc(256, 128);

// D[tensor memory of both CTAs] (+)= A[tensor memory of both CTAs] * B[shared memory of both CTAs].
__device__ __forceinline__ void umma_ts_pair(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Commit to the same barrier of both CTAs of the pair.
__device__ __forceinline__ void commit_both(uint32_t local_bar) {
    umma_commit_pair(local_bar);
    umma_commit_pair(map_to_rank(local_bar, 1));
}
// The eight K = 16 steps of one 256 x 128 x 128 product over the pair.  A: each CTA's 128-row query tile (two
// [128][64] blocks, 16 KB apart); B: each CTA's 64 rows of the K' tile (two [64][64] blocks, 8 KB apart).
__device__ __forceinline__ void issue_qk_pair(uint32_t d_tmem, uint32_t sQ, uint32_t sK, uint32_t idesc) {
    const uint64_t a0 = umma_smem_desc_k_sw128(sQ), b0 = umma_smem_desc_k_sw128(sK);
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
        const uint64_t off_a = (kk >> 2) * (kBlockBytes >> 4) + (kk & 3) * 2;
        const uint64_t off_b = (kk >> 2) * (kHalfBlockBytes >> 4) + (kk & 3) * 2;
        umma_ss_pair(d_tmem, a0 + off_a, b0 + off_b, idesc, kk > 0);
    }
}
// P.V over the pair.  The probabilities (fp16, two keys per cell) of keys [c, c + kColsPerThread) sit in the first
// half of the score columns [c, c + kColsPerThread) of the tile's own score buffer (every thread writes them over
// scores it has read itself); B is each CTA's 64 head-dim rows of V't (two [64][64 keys] blocks, 8 KB apart).
__device__ __forceinline__ void issue_pv_pair(uint32_t d_tmem, uint32_t p_tmem, uint32_t sV, bool accumulate) {
    const uint64_t b0 = umma_smem_desc_k_sw128(sV);
    constexpr int kGroups = kColsPerThread / 16;  // 16-key MMA steps per column group
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
        const uint64_t off = (kk >> 2) * (kHalfBlockBytes >> 4) + (kk & 3) * 2;
        umma_ts_pair(d_tmem, p_tmem + (kk / kGroups) * kColsPerThread + (kk % kGroups) * 8, b0 + off, kIdescPairF16,
                     accumulate || kk > 0);
    }
}

}  // namespace

// kQTma = false: the softmax warps fetch the bf16 query rows, rotate them and write the fp16 tile themselves.
// kQTma = true : the query tile is already in operand form in global memory (16-bit, same type as K', token-major)
//                and the TMA warp copies it; the softmax warps go straight to the first score tile.
// Grid: one cluster of two CTAs per work item of AttnParams (head x 256 query rows) and per key-range piece of the
// last items.  tmap_k / tmap_v have boxes of 64 rows (one CTA's half of a tile).
template <bool kQTma>
__global__ void __launch_bounds__(kThreads, 1)
attn_pair_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                   const __grid_constant__ CUtensorMap tmap_out, const __grid_constant__ CUtensorMap tmap_q,
                   const AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = smem_raw;
    if ((smem_u32(base) & 1023u) != 0) {  // the swizzled tiles need a 1024-byte aligned base (uniform over the grid)
        if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusInternal);
        return;
    }
    uint8_t* sQ = base;
    uint8_t* sKV = base + kTileBytes;
    PairBarriers* bar = reinterpret_cast<PairBarriers*>(base + kTileBytes + kPairStages * kHalfBytes);
    float (*xch)[kSplit] = reinterpret_cast<float (*)[kSplit]>(base + kTileBytes + kPairStages * kHalfBytes + 320);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint32_t tmem_base = 0;
    const WaitCtl ctl{&bar->abort_flag, p.status, kStatusTimeout, kWaitLimitNs};
    // work item, query tile and key-tile range of this CTA
    const int n_tiles_total = p.n_kv_pad / kTile;
    const int rank = static_cast<int>(cluster_rank());   // 0: leader of the pair (issues the MMAs)
    const int pair = static_cast<int>(cluster_id_x());
    const bool piece = pair >= p.n_full_items;         // one of several key-range pieces of an item
    const bool partial = piece || p.tok_o != nullptr;  // leaves an unnormalised result
    const int qt = rank;
    int item = pair, kv_tile0 = 0, n_tiles = n_tiles_total, piece_cta = 0;
    if (piece) {
        piece_cta = pair - p.n_full_items;
        item = p.n_full_items + piece_cta / p.split_k;
        kv_tile0 = (piece_cta % p.split_k) * p.tiles_per_piece;
        n_tiles = min(p.tiles_per_piece, n_tiles_total - kv_tile0);
    }
    const int head = item / p.pairs_per_head;
    const int q0 = (item % p.pairs_per_head) * 2 * kTile + qt * kTile;
    // (a second tile that does not exist still takes part: its query rows are zeros and nothing of it is stored)

    if (warp >= kMmaWarp) {
      setmaxnreg_dec<kControlRegs>();
      if (tid == kMmaWarp * 32) {
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(smem_u32(&bar->kv_full[s]), 1);
            mbar_init(smem_u32(&bar->kv_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar->q_full), kQTma ? 1 : 2);   // leader's: the bytes of both tiles / one arrival per CTA
        mbar_init(smem_u32(&bar->o_full[0]), 1);
        mbar_init(smem_u32(&bar->o_full[1]), 1);
        bar->sat_flag[0] = 0;
        bar->sat_flag[1] = 0;
        for (int b = 0; b < 3; ++b) {
            mbar_init(smem_u32(&bar->s_full[b]), 1);
            mbar_init(smem_u32(&bar->p_full[b]), 2 * (kSoftmaxThreads / 32));   // leader's: every softmax warp of the pair
        }
        // a sticky error from an earlier kernel makes this CTA skip its work (every bounded wait falls through)
        bar->abort_flag = (*reinterpret_cast<volatile int*>(p.status) != 0) ? 1 : 0;
        fence_mbar_init();
      }
      __syncwarp();
      if (warp == kMmaWarp) {
        tmem_alloc_pair(smem_u32(&bar->tmem_base), 512);
        tmem_relinquish_pair();
      }
      if (warp == kTmaWarp && elect_one()) {
        tma_prefetch_desc(&tmap_k);
        tma_prefetch_desc(&tmap_v);
        tma_prefetch_desc(&tmap_out);
        if (kQTma) tma_prefetch_desc(&tmap_q);
      }
      __syncwarp();
      tc_fence_before();
      // set-up is complete in this CTA; neither CTA may count bytes on, arrive at or commit to a barrier of the other
      // before that one has initialised it (the softmax warps join this barrier after loading their query tile)
      cluster_sync_all();
      tc_fence_after();
      tmem_base = bar->tmem_base;
      // The control warps run pass 0 (the optimistic run) and, only after a saturation in either CTA, pass 1 over the
      // same tiles; ring index and barrier phases run on.  Between the passes every warp of the pair meets at the
      // cluster barrier behind which the two CTAs' verdicts can be read (see the softmax warps).
      int c = 0;       // running ring index (producer: next slot to fill; issuer: next slot to consume)
      bool ok = true;
      for (int pass = 0; pass < 2; ++pass) {
        if (warp == kTmaWarp) {
          // ------------------------------------------------------------ TMA producer
          if (elect_one()) {
            if (kQTma && pass == 0) {  // rows past n_q lie outside the tensor map and arrive as zeros
                // the leader announces the bytes of both CTAs' tiles on its barrier; both CTAs' loads count there
                if (rank == 0) mbar_expect_tx(smem_u32(&bar->q_full), 2 * kTileBytes);
                const uint32_t full = map_to_rank(smem_u32(&bar->q_full), 0);
                tma_load_2d_pair(smem_u32(sQ), &tmap_q, head * kHeadDim, q0, full);
                tma_load_2d_pair(smem_u32(sQ) + kBlockBytes, &tmap_q, head * kHeadDim + 64, q0, full);
            }
            // this CTA's half of tile `j` of K' (is_v false) or V't (true) into the next ring slot
            auto fill = [&](bool is_v, int j) {
                const int slot = c % kPairStages, round = c / kPairStages;
                ++c;
                if (round > 0 && !mbar_wait(smem_u32(&bar->kv_empty[slot]), (round - 1) & 1, ctl)) {
                    ok = false;
                    return;
                }
                if (rank == 0) mbar_expect_tx(smem_u32(&bar->kv_full[slot]), 2 * kHalfBytes);
                const uint32_t full = map_to_rank(smem_u32(&bar->kv_full[slot]), 0);
                const uint32_t dst = smem_u32(sKV + slot * kHalfBytes);
                const int kv0 = (kv_tile0 + j) * kTile;
                if (!is_v) {   // keys kv0 + 64 rank .. + 63, all 128 head-dim columns
                    const int r0 = head * p.n_kv_pad + kv0 + rank * (kTile / 2);
                    tma_load_2d_pair(dst, &tmap_k, 0, r0, full);
                    tma_load_2d_pair(dst + kHalfBlockBytes, &tmap_k, 64, r0, full);
                } else {       // head-dim rows 64 rank .. + 63, all 128 keys of the tile
                    const int r0 = head * kHeadDim + rank * (kHeadDim / 2);
                    tma_load_2d_pair(dst, &tmap_v, kv0, r0, full);
                    tma_load_2d_pair(dst + kHalfBlockBytes, &tmap_v, kv0 + 64, r0, full);
                }
            };
            if (ok) fill(false, 0);
            if (ok && n_tiles > 1) fill(false, 1);
            for (int j = 0; ok && j < n_tiles; ++j) {
                fill(true, j);
                if (ok && j + 2 < n_tiles) fill(false, j + 2);
            }
          }
        } else if (warp == kMmaWarp) {
          // ------------------------------------------------------------ UMMA issuer (MMAs from the leader CTA only)
          if (rank == 0 && elect_one()) {
            const uint32_t sQa = smem_u32(sQ);
            const uint32_t idesc_qk = p.qk_bf16 ? kIdescPairBf16 : kIdescPairF16;
            if (pass == 0) ok = mbar_wait(smem_u32(&bar->q_full), 0, ctl);
            for (int b = 0; ok && b < 2 && b < n_tiles; ++b) {   // first two score tiles
                const int slot = c % kPairStages;
                ok = mbar_wait(smem_u32(&bar->kv_full[slot]), (c / kPairStages) & 1, ctl);
                ++c;
                if (!ok) break;
                tc_fence_after();
                issue_qk_pair(tmem_base + kPColS + b * 128, sQa, smem_u32(sKV + slot * kHalfBytes), idesc_qk);
                commit_both(smem_u32(&bar->s_full[b]));
                commit_both(smem_u32(&bar->kv_empty[slot]));
            }
            for (int j = 0; ok && j < n_tiles; ++j) {
                const int b = j % 3, b2 = (j + 2) % 3;   // score buffers of tile j (its probabilities) and of tile j + 2
                const bool more = j + 2 < n_tiles;
                const int slot_v = c % kPairStages, par_v = (c / kPairStages) & 1;
                ++c;
                const int slot_k = c % kPairStages, par_k = (c / kPairStages) & 1;
                if (more) ++c;
                ok = mbar_wait(smem_u32(&bar->kv_full[slot_v]), par_v, ctl);
                if (ok && more) ok = mbar_wait(smem_u32(&bar->kv_full[slot_k]), par_k, ctl);
                // the softmax warps of both CTAs have written P(j) and, before that, read S(j): S_b may be overwritten
                if (ok) ok = mbar_wait(smem_u32(&bar->p_full[b]), parity_of<3>(pass, j, n_tiles), ctl);
                if (!ok) break;
                tc_fence_after();
                // Scores first: the softmax warps then find tile j + 2 complete half a visit before they need it.
                // Its buffer last held the probabilities of tile j - 1, whose P.V was issued a hand-over ago: the
                // MMAs complete in the order they are issued, so that product has read them before these scores land.
                if (more) {
                    issue_qk_pair(tmem_base + kPColS + b2 * 128, sQa, smem_u32(sKV + slot_k * kHalfBytes), idesc_qk);
                    commit_both(smem_u32(&bar->s_full[b2]));
                }
                issue_pv_pair(tmem_base + kPColO, tmem_base + kPColS + b * 128, smem_u32(sKV + slot_v * kHalfBytes), j > 0);
                commit_both(smem_u32(&bar->o_full[j & 1]));
                commit_both(smem_u32(&bar->kv_empty[slot_v]));
                if (more) commit_both(smem_u32(&bar->kv_empty[slot_k]));
            }
          }
        }
        __syncwarp();
        if (pass == 0) {
            cluster_sync_all();   // the verdict barrier of the pair
            if (!(*reinterpret_cast<volatile int*>(&bar->sat_flag[0]) | *reinterpret_cast<volatile int*>(&bar->sat_flag[1])))
                break;
        }
      }
    } else {
        // ------------------------------------------------------------ softmax warps
        setmaxnreg_inc<kSoftmaxRegs>();
        const int part = warp >> 2;                      // which kColsPerThread key columns of a score row
        const int row = (warp & 3) * 32 + lane;          // row in the tile == TMEM lane
        // The softmax warps have nothing to publish at the set-up barrier of the pair: they arrive at once, fetch and
        // rotate their query tile while the control warps of both CTAs set up, and wait afterwards.
        cluster_arrive_relaxed();
        if (!kQTma) {
            load_rotate_q_tiles<kSoftmaxThreads, 1>(p, head, q0, sQ, tid);
            fence_proxy_async_smem();
        }
        cluster_wait();   // barriers and tensor memory of both CTAs exist from here on
        tc_fence_after();
        tmem_base = bar->tmem_base;
        if (!kQTma) {
            // This CTA's tile is complete (every thread's writes are fenced for the async proxy above): one arrival per
            // CTA on the leader's barrier.  The tile is read by this CTA's own half of the pair MMAs, so the arrival
            // needs no cluster-scope release (which costs several hundred cycles).
            softmax_barrier();
            if (tid == 0) mbar_arrive_peer(map_to_rank(smem_u32(&bar->q_full), 0));
        }
        const uint32_t p_full_leader = map_to_rank(smem_u32(&bar->p_full[0]), 0);
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const uint32_t t_O = lane_base + kPColO + part * kColsPerThread;
        const float scale = p.scale_log2;
        const uint64_t scale2 = pack2(scale, scale);
        const uint32_t opaque_zero = static_cast<uint32_t>(p.n_kv) >> 31;  // 0, but not to the compiler
        float m_ref = -INFINITY, l_run = 0.f;
        bool ok = true;  // false once a wait expired: keep the loop structure (named barriers) but skip the work
        bool sat = false;  // optimistic pass: one of this thread's partial row sums saturated
        // the one key tile of the sequence that is partly padding (if this CTA has it), and how many of this
        // thread's columns of that tile are real keys
        const int j_ragged = (p.n_kv % kTile != 0 && kv_tile0 + n_tiles == n_tiles_total) ? n_tiles - 1 : -1;
        const int valid_last = p.n_kv - (n_tiles_total - 1) * kTile - part * kColsPerThread;

        // One pass over the pair's key tiles.  kCareful = false: optimistic, a saturation is only recorded in `sat`;
        // true: the warps of a row group agree per tile and redo a saturated tile against a higher reference.
        auto run_pass = [&](auto careful_tag, const int pass) {
          constexpr bool kCareful = decltype(careful_tag)::value;
          m_ref = -INFINITY;
          l_run = 0.f;
          for (int j = 0; j < n_tiles; ++j) {
            const int b = j % 3;
            const uint32_t t_S = lane_base + kPColS + b * 128 + part * kColsPerThread;
            const uint32_t t_P = t_S;   // the probabilities overwrite this thread's own score columns
            if (ok) ok = mbar_wait(smem_u32(&bar->s_full[b]), parity_of<3>(pass, j, n_tiles), ctl);
            ok = __all_sync(0xffffffffu, ok);  // keep the warp-wide TMEM instructions below convergent
            tc_fence_after();
            // From the second tile on, the probabilities of each 32-column chunk are formed as soon as it
            // arrives, against the reference m_ref of the earlier tiles; no maximum is taken.  Probabilities
            // saturate at 65504 when rounded to fp16, and a saturated one makes the fp32 sum of its part reach
            // 65504.  Optimistic pass: the thread remembers it.  Careful pass: the threads of the row group agree on
            // it; only then (and on the first tile of either pass) the row maximum is taken, the reference raised, O
            // rescaled and the tile redone.
            uint32_t sr[kColsPerThread];
            uint64_t negm2 = pack2(-m_ref, -m_ref);
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
                        tmem_st16(t_P + cb * 16, pr);
                    }
                }
            }
            float part_sum;
            {
                float s0, s1;
                unpack2(add2(sum_a, sum_b), s0, s1);
                part_sum = s0 + s1;
            }
            // Careful pass: one barrier with an OR-reduction tells the threads sharing these 32 rows whether any part
            // of any row saturated (or this is the first tile); only then do they exchange anything.
            bool any_redo;
            if (kCareful) {
                any_redo = row_group_any(warp & 3, !stream || !(part_sum < 65504.0f));
            } else {
                any_redo = !stream;                               // uniform over the pair
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
                xch[row][part] = mx_part;
                row_group_barrier(warp & 3);
                float mx_row = mx_part;
#pragma unroll
                for (int o = 1; o < kSplit; ++o) mx_row = fmaxf(mx_row, xch[row][(part + o) % kSplit]);
                row_group_barrier(warp & 3);  // everyone has read xch before a later redo overwrites it
                const float m_tile = mx_row * scale;
                const bool raise = m_tile > m_ref;  // always on the first tile (reference starts at -inf)
                if (j > 0) {
                    // P.V(j - 1) is issued when every warp has handed the previous visit's probabilities over.  Its
                    // barrier's previous phase, P.V(j - 3), is complete (it was issued before the Q.K^T of this
                    // visit's scores), so the parity is unambiguous.
                    if (ok) ok = mbar_wait(smem_u32(&bar->o_full[(j - 1) & 1]), parity_of<2>(pass, j - 1, n_tiles), ctl);
                    ok = __all_sync(0xffffffffu, ok);
                    tc_fence_after();
                    const float alpha = raise ? ex2_approx(m_ref - m_tile) : 1.0f;
                    l_run *= alpha;
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
                if (raise) m_ref = m_tile;
                negm2 = pack2(-m_ref, -m_ref);
                sum_a = 0;
                sum_b = 0;
                if (ok) {
#pragma unroll
                    for (int cb = 0; cb < kChunks; ++cb) {
                        uint32_t pr[16];
                        exp_chunk<kPolyMask>(sr + cb * 32, scale2, negm2, pr, sum_a, sum_b, opaque_zero);
                        tmem_st16(t_P + cb * 16, pr);
                    }
                }
            }
            float s0, s1;
            unpack2(add2(sum_a, sum_b), s0, s1);
            l_run += s0 + s1;
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_peer(p_full_leader + 8 * b);
          }
        };
        run_pass(std::false_type{}, 0);
        // Verdict on the optimistic pass: first over this CTA's softmax warps, then over the pair (either CTA's
        // saturation sends both through the careful pass, because the MMAs are issued for both at once).  A CTA that
        // saw a saturation sets its flag in both CTAs' shared memory; then every warp of the pair -- these, and the
        // control warps after their pass -- meets at the cluster barrier, behind which everyone reads the same flags.
        const bool mine = softmax_any(sat);
        if (mine && tid == 0) {
            for (uint32_t r = 0; r < 2; ++r) st_shared_peer(map_to_rank(smem_u32(&bar->sat_flag[rank]), r), 1u);
        }
        cluster_sync_all();
        const bool again = (*reinterpret_cast<volatile int*>(&bar->sat_flag[0]) |
                            *reinterpret_cast<volatile int*>(&bar->sat_flag[1])) != 0;
        if (again) run_pass(std::true_type{}, 1);
        const int last_pass = again ? 1 : 0;

        // epilogue: O / l -> bf16 -> out; each thread owns kColsPerThread of the 128 output columns of its row
        {
            xch[row][part] = l_run;
            softmax_barrier();
            float l_row = 0.f;
#pragma unroll
            for (int o = 0; o < kSplit; ++o) l_row += xch[row][o];
            const float inv_l = 1.0f / l_row;
            // A warp that is done with its last visit can be three P.V products ahead of the tensor core (the scores of
            // tile j were issued before P.V(j - 2)): only P.V(n - 4) is known to be complete.  The last but one product
            // first (its barrier's previous phase is P.V(n - 4)), then the last one (previous phase P.V(n - 3), which
            // completes before P.V(n - 2)): both parities are then unambiguous.
            if (ok && n_tiles >= 2)
                ok = mbar_wait(smem_u32(&bar->o_full[(n_tiles - 2) & 1]), parity_of<2>(last_pass, n_tiles - 2, n_tiles), ctl);
            if (ok) ok = mbar_wait(smem_u32(&bar->o_full[(n_tiles - 1) & 1]), parity_of<2>(last_pass, n_tiles - 1, n_tiles), ctl);
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();
            const int n_row = q0 + row;  // query row of this thread
            const size_t part_row = (size_t)piece_cta * 2 * kTile + qt * kTile + row;
            if (partial && part == 0) {
                if (piece) p.part_ml[part_row] = make_float2(m_ref, l_row);
                else if (n_row < p.n_q) p.tok_ml[(size_t)n_row * p.h + head] = make_float2(m_ref, l_row);
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
                    float* row_o = piece ? p.part_o + part_row * kHeadDim : p.tok_o + ((size_t)n_row * p.h + head) * kHeadDim;
                    uint4* dst = reinterpret_cast<uint4*>(row_o + part * kColsPerThread + cb * 32);
                    if (piece || n_row < p.n_q) {
#pragma unroll
                        for (int c = 0; c < 8; ++c) dst[c] = make_uint4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]);
                    }
                } else if (ok) {
                    // normalised bf16 row part into the (now idle) query tile buffer, in the swizzled layout of a
                    // TMA box {64 columns, 128 rows}; one tiled store per 64-column block writes the tile out
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(o[8 * c + 0]) * inv_l, __uint_as_float(o[8 * c + 1]) * inv_l);
                        w.y = pack_bf16x2(__uint_as_float(o[8 * c + 2]) * inv_l, __uint_as_float(o[8 * c + 3]) * inv_l);
                        w.z = pack_bf16x2(__uint_as_float(o[8 * c + 4]) * inv_l, __uint_as_float(o[8 * c + 5]) * inv_l);
                        w.w = pack_bf16x2(__uint_as_float(o[8 * c + 6]) * inv_l, __uint_as_float(o[8 * c + 7]) * inv_l);
                        const int col = part * kColsPerThread + cb * 32 + c * 8;  // first of 8 output columns
                        *reinterpret_cast<uint4*>(sQ + (col >> 6) * kBlockBytes + sw128_offset(row, (col >> 3) & 7)) = w;
                    }
                }
            }
            if (!partial) {
                fence_proxy_async_smem();
                softmax_barrier();
                if (tid == 0 && ok) {
                    const uint32_t src = smem_u32(sQ);
                    tma_store_2d(&tmap_out, head * kHeadDim, q0, src);
                    tma_store_2d(&tmap_out, head * kHeadDim + 64, q0, src + kBlockBytes);
                    tma_store_commit();
                    // the tiled stores read shared memory asynchronously: they must be done before the CTA may exit
                    tma_store_wait_read();
                }
            }
        }
        __syncwarp();
    }

    // ---------------------------------------------------------------- tear-down
    __syncwarp();  // lanes that left a single-lane role loop rejoin before the warp-wide instructions below
    tc_fence_before();
    __syncthreads();
    // both CTAs are done with each other's barriers and tensor memory before either releases it or exits
    cluster_sync_all();
    if (warp == kMmaWarp) {
        __syncwarp();
        if (bar->abort_flag) {
            // a wait expired: give copies and MMAs that may still be in flight time to land before TMEM is released
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
        __syncwarp();
        tmem_dealloc_pair(tmem_base, 512);
    }
}


namespace {
template <bool kQTma>
cudaError_t configure_pair_one() {
    cudaFuncAttributes attr;
    cudaError_t e = cudaFuncGetAttributes(&attr, attn_pair_kernel<kQTma>);
    if (e != cudaSuccess) return e;
    // the register hand-over above assumes the kernel was compiled to exactly kLaunchRegs registers per thread
    if (attr.numRegs != kLaunchRegs) return cudaErrorInvalidConfiguration;
    return cudaFuncSetAttribute(attn_pair_kernel<kQTma>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)kPairAttnSmem);
}
}  // namespace

cudaError_t configure_attn_pair() {
    cudaError_t e = configure_pair_one<false>();
    return e != cudaSuccess ? e : configure_pair_one<true>();
}

cudaError_t launch_attn_pair(const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, const CUtensorMap& tmap_out,
                             const CUtensorMap* tmap_q, const AttnParams& p, cudaStream_t stream) {
    const int n_items = p.pairs_per_head * p.h;
    const int n_pairs = p.n_full_items + (n_items - p.n_full_items) * p.split_k;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (unsigned)n_pairs);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kPairAttnSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (tmap_q) return cudaLaunchKernelEx(&cfg, attn_pair_kernel<true>, tmap_k, tmap_v, tmap_out, *tmap_q, p);
    return cudaLaunchKernelEx(&cfg, attn_pair_kernel<false>, tmap_k, tmap_v, tmap_out, tmap_out, p);
}

}  // namespace regenvc
