// Streaming, warp-specialised tcgen05 attention kernel for sm_100a on PAIRS of CTAs (clusters of two, cta_group::2),
// persistent: as many pairs as fit on the GPU walk over the work items, pair c taking items c, c + G, c + 2G, ...
// (a call with more items than the pairs' lists can hold is launched with one pair per item instead: same kernel).
//
// A work item is one head, 256 query rows and a range of key tiles; CTA r of the pair owns the query rows 128 r ..
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
//   warps 18-19 query warps: they write the finished output tile out (TMA store from the staging buffer) and prepare
//              the query tile of the item after the next one in the buffer that this frees
//
// Tensor memory of each CTA (512 columns x 128 lanes, fp32 cells):
//   [0,128) S_0  [128,256) S_1  [256,384) S_2  [384,512) O
// The key tiles of all of a pair's items form ONE stream of visits g = 0, 1, 2, ...  The scores of visit g go to
// S_(g%3); its probabilities (fp16, two keys per cell) overwrite them in place, every thread writing over score
// columns it has read itself.  Issue order of the tensor core: Q.K^T(0), Q.K^T(1), then, whenever the probabilities
// of visit g have been handed over: Q.K^T(g+2), P.V(g) -- across item boundaries too, so the first two score tiles of
// the next item are complete before the softmax warps have stored the current item's output.  Scores first, so that
// the scores a softmax visit needs are complete long before it starts and the only chain left between the softmax
// warps and the tensor core is P(g) -> P.V(g).  Three buffers make that order safe without anybody waiting for it:
// S_((g+2)%3) last held the probabilities of visit g - 1, whose P.V was issued one hand-over earlier, and the MMAs
// complete in the order they are issued.  (With two score buffers and the probabilities in columns of their own the
// same order let a visit overwrite probabilities that P.V(g-2) was still reading: about one wrong tile in ten
// thousand calls.)  The accumulator O needs no barrier of its own either: the first P.V of an item overwrites it
// after the hand-over of that item's first visit, which every softmax warp reaches only after it has read the
// previous item's O out of tensor memory.
// Shared memory of each CTA: two Q buffers (32 KB each, rotated, fp16, 128B-swizzled K-major blocks; item number n
// of the pair uses buffer n % 2, which is also the staging buffer of its finished output tile), then a ring of
// kPairStages 16 KB slots (one half tile each) filled in the order the tensor core consumes them: K'(0), K'(1),
// V't(0), K'(2), V't(1), K'(3), ...
// Who tells whom: both CTAs' loads count on the leader's kv_full / q_full; every softmax warp of both CTAs arrives
// on the leader's p_full once its probabilities are in tensor memory; the leader commits s_full, o_full and
// kv_empty to both CTAs; a CTA's softmax warps tell its query warps through stage_full that the item's output is
// staged (or written) and its Q buffer free.  Every load reads this GPU's own memory, every CTA fetches its own halves.
//
// Softmax keeps, per row, a reference m (log2 domain) and a row sum l.  m is set from the first tile's row
// maximum (plus kRefMargin of headroom) and afterwards only raised when a probability would leave the fp16 range
// (p = 2^(s - m) > 65504).  As in attn_pipelined.cu an item first runs optimistically (a thread only remembers a saturated partial sum).  A CTA that
// saw a saturation marks the item in a bit mask in its shared memory and carries on; after its last item the pair
// meets at a cluster barrier, reads both CTAs' masks and runs the marked items again carefully (per-tile agreement
// of a row group, row maximum, rescale of O, redo of the tile), overwriting what the optimistic run left.
#include "common.cuh"
#include "attn_core.cuh"
#include "cta_pair.cuh"
#include "rope.cuh"

#include <type_traits>

namespace regenvc {


namespace {

constexpr int kPairStages = 10;                  // ring slots of one half tile (16 KB) each
constexpr int kMaskWords = kPairMaxItemsPerPair / 32;   // words of the mask of items to run again
constexpr uint32_t kHalfBytes = kTileBytes / 2;  // this CTA's half of a K' or V't tile: two [64 rows][64] blocks
constexpr uint32_t kHalfBlockBytes = kHalfBytes / 2;
constexpr uint32_t kPairXchBytes = kTile * kSplit * 4;   // one [128 rows][kSplit] float array for every row exchange
constexpr uint32_t kPairBarBytes = 320;
// no alignment slack: the dynamic shared memory of a kernel without static shared memory starts on a 1024-byte
// boundary (checked at run time)
constexpr uint32_t kPairAttnSmem = 2 * kTileBytes + kPairStages * kHalfBytes + kPairBarBytes + kPairXchBytes;
static_assert(kPairAttnSmem <= 232448, "shared memory of one SM");
constexpr uint32_t kPColS = 0, kPColO = 384;   // tensor-memory columns: three score buffers, then the accumulator
constexpr int kQueryWarp0 = kTmaWarp + 1;      // first of the two query warps
constexpr int kQueryThreads = 64;

struct PairBarriers {
    uint64_t kv_full[kPairStages];
    uint64_t kv_empty[kPairStages];
    uint64_t q_full[2];      // leader's: the query tiles of both CTAs for item number n are in buffer n % 2: phase n / 2
    uint64_t stage_full[2];  // own: the softmax warps are done with buffer n % 2 (output staged or written): phase n / 2
    uint64_t s_full[3];      // scores of visit g complete: barrier g % 3, phase g / 3
    uint64_t p_full[3];      // probabilities of visit g in tensor memory (every softmax warp of the pair): same
    uint64_t o_full[2];      // P.V(g) complete: barrier g % 2, phase g / 2
    uint32_t tmem_base;
    int abort_flag;
    uint32_t redo_mask[kMaskWords];   // bit i: this CTA saw a saturated probability in the optimistic run of its
                                      // i-th item (read by both CTAs behind the cluster barrier that ends the pass)
};
static_assert(sizeof(PairBarriers) <= kPairBarBytes, "barrier block too large");

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
// The two query warps' own named barrier, plain and with an OR-reduction of one predicate per thread.
__device__ __forceinline__ void query_warps_barrier() { asm volatile("bar.sync 8, %0;" ::"n"(kQueryThreads) : "memory"); }
__device__ __forceinline__ bool query_warps_any(bool flag) {
    uint32_t any;
    asm volatile(
        "{\n\t.reg .pred pin, pout;\n\t"
        "setp.ne.u32 pin, %1, 0;\n\t"
        "bar.red.or.pred pout, 8, %2, pin;\n\t"
        "selp.u32 %0, 1, 0, pout;\n\t}"
        : "=r"(any)
        : "r"(static_cast<uint32_t>(flag)), "n"(kQueryThreads)
        : "memory");
    return any != 0;
}

// One unit of work as this CTA sees it: head, first query row of ITS tile, key tiles [kv_tile0, kv_tile0 + n_tiles);
// piece_cta >= 0: one of several key-range pieces of an item (its index among the pieces), which leaves a partial
// result for the merge kernel.
struct Work {
    int head, q0, kv_tile0, n_tiles, piece_cta;
};
__device__ __forceinline__ Work decode_work(const AttnParams& p, int unit, int rank, int n_tiles_total) {
    Work w;
    int item = unit;
    w.kv_tile0 = 0;
    w.n_tiles = n_tiles_total;
    w.piece_cta = -1;
    if (unit >= p.n_full_items) {
        w.piece_cta = unit - p.n_full_items;
        item = p.n_full_items + w.piece_cta / p.split_k;
        w.kv_tile0 = (w.piece_cta % p.split_k) * p.tiles_per_piece;
        w.n_tiles = min(p.tiles_per_piece, n_tiles_total - w.kv_tile0);
    }
    w.head = item / p.pairs_per_head;
    // (a second tile that does not exist still takes part: its query rows are zeros and nothing of it is stored)
    w.q0 = (item % p.pairs_per_head) * 2 * kTile + rank * kTile;
    return w;
}

// The items of a pass in the order every role of the pair walks them.  Pass 0: all n_local items of the pair
// (units unit_first + i * stride).  Pass 1: those marked in either CTA's mask.
struct Walk {
    const AttnParams* p;
    const PairBarriers* bar;
    uint32_t peer_mask;      // shared::cluster address of the other CTA's mask
    int unit_first, stride, n_local, rank, n_tiles_total;

    // local index of the first item of the pass that is >= i, or -1
    __device__ __forceinline__ int from(int pass, int i) const {
        if (pass == 0) return i < n_local ? i : -1;
        while (i < n_local) {
            const int wd = i >> 5;
            const uint32_t m = (*reinterpret_cast<const volatile uint32_t*>(&bar->redo_mask[wd]) |
                                ld_shared_peer(peer_mask + 4 * wd)) >> (i & 31);
            if (m) return i + __ffs(m) - 1;
            i = (wd + 1) << 5;
        }
        return -1;
    }
    __device__ __forceinline__ bool any_marked() const {
        uint32_t m = 0;
        for (int wd = 0; wd * 32 < n_local; ++wd)
            m |= *reinterpret_cast<const volatile uint32_t*>(&bar->redo_mask[wd]) | ld_shared_peer(peer_mask + 4 * wd);
        return m != 0;
    }
    __device__ __forceinline__ Work work(int i) const { return decode_work(*p, unit_first + i * stride, rank, n_tiles_total); }
};
// A position in a pass's stream of key tiles: item (local index i, ordinal k within the pass) and tile j of it.
struct Cursor {
    int i, k, j;
    Work w;
};
__device__ __forceinline__ Cursor cursor_begin(const Walk& walk, int pass) {
    Cursor c;
    c.i = walk.from(pass, 0);
    c.k = 0;
    c.j = 0;
    if (c.i >= 0) c.w = walk.work(c.i);
    return c;
}
__device__ __forceinline__ void cursor_advance(const Walk& walk, int pass, Cursor& c) {
    if (++c.j < c.w.n_tiles) return;
    c.j = 0;
    ++c.k;
    c.i = walk.from(pass, c.i + 1);
    if (c.i >= 0) c.w = walk.work(c.i);
}

}  // namespace

// kQTma = false: the query rows are bf16; the first item's are fetched, rotated and written as an fp16 tile by the
//                softmax warps, those of the later items by the query warps while the item before them runs.
// kQTma = true : the query tiles are already in operand form in global memory (16-bit, same type as K', token-major)
//                and the query warps copy them by TMA.
// Grid: G clusters of two CTAs; cluster c runs the units unit0 + c, unit0 + c + G, ... < unit0 + n_units of the work
// list of AttnParams (head x 256 query rows, then the key-range pieces of the last items), at most
// kPairMaxItemsPerPair of them.  tmap_k / tmap_v have boxes of 64 rows (one CTA's half of a tile).
template <bool kQTma>
__global__ void __launch_bounds__(kThreads, 1)
attn_pair_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                   const __grid_constant__ CUtensorMap tmap_out, const __grid_constant__ CUtensorMap tmap_q,
                   const AttnParams p, const int unit0, const int n_units) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = smem_raw;
    if ((smem_u32(base) & 1023u) != 0) {  // the swizzled tiles need a 1024-byte aligned base (uniform over the grid)
        if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusInternal);
        return;
    }
    uint8_t* sQ = base;                       // two buffers
    uint8_t* sKV = base + 2 * kTileBytes;
    PairBarriers* bar = reinterpret_cast<PairBarriers*>(sKV + kPairStages * kHalfBytes);
    float (*xch)[kSplit] = reinterpret_cast<float (*)[kSplit]>(sKV + kPairStages * kHalfBytes + kPairBarBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint32_t tmem_base = 0;
    const WaitCtl ctl{&bar->abort_flag, p.status, kStatusTimeout, kWaitLimitNs};
    const int rank = static_cast<int>(cluster_rank());   // 0: leader of the pair (issues the MMAs)
    Walk walk;
    walk.p = &p;
    walk.bar = bar;
    walk.peer_mask = map_to_rank(smem_u32(&bar->redo_mask[0]), rank ^ 1);
    walk.stride = static_cast<int>(n_clusters_x());
    walk.unit_first = unit0 + static_cast<int>(cluster_id_x());
    walk.n_local = (n_units - static_cast<int>(cluster_id_x()) + walk.stride - 1) / walk.stride;   // >= 1
    walk.rank = rank;
    walk.n_tiles_total = p.n_kv_pad / kTile;
    const bool always_partial = p.tok_o != nullptr;   // every unit leaves an unnormalised result

    if (warp >= kMmaWarp) {
      setmaxnreg_dec<kControlRegs>();
      if (tid == kMmaWarp * 32) {
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(smem_u32(&bar->kv_full[s]), 1);
            mbar_init(smem_u32(&bar->kv_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar->q_full[b]), kQTma ? 1 : 2);   // leader's: the bytes of both tiles / one arrival per CTA
            mbar_init(smem_u32(&bar->stage_full[b]), kSoftmaxThreads / 32);
            mbar_init(smem_u32(&bar->o_full[b]), 1);
        }
        for (int b = 0; b < 3; ++b) {
            mbar_init(smem_u32(&bar->s_full[b]), 1);
            mbar_init(smem_u32(&bar->p_full[b]), 2 * (kSoftmaxThreads / 32));   // leader's: every softmax warp of the pair
        }
        for (int wd = 0; wd < kMaskWords; ++wd) bar->redo_mask[wd] = 0;
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
      }
      if (warp == kQueryWarp0 && elect_one()) {
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
      // The control warps run pass 0 (the optimistic run of every item) and, only after a saturation, pass 1 over the
      // marked items; ring index, visit numbers and item numbers (hence all barrier phases) run on.  Between the
      // passes every warp of the pair meets at the cluster barrier behind which the two CTAs' masks can be read.
      int c = 0;            // running ring index (producer: next slot to fill; issuer: next slot to consume)
      int g_k = 0, g_v = 0; // issuer: running visit numbers of the score stream and of the P.V stream
      int n_before = 0;     // items of the earlier pass: item k of this pass is item number n_before + k of the pair
      bool ok = true;
      for (int pass = 0; pass < 2; ++pass) {
        if (warp == kTmaWarp) {
          // ------------------------------------------------------------ TMA producer
          if (elect_one()) {
            // this CTA's half of the cursor's tile of K' (is_v false) or V't (true) into the next ring slot
            auto fill = [&](bool is_v, const Cursor& cu) {
                const int slot = c % kPairStages, round = c / kPairStages;
                ++c;
                if (round > 0 && !mbar_wait(smem_u32(&bar->kv_empty[slot]), (round - 1) & 1, ctl)) {
                    ok = false;
                    return;
                }
                if (rank == 0) mbar_expect_tx(smem_u32(&bar->kv_full[slot]), 2 * kHalfBytes);
                const uint32_t full = map_to_rank(smem_u32(&bar->kv_full[slot]), 0);
                const uint32_t dst = smem_u32(sKV + slot * kHalfBytes);
                const int kv0 = (cu.w.kv_tile0 + cu.j) * kTile;
                if (!is_v) {   // keys kv0 + 64 rank .. + 63, all 128 head-dim columns
                    const int r0 = cu.w.head * p.n_kv_pad + kv0 + rank * (kTile / 2);
                    tma_load_2d_pair(dst, &tmap_k, 0, r0, full);
                    tma_load_2d_pair(dst + kHalfBlockBytes, &tmap_k, 64, r0, full);
                } else {       // head-dim rows 64 rank .. + 63, all 128 keys of the tile
                    const int r0 = cu.w.head * kHeadDim + rank * (kHeadDim / 2);
                    tma_load_2d_pair(dst, &tmap_v, kv0, r0, full);
                    tma_load_2d_pair(dst + kHalfBlockBytes, &tmap_v, kv0 + 64, r0, full);
                }
            };
            Cursor ck = cursor_begin(walk, pass);   // the K' stream runs two visits ahead of the V't stream
            Cursor cv = ck;
            for (int n = 0; ok && n < 2 && ck.i >= 0; ++n) {
                fill(false, ck);
                cursor_advance(walk, pass, ck);
            }
            while (ok && cv.i >= 0) {
                fill(true, cv);
                cursor_advance(walk, pass, cv);
                if (ok && ck.i >= 0) {
                    fill(false, ck);
                    cursor_advance(walk, pass, ck);
                }
            }
          }
        } else if (warp == kMmaWarp) {
          // ------------------------------------------------------------ UMMA issuer (MMAs from the leader CTA only)
          if (rank == 0 && elect_one()) {
            const uint32_t idesc_qk = p.qk_bf16 ? kIdescPairBf16 : kIdescPairF16;
            Cursor ck = cursor_begin(walk, pass);   // scores: two visits ahead of ...
            Cursor cv = ck;                         // ... the P.V products
            // the query tiles of the item the score cursor is entering are in shared memory
            auto wait_q = [&]() -> bool {
                if (ck.j != 0) return true;
                const int n = n_before + ck.k;
                return mbar_wait(smem_u32(&bar->q_full[n & 1]), (n >> 1) & 1, ctl);
            };
            // Q.K^T of the score cursor's tile, K' half tiles in ring slot `slot`, into the visit's score buffer
            auto issue_scores = [&](int slot) {
                const int n = n_before + ck.k, b = g_k % 3;
                issue_qk_pair(tmem_base + kPColS + b * 128, smem_u32(sQ) + (n & 1) * kTileBytes,
                              smem_u32(sKV + slot * kHalfBytes), idesc_qk);
                commit_both(smem_u32(&bar->s_full[b]));
                ++g_k;
            };
            for (int n = 0; ok && n < 2 && ck.i >= 0; ++n) {   // first two score tiles of the pass
                const int slot = c % kPairStages, par = (c / kPairStages) & 1;
                ++c;
                ok = wait_q() && mbar_wait(smem_u32(&bar->kv_full[slot]), par, ctl);
                if (!ok) break;
                tc_fence_after();
                issue_scores(slot);
                commit_both(smem_u32(&bar->kv_empty[slot]));
                cursor_advance(walk, pass, ck);
            }
            while (ok && cv.i >= 0) {
                const int b = g_v % 3;   // score buffer of visit g_v, which now holds its probabilities
                const bool more = ck.i >= 0;
                const int slot_v = c % kPairStages, par_v = (c / kPairStages) & 1;
                ++c;
                const int slot_k = c % kPairStages, par_k = (c / kPairStages) & 1;
                if (more) ++c;
                // P.V first at an item's last visit: its epilogue waits for that product, and the scores issued here
                // (the next item's second tile) are not needed before a whole visit has passed.  It is also what keeps
                // items of a single key tile from blocking: an item's query tile is prepared after the epilogue of the
                // item two before it, and with such items the score cursor is that far ahead.
                const bool pv_first = more && cv.j == cv.w.n_tiles - 1;
                ok = mbar_wait(smem_u32(&bar->kv_full[slot_v]), par_v, ctl);
                if (ok && more && !pv_first) ok = wait_q() && mbar_wait(smem_u32(&bar->kv_full[slot_k]), par_k, ctl);
                // the softmax warps of both CTAs have written P(g_v) and, before that, read S(g_v)
                if (ok) ok = mbar_wait(smem_u32(&bar->p_full[b]), (g_v / 3) & 1, ctl);
                if (!ok) break;
                tc_fence_after();
                // Scores first: the softmax warps then find visit g_v + 2 complete half a visit before they need it.
                // Its buffer last held the probabilities of visit g_v - 1, whose P.V was issued a hand-over ago: the
                // MMAs complete in the order they are issued, so that product has read them before these scores land.
                if (more && !pv_first) issue_scores(slot_k);
                issue_pv_pair(tmem_base + kPColO, tmem_base + kPColS + b * 128, smem_u32(sKV + slot_v * kHalfBytes), cv.j > 0);
                commit_both(smem_u32(&bar->o_full[g_v & 1]));
                commit_both(smem_u32(&bar->kv_empty[slot_v]));
                if (pv_first) {
                    ok = wait_q() && mbar_wait(smem_u32(&bar->kv_full[slot_k]), par_k, ctl);
                    if (!ok) break;
                    tc_fence_after();
                    issue_scores(slot_k);
                }
                if (more) commit_both(smem_u32(&bar->kv_empty[slot_k]));
                ++g_v;
                cursor_advance(walk, pass, cv);
                if (more) cursor_advance(walk, pass, ck);
            }
          }
        } else {
          // ------------------------------------------------------------ query warps
          const int qtid = tid - kQueryWarp0 * 32;
          int i_next = walk.from(pass, 0), k_next = 0;   // the next item whose query tile is to be prepared
          auto prepare_next = [&]() {
              const Work w = walk.work(i_next);
              const int n = n_before + k_next;
              uint8_t* dst = sQ + (n & 1) * kTileBytes;
              if (kQTma) {   // rows past n_q lie outside the tensor map and arrive as zeros
                  if (qtid == 0) {
                      // the leader announces the bytes of both CTAs' tiles on its barrier; both CTAs' loads count there
                      if (rank == 0) mbar_expect_tx(smem_u32(&bar->q_full[n & 1]), 2 * kTileBytes);
                      const uint32_t full = map_to_rank(smem_u32(&bar->q_full[n & 1]), 0);
                      tma_load_2d_pair(smem_u32(dst), &tmap_q, w.head * kHeadDim, w.q0, full);
                      tma_load_2d_pair(smem_u32(dst) + kBlockBytes, &tmap_q, w.head * kHeadDim + 64, w.q0, full);
                  }
              } else {
                  load_rotate_q_tile_batched<kQueryThreads, 4>(p, w.head, w.q0, dst, qtid);
                  fence_proxy_async_smem();
                  query_warps_barrier();
                  // This CTA's tile is complete: one arrival per CTA on the leader's barrier.  The tile is read by this
                  // CTA's own half of the pair MMAs, so the arrival needs no cluster-scope release.
                  if (qtid == 0) mbar_arrive_peer(map_to_rank(smem_u32(&bar->q_full[n & 1]), 0));
              }
              i_next = walk.from(pass, i_next + 1);
              ++k_next;
          };
          if (!kQTma && i_next >= 0) {   // the first item's tile is the softmax warps'
              i_next = walk.from(pass, i_next + 1);
              k_next = 1;
          }
          while (i_next >= 0 && k_next < 2) prepare_next();
          int k = 0;
          for (int i = walk.from(pass, 0); ok && i >= 0; i = walk.from(pass, i + 1), ++k) {
              const int n = n_before + k;
              // one lane polls, with pauses: an item takes a hundred thousand cycles, and a polling warp takes issue
              // slots from the softmax warps of its scheduler; the other warp sleeps at the named barrier
              if (qtid == 0) ok = mbar_wait_paused(smem_u32(&bar->stage_full[n & 1]), (n >> 1) & 1, ctl, 200);
              __syncwarp();
              if (query_warps_any(!ok)) {   // the two warps stay together: they share named barriers below
                  ok = false;
                  break;
              }
              const Work w = walk.work(i);
              if (qtid == 0 && !always_partial && w.piece_cta < 0) {
                  // the finished tile in the swizzled layout of a TMA box {64 columns, 128 rows}: one tiled store per
                  // 64-column block; they must have read the buffer before the next query tile is written into it
                  const uint32_t src = smem_u32(sQ) + (n & 1) * kTileBytes;
                  tma_store_2d(&tmap_out, w.head * kHeadDim, w.q0, src);
                  tma_store_2d(&tmap_out, w.head * kHeadDim + 64, w.q0, src + kBlockBytes);
                  tma_store_commit();
                  tma_store_wait_read();
              }
              query_warps_barrier();
              if (i_next >= 0) prepare_next();
          }
        }
        __syncwarp();
        if (pass == 0) {
            cluster_sync_all();   // both CTAs' masks are final
            if (!walk.any_marked()) break;
            n_before = walk.n_local;
            // the second pass stores some tiles again: the first pass's stores of this thread are complete (not just
            // done reading shared memory) before it issues another one
            if (tid == kQueryWarp0 * 32) tma_store_wait_all();
        }
      }
    } else {
        // ------------------------------------------------------------ softmax warps
        setmaxnreg_inc<kSoftmaxRegs>();
        const int part = warp >> 2;                      // which kColsPerThread key columns of a score row
        const int row = (warp & 3) * 32 + lane;          // row in the tile == TMEM lane
        // The softmax warps have nothing to publish at the set-up barrier of the pair: they arrive at once, fetch and
        // rotate the first item's query tile while the control warps of both CTAs set up, and wait afterwards.
        cluster_arrive_relaxed();
        const uint32_t p_full_leader = map_to_rank(smem_u32(&bar->p_full[0]), 0);
        uint32_t lane_base = 0, t_O = 0;                 // known once tensor memory exists
        const float scale = p.scale_log2;
        const uint64_t scale2 = pack2(scale, scale);
        const uint32_t opaque_zero = static_cast<uint32_t>(p.n_kv) >> 31;  // 0, but not to the compiler
        float m_ref = -INFINITY, l_run = 0.f;
        bool ok = true;  // false once a wait expired: keep the loop structure (named barriers) but skip the work
        bool sat = false;  // optimistic run: one of this thread's partial row sums saturated
        int g = 0, b = 0;       // running visit number of the pair, and g % 3
        uint32_t par3 = 0;      // (g / 3) & 1
        int n_item = 0;         // running item number of the pair
        // how many of this thread's columns of the sequence's last key tile are real keys
        const int valid_last = p.n_kv - (walk.n_tiles_total - 1) * kTile - part * kColsPerThread;

        // One pass over the pair's items.  kCareful = false: optimistic, a saturation is only recorded (in `sat`, then
        // in the item's bit of the mask); true: the warps of a row group agree per tile and redo a saturated tile
        // against a higher reference.
        auto run_pass = [&](auto careful_tag, const int pass) {
          constexpr bool kCareful = decltype(careful_tag)::value;
          int k = 0;
          for (int i = walk.from(pass, 0); i >= 0; i = walk.from(pass, i + 1), ++k, ++n_item) {
            const Work w = walk.work(i);
            uint8_t* sQn = sQ + (n_item & 1) * kTileBytes;
            if (k == 0) {
                if (!kQTma) {
                    load_rotate_q_tiles<kSoftmaxThreads, 1>(p, w.head, w.q0, sQn, tid);
                    fence_proxy_async_smem();
                }
                if (pass == 0) {
                    cluster_wait();   // barriers and tensor memory of both CTAs exist from here on
                    tc_fence_after();
                    tmem_base = bar->tmem_base;
                    lane_base = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
                    t_O = lane_base + kPColO + part * kColsPerThread;
                }
                if (!kQTma) {
                    // This CTA's tile is complete (every thread's writes are fenced for the async proxy above): one
                    // arrival per CTA on the leader's barrier.  The tile is read by this CTA's own half of the pair MMAs,
                    // so the arrival needs no cluster-scope release (which costs several hundred cycles).
                    softmax_barrier();
                    if (tid == 0) mbar_arrive_peer(map_to_rank(smem_u32(&bar->q_full[n_item & 1]), 0));
                }
            }
            const bool piece = w.piece_cta >= 0;
            const bool partial = piece || always_partial;   // leaves an unnormalised result
            const int n_tiles = w.n_tiles;
            // the one key tile of the sequence that is partly padding (if this unit has it)
            const int j_ragged = (p.n_kv % kTile != 0 && w.kv_tile0 + n_tiles == walk.n_tiles_total) ? n_tiles - 1 : -1;
            m_ref = -INFINITY;
            l_run = 0.f;
            for (int j = 0; j < n_tiles; ++j) {
              const uint32_t t_S = lane_base + kPColS + b * 128 + part * kColsPerThread;
              const uint32_t t_P = t_S;   // the probabilities overwrite this thread's own score columns
              if (ok) ok = mbar_wait(smem_u32(&bar->s_full[b]), par3, ctl);
              ok = __all_sync(0xffffffffu, ok);  // keep the warp-wide TMEM instructions below convergent
              tc_fence_after();
              // From the second tile on, the probabilities of each 32-column chunk are formed as soon as it
              // arrives, against the reference m_ref of the earlier tiles; no maximum is taken.  Probabilities
              // saturate at 65504 when rounded to fp16, and a saturated one makes the fp32 sum of its part reach
              // 65504.  Optimistic run: the thread remembers it.  Careful run: the threads of the row group agree on
              // it; only then (and on the first tile of either run) the row maximum is taken, the reference raised, O
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
              // Careful run: one barrier with an OR-reduction tells the threads sharing these 32 rows whether any part
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
                  row_group_barrier(warp & 3);  // everyone has read xch before a later exchange overwrites it
                  const float m_tile = mx_row * scale + kRefMargin;
                  const bool raise = m_tile > m_ref;  // always on the first tile (reference starts at -inf)
                  if (j > 0) {
                      // P.V(g - 1) is issued when every warp has handed the previous visit's probabilities over.  Its
                      // barrier's previous phase, P.V(g - 3), is complete (it was issued before the Q.K^T of this
                      // visit's scores), so the parity is unambiguous.
                      if (ok) ok = mbar_wait(smem_u32(&bar->o_full[(g - 1) & 1]), ((g - 1) >> 1) & 1, ctl);
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
              ++g;
              if (++b == 3) {
                  b = 0;
                  par3 ^= 1u;
              }
            }

            // epilogue: O / l -> bf16 -> out; each thread owns kColsPerThread of the 128 output columns of its row
            {
                xch[row][part] = l_run;
                // every part's row sum is in xch behind this barrier; in the optimistic run it also tells whether any
                // thread of this CTA saw a saturation in this item
                const bool mine = softmax_any(!kCareful && sat);
                if (!kCareful) {
                    if (mine && tid == 0) bar->redo_mask[i >> 5] |= 1u << (i & 31);
                    sat = false;
                }
                float l_row = 0.f;
#pragma unroll
                for (int o = 0; o < kSplit; ++o) l_row += xch[row][o];
                row_group_barrier(warp & 3);   // all four parts have read before the next item's first visit writes xch
                const float inv_l = 1.0f / l_row;
                // A warp that is done with its last visit can be three P.V products ahead of the tensor core (the scores
                // of visit g were issued before P.V(g - 2)): only P.V(g - 3) is known to be complete.  The last but one
                // product first (its barrier's previous phase is P.V(g - 3)), then the last one (previous phase
                // P.V(g - 2), which completes before P.V(g - 1)): both parities are then unambiguous.
                const int g_last = g - 1;
                if (ok && g_last >= 1) ok = mbar_wait(smem_u32(&bar->o_full[(g_last - 1) & 1]), ((g_last - 1) >> 1) & 1, ctl);
                if (ok) ok = mbar_wait(smem_u32(&bar->o_full[g_last & 1]), (g_last >> 1) & 1, ctl);
                ok = __all_sync(0xffffffffu, ok);
                tc_fence_after();
                const int n_row = w.q0 + row;  // query row of this thread
                const size_t part_row = piece ? (size_t)w.piece_cta * 2 * kTile + rank * kTile + row : 0;
                if (partial && part == 0) {
                    if (piece) p.part_ml[part_row] = make_float2(m_ref, l_row);
                    else if (n_row < p.n_q) p.tok_ml[(size_t)n_row * p.h + w.head] = make_float2(m_ref, l_row);
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
                        float* row_o = piece ? p.part_o + part_row * kHeadDim : p.tok_o + ((size_t)n_row * p.h + w.head) * kHeadDim;
                        uint4* dst = reinterpret_cast<uint4*>(row_o + part * kColsPerThread + cb * 32);
                        if (piece || n_row < p.n_q) {
#pragma unroll
                            for (int c = 0; c < 8; ++c) dst[c] = make_uint4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]);
                        }
                    } else if (ok) {
                        // normalised bf16 row part into the item's (now idle) query buffer, in the swizzled layout of a
                        // TMA box {64 columns, 128 rows}; the query warps write the tile out from there
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint4 wv;
                            wv.x = pack_bf16x2(__uint_as_float(o[8 * c + 0]) * inv_l, __uint_as_float(o[8 * c + 1]) * inv_l);
                            wv.y = pack_bf16x2(__uint_as_float(o[8 * c + 2]) * inv_l, __uint_as_float(o[8 * c + 3]) * inv_l);
                            wv.z = pack_bf16x2(__uint_as_float(o[8 * c + 4]) * inv_l, __uint_as_float(o[8 * c + 5]) * inv_l);
                            wv.w = pack_bf16x2(__uint_as_float(o[8 * c + 6]) * inv_l, __uint_as_float(o[8 * c + 7]) * inv_l);
                            const int col = part * kColsPerThread + cb * 32 + c * 8;  // first of 8 output columns
                            *reinterpret_cast<uint4*>(sQn + (col >> 6) * kBlockBytes + sw128_offset(row, (col >> 3) & 7)) = wv;
                        }
                    }
                }
                // this warp is done with the item's buffer and has read its part of O out of tensor memory
                if (!partial) fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar->stage_full[n_item & 1]));
            }
          }
        };
        run_pass(std::false_type{}, 0);
        // Both CTAs' masks of saturated items are final behind this barrier (the control warps join it after their
        // pass); an item marked by either CTA is run again by both, because the MMAs are issued for both at once.
        cluster_sync_all();
        if (walk.any_marked()) run_pass(std::true_type{}, 1);
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
cudaError_t configure_pair_one(int* max_clusters) {
    cudaFuncAttributes attr;
    cudaError_t e = cudaFuncGetAttributes(&attr, attn_pair_kernel<kQTma>);
    if (e != cudaSuccess) return e;
    // the register hand-over above assumes the kernel was compiled to exactly kLaunchRegs registers per thread
    if (attr.numRegs != kLaunchRegs) return cudaErrorInvalidConfiguration;
    e = cudaFuncSetAttribute(attn_pair_kernel<kQTma>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairAttnSmem);
    if (e != cudaSuccess) return e;
    // how many pairs the GPU holds at a time: the size of the persistent grid
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kPairAttnSmem;
    cudaLaunchAttribute la[1];
    la[0].id = cudaLaunchAttributeClusterDimension;
    la[0].val.clusterDim.x = 2;
    la[0].val.clusterDim.y = 1;
    la[0].val.clusterDim.z = 1;
    cfg.attrs = la;
    cfg.numAttrs = 1;
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, attn_pair_kernel<kQTma>, &cfg);
    if (e != cudaSuccess || n < 1) {
        // no answer: the caller falls back to one pair per two SMs (the grid size only sets how the units are handed
        // out; any number of pairs computes the same result)
        (void)cudaGetLastError();
        n = 0;
    }
    if (n > 0 && (*max_clusters == 0 || n < *max_clusters)) *max_clusters = n;
    return cudaSuccess;
}
}  // namespace

cudaError_t configure_attn_pair(int* max_clusters) {
    *max_clusters = 0;
    cudaError_t e = configure_pair_one<false>(max_clusters);
    return e != cudaSuccess ? e : configure_pair_one<true>(max_clusters);
}

cudaError_t launch_attn_pair(const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, const CUtensorMap& tmap_out,
                             const CUtensorMap* tmap_q, const AttnParams& p, int max_clusters, cudaStream_t stream) {
    const int n_items = p.pairs_per_head * p.h;
    const int n_units = p.n_full_items + (n_items - p.n_full_items) * p.split_k;
    // A persistent grid: the pairs the GPU holds at a time, the units handed out statically (pair c: c, c + G, ...).  Only
    // a call with more units than the pairs' lists can hold gets one cluster per unit instead.
    // (max_clusters < 0, a test aid: a grid of at most -max_clusters pairs)
    if (max_clusters < 0) max_clusters = -max_clusters;
    const bool persistent = (long long)n_units <= (long long)kPairMaxItemsPerPair * max_clusters;
    const int n_clusters = (!persistent || n_units < max_clusters) ? n_units : max_clusters;
    if (n_clusters < 1 || (long long)n_clusters * kPairMaxItemsPerPair < n_units) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (unsigned)n_clusters);
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
    if (tmap_q) return cudaLaunchKernelEx(&cfg, attn_pair_kernel<true>, tmap_k, tmap_v, tmap_out, *tmap_q, p, 0, n_units);
    return cudaLaunchKernelEx(&cfg, attn_pair_kernel<false>, tmap_k, tmap_v, tmap_out, tmap_out, p, 0, n_units);
}

}  // namespace regenvc
