// Persistent form of the attention kernel for calls whose work items are short (cross-attention to a few hundred
// conditioning tokens): with four key tiles per item the one-CTA-per-item kernel spends half of each CTA's life
// outside its loop (query load, set-up, drain, epilogue, exit).  Here one CTA per SM walks over its items
// (item = blockIdx.x, + gridDim.x, ...) and overlaps those phases across items:
//   * the query tiles are already in operand form in global memory, so the TMA warp fetches the NEXT item's tiles
//     as soon as the last Q.K^T of the current item has been issued and completed (q_empty);
//   * the next item's first Q.K^T runs on the tensor core while the softmax warps are still normalising and
//     storing the current item's output (the score columns are free once the last P.V has read them; the
//     accumulator columns are handed back through o_free when the softmax warps have loaded them);
//   * barriers, tensor memory and the tensor maps are set up once per CTA.
// Roles, tensor-memory map and the UMMA sequences are those of attn_pipelined.cu; the softmax is that kernel's careful
// form (the warps of a row group agree on a saturation tile by tile; there is no optimistic pass here, because by the
// time an item's verdict would be known the control warps are already streaming the next item).  Shared memory:
// Q0, Q1, a 4-slot K'/V't ring and one 32 KB staging tile for the output (the query buffers cannot double as
// staging here because the next item's tiles arrive while the epilogue runs; writing the output rows straight
// from registers, 16 bytes per thread and store, was measured 13 us slower per call at the 480x832 window).
// That is 7 tiles of 32 KB; with the barriers and one 2 KB row-exchange array it fits only because the dynamic
// shared memory of a kernel without static shared memory starts on a 1024-byte boundary (checked at run time).
// Work items: the first n_full_items are (head, 256 query rows); the items after them are single 128-row query
// tiles, which the host uses for the last, incomplete round so that it is spread over twice as many SMs.
// Only normalised bf16 output is produced (no key-range pieces, no token-major partial results).
#include "attn_core.cuh"
#include "common.cuh"

namespace regenvc {

namespace {

constexpr int kPStages = 4;
constexpr uint32_t kPXchBytes = kTile * kSplit * 4;   // one [128 rows][kSplit] float array for every row exchange
constexpr uint32_t kPSmemBytes = (2 + kPStages + 1) * kTileBytes + 256 /*barriers*/ + kPXchBytes;
static_assert(kPSmemBytes <= 232448, "shared memory of one SM");

// A work item of the persistent kernel: head, first query row, number of 128-row query tiles (2, 1 or 0).
struct PItem {
    int head, q0, n_active;
};
__device__ __forceinline__ PItem decode_item(int item, const AttnParams& p) {
    PItem w;
    if (item < p.n_full_items) {
        w.head = item / p.pairs_per_head;
        w.q0 = (item % p.pairs_per_head) * 2 * kTile;
        w.n_active = w.q0 + kTile < p.n_q ? 2 : 1;
    } else {
        const int hx = item - p.n_full_items, pair = p.n_full_items + (hx >> 1);
        w.head = pair / p.pairs_per_head;
        w.q0 = (pair % p.pairs_per_head) * 2 * kTile + (hx & 1) * kTile;
        w.n_active = w.q0 < p.n_q ? 1 : 0;   // the second half of a pair whose second tile does not exist: no work
    }
    return w;
}

struct PBarriers {
    uint64_t kv_full[kPStages];
    uint64_t kv_empty[kPStages];
    uint64_t q_full[2];
    uint64_t q_empty[2];
    uint64_t s_full[2];
    uint64_t p_full[2];
    uint64_t o_full[2];
    uint64_t o_free[2];
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(PBarriers) <= 256, "barrier block too large");

// Byte offsets of the barriers inside PBarriers, for code that addresses them from one 32-bit shared address.
constexpr uint32_t kOffSFull = offsetof(PBarriers, s_full), kOffPFull = offsetof(PBarriers, p_full);
constexpr uint32_t kOffOFull = offsetof(PBarriers, o_full), kOffOFree = offsetof(PBarriers, o_free);
constexpr uint32_t kOffAbort = offsetof(PBarriers, abort_flag);

// Bounded wait of the softmax warps with few live registers: everything except the barrier address and the parity
// is re-derived in the slow path (the CTA's barrier block address, the status pointer from the kernel parameters).
__device__ __forceinline__ bool mbar_wait_lean(uint32_t bar_block, uint32_t off, uint32_t parity, int* status) {
    if (mbar_try_wait(bar_block + off, parity)) return true;
    uint64_t t0 = 0;
    uint32_t spins = 0;
    while (true) {
        if (mbar_try_wait(bar_block + off, parity)) return true;
        if ((++spins & 255u) == 0) {
            int aborted;
            asm volatile("ld.volatile.shared.s32 %0, [%1];" : "=r"(aborted) : "r"(bar_block + kOffAbort) : "memory");
            if (aborted) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > kWaitLimitNs) {
                asm volatile("st.volatile.shared.s32 [%0], %1;" ::"r"(bar_block + kOffAbort), "r"(1) : "memory");
                atomicCAS(status, 0, kStatusTimeout);
                return false;
            }
        }
    }
}
__device__ __forceinline__ void mbar_arrive_at(uint32_t bar_block, uint32_t off) { mbar_arrive(bar_block + off); }

}  // namespace

__global__ void __launch_bounds__(kThreads, 1)
attn_persistent_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                       const __grid_constant__ CUtensorMap tmap_out, const __grid_constant__ CUtensorMap tmap_q,
                       const AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = smem_raw;
    if ((smem_u32(base) & 1023u) != 0) {  // the swizzled tiles need a 1024-byte aligned base (uniform over the grid)
        if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusInternal);
        return;
    }
    uint8_t* sQ = base;                                   // 2 tiles
    uint8_t* sKV = base + 2 * kTileBytes;                 // ring
    uint8_t* sOut = base + (2 + kPStages) * kTileBytes;   // staging tile of the epilogue
    PBarriers* bar = reinterpret_cast<PBarriers*>(base + (3 + kPStages) * kTileBytes);
    // values the kSplit threads of a row hand each other (tile maxima on the redo path, row sums in the epilogue;
    // every use is fenced off from the next by a barrier of the threads involved, so one array serves all)
    float (*xch)[kSplit] = reinterpret_cast<float (*)[kSplit]>(base + (3 + kPStages) * kTileBytes + 256);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint32_t tmem_base = 0;
    const WaitCtl ctl{&bar->abort_flag, p.status, kStatusTimeout, kWaitLimitNs};
    const int n_tiles = p.n_kv_pad / kTile;
    const int n_pairs = p.pairs_per_head * p.h;
    const int n_items = p.n_full_items + 2 * (n_pairs - p.n_full_items);
    const int first_item = blockIdx.x, item_step = gridDim.x;

    if (warp >= kMmaWarp) {
      setmaxnreg_dec<kControlRegs>();
      if (tid == kMmaWarp * 32) {
        for (int s = 0; s < kPStages; ++s) {
            mbar_init(smem_u32(&bar->kv_full[s]), 1);
            mbar_init(smem_u32(&bar->kv_empty[s]), 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_u32(&bar->q_full[t]), 1);
            mbar_init(smem_u32(&bar->q_empty[t]), 1);
            mbar_init(smem_u32(&bar->s_full[t]), 1);
            mbar_init(smem_u32(&bar->p_full[t]), kSoftmaxThreads);
            mbar_init(smem_u32(&bar->o_full[t]), 1);
            mbar_init(smem_u32(&bar->o_free[t]), kSoftmaxThreads);
        }
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
        tma_prefetch_desc(&tmap_q);
      }
      __syncwarp();
      tc_fence_before();
      control_barrier();
      tc_fence_after();
      setup_done_arrive();
      tmem_base = bar->tmem_base;
      if (warp == kTmaWarp) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            int kv_i = 0, it = 0;  // running ring index over all items, item count
            bool ok = true;
            for (int item = first_item; ok && item < n_items; item += item_step) {
                const PItem w = decode_item(item, p);
                const int head = w.head, q0 = w.q0, n_active = w.n_active;
                if (n_active == 0) continue;  // every role skips an empty item the same way
                for (int t = 0; ok && t < n_active; ++t) {
                    if (it > 0) ok = mbar_wait(smem_u32(&bar->q_empty[t]), (it - 1) & 1, ctl);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&bar->q_full[t]);
                    const uint32_t dst = smem_u32(sQ + t * kTileBytes);
                    mbar_expect_tx(full, kTileBytes);  // rows past n_q lie outside the tensor map: zeros
                    tma_load_2d(dst, &tmap_q, head * kHeadDim, q0 + t * kTile, full);
                    tma_load_2d(dst + kBlockBytes, &tmap_q, head * kHeadDim + 64, q0 + t * kTile, full);
                }
                for (int i = 0; ok && i < 2 * n_tiles; ++i, ++kv_i) {
                    const int slot = kv_i % kPStages, round = kv_i / kPStages;
                    if (round > 0) ok = mbar_wait(smem_u32(&bar->kv_empty[slot]), (round - 1) & 1, ctl);
                    if (!ok) break;
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
                ++it;
            }
        }
      } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------ UMMA issuer
        if (elect_one()) {
            const uint32_t sQ0 = smem_u32(sQ), sQ1 = smem_u32(sQ) + kTileBytes;
            const uint32_t idesc_qk = p.qk_bf16 ? kIdescBf16 : kIdesc;
            int kv_c = 0, it = 0;       // ring index of the next tile to consume, item count
            int visit = 0;              // key tiles done so far over all items: the phase of s/p/o_full of BOTH tiles
            bool ok = true;
            for (int item = first_item; ok && item < n_items; item += item_step) {
                const int n_active = decode_item(item, p).n_active;
                if (n_active == 0) continue;
                for (int t = 0; ok && t < n_active; ++t) ok = mbar_wait(smem_u32(&bar->q_full[t]), it & 1, ctl);
                if (ok) ok = mbar_wait(smem_u32(&bar->kv_full[kv_c % kPStages]), (kv_c / kPStages) & 1, ctl);
                if (!ok) break;
                tc_fence_after();
                // first scores of the item: the score columns are free (the previous item's last P.V, issued
                // earlier by this thread, reads them before these MMAs run)
                // (a query tile that does not exist still takes part in every barrier, without MMAs, so that the
                // phases of both tiles stay equal to the running visit count)
                for (int t = 0; t < 2; ++t) {
                    if (t < n_active)
                        issue_qk(tmem_base + t * 128, t ? sQ1 : sQ0, smem_u32(sKV + (kv_c % kPStages) * kTileBytes), idesc_qk);
                    umma_commit(smem_u32(&bar->s_full[t]));
                }
                umma_commit(smem_u32(&bar->kv_empty[kv_c % kPStages]));
                if (n_tiles == 1) {
                    umma_commit(smem_u32(&bar->q_empty[0]));
                    umma_commit(smem_u32(&bar->q_empty[1]));
                }
                ++kv_c;
                for (int j = 0; ok && j < n_tiles; ++j) {
                    const int slot_v = kv_c % kPStages, slot_k = (kv_c + 1) % kPStages;
                    const bool more = j + 1 < n_tiles;
                    ok = mbar_wait(smem_u32(&bar->kv_full[slot_v]), (kv_c / kPStages) & 1, ctl);
                    if (ok && more) ok = mbar_wait(smem_u32(&bar->kv_full[slot_k]), ((kv_c + 1) / kPStages) & 1, ctl);
                    for (int t = 0; ok && t < 2; ++t) {
                        ok = mbar_wait(smem_u32(&bar->p_full[t]), visit & 1, ctl);
                        if (!ok) break;
                        // the accumulator of the previous item must have been read out before it is overwritten
                        if (j == 0 && it > 0) ok = mbar_wait(smem_u32(&bar->o_free[t]), (it - 1) & 1, ctl);
                        if (!ok) break;
                        tc_fence_after();
                        if (t < n_active)
                            issue_pv(tmem_base + 256 + t * 128, tmem_base + t * 128, smem_u32(sKV + slot_v * kTileBytes), j > 0);
                        umma_commit(smem_u32(&bar->o_full[t]));
                        if (more) {
                            if (t < n_active)
                                issue_qk(tmem_base + t * 128, t ? sQ1 : sQ0, smem_u32(sKV + slot_k * kTileBytes), idesc_qk);
                            umma_commit(smem_u32(&bar->s_full[t]));
                        }
                    }
                    ++visit;
                    if (ok) {
                        umma_commit(smem_u32(&bar->kv_empty[slot_v]));
                        if (more) umma_commit(smem_u32(&bar->kv_empty[slot_k]));
                        // after the item's last Q.K^T the query buffers may be refilled (both barriers advance once
                        // per item whether or not the second tile exists)
                        if (j + 2 == n_tiles) {
                            umma_commit(smem_u32(&bar->q_empty[0]));
                            umma_commit(smem_u32(&bar->q_empty[1]));
                        }
                    }
                    kv_c += more ? 2 : 1;
                }
                ++it;
            }
        }
      }
    } else {
        // ------------------------------------------------------------ softmax warps
        setmaxnreg_inc<kSoftmaxRegs>();
        const int part = warp >> 2;
        const int row = (warp & 3) * 32 + lane;
        setup_done_wait();
        tc_fence_after();
        tmem_base = bar->tmem_base;
        // this thread's first score column of tile 0: lane (row) and column part folded into one address
        const uint32_t t_S0 = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16) + part * kColsPerThread;
        const uint32_t bars = smem_u32(bar);
        const float scale = p.scale_log2;
        const uint64_t scale2 = pack2(scale, scale);
        const uint32_t opaque_zero = static_cast<uint32_t>(p.n_kv) >> 31;
        bool ok = true;
        int visit = 0;  // key tiles done so far over all items = completed phases of s_full, p_full, o_full (both tiles)

        for (int item = first_item; item < n_items; item += item_step) {
            const PItem wi = decode_item(item, p);   // kept for the stores at the end: the divisions stay off that path
            const int n_active = wi.n_active;
            if (n_active == 0) continue;
            float m_ref[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

            for (int j = 0; j < n_tiles; ++j, ++visit) {
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (t >= n_active) {  // no such query tile: keep its barriers in step and move on
                        mbar_arrive_at(bars, kOffPFull + 8 * t);
                        continue;
                    }
                    const uint32_t t_S = t_S0 + t * 128;
                    const uint32_t t_O = t_S0 + 256 + t * 128;
                    if (ok) ok = mbar_wait_lean(bars, kOffSFull + 8 * t, visit & 1, p.status);
                    ok = __all_sync(0xffffffffu, ok);
                    tc_fence_after();
                    uint32_t sr[kColsPerThread];
                    uint64_t negm2 = pack2(-m_ref[t], -m_ref[t]);
                    uint64_t sum_a = 0, sum_b = 0;
                    const bool stream = j > 0;
                    if (ok) {
                        tmem_ld32(t_S, sr);
#pragma unroll
                        for (int cb = 0; cb < kChunks; ++cb) {
                            tmem_wait_ld();
                            if (cb + 1 < kChunks) tmem_ld32(t_S + 32 * (cb + 1), sr + 32 * (cb + 1));
                            if (j == n_tiles - 1 && (p.n_kv & (kTile - 1)) != 0) {  // the partly padded last key tile
                                const int valid_last = p.n_kv - (n_tiles - 1) * kTile - part * kColsPerThread;
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
                    const bool any_redo = row_group_any(warp & 3, !stream || !(part_sum < 65504.0f));
                    if (any_redo) {
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
                        row_group_barrier(warp & 3);
                        const float m_tile = mx_row * scale + kRefMargin;
                        const bool raise = m_tile > m_ref[t];
                        if (j > 0) {
                            if (ok) ok = mbar_wait_lean(bars, kOffOFull + 8 * t, (visit - 1) & 1, p.status);
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
                    mbar_arrive_at(bars, kOffPFull + 8 * t);
                }
            }

            // epilogue of the item: O / l -> bf16 -> staging tile -> tiled store, one query tile at a time
#pragma unroll 1
            for (int t = 0; t < 2; ++t) {
                if (t < n_active) {
                    xch[row][part] = l_run[t];
                    softmax_barrier();
                    float l_row = 0.f;
#pragma unroll
                    for (int o = 0; o < kSplit; ++o) l_row += xch[row][o];
                    const float inv_l = 1.0f / l_row;
                    if (ok) ok = mbar_wait_lean(bars, kOffOFull + 8 * t, (visit - 1) & 1, p.status);
                    ok = __all_sync(0xffffffffu, ok);
                    tc_fence_after();
                    static_assert(kChunks == 1, "the epilogue keeps one 32-column chunk per thread in registers");
                    uint4 w[4];
                    if (ok) {
                        uint32_t o[32];
                        tmem_ld32(t_S0 + 256 + t * 128, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            w[c].x = pack_bf16x2(__uint_as_float(o[8 * c + 0]) * inv_l, __uint_as_float(o[8 * c + 1]) * inv_l);
                            w[c].y = pack_bf16x2(__uint_as_float(o[8 * c + 2]) * inv_l, __uint_as_float(o[8 * c + 3]) * inv_l);
                            w[c].z = pack_bf16x2(__uint_as_float(o[8 * c + 4]) * inv_l, __uint_as_float(o[8 * c + 5]) * inv_l);
                            w[c].w = pack_bf16x2(__uint_as_float(o[8 * c + 6]) * inv_l, __uint_as_float(o[8 * c + 7]) * inv_l);
                        }
                    }
                    // the accumulator columns of this tile may now be overwritten by the next item
                    tc_fence_before();
                    mbar_arrive_at(bars, kOffOFree + 8 * t);
                    // the staging tile is free once the previous store has read it (thread 0 issued that store); by now
                    // that read has had the time of the row-sum exchange and of the accumulator load to finish
                    if (tid == 0) tma_store_wait_read();
                    softmax_barrier();
                    if (ok) {
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const int col = part * kColsPerThread + c * 8;
                            *reinterpret_cast<uint4*>(sOut + (col >> 6) * kBlockBytes + sw128_offset(row, (col >> 3) & 7)) = w[c];
                        }
                    }
                    fence_proxy_async_smem();
                    softmax_barrier();
                    if (tid == 0 && ok) {
                        const uint32_t src = smem_u32(sOut);
                        tma_store_2d(&tmap_out, wi.head * kHeadDim, wi.q0 + t * kTile, src);
                        tma_store_2d(&tmap_out, wi.head * kHeadDim + 64, wi.q0 + t * kTile, src + kBlockBytes);
                        tma_store_commit();
                    }
                } else {
                    // a tile that does not exist still arrives, so that the barrier's phase follows the item count
                    mbar_arrive_at(bars, kOffOFree + 8 * t);
                }
            }
        }
        if (tid == 0) tma_store_wait_read();
        __syncwarp();
    }

    // ---------------------------------------------------------------- tear-down
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        __syncwarp();
        if (bar->abort_flag) {
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

cudaError_t configure_attn_persistent() {
    cudaFuncAttributes attr;
    cudaError_t e = cudaFuncGetAttributes(&attr, attn_persistent_kernel);
    if (e != cudaSuccess) return e;
    if (attr.numRegs != kLaunchRegs) return cudaErrorInvalidConfiguration;  // the register hand-over assumes it
    return cudaFuncSetAttribute(attn_persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPSmemBytes);
}

cudaError_t launch_attn_persistent(const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, const CUtensorMap& tmap_out,
                                   const CUtensorMap& tmap_q, const AttnParams& p, int n_ctas, cudaStream_t stream) {
    attn_persistent_kernel<<<n_ctas, kThreads, kPSmemBytes, stream>>>(tmap_k, tmap_v, tmap_out, tmap_q, p);
    return cudaGetLastError();
}

}  // namespace regenvc
