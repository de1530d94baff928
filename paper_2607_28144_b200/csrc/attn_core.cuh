// Pieces shared by the attention kernels: the split of the CTA into softmax warps and a control warpgroup, the
// register hand-over, the packed exponential (MUFU / polynomial split), the named barriers of the softmax warps and
// the UMMA issue sequences of one 128 x 128 x 128 product.
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include "q_tile.cuh"
#include "umma_desc.cuh"

namespace regenvc {

namespace {

#ifndef REGENVC_ROW_SPLIT
#define REGENVC_ROW_SPLIT 4
#endif
constexpr int kSplit = REGENVC_ROW_SPLIT;          // threads sharing one score row (2 or 4)
constexpr int kColsPerThread = kTile / kSplit;     // key columns of a score tile per thread (64 or 32)
constexpr int kChunks = kColsPerThread / 32;       // 32-column TMEM loads per thread and tile
constexpr int kSoftmaxThreads = 128 * kSplit;
constexpr int kThreads = kSoftmaxThreads + 128;    // + one warpgroup holding the UMMA and TMA warps
// Register hand-over between the warpgroups (setmaxnreg): what the softmax warps take must fit in what
// the CTA got at launch (kLaunchRegs per thread, checked against the compiled kernel on the host)
// minus what the control warpgroup keeps; an over-ask would block the last softmax warpgroup forever.
constexpr int kLaunchRegs = (65536 / kThreads) / 8 * 8;   // 168 for 384 threads, 96 for 640
constexpr int kControlRegs = 64;
constexpr int kSoftmaxRegs = ((kLaunchRegs * kThreads - kControlRegs * 128) / kSoftmaxThreads) / 8 * 8;  // 232 / 104
static_assert(kSoftmaxRegs * kSoftmaxThreads + kControlRegs * 128 <= kLaunchRegs * kThreads, "register budget");
static_assert(kSoftmaxRegs >= kLaunchRegs && kSoftmaxRegs <= 255, "setmaxnreg.inc must not shrink");
constexpr int kMmaWarp = kSoftmaxThreads / 32, kTmaWarp = kMmaWarp + 1;
#ifndef REGENVC_POLY_MASK
#define REGENVC_POLY_MASK 0x04
#endif
// bit i set: pair i of every eight probability pairs takes the polynomial 2^x instead of the MUFU.  One pair in
// eight: with the per-tile agreement barrier gone from the common path (optimistic pass) the softmax warps' issue
// slots weigh more than their MUFU time, and two in eight is 1 % slower, in isolated launches and under the power cap.
constexpr uint32_t kPolyMask = REGENVC_POLY_MASK;
constexpr uint32_t kIdesc = umma_idesc_f16_f32acc(128, 128);           // fp16 x fp16 -> fp32
constexpr uint32_t kIdescBf16 = umma_idesc_bf16_f32acc(128, 128);      // bf16 x bf16 -> fp32
constexpr uint64_t kWaitLimitNs = 500000000ull;   // 0.5 s per wait
// Headroom of the softmax reference (log2 units): whenever the reference of a row is set from a tile's row maximum it
// is set this far above it, so the largest probability is 2^-4 and a later score may exceed that maximum by 20 log2
// units (13.9 nats) instead of 16 before a probability leaves the fp16 range and the item has to be run again.  The
// cost is at the other end: probabilities more than 10 (instead of 14) log2 units below the largest are subnormal
// in fp16 and those more than 20 (instead of 24) below it vanish from P.V (never from the fp32 row sum), at most
// 2^-20 of the largest term each.  With scores of standard deviation 4 nats (the 40-head workload's heads with twice
// the unit scale) a third of the work items of such a head saturated without the headroom, practically none with it.
constexpr float kRefMargin = 4.0f;


// Values the threads of a row hand each other through shared memory (redo path and epilogue only).
struct RowExchange {
    float m[2][kTile][kSplit];     // partial tile maxima (redo path): [tile][row][part]
    float l[2][kTile][kSplit];     // row sums at the end: [tile][row][part]
};

// sign(x) * min(|x|, bound), bound > 0: the clamp to [-bound, bound] in one instruction.
__device__ __forceinline__ float clamp_sym(float x, float bound) {
    float y;
    asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(y) : "f"(x), "f"(bound));
    return y;
}

// 2^x for a packed pair on the FMA/ALU pipes: x = n + f with n = round(x), f in [-0.5, 0.5];
// 2^f by a degree-3 minimax polynomial (max relative error 7.5e-5, below fp16 rounding of P),
// 2^n by adding n to the exponent field.  x is clamped to [-125, 125] so that the exponent cannot wrap at
// either end: a score far above the reference then still gives a probability of about 2^125, which saturates
// the fp16 conversion, pushes the part's row sum past 65504 and so requests the raise of the reference, exactly
// as the infinity of the MUFU path does.
__device__ __forceinline__ uint64_t exp2_poly2(uint64_t x2) {
    float x0, x1;
    unpack2(x2, x0, x1);
    x2 = pack2(clamp_sym(x0, 125.0f), clamp_sym(x1, 125.0f));
    const float kMagic = 12582912.0f;  // 1.5 * 2^23: adding it leaves round(x) in the low mantissa bits
    const uint64_t r2 = add2(x2, pack2(kMagic, kMagic));
    const uint64_t n2 = add2(r2, pack2(-kMagic, -kMagic));
    const uint64_t f2 = fma2(n2, pack2(-1.0f, -1.0f), x2);
    uint64_t q2 = fma2(f2, pack2(0.0551716685f, 0.0551716685f), pack2(0.242611125f, 0.242611125f));
    q2 = fma2(q2, f2, pack2(0.693260968f, 0.693260968f));
    q2 = fma2(q2, f2, pack2(0.999928057f, 0.999928057f));
    float q0, q1, r0, r1;
    unpack2(q2, q0, q1);
    unpack2(r2, r0, r1);
    q0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(r0) << 23));
    q1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(r1) << 23));
    return pack2(q0, q1);
}

// Named barrier over all softmax warps (barrier 0 is __syncthreads).
__device__ __forceinline__ void softmax_barrier() {
    asm volatile("bar.sync 1, %0;" ::"n"(kSoftmaxThreads) : "memory");
}
// Barrier 1 with an OR-reduction of one predicate per thread: every softmax thread learns whether any of them
// raised the flag.
__device__ __forceinline__ bool softmax_any(bool flag) {
    uint32_t any;
    asm volatile(
        "{\n\t.reg .pred pin, pout;\n\t"
        "setp.ne.u32 pin, %1, 0;\n\t"
        "bar.red.or.pred pout, 1, %2, pin;\n\t"
        "selp.u32 %0, 1, 0, pout;\n\t}"
        : "=r"(any)
        : "r"(static_cast<uint32_t>(flag)), "n"(kSoftmaxThreads)
        : "memory");
    return any != 0;
}
// A row group's barrier with an OR-reduction of one predicate per thread: every thread of the row group learns
// whether any of them raised the flag, without touching shared memory.
__device__ __forceinline__ bool row_group_any(int g, bool flag) {
    uint32_t any;
    asm volatile(
        "{\n\t.reg .pred pin, pout;\n\t"
        "setp.ne.u32 pin, %1, 0;\n\t"
        "bar.red.or.pred pout, %2, %3, pin;\n\t"
        "selp.u32 %0, 1, 0, pout;\n\t}"
        : "=r"(any)
        : "r"(static_cast<uint32_t>(flag)), "r"(2 + g), "n"(32 * kSplit)
        : "memory");
    return any != 0;
}
// Barrier 6: the four warps of the control warpgroup.  Barrier 7, used once at start-up: the control warps arrive
// without waiting once set-up is done, the softmax warps wait there after loading their query tiles.  (Not
// barrier 0: the idle control warps go straight on to the __syncthreads of the tear-down, and a warp must not
// arrive twice at a barrier whose current phase is still open.)
__device__ __forceinline__ void control_barrier() { asm volatile("bar.sync 6, 128;" ::: "memory"); }
__device__ __forceinline__ void setup_done_arrive() { asm volatile("bar.arrive 7, %0;" ::"n"(kThreads) : "memory"); }
__device__ __forceinline__ void setup_done_wait() { asm volatile("bar.sync 7, %0;" ::"n"(kThreads) : "memory"); }
// Named barrier over the kSplit warps that share the 32 rows of lane group g (barriers 2..5).
__device__ __forceinline__ void row_group_barrier(int g) {
    asm volatile("bar.sync %0, %1;" ::"r"(2 + g), "n"(32 * kSplit) : "memory");
}

// 32 scores of one row -> 16 packed fp16 probability pairs p = 2^(s * scale - m_ref).  The FMA is done on
// packed fp32 pairs; pair c of every eight uses the polynomial when bit (c % 8) of kMask is set, the MUFU
// otherwise, which splits the exponentials between the two pipes.  The fp32 probabilities are also added
// into two packed partial row sums.
// The 16 pairs are worked off as two groups of eight: the second group's FMAs are made to depend on the first
// group's last conversion (through `zero`, a value that is 0 but that the compiler cannot know), which keeps the
// compiler from gathering all FMAs, then all MUFU operations, then all additions and conversions of the chunk
// into three long phases; the warps of a scheduler then meet on the same pipe less often.  Measured on the shipped
// kernel: groups of eight 0.559 ms, no grouping 0.572 ms, groups of four 0.578 ms (480x832 window).
#ifndef REGENVC_EXP_GROUP
#define REGENVC_EXP_GROUP 8
#endif
constexpr int kExpGroup = REGENVC_EXP_GROUP;
template <uint32_t kMask>
__device__ __forceinline__ void exp_chunk(const uint32_t* s, uint64_t scale2, uint64_t negm2_in, uint32_t* pr,
                                          uint64_t& sum_a, uint64_t& sum_b, uint32_t zero) {
    uint64_t negm2 = negm2_in;
#pragma unroll
    for (int c = 0; c < 16; ++c) {
        if (kExpGroup < 16 && c > 0 && c % kExpGroup == 0) {
            float lo, hi;
            unpack2(negm2_in, lo, hi);
            const uint32_t dep = pr[c - 1] & zero;
            negm2 = pack2(__uint_as_float(__float_as_uint(lo) | dep), __uint_as_float(__float_as_uint(hi) | dep));
        }
        const uint64_t x2 = fma2(pack2(__uint_as_float(s[2 * c]), __uint_as_float(s[2 * c + 1])), scale2, negm2);
        uint64_t p2;
        if ((kMask >> (c & 7)) & 1u) {
            p2 = exp2_poly2(x2);
        } else {
            float x0, x1;
            unpack2(x2, x0, x1);
            p2 = pack2(ex2_approx(x0), ex2_approx(x1));
        }
        if (c & 1) sum_b = add2(sum_b, p2);
        else sum_a = add2(sum_a, p2);
        float p0, p1;
        unpack2(p2, p0, p1);
        pr[c] = pack_f16x2_sat(p0, p1);
    }
}

// The eight K = 16 steps of one 128 x 128 x 128 product.  Descriptors differ only in the start-address
// field: +2 (32 bytes) per K step inside a 128-byte row, +1024 (16 KB) for the second 64-element block.
__device__ __forceinline__ void issue_qk(uint32_t d_tmem, uint32_t sQ, uint32_t sK, uint32_t idesc) {
    const uint64_t a0 = umma_smem_desc_k_sw128(sQ), b0 = umma_smem_desc_k_sw128(sK);
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
        const uint64_t off = (kk >> 2) * (kBlockBytes >> 4) + (kk & 3) * 2;
        umma_ss(d_tmem, a0 + off, b0 + off, idesc, kk > 0);
    }
}
__device__ __forceinline__ void issue_pv(uint32_t d_tmem, uint32_t p_tmem, uint32_t sV, bool accumulate) {
    const uint64_t b0 = umma_smem_desc_k_sw128(sV);
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
        const uint64_t off = (kk >> 2) * (kBlockBytes >> 4) + (kk & 3) * 2;
        // P of keys [c, c + kColsPerThread) sits in the first half of score columns [c, c + kColsPerThread)
        constexpr int kGroups = kColsPerThread / 16;  // 16-key MMA steps per column group
        umma_ts(d_tmem, p_tmem + (kk / kGroups) * kColsPerThread + (kk % kGroups) * 8, b0 + off, kIdesc,
                accumulate || kk > 0);
    }
}

}  // namespace

}  // namespace regenvc
