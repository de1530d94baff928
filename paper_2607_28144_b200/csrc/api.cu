// Host side of the C ABI: argument validation, per-device state (status word,
// rotary tables, workspaces, staging buffers), TMA tensor maps and launches.
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <thread>
#include <vector>

#include "../../include/regenvc_attn.h"
#include "common.cuh"


namespace {

using namespace regenvc;

struct Buf {
    void* ptr = nullptr;
    size_t bytes = 0;
};
// A default workspace remembers the stream of its last user and an event recorded behind that user's kernels,
// so that a call on another stream is ordered after them instead of overwriting operands still being read.
struct Workspace {
    Buf buf;
    cudaEvent_t last_use = nullptr;
    cudaStream_t last_stream = nullptr;
    bool used = false;
};
struct RopeEntry {
    int T, H, W;
    float theta;
    float2* dev;
};
// Streams and events of the host-buffer entry points: copies in, kernels and copies out run on three streams
// so that the transfer of one block of query rows overlaps the attention of the previous one.
constexpr int kMaxHostChunks = 8;
struct HostPipe {
    bool made = false;
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, kv = nullptr, fin = nullptr;
    cudaEvent_t q[kMaxHostChunks] = {}, done[kMaxHostChunks] = {};
};
struct DeviceState {
    bool checked = false, supported = false;
    int* status = nullptr;
    int sm_count = 0;
    int pair_clusters = 0;   // pairs of CTAs of the attention kernel on pairs that the device holds at a time
    std::vector<RopeEntry> ropes;
    std::map<std::thread::id, Workspace> workspace;
    std::map<std::thread::id, std::vector<Buf>> staging;  // q, k, v, out
    std::map<std::thread::id, HostPipe> pipes;
};

std::mutex g_mu;
std::map<int, DeviceState> g_dev;
std::atomic<unsigned long long> g_launches{0};
thread_local std::string tl_cuda_error;
thread_local Buf tl_user_ws;
thread_local int tl_phases = 3;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

int cuda_fail(cudaError_t e, const char* what) {
    tl_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
    (void)cudaGetLastError();
    return REGENVC_ERR_CUDA;
}
void launched() { g_launches.fetch_add(1, std::memory_order_relaxed); }
#define CUDA_TRY(expr)                                   \
    do {                                                 \
        cudaError_t e_ = (expr);                         \
        if (e_ != cudaSuccess) return cuda_fail(e_, #expr); \
    } while (0)

bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + nb && b0 < a0 + na;
}

// Validation common to both operations; no CUDA call is made here.
int validate(const void* q, const void* k, const void* v, void* out, long long n_q, long long n_kv, int n_heads,
             int head_dim, bool device_ptrs) {
    if (!q || !k || !v || !out) return REGENVC_ERR_NULL_POINTER;
    if (n_q < 1 || n_kv < 1 || n_heads < 1 || head_dim < 1) return REGENVC_ERR_BAD_SHAPE;
    // token * head row indices (including the padded key rows of the workspace) are 32-bit in the TMA coordinates
    const long long kv_pad = (n_kv + kTile - 1) / kTile * kTile;
    if (n_q > (1ll << 30) || n_kv > (1ll << 30) || n_heads > 65535 || kv_pad * n_heads >= (1ll << 31) ||
        n_q * n_heads >= (1ll << 31))
        return REGENVC_ERR_BAD_SHAPE;
    if (head_dim != kHeadDim) return REGENVC_ERR_UNSUPPORTED;
    if (device_ptrs) {
        if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15) return REGENVC_ERR_MISALIGNED;
    }
    const size_t qb = (size_t)n_q * n_heads * head_dim * 2, kb = (size_t)n_kv * n_heads * head_dim * 2;
    if (overlaps(out, qb, q, qb) || overlaps(out, qb, k, kb) || overlaps(out, qb, v, kb)) return REGENVC_ERR_ALIASING;
    return REGENVC_OK;
}

int device_state(int* dev_out, DeviceState** st_out) {
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    DeviceState& st = g_dev[dev];
    if (!st.checked) {
        int major = 0;
        CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        CUDA_TRY(cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, dev));
        st.supported = (major == 10);
        if (st.supported) {
            if (!g_encode) {
                void* fn = nullptr;
                cudaDriverEntryPointQueryResult qres;
                CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
                if (!fn || qres != cudaDriverEntryPointSuccess) {
                    tl_cuda_error = "cuTensorMapEncodeTiled is not available in this driver";
                    return REGENVC_ERR_CUDA;
                }
                g_encode = (EncodeTiledFn)fn;
            }
            CUDA_TRY(configure_attn_pipelined());
            CUDA_TRY(configure_attn_pair(&st.pair_clusters));
            if (st.pair_clusters < 1) st.pair_clusters = st.sm_count / 2 > 0 ? st.sm_count / 2 : 1;
            CUDA_TRY(configure_qkv_project_pair());
            CUDA_TRY(configure_out_project());
            CUDA_TRY(configure_attn_persistent());
            CUDA_TRY(cudaMalloc(&st.status, sizeof(int)));
            CUDA_TRY(cudaMemset(st.status, 0, sizeof(int)));
        }
        st.checked = true;
    }
    *dev_out = dev;
    *st_out = &st;
    return st.supported ? REGENVC_OK : REGENVC_ERR_UNSUPPORTED;
}

// True when `stream` is being captured into a graph (or its state cannot be queried): events of the library
// are then left alone, and ordering against other streams stays with the caller.
bool capturing(cudaStream_t stream) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cs) != cudaSuccess) {
        (void)cudaGetLastError();
        return true;
    }
    return cs != cudaStreamCaptureStatusNone;
}

// Two calls of one host thread on different streams would share the thread's default workspace while both are
// in flight.  The second one is made to wait (on the GPU, not on the host) for the first one's kernels.
int order_after_last_user(Workspace& w, cudaStream_t stream) {
    if (!w.used || w.last_stream == stream || capturing(stream)) return REGENVC_OK;
    CUDA_TRY(cudaStreamWaitEvent(stream, w.last_use, 0));
    return REGENVC_OK;
}
int note_use(Workspace& w, cudaStream_t stream) {
    if (capturing(stream)) return REGENVC_OK;
    if (!w.last_use) CUDA_TRY(cudaEventCreateWithFlags(&w.last_use, cudaEventDisableTiming));
    CUDA_TRY(cudaEventRecord(w.last_use, stream));
    w.last_stream = stream;
    w.used = true;
    return REGENVC_OK;
}

int grow(Buf& b, size_t bytes) {
    if (b.bytes >= bytes) return REGENVC_OK;
    if (b.ptr) CUDA_TRY(cudaFree(b.ptr));  // waits for work that may still use it
    b.ptr = nullptr;
    b.bytes = 0;
    CUDA_TRY(cudaMalloc(&b.ptr, bytes));
    b.bytes = bytes;
    return REGENVC_OK;
}

// cos/sin of every (axis position, pair) in double precision, stored as float2.
int rope_table(DeviceState& st, int T, int H, int W, float theta, const float2** out) {
    for (const RopeEntry& e : st.ropes)
        if (e.T == T && e.H == H && e.W == W && e.theta == theta) {
            *out = e.dev;
            return REGENVC_OK;
        }
    std::vector<float2> host((size_t)T * kPairsT + (size_t)H * kPairsY + (size_t)W * kPairsX);
    size_t at = 0;
    const int extent[3] = {T, H, W};
    const int pairs[3] = {kPairsT, kPairsY, kPairsX};
    for (int axis = 0; axis < 3; ++axis)
        for (int pos = 0; pos < extent[axis]; ++pos)
            for (int i = 0; i < pairs[axis]; ++i) {
                const double freq = std::pow((double)theta, -(double)i / (double)pairs[axis]);
                const double ang = (double)pos * freq;
                host[at++] = make_float2((float)std::cos(ang), (float)std::sin(ang));
            }
    float2* dev = nullptr;
    CUDA_TRY(cudaMalloc(&dev, host.size() * sizeof(float2)));
    cudaError_t e = cudaMemcpy(dev, host.data(), host.size() * sizeof(float2), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        cudaFree(dev);
        return cuda_fail(e, "cudaMemcpy(rope table)");
    }
    st.ropes.push_back(RopeEntry{T, H, W, theta, dev});
    *out = dev;
    return REGENVC_OK;
}

int make_tmap(CUtensorMap* m, void* base, uint64_t inner, uint64_t outer, uint64_t row_bytes,
              CUtensorMapDataType type = CU_TENSOR_MAP_DATA_TYPE_FLOAT16, int box_rows = 128) {
    const cuuint64_t gdim[2] = {inner, outer};
    const cuuint64_t gstride[1] = {row_bytes};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(m, type, 2, base, gdim, gstride, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        tl_cuda_error = "cuTensorMapEncodeTiled failed with CUresult " + std::to_string((int)r);
        return REGENVC_ERR_CUDA;
    }
    return REGENVC_OK;
}

size_t operand_bytes(long long n_kv, int n_heads) {
    const size_t kv_pad = (size_t)((n_kv + kTile - 1) / kTile * kTile);
    return 2 * (size_t)n_heads * kv_pad * kHeadDim * sizeof(__half);
}
size_t workspace_need(long long n_kv, int n_heads) { return operand_bytes(n_kv, n_heads) + kSplitScratchBytes; }

// Enqueues the two kernels.  Arguments are already validated; pointers are device pointers.
// Block-wise use: q and k/v are contiguous token ranges of the T x H x W grid starting at these tokens, and the
// unnormalised result goes to token-major fp32 buffers instead of `out`.
struct BlockArgs {
    int q_token0 = 0, kv_token0 = 0;
    float* tok_o = nullptr;
    float2* tok_ml = nullptr;
    int phases = -1;  // bit 0: preparation pass, bit 1: attention; -1: the calling thread's debug setting
    // Caller-owned operand buffer (K' then V't, regenvc_prepared_bytes()): the preparation pass writes it and the
    // attention kernel reads it instead of the workspace, which then only serves the split-key scratch.
    void* prepared = nullptr;
    // q is a 16-bit tensor already in operand form (rotated where that applies, same type as K'): the kernel's
    // TMA warp copies the query tiles; qk_bf16 says whether that type is bf16 (else fp16).
    bool q_operand = false;
    bool qk_bf16 = false;
};

int enqueue(const void* q, const void* k, const void* v, void* out, int n_q, int n_kv, int n_heads, bool rope, int T,
            int H, int W, float theta, cudaStream_t stream, const BlockArgs& blk = BlockArgs()) {
    std::lock_guard<std::mutex> lock(g_mu);
    int dev = 0;
    DeviceState* st = nullptr;
    int rc = device_state(&dev, &st);
    if (rc != REGENVC_OK) return rc;

    const int phases = blk.phases >= 0 ? blk.phases : tl_phases;
    const size_t need = !blk.prepared ? workspace_need(n_kv, n_heads) : ((phases & 2) ? kSplitScratchBytes : 0);
    void* ws = nullptr;
    Workspace* own = nullptr;  // the library's workspace of this thread, when the caller supplied none
    if (tl_user_ws.ptr) {
        if (tl_user_ws.bytes < need) return REGENVC_ERR_WORKSPACE;
        ws = tl_user_ws.ptr;
    } else {
        own = &st->workspace[std::this_thread::get_id()];
        rc = grow(own->buf, need);
        if (rc != REGENVC_OK) return rc;
        ws = own->buf.ptr;
        rc = order_after_last_user(*own, stream);
        if (rc != REGENVC_OK) return rc;
    }
    const int kv_pad = round_up(n_kv, kTile);
    __half* kp = reinterpret_cast<__half*>(blk.prepared ? blk.prepared : ws);
    __half* vt = kp + (size_t)n_heads * kv_pad * kHeadDim;
    // Without rotation the queries need no arithmetic before Q.K^T: both they and the keys stay bf16 (their
    // products are then exact) and the query tiles are copied by TMA straight from the caller's tensor.
    const bool q_operand = blk.q_operand || !rope;
    const bool qk_bf16 = blk.q_operand ? blk.qk_bf16 : !rope;

    RopeGrid grid{nullptr, T, H, W};
    if (rope) {
        rc = rope_table(*st, T, H, W, theta, &grid.tab);
        if (rc != REGENVC_OK) return rc;
    }

    // Which attention kernel.  Long key sequences with at least one full round of work items go to the persistent
    // kernel on pairs of CTAs (a pair per item, each CTA one query tile and half of every K' / V't tile; the pairs walk
    // over the items, so the fixed cost of an item overlaps the end of the one before it); short key sequences with
    // query tiles in operand form to the persistent kernel for those; everything else to one CTA per item.  Debug bits
    // 8 / 16 force / forbid the first (32: force it with a grid of two pairs only, so that small shapes take many
    // items per pair).
    const int n_tiles = kv_pad / kTile;
    const int n_items = ((n_q + 2 * kTile - 1) / (2 * kTile)) * n_heads;
    const bool use_pair = (tl_phases & 40) || (!(tl_phases & 16) && n_tiles >= kPairMinTiles && n_items >= st->pair_clusters);
    const int kv_box_rows = use_pair ? 64 : 128;
    CUtensorMap tmap_k, tmap_v;
    rc = make_tmap(&tmap_k, kp, kHeadDim, (uint64_t)n_heads * kv_pad, kHeadDim * sizeof(__half),
                   qk_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, kv_box_rows);
    if (rc != REGENVC_OK) return rc;
    rc = make_tmap(&tmap_v, vt, (uint64_t)kv_pad, (uint64_t)n_heads * kHeadDim, (uint64_t)kv_pad * sizeof(__half),
                   CU_TENSOR_MAP_DATA_TYPE_FLOAT16, kv_box_rows);
    if (rc != REGENVC_OK) return rc;

    PrepParams pp;
    pp.k = reinterpret_cast<const __nv_bfloat16*>(k);
    pp.v = reinterpret_cast<const __nv_bfloat16*>(v);
    pp.kp = kp;
    pp.vt = vt;
    pp.n_kv = n_kv;
    pp.n_kv_pad = kv_pad;
    pp.h = n_heads;
    pp.rope = rope ? 1 : 0;
    pp.k_bf16 = qk_bf16 ? 1 : 0;
    pp.grid = grid;
    pp.pos_offset = blk.kv_token0;
    pp.status = st->status;
    if (phases & 1) {
        CUDA_TRY(launch_prep_kv(pp, stream));
        launched();
    }
    if (!(phases & 2)) return own ? note_use(*own, stream) : REGENVC_OK;

    AttnParams ap;
    ap.q = reinterpret_cast<const __nv_bfloat16*>(q);
    ap.out = reinterpret_cast<__nv_bfloat16*>(out);
    ap.n_q = n_q;
    ap.n_kv = n_kv;
    ap.n_kv_pad = kv_pad;
    ap.h = n_heads;
    ap.rope = rope ? 1 : 0;
    ap.qk_bf16 = qk_bf16 ? 1 : 0;
    ap.grid = grid;
    ap.q_pos_offset = blk.q_token0;
    ap.tok_o = blk.tok_o;
    ap.tok_ml = blk.tok_ml;
    ap.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)kHeadDim));
    ap.status = st->status;
    ap.sm_count = st->sm_count;
    // Work decomposition: one CTA (or pair of CTAs) per (head, 256 query rows).  The items of the last, incomplete
    // wave are cut along the key axis into split_k pieces each so that the pieces fill the SMs; a merge kernel
    // combines them.
    ap.pairs_per_head = (n_q + 2 * kTile - 1) / (2 * kTile);
    ap.n_full_items = n_items;
    ap.split_k = 1;
    ap.tiles_per_piece = n_tiles;
    ap.part_o = reinterpret_cast<float*>(reinterpret_cast<char*>(ws) + (blk.prepared ? 0 : operand_bytes(n_kv, n_heads)));
    ap.part_ml = reinterpret_cast<float2*>(ap.part_o + (size_t)kMaxPieceCtas * 2 * kTile * kHeadDim);
    // Short key sequences with query tiles in operand form: one persistent CTA per SM walks over the items and
    // overlaps their fixed costs (no key-range pieces in that form).
    const bool persistent = !use_pair && q_operand && blk.tok_o == nullptr && n_tiles <= kPersistentMaxTiles && !(tl_phases & 4);
    const int slots = use_pair ? st->pair_clusters : st->sm_count;   // work items that run at a time
    const int rem = n_items % slots;
    if (!persistent && rem > 0 && st->sm_count <= kMaxPieceCtas && blk.tok_o == nullptr) {
        int k = slots / rem;
        if (k > 8) k = 8;
        if (k > n_tiles / 4) k = n_tiles / 4;
        if (k >= 2) {
            ap.tiles_per_piece = (n_tiles + k - 1) / k;
            ap.split_k = (n_tiles + ap.tiles_per_piece - 1) / ap.tiles_per_piece;  // no empty piece
            ap.n_full_items = n_items - rem;
        }
    }
    // out seen as [n_q rows][n_heads * 128 columns] bf16 for the tiled stores of finished query tiles
    CUtensorMap tmap_out;
    rc = make_tmap(&tmap_out, out != nullptr ? out : const_cast<void*>(q), (uint64_t)n_heads * kHeadDim, (uint64_t)n_q,
                   (uint64_t)n_heads * kHeadDim * sizeof(__nv_bfloat16), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
    if (rc != REGENVC_OK) return rc;
    CUtensorMap tmap_q;
    if (q_operand) {
        rc = make_tmap(&tmap_q, const_cast<void*>(q), (uint64_t)n_heads * kHeadDim, (uint64_t)n_q,
                       (uint64_t)n_heads * kHeadDim * 2,
                       qk_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16);
        if (rc != REGENVC_OK) return rc;
    }
    if (persistent) {
        // a last round that would keep at most half of the SMs busy is handed out as single 128-row query tiles
        int n_ctas = n_items < st->sm_count ? n_items : st->sm_count;
        if (n_items > st->sm_count && rem > 0 && 2 * rem <= st->sm_count) ap.n_full_items = n_items - rem;
        if (n_items <= st->sm_count / 2) {
            ap.n_full_items = 0;
            n_ctas = 2 * n_items;
        }
        CUDA_TRY(launch_attn_persistent(tmap_k, tmap_v, tmap_out, tmap_q, ap, n_ctas, stream));
    } else {
        if (use_pair) CUDA_TRY(launch_attn_pair(tmap_k, tmap_v, tmap_out, q_operand ? &tmap_q : nullptr, ap,
                                                    (tl_phases & 32) ? -2 : st->pair_clusters, stream));
        else CUDA_TRY(launch_attn_pipelined(tmap_k, tmap_v, tmap_out, q_operand ? &tmap_q : nullptr, ap, stream));
    }
    launched();
    if (ap.split_k > 1) {
        MergeParams mp;
        mp.part_o = ap.part_o;
        mp.part_ml = ap.part_ml;
        mp.out = ap.out;
        mp.n_q = n_q;
        mp.h = n_heads;
        mp.pairs_per_head = ap.pairs_per_head;
        mp.n_full_items = ap.n_full_items;
        mp.split_k = ap.split_k;
        mp.n_split_items = n_items - ap.n_full_items;
        CUDA_TRY(launch_merge_partials(mp, stream));
        launched();
    }
    return own ? note_use(*own, stream) : REGENVC_OK;
}

int make_pipe(HostPipe& hp) {
    if (hp.made) return REGENVC_OK;
    CUDA_TRY(cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking));
    CUDA_TRY(cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking));
    CUDA_TRY(cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming));
    CUDA_TRY(cudaEventCreateWithFlags(&hp.kv, cudaEventDisableTiming));
    CUDA_TRY(cudaEventCreateWithFlags(&hp.fin, cudaEventDisableTiming));
    for (int c = 0; c < kMaxHostChunks; ++c) {
        CUDA_TRY(cudaEventCreateWithFlags(&hp.q[c], cudaEventDisableTiming));
        CUDA_TRY(cudaEventCreateWithFlags(&hp.done[c], cudaEventDisableTiming));
    }
    hp.made = true;
    return REGENVC_OK;
}

// Host-buffer variant: stage in, run, stage out, wait.  K and V go first (the preparation pass needs them whole);
// the query rows follow in blocks of whole waves of work items, and each block's attention and the copy of its
// result back overlap the transfer of the next block.
int run_host(const void* q, const void* k, const void* v, void* out, int n_q, int n_kv, int n_heads, bool rope, int T,
             int H, int W, float theta, cudaStream_t stream) {
    const size_t row_bytes = (size_t)n_heads * kHeadDim * 2;
    const size_t qb = (size_t)n_q * row_bytes, kb = (size_t)n_kv * row_bytes;
    char *dq, *dout;
    void *dk, *dv;
    HostPipe* hp = nullptr;
    int sm_count = 1;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        int dev = 0;
        DeviceState* st = nullptr;
        int rc = device_state(&dev, &st);
        if (rc != REGENVC_OK) return rc;
        std::vector<Buf>& s = st->staging[std::this_thread::get_id()];
        s.resize(4);
        const size_t need[4] = {qb, kb, kb, qb};
        for (int i = 0; i < 4; ++i) {
            rc = grow(s[i], need[i]);
            if (rc != REGENVC_OK) return rc;
        }
        dq = (char*)s[0].ptr; dk = s[1].ptr; dv = s[2].ptr; dout = (char*)s[3].ptr;
        hp = &st->pipes[std::this_thread::get_id()];
        rc = make_pipe(*hp);
        if (rc != REGENVC_OK) return rc;
        sm_count = st->sm_count > 0 ? st->sm_count : 1;
    }
    // blocks of query rows: about one wave of (head x 256 rows) work items each, at most kMaxHostChunks
    // (measured at the 480x832 window: 1 block 4.43 ms per self + cross step, 2: 3.63, 3: 3.37, 4: 3.25, 8: 3.26)
    const int pairs = (n_q + 2 * kTile - 1) / (2 * kTile);
    int n_chunks = (int)(((long long)pairs * n_heads + sm_count - 1) / sm_count);
    if (n_chunks < 1) n_chunks = 1;
    if (n_chunks > kMaxHostChunks) n_chunks = kMaxHostChunks;
    if (n_chunks > pairs) n_chunks = pairs;
    const int rows_per_chunk = (pairs + n_chunks - 1) / n_chunks * 2 * kTile;

    // the copies start after whatever the caller has already put on its stream
    CUDA_TRY(cudaEventRecord(hp->start, stream));
    CUDA_TRY(cudaStreamWaitEvent(hp->in, hp->start, 0));
    CUDA_TRY(cudaStreamWaitEvent(hp->out, hp->start, 0));
    CUDA_TRY(cudaMemcpyAsync(dk, k, kb, cudaMemcpyHostToDevice, hp->in));
    CUDA_TRY(cudaMemcpyAsync(dv, v, kb, cudaMemcpyHostToDevice, hp->in));
    CUDA_TRY(cudaEventRecord(hp->kv, hp->in));
    CUDA_TRY(cudaStreamWaitEvent(stream, hp->kv, 0));
    BlockArgs prep;
    prep.phases = 1;
    int rc = enqueue(dq, dk, dv, dout, n_q, n_kv, n_heads, rope, T, H, W, theta, stream, prep);
    if (rc != REGENVC_OK) return rc;
    int c = 0;
    for (int r0 = 0; r0 < n_q; r0 += rows_per_chunk, ++c) {
        const int rows = n_q - r0 < rows_per_chunk ? n_q - r0 : rows_per_chunk;
        const size_t off = (size_t)r0 * row_bytes, bytes = (size_t)rows * row_bytes;
        CUDA_TRY(cudaMemcpyAsync(dq + off, (const char*)q + off, bytes, cudaMemcpyHostToDevice, hp->in));
        CUDA_TRY(cudaEventRecord(hp->q[c], hp->in));
        CUDA_TRY(cudaStreamWaitEvent(stream, hp->q[c], 0));
        BlockArgs blk;
        blk.phases = 2;
        blk.q_token0 = r0;
        rc = enqueue(dq + off, dk, dv, dout + off, rows, n_kv, n_heads, rope, T, H, W, theta, stream, blk);
        if (rc != REGENVC_OK) return rc;
        CUDA_TRY(cudaEventRecord(hp->done[c], stream));
        CUDA_TRY(cudaStreamWaitEvent(hp->out, hp->done[c], 0));
        CUDA_TRY(cudaMemcpyAsync((char*)out + off, dout + off, bytes, cudaMemcpyDeviceToHost, hp->out));
    }
    CUDA_TRY(cudaEventRecord(hp->fin, hp->out));
    CUDA_TRY(cudaStreamWaitEvent(stream, hp->fin, 0));
    CUDA_TRY(cudaStreamSynchronize(stream));
    return REGENVC_OK;
}

int check_self_args(int T, int H, int W, float theta, long long* n_out) {
    if (T < 1 || H < 1 || W < 1) return REGENVC_ERR_BAD_SHAPE;
    const long long n = (long long)T * H * W;
    if (n > (1ll << 30)) return REGENVC_ERR_BAD_SHAPE;
    *n_out = n;
    (void)theta;
    return REGENVC_OK;
}

}  // namespace

namespace regenvc {
void count_launch() { launched(); }
int record_cuda_failure(cudaError_t e, const char* what) { return cuda_fail(e, what); }
}  // namespace regenvc

extern "C" {

int regenvc_attn_forward(const void* q, const void* k, const void* v, void* out, int T, int H, int W, int n_heads,
                         int head_dim, float rope_theta, void* stream) {
    if (!q || !k || !v || !out) return REGENVC_ERR_NULL_POINTER;
    long long n = 0;
    int rc = check_self_args(T, H, W, rope_theta, &n);
    if (rc != REGENVC_OK) return rc;
    rc = validate(q, k, v, out, n, n, n_heads, head_dim, true);
    if (rc != REGENVC_OK) return rc;
    if (!(rope_theta > 0.0f) || !std::isfinite(rope_theta)) return REGENVC_ERR_UNSUPPORTED;
    return enqueue(q, k, v, out, (int)n, (int)n, n_heads, true, T, H, W, rope_theta, (cudaStream_t)stream);
}

int regenvc_cross_attn_forward(const void* q, const void* k, const void* v, void* out, int n_q, int n_kv, int n_heads,
                               int head_dim, void* stream) {
    int rc = validate(q, k, v, out, n_q, n_kv, n_heads, head_dim, true);
    if (rc != REGENVC_OK) return rc;
    return enqueue(q, k, v, out, n_q, n_kv, n_heads, false, 1, 1, 1, 1.0f, (cudaStream_t)stream);
}

size_t regenvc_prepared_bytes(int n_kv, int n_heads, int head_dim) {
    if (n_kv < 1 || n_heads < 1 || head_dim != kHeadDim) return 0;
    return operand_bytes(n_kv, n_heads);
}

int regenvc_cross_kv_prepare(const void* k, const void* v, void* prepared, int n_kv, int n_heads, int head_dim,
                             void* stream) {
    // the ordinary checks with a one-row stand-in for q/out: `prepared` must not overlap k or v
    if (!k || !v || !prepared) return REGENVC_ERR_NULL_POINTER;
    if (n_kv < 1 || n_heads < 1 || head_dim < 1) return REGENVC_ERR_BAD_SHAPE;
    const long long kv_pad = ((long long)n_kv + kTile - 1) / kTile * kTile;
    if (n_kv > (1 << 30) || n_heads > 65535 || kv_pad * n_heads >= (1ll << 31)) return REGENVC_ERR_BAD_SHAPE;
    if (head_dim != kHeadDim) return REGENVC_ERR_UNSUPPORTED;
    if (((uintptr_t)k | (uintptr_t)v) & 15) return REGENVC_ERR_MISALIGNED;
    if ((uintptr_t)prepared & 255) return REGENVC_ERR_MISALIGNED;
    const size_t kb = (size_t)n_kv * n_heads * kHeadDim * 2, pb = operand_bytes(n_kv, n_heads);
    if (overlaps(prepared, pb, k, kb) || overlaps(prepared, pb, v, kb)) return REGENVC_ERR_ALIASING;
    BlockArgs blk;
    blk.phases = 1;
    blk.prepared = prepared;
    return enqueue(nullptr, k, v, nullptr, 1, n_kv, n_heads, false, 1, 1, 1, 1.0f, (cudaStream_t)stream, blk);
}

namespace {
// Checks shared by the two calls that run attention on operands prepared earlier.
int validate_prepared(const void* q, const void* prepared, void* out, int n_q, int n_kv, int n_heads, int head_dim) {
    if (!q || !prepared || !out) return REGENVC_ERR_NULL_POINTER;
    if (n_q < 1 || n_kv < 1 || n_heads < 1 || head_dim < 1) return REGENVC_ERR_BAD_SHAPE;
    const long long kv_pad = ((long long)n_kv + kTile - 1) / kTile * kTile;
    if (n_q > (1 << 30) || n_kv > (1 << 30) || n_heads > 65535 || kv_pad * n_heads >= (1ll << 31) ||
        (long long)n_q * n_heads >= (1ll << 31))
        return REGENVC_ERR_BAD_SHAPE;
    if (head_dim != kHeadDim) return REGENVC_ERR_UNSUPPORTED;
    if (((uintptr_t)q | (uintptr_t)out) & 15) return REGENVC_ERR_MISALIGNED;
    if ((uintptr_t)prepared & 255) return REGENVC_ERR_MISALIGNED;
    const size_t qb = (size_t)n_q * n_heads * kHeadDim * 2, pb = operand_bytes(n_kv, n_heads);
    if (overlaps(out, qb, q, qb) || overlaps(out, qb, prepared, pb)) return REGENVC_ERR_ALIASING;
    return REGENVC_OK;
}
}  // namespace

int regenvc_cross_attn_forward_prepared(const void* q, const void* prepared, void* out, int n_q, int n_kv,
                                        int n_heads, int head_dim, void* stream) {
    int rc = validate_prepared(q, prepared, out, n_q, n_kv, n_heads, head_dim);
    if (rc != REGENVC_OK) return rc;
    BlockArgs blk;
    blk.phases = 2;
    blk.prepared = const_cast<void*>(prepared);
    return enqueue(q, nullptr, nullptr, out, n_q, n_kv, n_heads, false, 1, 1, 1, 1.0f, (cudaStream_t)stream, blk);
}

int regenvc_attn_forward_prepared(const void* q_rot, const void* prepared, void* out, int n_q, int n_kv, int n_heads,
                                  int head_dim, void* stream) {
    int rc = validate_prepared(q_rot, prepared, out, n_q, n_kv, n_heads, head_dim);
    if (rc != REGENVC_OK) return rc;
    BlockArgs blk;
    blk.phases = 2;
    blk.prepared = const_cast<void*>(prepared);
    blk.q_operand = true;   // fp16 queries, rotated by whoever produced them
    blk.qk_bf16 = false;
    return enqueue(q_rot, nullptr, nullptr, out, n_q, n_kv, n_heads, false, 1, 1, 1, 1.0f, (cudaStream_t)stream, blk);
}

int regenvc_qkv_rope_project(const void* x, const void* w_qkv, const void* b_qkv, const void* g_q, const void* g_k,
                             float eps, void* q_rot, void* prepared, int T, int H, int W, int n_heads, int head_dim,
                             float rope_theta, void* stream) {
    if (!x || !w_qkv || !q_rot || !prepared) return REGENVC_ERR_NULL_POINTER;
    long long n = 0;
    int rc = check_self_args(T, H, W, rope_theta, &n);
    if (rc != REGENVC_OK) return rc;
    if (n_heads < 1 || head_dim < 1) return REGENVC_ERR_BAD_SHAPE;
    const long long n_pad = (n + kTile - 1) / kTile * kTile;
    if (n_heads > 65535 || n_pad * n_heads >= (1ll << 31)) return REGENVC_ERR_BAD_SHAPE;
    if (head_dim != kHeadDim || n_heads % kProjHeadsPerCta != 0) return REGENVC_ERR_UNSUPPORTED;
    if (!(rope_theta > 0.0f) || !std::isfinite(rope_theta) || !(eps >= 0.0f) || !std::isfinite(eps))
        return REGENVC_ERR_UNSUPPORTED;
    if (((uintptr_t)x | (uintptr_t)w_qkv | (uintptr_t)q_rot | (uintptr_t)b_qkv | (uintptr_t)g_q | (uintptr_t)g_k) & 15)
        return REGENVC_ERR_MISALIGNED;
    if ((uintptr_t)prepared & 255) return REGENVC_ERR_MISALIGNED;
    const size_t C = (size_t)n_heads * kHeadDim;
    const size_t xb = (size_t)n * C * 2, wb = 3 * C * C * 2, pb = operand_bytes(n, n_heads);
    if (overlaps(q_rot, xb, x, xb) || overlaps(q_rot, xb, w_qkv, wb) || overlaps(prepared, pb, x, xb) ||
        overlaps(prepared, pb, w_qkv, wb) || overlaps(prepared, pb, q_rot, xb))
        return REGENVC_ERR_ALIASING;

    std::lock_guard<std::mutex> lock(g_mu);
    int dev = 0;
    DeviceState* st = nullptr;
    rc = device_state(&dev, &st);
    if (rc != REGENVC_OK) return rc;
    // scratch for the norm's sums: the caller's workspace if one is set, else this thread's own
    const size_t need = proj_scratch_bytes(n, n_heads);
    char* ws = nullptr;
    Workspace* own = nullptr;
    if (tl_user_ws.ptr) {
        if (tl_user_ws.bytes < need) return REGENVC_ERR_WORKSPACE;
        ws = reinterpret_cast<char*>(tl_user_ws.ptr);
    } else {
        own = &st->workspace[std::this_thread::get_id()];
        rc = grow(own->buf, need);
        if (rc != REGENVC_OK) return rc;
        ws = reinterpret_cast<char*>(own->buf.ptr);
        rc = order_after_last_user(*own, (cudaStream_t)stream);
        if (rc != REGENVC_OK) return rc;
    }
    ProjParams pp;
    pp.unit_sums = reinterpret_cast<float*>(ws);
    pp.bias = reinterpret_cast<const float*>(b_qkv);
    pp.g_q = reinterpret_cast<const float*>(g_q);
    pp.g_k = reinterpret_cast<const float*>(g_k);
    pp.eps = eps;
    pp.n_tokens = (int)n;
    pp.n_pad = (int)n_pad;
    pp.C = (int)C;
    pp.h = n_heads;
    pp.grid = RopeGrid{nullptr, T, H, W};
    pp.status = st->status;
    rc = rope_table(*st, T, H, W, rope_theta, &pp.grid.tab);
    if (rc != REGENVC_OK) return rc;
    __half* kp = reinterpret_cast<__half*>(prepared);
    __half* vt = kp + (size_t)n_heads * n_pad * kHeadDim;
    CUtensorMap tmap_x, tmap_w, tmap_q, tmap_k, tmap_v;
    rc = make_tmap(&tmap_x, const_cast<void*>(x), C, (uint64_t)n, C * 2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
    if (rc == REGENVC_OK)
        rc = make_tmap(&tmap_w, const_cast<void*>(w_qkv), C, 3 * C, C * 2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
    if (rc == REGENVC_OK) rc = make_tmap(&tmap_q, q_rot, C, (uint64_t)n, C * 2);
    if (rc == REGENVC_OK) rc = make_tmap(&tmap_k, kp, kHeadDim, (uint64_t)n_heads * n_pad, kHeadDim * sizeof(__half));
    if (rc == REGENVC_OK)
        rc = make_tmap(&tmap_v, vt, (uint64_t)n_pad, (uint64_t)n_heads * kHeadDim, (uint64_t)n_pad * sizeof(__half));
    if (rc != REGENVC_OK) return rc;
    CUDA_TRY(launch_qkv_project_pair(tmap_x, tmap_w, tmap_q, tmap_k, tmap_v, pp, st->sm_count, (cudaStream_t)stream));
    launched();
    return own ? note_use(*own, (cudaStream_t)stream) : REGENVC_OK;
}

int regenvc_out_project(const void* attn_out, const void* w_o, const void* b_o, void* y, int n_tokens,
                        int n_heads, int head_dim, void* stream) {
    if (!attn_out || !w_o || !y) return REGENVC_ERR_NULL_POINTER;
    if (n_tokens < 1 || n_tokens > (1 << 30) || n_heads < 1 || n_heads > 65535 || head_dim < 1)
        return REGENVC_ERR_BAD_SHAPE;
    if (head_dim != kHeadDim || n_heads % kProjHeadsPerCta != 0) return REGENVC_ERR_UNSUPPORTED;
    if (((uintptr_t)attn_out | (uintptr_t)w_o | (uintptr_t)y | (uintptr_t)b_o) & 15) return REGENVC_ERR_MISALIGNED;
    const size_t C = (size_t)n_heads * kHeadDim;
    const size_t ob = (size_t)n_tokens * C * 2, wb = C * C * 2;
    if (overlaps(y, ob, attn_out, ob) || overlaps(y, ob, w_o, wb) || (b_o && overlaps(y, ob, b_o, C * 4)))
        return REGENVC_ERR_ALIASING;

    std::lock_guard<std::mutex> lock(g_mu);
    int dev = 0;
    DeviceState* st = nullptr;
    int rc = device_state(&dev, &st);
    if (rc != REGENVC_OK) return rc;
    ProjParams pp{};
    pp.bias = reinterpret_cast<const float*>(b_o);
    pp.n_tokens = n_tokens;
    pp.n_pad = (int)(((long long)n_tokens + kTile - 1) / kTile * kTile);
    pp.C = (int)C;
    pp.h = n_heads;
    pp.grid = RopeGrid{nullptr, 1, 1, 1};
    pp.status = st->status;
    CUtensorMap tmap_o, tmap_w, tmap_y;
    rc = make_tmap(&tmap_o, const_cast<void*>(attn_out), C, (uint64_t)n_tokens, C * 2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
    if (rc == REGENVC_OK)
        rc = make_tmap(&tmap_w, const_cast<void*>(w_o), C, C, C * 2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
    if (rc == REGENVC_OK) rc = make_tmap(&tmap_y, y, C, (uint64_t)n_tokens, C * 2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
    if (rc != REGENVC_OK) return rc;
    CUDA_TRY(launch_out_project(tmap_o, tmap_w, tmap_y, pp, st->sm_count, (cudaStream_t)stream));
    launched();
    return REGENVC_OK;
}

int regenvc_attn_forward_host(const void* q, const void* k, const void* v, void* out, int T, int H, int W, int n_heads,
                              int head_dim, float rope_theta, void* stream) {
    if (!q || !k || !v || !out) return REGENVC_ERR_NULL_POINTER;
    long long n = 0;
    int rc = check_self_args(T, H, W, rope_theta, &n);
    if (rc != REGENVC_OK) return rc;
    rc = validate(q, k, v, out, n, n, n_heads, head_dim, false);
    if (rc != REGENVC_OK) return rc;
    if (!(rope_theta > 0.0f) || !std::isfinite(rope_theta)) return REGENVC_ERR_UNSUPPORTED;
    return run_host(q, k, v, out, (int)n, (int)n, n_heads, true, T, H, W, rope_theta, (cudaStream_t)stream);
}

int regenvc_cross_attn_forward_host(const void* q, const void* k, const void* v, void* out, int n_q, int n_kv,
                                    int n_heads, int head_dim, void* stream) {
    int rc = validate(q, k, v, out, n_q, n_kv, n_heads, head_dim, false);
    if (rc != REGENVC_OK) return rc;
    return run_host(q, k, v, out, n_q, n_kv, n_heads, false, 1, 1, 1, 1.0f, (cudaStream_t)stream);
}

int regenvc_attn_partial(const void* q, const void* k, const void* v, void* o_part, void* ml, int T, int H, int W,
                         int q_token0, int n_q, int kv_token0, int n_kv, int n_heads, int head_dim, float rope_theta,
                         void* stream) {
    if (!q || !k || !v || !o_part || !ml) return REGENVC_ERR_NULL_POINTER;
    long long n = 0;
    int rc = check_self_args(T, H, W, rope_theta, &n);
    if (rc != REGENVC_OK) return rc;
    if (q_token0 < 0 || kv_token0 < 0 || n_q < 1 || n_kv < 1 || (long long)q_token0 + n_q > n ||
        (long long)kv_token0 + n_kv > n)
        return REGENVC_ERR_BAD_SHAPE;
    // the ordinary checks, with o_part standing in for out (it is larger, so an overlap test on it is stricter)
    rc = validate(q, k, v, o_part, n_q, n_kv, n_heads, head_dim, true);
    if (rc != REGENVC_OK) return rc;
    if (((uintptr_t)ml) & 15) return REGENVC_ERR_MISALIGNED;
    const size_t qb = (size_t)n_q * n_heads * head_dim * 2, kb = (size_t)n_kv * n_heads * head_dim * 2;
    const size_t ob = 2 * qb, mb = (size_t)n_q * n_heads * sizeof(float2);
    if (overlaps(o_part, ob, q, qb) || overlaps(o_part, ob, k, kb) || overlaps(o_part, ob, v, kb) ||
        overlaps(ml, mb, q, qb) || overlaps(ml, mb, k, kb) || overlaps(ml, mb, v, kb) || overlaps(ml, mb, o_part, ob))
        return REGENVC_ERR_ALIASING;
    if (!(rope_theta > 0.0f) || !std::isfinite(rope_theta)) return REGENVC_ERR_UNSUPPORTED;
    BlockArgs blk;
    blk.q_token0 = q_token0;
    blk.kv_token0 = kv_token0;
    blk.tok_o = reinterpret_cast<float*>(o_part);
    blk.tok_ml = reinterpret_cast<float2*>(ml);
    return enqueue(q, k, v, nullptr, n_q, n_kv, n_heads, true, T, H, W, rope_theta, (cudaStream_t)stream, blk);
}

int regenvc_attn_merge(const void* const* o_parts, const void* const* mls, int n_parts, void* out, int n_q,
                       int n_heads, int head_dim, void* stream) {
    if (!o_parts || !mls || !out) return REGENVC_ERR_NULL_POINTER;
    if (n_parts < 1 || n_parts > kMaxMergeParts || n_q < 1 || n_heads < 1) return REGENVC_ERR_BAD_SHAPE;
    if (n_q > (1 << 30) || n_heads > 65535 || (long long)n_q * n_heads >= (1ll << 31)) return REGENVC_ERR_BAD_SHAPE;
    if (head_dim != kHeadDim) return REGENVC_ERR_UNSUPPORTED;
    TokenMergeParams mp;
    const size_t rows = (size_t)n_q * n_heads;
    for (int i = 0; i < n_parts; ++i) {
        if (!o_parts[i] || !mls[i]) return REGENVC_ERR_NULL_POINTER;
        if ((((uintptr_t)o_parts[i]) | ((uintptr_t)mls[i])) & 15) return REGENVC_ERR_MISALIGNED;
        if (overlaps(out, rows * kHeadDim * 2, o_parts[i], rows * kHeadDim * 4) ||
            overlaps(out, rows * kHeadDim * 2, mls[i], rows * sizeof(float2)))
            return REGENVC_ERR_ALIASING;
        mp.o[i] = reinterpret_cast<const float*>(o_parts[i]);
        mp.ml[i] = reinterpret_cast<const float2*>(mls[i]);
    }
    if (((uintptr_t)out) & 15) return REGENVC_ERR_MISALIGNED;
    mp.n_parts = n_parts;
    mp.out = reinterpret_cast<__nv_bfloat16*>(out);
    mp.n_rows = (long long)rows;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        int dev = 0;
        DeviceState* st = nullptr;
        int rc = device_state(&dev, &st);
        if (rc != REGENVC_OK) return rc;
    }
    CUDA_TRY(launch_merge_token_partials(mp, (cudaStream_t)stream));
    launched();
    return REGENVC_OK;
}

int regenvc_ulysses_scatter_heads(const void* x_local, void* const* dst, int world, int n_local, int dst_token0,
                                  int n_heads, int head_dim, void* stream) {
    if (!x_local || !dst) return REGENVC_ERR_NULL_POINTER;
    if (world < 1 || world > kMaxReshardPeers || n_local < 0 || dst_token0 < 0 || n_heads < 1 || n_heads % world != 0)
        return REGENVC_ERR_BAD_SHAPE;
    if ((long long)(dst_token0 + (long long)n_local) * n_heads >= (1ll << 31)) return REGENVC_ERR_BAD_SHAPE;
    if (head_dim != kHeadDim) return REGENVC_ERR_UNSUPPORTED;
    if ((uintptr_t)x_local & 15) return REGENVC_ERR_MISALIGNED;
    ReshardParams rp{};
    rp.src = reinterpret_cast<const uint4*>(x_local);
    rp.world = world;
    rp.h_src = n_heads;
    rp.h_dst = n_heads / world;
    rp.dst_row0 = dst_token0;
    rp.dst_head0 = 0;
    const size_t src_bytes = (size_t)n_local * n_heads * kHeadDim * 2;
    for (int r = 0; r < world; ++r) {
        if (!dst[r]) return REGENVC_ERR_NULL_POINTER;
        if ((uintptr_t)dst[r] & 15) return REGENVC_ERR_MISALIGNED;
        const char* first = (const char*)dst[r] + (size_t)dst_token0 * rp.h_dst * kHeadDim * 2;
        if (overlaps(first, src_bytes / world, x_local, src_bytes)) return REGENVC_ERR_ALIASING;
        rp.dst[r] = reinterpret_cast<uint4*>(dst[r]);
        rp.row0[r] = 0;
        rp.rows[r] = n_local;
    }
    int sm_count = 0;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        int dev = 0;
        DeviceState* st = nullptr;
        int rc = device_state(&dev, &st);
        if (rc != REGENVC_OK) return rc;
        sm_count = st->sm_count;
    }
    if (n_local == 0) return REGENVC_OK;
    CUDA_TRY(launch_scatter_heads(rp, sm_count, (cudaStream_t)stream));
    launched();
    return REGENVC_OK;
}

int regenvc_ulysses_gather_heads(const void* x_heads, void* const* dst, const int* token0, const int* n_tokens,
                                 int world, int n_heads_local, int n_heads_dst, int dst_head0, int head_dim,
                                 void* stream) {
    if (!x_heads || !dst || !token0 || !n_tokens) return REGENVC_ERR_NULL_POINTER;
    if (world < 1 || world > kMaxReshardPeers || n_heads_local < 1 || n_heads_dst < n_heads_local || dst_head0 < 0 ||
        dst_head0 + n_heads_local > n_heads_dst)
        return REGENVC_ERR_BAD_SHAPE;
    if (head_dim != kHeadDim) return REGENVC_ERR_UNSUPPORTED;
    if ((uintptr_t)x_heads & 15) return REGENVC_ERR_MISALIGNED;
    ReshardParams rp{};
    rp.src = reinterpret_cast<const uint4*>(x_heads);
    rp.world = world;
    rp.h_src = n_heads_local;
    rp.h_dst = n_heads_dst;
    rp.dst_row0 = 0;
    rp.dst_head0 = dst_head0;
    long long total = 0;
    for (int r = 0; r < world; ++r) {
        if (!dst[r]) return REGENVC_ERR_NULL_POINTER;
        if ((uintptr_t)dst[r] & 15) return REGENVC_ERR_MISALIGNED;
        if (token0[r] < 0 || n_tokens[r] < 0) return REGENVC_ERR_BAD_SHAPE;
        if (((long long)token0[r] + n_tokens[r]) * n_heads_dst >= (1ll << 31)) return REGENVC_ERR_BAD_SHAPE;
        const char* from = (const char*)x_heads + (size_t)token0[r] * n_heads_local * kHeadDim * 2;
        if (overlaps(dst[r], (size_t)n_tokens[r] * n_heads_dst * kHeadDim * 2, from,
                     (size_t)n_tokens[r] * n_heads_local * kHeadDim * 2))
            return REGENVC_ERR_ALIASING;
        rp.dst[r] = reinterpret_cast<uint4*>(dst[r]);
        rp.row0[r] = token0[r];
        rp.rows[r] = n_tokens[r];
        total += n_tokens[r];
    }
    int sm_count = 0;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        int dev = 0;
        DeviceState* st = nullptr;
        int rc = device_state(&dev, &st);
        if (rc != REGENVC_OK) return rc;
        sm_count = st->sm_count;
    }
    if (total == 0) return REGENVC_OK;
    CUDA_TRY(launch_gather_heads(rp, sm_count, (cudaStream_t)stream));
    launched();
    return REGENVC_OK;
}

size_t regenvc_workspace_bytes(int n_kv, int n_heads, int head_dim) {
    if (n_kv < 1 || n_heads < 1 || head_dim != kHeadDim) return 0;
    return workspace_need(n_kv, n_heads);
}

int regenvc_set_workspace(void* dev_ptr, size_t bytes) {
    if (!dev_ptr || bytes == 0) {
        tl_user_ws = Buf{};
        return REGENVC_OK;
    }
    if ((uintptr_t)dev_ptr & 255) return REGENVC_ERR_WORKSPACE;
    tl_user_ws.ptr = dev_ptr;
    tl_user_ws.bytes = bytes;
    return REGENVC_OK;
}

int regenvc_device_status(void* stream, int* status_out) {
    if (!status_out) return REGENVC_ERR_NULL_POINTER;
    std::lock_guard<std::mutex> lock(g_mu);
    int dev = 0;
    DeviceState* st = nullptr;
    int rc = device_state(&dev, &st);
    if (rc != REGENVC_OK) return rc;
    CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    int h = 0;
    CUDA_TRY(cudaMemcpy(&h, st->status, sizeof(int), cudaMemcpyDeviceToHost));
    if (h != 0) CUDA_TRY(cudaMemset(st->status, 0, sizeof(int)));
    *status_out = h;
    return REGENVC_OK;
}

int regenvc_debug_set_phases(int mask) {
    if (mask < 1 || mask > 63 || !(mask & 3) || (mask & 24) == 24 || (mask & 48) == 48) return REGENVC_ERR_BAD_SHAPE;
    tl_phases = mask;
    return REGENVC_OK;
}

int regenvc_debug_expire_wait(int limit_us, void* stream) {
    if (limit_us < 1 || limit_us > 100000) return REGENVC_ERR_BAD_SHAPE;
    int* status = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        int dev = 0;
        DeviceState* st = nullptr;
        int rc = device_state(&dev, &st);
        if (rc != REGENVC_OK) return rc;
        status = st->status;
    }
    CUDA_TRY(launch_expire_wait(status, (unsigned long long)limit_us * 1000ull, (cudaStream_t)stream));
    launched();
    return REGENVC_OK;
}

const char* regenvc_status_string(int status) {
    switch (status) {
        case REGENVC_OK: return "ok";
        case REGENVC_ERR_NULL_POINTER: return "null pointer";
        case REGENVC_ERR_BAD_SHAPE: return "bad shape";
        case REGENVC_ERR_UNSUPPORTED: return "unsupported (head_dim must be 128, theta > 0, device sm_100)";
        case REGENVC_ERR_MISALIGNED: return "device pointer not 16-byte aligned";
        case REGENVC_ERR_ALIASING: return "out overlaps an input";
        case REGENVC_ERR_CUDA: return "CUDA call failed";
        case REGENVC_ERR_TIMEOUT: return "device-side bounded wait expired";
        case REGENVC_ERR_WORKSPACE: return "workspace too small or misaligned";
        case REGENVC_ERR_RANGE: return "input outside the fp16 operand range";
        case REGENVC_ERR_STATIC_LIMIT: return "shape exceeds the built-in scratch of the allocation-free entry point";
        case REGENVC_ERR_INTERNAL: return "a kernel found its launch assumptions broken and did no work";
        default: return "unknown status";
    }
}

const char* regenvc_last_cuda_error(void) { return tl_cuda_error.c_str(); }

const char* regenvc_version(void) { return "regenvc-attn 0.1 (sm_100a)"; }

unsigned long long regenvc_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

void regenvc_shutdown(void) {
    std::lock_guard<std::mutex> lock(g_mu);
    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess) {
        (void)cudaGetLastError();
        g_dev.clear();
        return;
    }
    for (auto& kv : g_dev) {
        if (cudaSetDevice(kv.first) != cudaSuccess) continue;
        DeviceState& st = kv.second;
        if (st.status) cudaFree(st.status);
        for (RopeEntry& e : st.ropes) cudaFree(e.dev);
        for (auto& w : st.workspace) {
            cudaFree(w.second.buf.ptr);
            if (w.second.last_use) cudaEventDestroy(w.second.last_use);
        }
        for (auto& s : st.staging)
            for (Buf& b : s.second) cudaFree(b.ptr);
        for (auto& hp : st.pipes) {
            HostPipe& h = hp.second;
            if (!h.made) continue;
            cudaStreamDestroy(h.in);
            cudaStreamDestroy(h.out);
            cudaEventDestroy(h.start);
            cudaEventDestroy(h.kv);
            cudaEventDestroy(h.fin);
            for (int c = 0; c < kMaxHostChunks; ++c) {
                cudaEventDestroy(h.q[c]);
                cudaEventDestroy(h.done[c]);
            }
        }
    }
    g_dev.clear();
    cudaSetDevice(prev);
    (void)cudaGetLastError();
}

}  // extern "C"
