// Internal declarations shared by the host API and the kernels' launchers.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace regenvc {

constexpr int kHeadDim = 128;
constexpr int kTile = 128;          // keys per K/V tile and query rows per Q tile
constexpr int kPairsT = 22;         // rotary pairs on the t axis (width 44)
constexpr int kPairsY = 21;         // y axis (width 42)
constexpr int kPairsX = 21;         // x axis (width 42)

// Sticky device status codes (mirror regenvc_status).
constexpr int kStatusTimeout = 7;
constexpr int kStatusRange = 9;
constexpr int kStatusInternal = 11;

// cos/sin table of one (T, H, W, theta): float2 (cos, sin) entries,
// [T][22] then [H][21] then [W][21].
struct RopeGrid {
    const float2* tab;
    int T, H, W;
};

__host__ __device__ inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

struct PrepParams {
    const __nv_bfloat16* k;   // [n_kv, h, 128]
    const __nv_bfloat16* v;   // [n_kv, h, 128]
    __half* kp;               // [h][n_kv_pad][128]
    __half* vt;               // [h][128][n_kv_pad]
    int n_kv, n_kv_pad, h;
    int rope;                 // 1: rotate k by the 3D rotary embedding
    int k_bf16;               // 1: K' keeps the bf16 bits of k (no rotation, no conversion); 0: fp16
    RopeGrid grid;
    int pos_offset;           // token index (in the T x H x W grid) of row 0 of k
    int* status;
};

struct AttnParams {
    const __nv_bfloat16* q;   // [n_q, h, 128]
    __nv_bfloat16* out;       // [n_q, h, 128]
    int n_q, n_kv, n_kv_pad, h;
    int rope;
    int qk_bf16;              // 1: the query tiles and K' are bf16 (Q.K^T runs bf16 x bf16), 0: fp16
    RopeGrid grid;
    float scale_log2;         // log2(e) / sqrt(head_dim)
    int* status;
    int sm_count;
    // Work decomposition of the pipelined kernel.  A work item is one head and 256 query rows; items are
    // numbered head-major.  The first n_full_items CTAs each run one item over all keys.  Each of the remaining
    // items is cut into split_k pieces of tiles_per_piece key tiles, one CTA per piece, which leave
    // unnormalised partial results in part_o / part_ml for the merge kernel.
    int pairs_per_head;       // items per head = ceil(n_q / 256)
    int n_full_items;
    int split_k;              // >= 1
    int tiles_per_piece;
    int q_pos_offset;         // token index (in the T x H x W grid) of row 0 of q
    // Token-major partial output (block-wise attention for ring-style merging): when tok_o is not null every
    // CTA leaves its unnormalised result here instead of writing `out`.
    float* tok_o;             // [n_q, h, 128] fp32, sum_m 2^(s_m c - m_row) v_m
    float2* tok_ml;           // [n_q, h] (m_row in log2 units, l_row)
    float* part_o;            // [piece CTA][256 rows][128] fp32, sum_m p_m v_m against the piece's reference
    float2* part_ml;          // [piece CTA][256 rows] (reference m in log2 units, row sum l)
};

// QKV projection with fused norm / rotation / operand-layout epilogue (producer of the attention operands), on pairs
// of CTAs (qkv_project_pair.cu).
constexpr int kProjHeadsPerCta = 2;   // a slice of the projection kernels is 256 output features = two heads
struct ProjParams {
    const float* bias;        // [3C] or nullptr
    const float* g_q;         // [C] RMS-norm gains of q (nullptr: ones)
    const float* g_k;         // [C]
    float eps;
    int n_tokens, n_pad, C, h;
    RopeGrid grid;
    int* status;
    // scratch of the norm's sum over all features: the partial row sums of every (128-token tile, q/k/v) unit and
    // slice, [unit][slice][128 tokens]; a slot that still holds the all-ones pattern has not been written yet
    float* unit_sums;
};
// Bytes of that scratch for n_tokens tokens and h heads.
inline size_t proj_scratch_bytes(long long n_tokens, int h) {
    const size_t n_units = 3 * (size_t)((n_tokens + kTile - 1) / kTile);
    return n_units * (size_t)(h / kProjHeadsPerCta) * kTile * sizeof(float);
}
cudaError_t configure_qkv_project_pair();
cudaError_t launch_qkv_project_pair(const CUtensorMap& tmap_x, const CUtensorMap& tmap_w, const CUtensorMap& tmap_q,
                                    const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, const ProjParams& p,
                                    int sm_count, cudaStream_t stream);
// Output projection y = o W_o^T + b_o (bf16 in, bf16 out) on pairs of CTAs (out_project_pair.cu); of ProjParams it
// reads bias ([C] or nullptr), n_tokens, C, h and status.
cudaError_t configure_out_project();
cudaError_t launch_out_project(const CUtensorMap& tmap_o, const CUtensorMap& tmap_w, const CUtensorMap& tmap_y,
                               const ProjParams& p, int sm_count, cudaStream_t stream);

// Merge of token-major partial results of several key/value blocks.
constexpr int kMaxMergeParts = 8;
struct TokenMergeParams {
    const float* o[kMaxMergeParts];
    const float2* ml[kMaxMergeParts];
    int n_parts;
    __nv_bfloat16* out;       // [n_q, h, 128]
    long long n_rows;         // n_q * h
};

struct MergeParams {
    const float* part_o;
    const float2* part_ml;
    __nv_bfloat16* out;       // [n_q, h, 128]
    int n_q, h;
    int pairs_per_head, n_full_items, split_k, n_split_items;
};

// Head <-> sequence resharding (Ulysses, Sec. 3.5).  Rows are (token, head) vectors of 128 bf16 = 16 uint4.
//   scatter: src [n_rows][h_src] -> for every destination r: dst[r][(dst_row0 + n)][h_dst] = src[n][r * h_dst + .]
//   gather : src [.][h_src]      -> for every destination r: dst[r][n][dst_head0 + .] = src[row0[r] + n][.],
//            n < rows[r], destination rows holding h_dst heads
constexpr int kMaxReshardPeers = 16;
struct ReshardParams {
    const uint4* src;
    uint4* dst[kMaxReshardPeers];
    int row0[kMaxReshardPeers];   // gather: first source row of destination r
    int rows[kMaxReshardPeers];   // rows copied to destination r (scatter: all equal to the source's row count)
    int world;
    int h_src, h_dst;
    int dst_row0;                 // scatter only
    int dst_head0;                // gather only
};
cudaError_t launch_scatter_heads(const ReshardParams& p, int sm_count, cudaStream_t stream);
cudaError_t launch_gather_heads(const ReshardParams& p, int sm_count, cudaStream_t stream);

// One warp that waits `limit_ns` on a barrier nothing completes and then records kStatusTimeout (test aid).
cudaError_t launch_expire_wait(int* status, unsigned long long limit_ns, cudaStream_t stream);

// Host-side bookkeeping shared by the files that implement entry points: every kernel launch is counted
// (regenvc_kernel_launch_count), and a failing CUDA call leaves its text for regenvc_last_cuda_error(), clears the
// runtime's error state and maps to REGENVC_ERR_CUDA.
void count_launch();
int record_cuda_failure(cudaError_t e, const char* what);

// Launchers (each returns the launch error, enqueues on `stream`).
cudaError_t launch_prep_kv(const PrepParams& p, cudaStream_t stream);
// tmap_q != nullptr: the query tiles are copied by TMA from a 16-bit tensor already in operand form (same type as
// K'); nullptr: the kernel reads p.q (bf16), rotates if p.rope and converts to fp16 itself.
cudaError_t launch_attn_pipelined(const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, const CUtensorMap& tmap_out,
                                  const CUtensorMap* tmap_q, const AttnParams& p, cudaStream_t stream);
// Persistent form for short key sequences (one CTA per SM walks over its work items; query tiles by TMA only).
constexpr int kPersistentMaxTiles = 8;
cudaError_t configure_attn_persistent();
cudaError_t launch_attn_persistent(const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, const CUtensorMap& tmap_out,
                                   const CUtensorMap& tmap_q, const AttnParams& p, int n_ctas, cudaStream_t stream);
// Kernel on pairs of CTAs (attn_pair.cu): a persistent grid of clusters of two walks over the work items; tmap_k /
// tmap_v with boxes of 64 rows.  The host uses it for key sequences of at least kPairMinTiles tiles.
// configure_attn_pair reports how many pairs the device holds at a time (the grid size); a launch covers at most
// that many times kPairMaxItemsPerPair units of work as a persistent grid (more: one cluster per unit).  (max_clusters
// < 0 in launch_attn_pair, a test aid: a grid of at most -max_clusters pairs.)
constexpr int kPairMinTiles = 32;
constexpr int kPairMaxItemsPerPair = 256;
cudaError_t configure_attn_pair(int* max_clusters);
cudaError_t launch_attn_pair(const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, const CUtensorMap& tmap_out,
                             const CUtensorMap* tmap_q, const AttnParams& p, int max_clusters, cudaStream_t stream);
cudaError_t configure_attn_pipelined();   // once per device: register hand-over check, large dynamic shared memory
cudaError_t launch_merge_partials(const MergeParams& p, cudaStream_t stream);
cudaError_t launch_merge_token_partials(const TokenMergeParams& p, cudaStream_t stream);

// Bytes of the partial-result scratch that follows K' and V't in the workspace: room for up to
// kMaxPieceCtas piece CTAs (never more than one wave of SMs is cut into pieces).
constexpr int kMaxPieceCtas = 160;
constexpr size_t kPieceBytes = 2 * kTile * kHeadDim * sizeof(float) + 2 * kTile * sizeof(float2);
constexpr size_t kSplitScratchBytes = kMaxPieceCtas * kPieceBytes;

}  // namespace regenvc
