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
    RopeGrid grid;
    int* status;
};

struct AttnParams {
    const __nv_bfloat16* q;   // [n_q, h, 128]
    __nv_bfloat16* out;       // [n_q, h, 128]
    int n_q, n_kv, n_kv_pad, h;
    int rope;
    RopeGrid grid;
    float scale_log2;         // log2(e) / sqrt(head_dim)
    int* status;
    int sm_count;
};

// Launchers (each returns the launch error, enqueues on `stream`).
cudaError_t launch_prep_kv(const PrepParams& p, cudaStream_t stream);

}  // namespace regenvc
