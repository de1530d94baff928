// Cross-attention entry point that performs no device allocation: its scratch (the fp16 operand forms of
// the conditioning keys and values) lives in a fixed array inside the library image.
#include <cmath>
#include <map>
#include <mutex>
#include <string>

#include "../../include/regenvc_attn.h"
#include "common.cuh"

namespace {

using namespace regenvc;

// Scratch of the allocation-free entry point.  Every GPU that loads the library holds these bytes from
// load to exit.  In HOST code the names below are only handles of the symbols, not device addresses: the
// device addresses are fetched once per device with cudaGetSymbolAddress() and passed to the kernels.
static __device__ __align__(256) unsigned char g_static_scratch[REGENVC_STATIC_SCRATCH_BYTES];
static __device__ int g_static_status;  // sticky device status of this entry point (0 = ok)

struct StaticDevice {
    unsigned char* scratch = nullptr;  // device address of g_static_scratch on this device
    int* status = nullptr;             // device address of g_static_status on this device
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

std::mutex g_static_mu;
std::map<int, StaticDevice> g_static_dev;
EncodeTiledFn g_static_encode = nullptr;

// One-time set-up for the current device: capability check, kernel attributes, symbol addresses.  Nothing here
// allocates device memory.
int static_setup(StaticDevice** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_failure(e, "cudaGetDevice");
    auto it = g_static_dev.find(dev);
    if (it != g_static_dev.end()) {
        *out = &it->second;
        return REGENVC_OK;
    }
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return record_cuda_failure(e, "cudaDeviceGetAttribute");
    if (major != 10) return REGENVC_ERR_UNSUPPORTED;
    if (!g_static_encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || !fn || qres != cudaDriverEntryPointSuccess)
            return record_cuda_failure(e == cudaSuccess ? cudaErrorNotSupported : e, "cuTensorMapEncodeTiled lookup");
        g_static_encode = (EncodeTiledFn)fn;
    }
    e = configure_attn_pipelined();
    if (e != cudaSuccess) return record_cuda_failure(e, "kernel attributes of the attention kernel");
    StaticDevice d;
    e = cudaGetSymbolAddress((void**)&d.scratch, g_static_scratch);
    if (e != cudaSuccess || !d.scratch)
        return record_cuda_failure(e == cudaSuccess ? cudaErrorInvalidSymbol : e, "cudaGetSymbolAddress(scratch array)");
    e = cudaGetSymbolAddress((void**)&d.status, g_static_status);
    if (e != cudaSuccess || !d.status)
        return record_cuda_failure(e == cudaSuccess ? cudaErrorInvalidSymbol : e, "cudaGetSymbolAddress(status word)");
    *out = &(g_static_dev[dev] = d);
    return REGENVC_OK;
}

bool ranges_overlap(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + nb && b0 < a0 + na;
}

int encode_map(CUtensorMap* m, CUtensorMapDataType type, void* base, uint64_t inner, uint64_t outer, uint64_t row_bytes) {
    const cuuint64_t gdim[2] = {inner, outer};
    const cuuint64_t gstride[1] = {row_bytes};
    const cuuint32_t box[2] = {64, 128};
    const cuuint32_t estr[2] = {1, 1};
    if (g_static_encode(m, type, 2, base, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return record_cuda_failure(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return REGENVC_OK;
}

}  // namespace

extern "C" int regenvc_cross_attn_forward_static(const void* q, const void* k, const void* v, void* out, int n_q,
                                                 int n_kv, int n_heads, int head_dim, void* stream) {
    if (!q || !k || !v || !out) return REGENVC_ERR_NULL_POINTER;
    if (n_q < 1 || n_kv < 1 || n_heads < 1 || head_dim < 1) return REGENVC_ERR_BAD_SHAPE;
    if (n_q > (1 << 30) || n_kv > (1 << 30) || n_heads > 65535 || (long long)n_q * n_heads >= (1ll << 31))
        return REGENVC_ERR_BAD_SHAPE;
    if (head_dim != kHeadDim) return REGENVC_ERR_UNSUPPORTED;
    if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15) return REGENVC_ERR_MISALIGNED;
    const size_t qb = (size_t)n_q * n_heads * kHeadDim * 2, kb = (size_t)n_kv * n_heads * kHeadDim * 2;
    if (ranges_overlap(out, qb, q, qb) || ranges_overlap(out, qb, k, kb) || ranges_overlap(out, qb, v, kb))
        return REGENVC_ERR_ALIASING;
    const long long kv_pad = ((long long)n_kv + kTile - 1) / kTile * kTile;
    const unsigned long long need = 2ull * (unsigned long long)n_heads * (unsigned long long)kv_pad * kHeadDim * sizeof(__half);
    if (need > (unsigned long long)REGENVC_STATIC_SCRATCH_BYTES) return REGENVC_ERR_STATIC_LIMIT;

    std::lock_guard<std::mutex> lock(g_static_mu);
    StaticDevice* dev = nullptr;
    int rc = static_setup(&dev);
    if (rc != REGENVC_OK) return rc;

    __half* kp = reinterpret_cast<__half*>(dev->scratch);
    __half* vt = kp + (size_t)n_heads * kv_pad * kHeadDim;
    // as in regenvc_cross_attn_forward(): queries and keys stay bf16, the query tiles are copied by TMA
    CUtensorMap tmap_k, tmap_v, tmap_out, tmap_q;
    rc = encode_map(&tmap_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, kp, kHeadDim, (uint64_t)n_heads * kv_pad,
                    kHeadDim * sizeof(__half));
    if (rc == REGENVC_OK)
        rc = encode_map(&tmap_v, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, vt, (uint64_t)kv_pad, (uint64_t)n_heads * kHeadDim,
                        (uint64_t)kv_pad * sizeof(__half));
    if (rc == REGENVC_OK)
        rc = encode_map(&tmap_out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, out, (uint64_t)n_heads * kHeadDim, (uint64_t)n_q,
                        (uint64_t)n_heads * kHeadDim * sizeof(__nv_bfloat16));
    if (rc == REGENVC_OK)
        rc = encode_map(&tmap_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, const_cast<void*>(q), (uint64_t)n_heads * kHeadDim,
                        (uint64_t)n_q, (uint64_t)n_heads * kHeadDim * sizeof(__nv_bfloat16));
    if (rc != REGENVC_OK) return rc;

    PrepParams pp;
    pp.k = reinterpret_cast<const __nv_bfloat16*>(k);
    pp.v = reinterpret_cast<const __nv_bfloat16*>(v);
    pp.kp = kp;
    pp.vt = vt;
    pp.n_kv = n_kv;
    pp.n_kv_pad = (int)kv_pad;
    pp.h = n_heads;
    pp.rope = 0;
    pp.k_bf16 = 1;
    pp.grid = RopeGrid{nullptr, 1, 1, 1};
    pp.pos_offset = 0;
    pp.status = dev->status;
    cudaError_t e = launch_prep_kv(pp, (cudaStream_t)stream);
    if (e != cudaSuccess) return record_cuda_failure(e, "launch of the key/value preparation kernel");
    count_launch();

    AttnParams ap;
    ap.q = reinterpret_cast<const __nv_bfloat16*>(q);
    ap.out = reinterpret_cast<__nv_bfloat16*>(out);
    ap.n_q = n_q;
    ap.n_kv = n_kv;
    ap.n_kv_pad = (int)kv_pad;
    ap.h = n_heads;
    ap.rope = 0;
    ap.qk_bf16 = 1;
    ap.grid = pp.grid;
    ap.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)kHeadDim));
    ap.status = dev->status;
    ap.sm_count = 0;
    ap.pairs_per_head = (n_q + 2 * kTile - 1) / (2 * kTile);
    ap.n_full_items = ap.pairs_per_head * n_heads;  // no key-range pieces: they would need more scratch
    ap.split_k = 1;
    ap.tiles_per_piece = (int)(kv_pad / kTile);
    ap.q_pos_offset = 0;
    ap.tok_o = nullptr;
    ap.tok_ml = nullptr;
    ap.part_o = nullptr;
    ap.part_ml = nullptr;
    e = launch_attn_pipelined(tmap_k, tmap_v, tmap_out, &tmap_q, ap, (cudaStream_t)stream);
    if (e != cudaSuccess) return record_cuda_failure(e, "launch of the attention kernel");
    count_launch();
    return REGENVC_OK;
}

extern "C" int regenvc_static_device_status(void* stream, int* status_out) {
    if (!status_out) return REGENVC_ERR_NULL_POINTER;
    std::lock_guard<std::mutex> lock(g_static_mu);
    StaticDevice* dev = nullptr;
    int rc = static_setup(&dev);
    if (rc != REGENVC_OK) return rc;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return record_cuda_failure(e, "cudaStreamSynchronize");
    int h = 0;
    e = cudaMemcpy(&h, dev->status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return record_cuda_failure(e, "cudaMemcpy(status word of the built-in scratch)");
    if (h != 0) {
        e = cudaMemset(dev->status, 0, sizeof(int));
        if (e != cudaSuccess) return record_cuda_failure(e, "cudaMemset(status word of the built-in scratch)");
    }
    *status_out = h;
    return REGENVC_OK;
}
