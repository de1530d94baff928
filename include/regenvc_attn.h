/*
 * regenvc_attn.h -- C ABI of the B200 (sm_100a) fused 3D-RoPE attention library.
 *
 * The operation is the attention step of the paper's real-time decoder: every
 * block of the four-step diffusion transformer runs exact, non-causal
 * multi-head softmax attention over the whole flattened T x H x W latent-token
 * sequence of a 25-frame window (Sec. 3.5: after the Ulysses exchange a
 * device holds some of the heads and attends over the whole sequence for
 * them; here that is done for all heads on one GPU with no sharding), and
 * cross-attention of the same queries to the short, precomputed text/image
 * conditioning key/value tensors (Sec. 3.9).  The backbone's 3D rotary
 * position embedding is applied to queries and keys inside the call.
 *
 * Conventions common to every entry point
 *   - Tensors are bf16, contiguous, layout [tokens, n_heads, head_dim];
 *     token n of a T x H x W grid is n = (t*H + y)*W + x.  Batch is 1; a
 *     caller with several windows loops (or gives each GPU its own window).
 *   - head_dim must be 128.  Rotary pairs are the adjacent elements
 *     (2j, 2j+1); head_dim is split 44/42/42 over (t, y, x), each axis a 1-D
 *     rotary embedding of its own width with frequencies theta^(-2i/width).
 *     Scores are scaled by 1/sqrt(head_dim).  No mask.
 *   - Arithmetic: inputs are widened exactly; rotated Q/K, V and the softmax
 *     probabilities are rounded to fp16 tensor-core operands (inputs must
 *     therefore be finite with |x| <= 65504); where nothing is rotated
 *     (cross-attention) Q and K enter Q.K^T as the bf16 values they are; all
 *     accumulation is fp32; the output is rounded once to bf16 (nearest
 *     even).  NaN/Inf inputs give unspecified results.
 *   - Pointers marked "device" must be valid on the current CUDA device and
 *     16-byte aligned; the caller owns them, and the library neither frees
 *     nor keeps them beyond the stream-ordered work of the call.
 *   - Device entry points are asynchronous on `stream` (a cudaStream_t cast
 *     to void*, NULL = legacy default stream) and never synchronise the host
 *     once the workspace and the rotary table for the shape exist.  Such a
 *     warm call only enqueues kernels (their parameters, tensor maps
 *     included, travel by value), so a sequence of warm calls can be
 *     recorded into a CUDA graph and replayed on new values in the same
 *     buffers (regenvc_attn_forward, regenvc_cross_attn_forward,
 *     regenvc_attn_partial, regenvc_attn_merge, the resharding calls; not
 *     the *_host variants, which copy and wait).
 *   - Errors are return codes only; arguments are validated before any CUDA
 *     work is enqueued, and a failing call enqueues nothing.
 *   - There is no CPU path: on a machine without an sm_100 GPU every compute
 *     entry point returns REGENVC_ERR_UNSUPPORTED or REGENVC_ERR_CUDA.
 *   - Calls on one stream are ordered as usual.  Calls that overlap on the
 *     GPU (different streams) must not share a workspace: give each stream
 *     its own with regenvc_set_workspace() from the thread that launches on
 *     it (the setting is per host thread), or serialise them.
 */
#ifndef REGENVC_ATTN_H
#define REGENVC_ATTN_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    REGENVC_OK = 0,
    REGENVC_ERR_NULL_POINTER = 1,
    REGENVC_ERR_BAD_SHAPE = 2,   /* a dimension < 1 or a size that overflows */
    REGENVC_ERR_UNSUPPORTED = 3, /* head_dim != 128, theta <= 0, device is not sm_100 */
    REGENVC_ERR_MISALIGNED = 4,  /* a device pointer is not 16-byte aligned */
    REGENVC_ERR_ALIASING = 5,    /* out overlaps q, k or v */
    REGENVC_ERR_CUDA = 6,        /* a CUDA call failed: see regenvc_last_cuda_error() */
    REGENVC_ERR_TIMEOUT = 7,     /* a bounded device-side wait expired (sticky device status) */
    REGENVC_ERR_WORKSPACE = 8,   /* caller-supplied workspace too small or misaligned */
    REGENVC_ERR_RANGE = 9,       /* an input exceeded the fp16 operand range (sticky device status) */
    REGENVC_ERR_STATIC_LIMIT = 10, /* regenvc_cross_attn_forward_static(): the shape needs more than the built-in scratch */
    REGENVC_ERR_INTERNAL = 11     /* a kernel found an assumption about its launch broken and did no work (sticky device
                                     status): the dynamic shared memory of the persistent attention kernel did not
                                     start on a 1024-byte boundary */
} regenvc_status;

/*
 * Self-attention with fused 3D RoPE (Sec. 3.5; rotary convention as above).
 *   q, k, v : device, bf16 [T*H*W, n_heads, head_dim]           (read only)
 *   out     : device, bf16 [T*H*W, n_heads, head_dim]           (written; must not overlap q/k/v)
 *   rope_theta : rotary base (> 0), 10000 for the paper's backbone
 * out[n, a, :] = sum_m softmax_m( <R(n) q[n,a], R(m) k[m,a]> / sqrt(head_dim) ) v[m,a, :]
 * Returns REGENVC_OK once the work is enqueued on `stream`.
 */
int regenvc_attn_forward(const void* q, const void* k, const void* v, void* out,
                         int T, int H, int W, int n_heads, int head_dim,
                         float rope_theta, void* stream);

/*
 * Cross-attention to a short conditioning sequence (Sec. 3.9: keys/values of
 * the 512 text tokens or the 257 image tokens, computed once per sequence).
 * No rotation, no mask.
 *   q, out : device, bf16 [n_q, n_heads, head_dim]
 *   k, v   : device, bf16 [n_kv, n_heads, head_dim]
 */
int regenvc_cross_attn_forward(const void* q, const void* k, const void* v, void* out,
                               int n_q, int n_kv, int n_heads, int head_dim, void* stream);

/*
 * Conditioning keys/values prepared once (Sec. 3.9: the text and image conditioning key/value tensors are
 * computed once per sequence and reused by every block, step and window).  regenvc_cross_attn_forward()
 * rewrites k and v into tensor-core operand form on every call; these three calls split that off:
 *
 * regenvc_prepared_bytes(): size of the operand buffer for n_kv keys (0 for invalid arguments):
 *   K' : 16-bit [n_heads][n_kv_pad][128], then V't : fp16 [n_heads][128][n_kv_pad], n_kv_pad = n_kv rounded up
 *   to a multiple of 128, padding zero.
 * regenvc_cross_kv_prepare(): fills `prepared` (device, caller-owned, 256-byte aligned, at least
 *   regenvc_prepared_bytes() bytes, not overlapping k or v) from k, v [n_kv, n_heads, head_dim] bf16.  K' keeps
 *   the bf16 bits of k; V't is v converted to fp16 and transposed.  An element of v beyond the fp16 range sets
 *   the sticky REGENVC_ERR_RANGE status.
 * regenvc_cross_attn_forward_prepared(): regenvc_cross_attn_forward() on a buffer filled by the call above
 *   (same n_kv and n_heads); bit-identical result, one kernel instead of two.  `prepared` is only read, so
 *   calls on different streams may share it; the thread's workspace is still used for split-key scratch.
 *
 * regenvc_attn_forward_prepared(): attention on operands a producer has already written in operand form
 *   (a fused QKV-projection epilogue: regenvc_qkv_rope_project()):
 *   q_rot    : device, fp16 [n_q, n_heads, 128], rotated queries
 *   prepared : K' fp16 (rotated keys) and V't fp16 in the layout above; the padding columns of V't must be finite
 *   out      : device, bf16 [n_q, n_heads, 128]
 *   No rotation, conversion or preparation pass happens inside the call.
 */
size_t regenvc_prepared_bytes(int n_kv, int n_heads, int head_dim);
int regenvc_cross_kv_prepare(const void* k, const void* v, void* prepared,
                             int n_kv, int n_heads, int head_dim, void* stream);
int regenvc_cross_attn_forward_prepared(const void* q, const void* prepared, void* out,
                                        int n_q, int n_kv, int n_heads, int head_dim, void* stream);
int regenvc_attn_forward_prepared(const void* q_rot, const void* prepared, void* out,
                                  int n_q, int n_kv, int n_heads, int head_dim, void* stream);

/*
 * Producer fusion: the QKV projection of a transformer block with the steps between it and the attention
 * kernel fused into its epilogue.  The paper takes the backbone by reference (Sec. 3.2, 3.4); in that block
 *     y_q = x W_q^T + b_q,  y_k = x W_k^T + b_k,  v = x W_v^T + b_v,
 *     q = y_q * g_q / sqrt(mean_c y_q[c]^2 + eps)   (RMS norm over ALL n_heads * 128 features of a token), k alike,
 * heads are consecutive blocks of 128 features, and q, k are then rotated by the 3D rotary embedding.  This call
 * computes all of it in one pass and writes the results directly in the operand form
 * regenvc_attn_forward_prepared() consumes, so that neither a preparation pass nor a bf16 round trip of q, k, v
 * exists on this path:
 *   x        : device, bf16 [T*H*W, C], C = n_heads * 128                     (read only)
 *   w_qkv    : device, bf16 [3C, C]; row f = weights of output feature f; rows 0..C-1 q, C..2C-1 k, 2C..3C-1 v
 *   b_qkv    : device, fp32 [3C], or NULL for no bias
 *   g_q, g_k : device, fp32 [C] norm gains, or NULL for ones;  eps >= 0
 *   q_rot    : device, fp16 [T*H*W, n_heads, 128]                              (written)
 *   prepared : device, 256-byte aligned, regenvc_prepared_bytes(T*H*W, n_heads, 128) bytes: K' then V't (written,
 *              padding zero)
 * Arithmetic: bf16 products accumulated in fp32, norm and rotation in fp32, one rounding to fp16.  A result
 * beyond the fp16 range sets the sticky REGENVC_ERR_RANGE status.  n_heads must be even (a thread block computes two
 * heads of a token tile): otherwise REGENVC_ERR_UNSUPPORTED.  The thread blocks that share a token tile exchange
 * their partial sums of squares through 6 * n_pad * n_heads bytes (n_pad = T*H*W rounded up to 128) of the calling
 * thread's workspace -- regenvc_workspace_bytes(T*H*W, n_heads, 128) is always enough for a caller-supplied one --
 * and wait for each other with the same bounded waits as everything else (the grid never exceeds what the device
 * holds at once; REGENVC_ERR_TIMEOUT if the GPU is shared with work that keeps part of it from becoming resident for
 * half a second).  Asynchronous on `stream`; allocates
 * only the rotary table of a new (T, H, W, theta) and, the first time, the workspace.  Typical use:
 *     regenvc_qkv_rope_project(x, w, b, gq, gk, eps, q_rot, prepared, T, H, W, h, 128, theta, s);
 *     regenvc_attn_forward_prepared(q_rot, prepared, out, T*H*W, T*H*W, h, 128, s);
 */
int regenvc_qkv_rope_project(const void* x, const void* w_qkv, const void* b_qkv,
                             const void* g_q, const void* g_k, float eps,
                             void* q_rot, void* prepared,
                             int T, int H, int W, int n_heads, int head_dim,
                             float rope_theta, void* stream);

/*
 * The step behind the attention in the same block (backbone by reference, Sec. 3.2 / 3.4): its output projection
 *     y = o W_o^T + b_o
 * on the attention output exactly as the attention entry points leave it (the heads of a token side by side are
 * one row of C = n_heads * 128 features), with the bias and the rounding to bf16 in the epilogue:
 *   attn_out : device, bf16 [n_tokens, n_heads, 128]                           (read only)
 *   w_o      : device, bf16 [C, C]; row f = weights of output feature f
 *   b_o      : device, fp32 [C], or NULL for no bias
 *   y        : device, bf16 [n_tokens, C]                (written; must not overlap the inputs)
 * Arithmetic: bf16 products accumulated in fp32, bias added in fp32, one rounding to bf16.  n_heads must be even
 * (REGENVC_ERR_UNSUPPORTED otherwise).  No workspace, no allocation, asynchronous on `stream`.
 */
int regenvc_out_project(const void* attn_out, const void* w_o, const void* b_o, void* y,
                        int n_tokens, int n_heads, int head_dim, void* stream);

/*
 * Block-wise attention for sequence-parallel use (Sec. 3.5: Ring attention streams key/value blocks around
 * the devices and combines the per-block results by the online-softmax rule; the result is unsharded
 * attention, only summed in another order).
 *
 * regenvc_attn_partial(): attention of a contiguous range of query tokens against ONE contiguous range of
 * key/value tokens of the same T x H x W grid, left unnormalised.
 *   q            : device, bf16 [n_q, n_heads, head_dim], tokens q_token0 .. q_token0 + n_q - 1 of the grid
 *   k, v         : device, bf16 [n_kv, n_heads, head_dim], tokens kv_token0 .. kv_token0 + n_kv - 1
 *   o_part       : device, fp32 [n_q, n_heads, head_dim]  = sum_m 2^(s_m c - m_row) v_m over the block
 *                  (c = log2(e) / sqrt(head_dim), s_m the rotated score)
 *   ml           : device, float pairs [n_q, n_heads]     = (m_row in log2 units, l_row = sum_m 2^(s_m c - m_row))
 * Rotary positions are those of the tokens in the whole grid, so blocks computed on different devices merge
 * exactly.  m_row is a reference between 16 log2 units below and 4 above the block's row maximum (not
 * necessarily the maximum itself).
 *
 * regenvc_attn_merge(): out[n, a, :] = sum_i w_i o_i / sum_i w_i l_i with w_i = 2^(m_i - max_i m_i), rounded to
 * bf16, for n_parts (1..8) partial results of the same query range.  o_parts / mls are HOST arrays of device
 * pointers.  Merging the partials of a partition of the key range reproduces regenvc_attn_forward().
 */
int regenvc_attn_partial(const void* q, const void* k, const void* v, void* o_part, void* ml,
                         int T, int H, int W, int q_token0, int n_q, int kv_token0, int n_kv,
                         int n_heads, int head_dim, float rope_theta, void* stream);
int regenvc_attn_merge(const void* const* o_parts, const void* const* mls, int n_parts, void* out,
                       int n_q, int n_heads, int head_dim, void* stream);

/*
 * Head <-> sequence resharding of the Ulysses scheme (Sec. 3.5: an all-to-all moves the sequence sharding
 * into the head dimension before attention and back afterwards, so that each GPU attends over the whole
 * sequence for a subset of the heads).  These two calls are the data movement of that all-to-all for one
 * GPU of a group of `world` (1..16) GPUs; all tensors are bf16 with head_dim = 128, device pointers, 16-byte
 * aligned.  `dst` is a HOST array of `world` device pointers.  A destination may be memory of this GPU (a
 * send buffer that a collective ships afterwards) or a peer GPU's buffer mapped into this process: then the
 * stores cross NVLink and the call is the exchange itself.  The library only writes; ordering between GPUs
 * (nobody reads a buffer before all writers have finished, nobody overwrites one that is still being read)
 * is the caller's, by stream events or a barrier.  Asynchronous on `stream`; no allocation.
 *
 * regenvc_ulysses_scatter_heads(): x_local is this GPU's token range [n_local, n_heads, 128].  For every
 *   r < world: dst[r][dst_token0 + n, a, :] = x_local[n, r * n_heads / world + a, :], dst[r] laid out
 *   [tokens of the group, n_heads / world, 128].  n_heads must be a multiple of world.
 * regenvc_ulysses_gather_heads(): x_heads is this GPU's head range of all tokens of the group
 *   [*, n_heads_local, 128].  For every r < world: dst[r][n, dst_head0 + a, :] = x_heads[token0[r] + n, a, :]
 *   for n < n_tokens[r], dst[r] laid out [n_tokens[r], n_heads_dst, 128].  token0 / n_tokens are HOST arrays.
 * Errors: NULL_POINTER, BAD_SHAPE (world, head counts, negative sizes, 32-bit row index overflow),
 * UNSUPPORTED (head_dim), MISALIGNED, ALIASING (a destination range overlaps the source), CUDA.
 */
int regenvc_ulysses_scatter_heads(const void* x_local, void* const* dst, int world, int n_local,
                                  int dst_token0, int n_heads, int head_dim, void* stream);
int regenvc_ulysses_gather_heads(const void* x_heads, void* const* dst, const int* token0,
                                 const int* n_tokens, int world, int n_heads_local, int n_heads_dst,
                                 int dst_head0, int head_dim, void* stream);

/*
 * The same two operations for callers whose tensors live in HOST memory
 * (pinned memory gives asynchronous copies; pageable memory works but is
 * staged by the driver).  The call copies q, k, v to device staging buffers
 * that the library owns and reuses, runs the device path, copies the result
 * back into `out` and waits for `stream` before returning.  K and V are
 * copied first; the query rows follow in up to 8 blocks of about one wave
 * of work items, and the library's own copy-in and copy-out streams overlap
 * the transfer of a block with the attention of the previous one (all of it
 * ordered after the work already on `stream`).  The result equals the device
 * call's to the last bf16 step: a block is cut into work items of its own, so
 * a row can see another rounding of its fp16 probabilities.
 */
int regenvc_attn_forward_host(const void* q, const void* k, const void* v, void* out,
                              int T, int H, int W, int n_heads, int head_dim,
                              float rope_theta, void* stream);
int regenvc_cross_attn_forward_host(const void* q, const void* k, const void* v, void* out,
                                    int n_q, int n_kv, int n_heads, int head_dim, void* stream);

/*
 * Cross-attention for callers that must not allocate device memory.  (The paper has no counterpart: this
 * is a deployment variant of regenvc_cross_attn_forward(), same arguments, same result.)
 *
 * Who needs it: code in the steady-state window loop of a real-time decoder.  cudaMalloc and cudaFree
 * synchronise the whole device, so one allocation made on behalf of this library would stall the decode and
 * encode streams running beside it and break the per-window time budget; and a serving process whose
 * framework has already claimed nearly all device memory for its own pool may simply get an out-of-memory
 * error from a raw cudaMalloc.  regenvc_cross_attn_forward() can do both on its first call or when its
 * workspace has to grow.  This entry point never calls cudaMalloc, cudaFree or any allocating routine: the
 * fp16 operand forms of k and v go into a fixed REGENVC_STATIC_SCRATCH_BYTES array that is part of the
 * library image, so every GPU that loads the library holds those bytes until the process exits.
 *
 *   - Limit: 2 * n_heads * n_kv_pad * 256 bytes (n_kv_pad = n_kv rounded up to 128) must fit in the array,
 *     i.e. n_heads * n_kv_pad <= 32768 (12 heads x 2688 keys, 40 heads x 768 keys).  Larger shapes are
 *     rejected with REGENVC_ERR_STATIC_LIMIT and nothing is enqueued.  The key range is never cut into
 *     pieces here (that path needs extra scratch), so very long conditioning sequences run slower than
 *     through regenvc_cross_attn_forward().
 *   - The first call on each device looks up the device address of the array (and sets kernel attributes);
 *     make that call during start-up, before any stream capture is begun.
 *   - All calls on a device share the one array, which still holds the previous call's operands when the
 *     next call starts.  Each call rewrites everything it later reads (padding rows included), so nothing
 *     needs clearing between calls; but two calls that overlap on the GPU (different streams, or different
 *     host threads) race on the array and give wrong results: keep them on one stream or order them with
 *     events.  regenvc_set_workspace() has no effect here.
 *   - Device-side conditions of these calls (an input beyond the fp16 range, an expired bounded wait) are
 *     recorded in a status word that is also part of the image, not in the one regenvc_device_status() reads.
 *     The word is sticky: while it is set, later calls of this entry point on the device skip their work and
 *     leave `out` unspecified although they return REGENVC_OK.  regenvc_static_device_status() waits for
 *     `stream`, reports the word in *status_out (REGENVC_OK, REGENVC_ERR_RANGE or REGENVC_ERR_TIMEOUT) and
 *     clears it; it allocates nothing either (a stream synchronisation and a 4-byte copy).  A real-time loop
 *     should read it once per window, after the window's last call.
 *   - The call enqueues two kernels.  Arguments are validated before the first; if the launch of the second
 *     fails (REGENVC_ERR_CUDA), the first, which only rewrites the scratch array, has already been enqueued.
 */
#define REGENVC_STATIC_SCRATCH_BYTES (16u << 20)
int regenvc_cross_attn_forward_static(const void* q, const void* k, const void* v, void* out,
                                      int n_q, int n_kv, int n_heads, int head_dim, void* stream);
int regenvc_static_device_status(void* stream, int* status_out);

/*
 * Scratch memory.  Each call first rewrites the keys and values into
 * tensor-core operand form in a device workspace:
 *   K' : 16-bit [n_heads][n_kv_pad][128] rotated fp16 keys (self) or the bf16 keys as they are (cross)
 *   V't: fp16 [n_heads][128][n_kv_pad]   values, transposed so that keys are contiguous
 * with n_kv_pad = n_kv rounded up to a multiple of 128 (padding is zero),
 * K' first, V't directly after it, followed by a fixed 21,299,200-byte area
 * for the partial results of query tiles whose key range is cut into pieces
 * (fp32 accumulators, references and row sums that a merge kernel combines).
 * regenvc_workspace_bytes() returns the total this needs (0 for invalid
 * arguments).  By default the library keeps
 * one workspace per device and host thread and grows it on demand with
 * cudaMalloc (which synchronises: do a warm-up call before capturing a CUDA
 * graph).  regenvc_set_workspace() makes the calling host thread use a
 * caller-owned device buffer instead (256-byte aligned; NULL/0 returns to the
 * internal one); a call that needs more than `bytes` then fails with
 * REGENVC_ERR_WORKSPACE.
 */
size_t regenvc_workspace_bytes(int n_kv, int n_heads, int head_dim);
int regenvc_set_workspace(void* dev_ptr, size_t bytes);

/*
 * Waits for `stream` and reports the sticky device-side status of the current
 * device in *status_out: REGENVC_OK, REGENVC_ERR_TIMEOUT (a kernel gave up on
 * a bounded wait; its output is invalid) or REGENVC_ERR_RANGE.  The status is
 * cleared by the call.  Returns REGENVC_OK or the error of the query itself.
 */
int regenvc_device_status(void* stream, int* status_out);

/*
 * Profiling aid: selects which of the two kernels later calls from this host
 * thread enqueue.  Bit 0 = key/value preparation pass, bit 1 = attention
 * kernel; the default is 3 (both).  With bit 0 clear the workspace must still
 * hold the prepared operands of the same k, v and shape (from an earlier full
 * call), which lets a benchmark time the attention kernel alone.  Bit 2 (value
 * 4, together with bit 0 and/or 1) makes calls with short key sequences use
 * one thread block per work item instead of the persistent form they
 * normally take (same results; for measuring the difference).  Bit 3 (value
 * 8) sends every call to the attention kernel that runs on pairs of thread
 * blocks, which the library otherwise picks for long key sequences only, bit
 * 4 (value 16) keeps every call away from it (same results within rounding
 * of the split into key-range pieces; for tests and for measuring the
 * difference).  Bit 5 (value 32) sends every call to that kernel too, with a
 * grid of two pairs of thread blocks only, so that even a small call makes
 * each pair walk over many work items (for tests of that walk).  Returns
 * REGENVC_ERR_BAD_SHAPE for a mask outside 1..63, without bit 0 and bit 1, or
 * with bit 4 together with bit 3 or bit 5.
 */
int regenvc_debug_set_phases(int mask);

/*
 * Test aid for the bounded waits inside the kernels: enqueues one warp that
 * waits on a barrier nothing ever completes.  After limit_us microseconds
 * (1..100000) the wait gives up exactly as a wait in the attention kernels
 * would, the kernel returns normally and the sticky status word holds
 * REGENVC_ERR_TIMEOUT until regenvc_device_status() reads it.  Kernels of this
 * library that start while the word is set skip their work (their bounded
 * waits fall through) and leave `out` unspecified.  Nothing faults or hangs.
 */
int regenvc_debug_expire_wait(int limit_us, void* stream);

const char* regenvc_status_string(int status);
/* Text of the last failing CUDA call on this host thread ("" if none). */
const char* regenvc_last_cuda_error(void);
const char* regenvc_version(void);
/* Number of kernels the library has launched from this process (all threads). */
unsigned long long regenvc_kernel_launch_count(void);
/* Frees cached rotary tables, staging buffers and internal workspaces of every
 * device.  No library work may be in flight. */
void regenvc_shutdown(void);

#ifdef __cplusplus
}
#endif
#endif /* REGENVC_ATTN_H */
