/*
 * hmar.h - C ABI of the B200 (sm_100a) library for HMAR's Markovian block-sparse attention.
 *
 * The operation (paper Sec. 4.1 "I/O-Aware Windowed Attention", Fig. attn-mask, App. B.3/B.4):
 * exact softmax attention over the flattened multi-scale token sequence, where the K resolution
 * scales of side_k x side_k tokens are laid out one after another (Sec. 3) and a token of scale k
 * attends to every token of scales k-1 and k and to nothing else (Sec. 4.1, Markovian next-scale
 * prediction); attention inside a scale is bidirectional (Sec. 3).  The first scale has no
 * predecessor and attends to itself only.
 *
 * Conventions shared by every entry point
 *   - n_k = side_lens[k]^2 tokens in scale k, L = sum n_k, tokens ordered scale after scale.
 *   - Tensors are [B, H, rows, D] contiguous with D innermost, rows = L for the training calls.
 *     D must be 64 (the paper's head dimension, App. B.4); anything else is HMAR_ERR_UNSUPPORTED.
 *   - Entry points without suffix take bf16 tensors (raw 16-bit storage) and compute with bf16 tensor
 *     core inputs, fp32 accumulation and fp32 softmax.  The `_f32` entry points are the debug build:
 *     float tensors and plain fp32 FMA arithmetic everywhere.
 *   - softmax_scale must be positive and finite (HMAR_ERR_BAD_ARG otherwise).
 *   - lse[b,h,i] = ln sum_j exp(softmax_scale * q_i . k_j) over the allowed j (natural log), fp32.
 *   - Every tensor pointer is DEVICE memory owned by the caller, 16-byte aligned.  `side_lens` is a
 *     HOST array read during the call.  The library allocates no per-call device memory; it owns a
 *     small per-schedule plan cache (device work lists), created on the first call that uses a new
 *     side_lens list and released by hmar_shutdown().  That first call synchronises an internal
 *     stream and must therefore not be issued while `stream` is being captured.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *     They return HMAR_OK or a negative hmar_status.  Argument errors are found before any launch
 *     and leave the outputs untouched.  No entry point throws, traps or synchronises the device.
 *   - Every wait inside the kernels is bounded; a wait that runs out makes the kernel stop cleanly
 *     and record a code that hmar_device_status() reports.
 */
#ifndef HMAR_H_
#define HMAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    HMAR_OK = 0,
    HMAR_ERR_BAD_ARG = -1,        /* null pointer, non-positive size, misaligned pointer, too many scales */
    HMAR_ERR_UNSUPPORTED = -2,    /* head dimension not offered by this entry point, or the device is not sm_100 */
    HMAR_ERR_CUDA = -3,           /* a CUDA runtime / driver call failed */
    HMAR_ERR_WORKSPACE = -4,      /* workspace missing or smaller than hmar_attn_bwd_workspace_bytes() */
    HMAR_ERR_DEVICE_TIMEOUT = -5, /* a bounded wait inside a kernel ran out (see hmar_device_status) */
    HMAR_ERR_BOUNDS = -6          /* checking build only: a kernel formed an address outside its tensor (hmar_device_status) */
} hmar_status;

#define HMAR_MAX_SCALES 64

/* Which scales a token of scale k attends to.  All four are block masks over the same flattened
 * sequence in which the allowed keys of a query are one contiguous range, so one scheduler and one set
 * of kernels serves them.
 *   HMAR_WINDOW_MARKOV : scales k-1 and k - HMAR's Markovian mask (Sec. 4.1, Fig. attn-mask); what the
 *                        entry points without `_window` compute.
 *   HMAR_WINDOW_CAUSAL : scales 1..k - VAR's block-causal mask (Sec. 3, Fig. attn-mask), the workload the
 *                        paper's attention benchmark compares against (App. B.4).
 *   HMAR_WINDOW_SELF   : scale k only - the literal "block-diagonal" reading of Sec. 1 / App. B.3.
 *   HMAR_WINDOW_PREV   : scale k-1 only - App. B.3's literal "only the immediately preceding scale"; the first
 *                        scale, which has no predecessor, attends to itself.  No query looks at the keys of the
 *                        last scale, so the backward returns zeros for their dK and dV. */
typedef enum { HMAR_WINDOW_MARKOV = 0, HMAR_WINDOW_CAUSAL = 1, HMAR_WINDOW_SELF = 2, HMAR_WINDOW_PREV = 3 } hmar_window;

/* Head dimension D.  The tensor-core kernels exist for D = 64 (the paper's attention benchmark, App. B.4, and
 * every config).  hmar_attn_fwd, hmar_attn_bwd, their _window and _f32 forms, hmar_attn_bwd_workspace_bytes and
 * hmar_attn_scale_step(_f32) also accept D = 32 and D = 128, which run on the plain-FMA kernels of the debug
 * build (same results within the same tolerances, a small fraction of the speed).  The packed, strided and
 * no-allocation entry points take D = 64 only.  Anything else is HMAR_ERR_UNSUPPORTED. */

/* Training forward (Sec. 4.1; App. B.4 benchmarks this pass).
 *   q, k, v : [B,H,L,D] in;  out : [B,H,L,D] out;  lse : [B,H,L] fp32 out.
 *   side_lens : host array of n_scales positive side lengths (any order of sizes is accepted). */
int hmar_attn_fwd(const void* q, const void* k, const void* v, void* out, float* lse,
                  int B, int H, int D, int n_scales, const int* side_lens,
                  float softmax_scale, void* stream);
int hmar_attn_fwd_f32(const float* q, const float* k, const float* v, float* out, float* lse,
                      int B, int H, int D, int n_scales, const int* side_lens,
                      float softmax_scale, void* stream);

/* Training forward on the packed output of the QKV projection (Sec. 4.1: the kernel sits between the
 * transformer block's QKV projection and its output projection; reading the projection's layout saves the
 * transposing copies around the kernel).  bf16 only, Markovian mask.
 *   qkv : [B,L,3,H,D] in (q, k, v of a token side by side);  out : [B,L,H,D] out (the layout the output
 *   projection reads);  lse : [B,H,L] fp32 out, as for hmar_attn_fwd.  All pointers device, 16-byte aligned.  HMAR_ERR_UNSUPPORTED while the
 *   fall-back kernels are forced (they read contiguous tensors only); other errors as for hmar_attn_fwd. */
int hmar_attn_fwd_packed(const void* qkv, void* out, float* lse, int B, int H, int D, int n_scales,
                         const int* side_lens, float softmax_scale, void* stream);

/* The same forward under another block mask of the same family (see hmar_window).  Everything else -
 * layouts, lse convention, precision, errors - is as for hmar_attn_fwd; an unknown `window` is
 * HMAR_ERR_BAD_ARG. */
int hmar_attn_fwd_window(const void* q, const void* k, const void* v, void* out, float* lse,
                         int B, int H, int D, int n_scales, const int* side_lens, int window,
                         float softmax_scale, void* stream);
int hmar_attn_fwd_window_f32(const float* q, const float* k, const float* v, float* out, float* lse,
                             int B, int H, int D, int n_scales, const int* side_lens, int window,
                             float softmax_scale, void* stream);

/* Training backward on the packed layouts of hmar_attn_fwd_packed, so that a training step needs no
 * transposing copy on either side of the attention (Sec. 4.1).  bf16 only, Markovian mask.
 *   qkv : [B,L,3,H,D] in;  out, dout : [B,L,H,D] in;  lse : [B,H,L] in (from hmar_attn_fwd_packed);
 *   dqkv : [B,L,3,H,D] out (dq, dk, dv of a token side by side, the layout the projection's backward reads).
 *   workspace : as for hmar_attn_bwd (same size).  Same arithmetic as hmar_attn_bwd: dk and dv carry the very
 *   bits the contiguous entry point gives for the same values.  Errors as for hmar_attn_fwd_packed. */
int hmar_attn_bwd_packed(const void* qkv, const void* out, const float* lse, const void* dout, void* dqkv,
                         void* workspace, size_t workspace_bytes, int B, int H, int D, int n_scales,
                         const int* side_lens, float softmax_scale, void* stream);

/* Bytes of caller-provided device scratch the backward needs for this problem (0 on bad arguments).
 * The scratch holds delta = rowsum(dO o O) and the fp32 dQ accumulator; its contents on entry do not
 * matter and are undefined on return. */
size_t hmar_attn_bwd_workspace_bytes(int B, int H, int D, int n_scales, const int* side_lens);

/* Training backward (App. B.4 benchmarks this pass; the gradient of the exact attention above).
 *   in : q, k, v, out, dout [B,H,L,D]; lse [B,H,L] as written by the forward.
 *   out: dq, dk, dv [B,H,L,D] (fully overwritten).
 *   workspace : device scratch of at least hmar_attn_bwd_workspace_bytes() bytes, 256-byte aligned.
 * dQ is accumulated in fp32 by bulk tensor reductions into global memory (cp.reduce.async.bulk.tensor),
 * whose order is not fixed, so its low-order bits may differ between runs. */
int hmar_attn_bwd(const void* q, const void* k, const void* v, const void* out, const float* lse,
                  const void* dout, void* dq, void* dk, void* dv,
                  void* workspace, size_t workspace_bytes,
                  int B, int H, int D, int n_scales, const int* side_lens,
                  float softmax_scale, void* stream);
int hmar_attn_bwd_f32(const float* q, const float* k, const float* v, const float* out, const float* lse,
                      const float* dout, float* dq, float* dk, float* dv,
                      void* workspace, size_t workspace_bytes,
                      int B, int H, int D, int n_scales, const int* side_lens,
                      float softmax_scale, void* stream);

/* The same backward under another block mask of the same family (see hmar_window); `lse` and `out` must
 * come from hmar_attn_fwd_window with the same `window`.  Workspace as for hmar_attn_bwd. */
int hmar_attn_bwd_window(const void* q, const void* k, const void* v, const void* out, const float* lse,
                         const void* dout, void* dq, void* dk, void* dv,
                         void* workspace, size_t workspace_bytes,
                         int B, int H, int D, int n_scales, const int* side_lens, int window,
                         float softmax_scale, void* stream);
int hmar_attn_bwd_window_f32(const float* q, const float* k, const float* v, const float* out, const float* lse,
                             const float* dout, float* dq, float* dk, float* dv,
                             void* workspace, size_t workspace_bytes,
                             int B, int H, int D, int n_scales, const int* side_lens, int window,
                             float softmax_scale, void* stream);

/* Backward for callers that cannot allocate device memory (the paper has no counterpart; this is a
 * library convenience).  Same inputs, outputs and arithmetic as hmar_attn_bwd (bf16), but no workspace
 * argument and no plan cache: the work list, delta and the fp32 dQ accumulator live in one fixed
 * device array inside the library image (about 8.6 MB, held by every GPU that loads the library until
 * the process exits).  It is meant for code that runs where cudaMalloc is off limits: under a framework
 * that owns all device memory through its own pool, inside a server plug-in that must not grow after
 * start-up, or wherever cudaMalloc / cudaFree are forbidden because they may synchronise the device.
 *   - Limit: B * H * L <= HMAR_NOALLOC_MAX_ROWS; larger problems are rejected with HMAR_ERR_WORKSPACE
 *     before anything is launched.
 *   - The call itself never calls cudaMalloc, cudaFree or any allocating routine, and copies nothing from
 *     host memory: the work list travels as kernel parameters.  Its first call on a device looks up the
 *     array's device address (cudaGetSymbolAddress); make that first call outside any stream capture.
 *   - All calls on a device share the array.  The array keeps whatever the previous call left in it;
 *     each call overwrites the work list and delta and clears the accumulator itself.  Two calls whose
 *     GPU work may overlap (different streams without an ordering between them) race on it: keep
 *     calls to this entry point on one stream, or order them with events.
 *   - Kernel waits that run out are not reported through hmar_device_status() for this entry point. */
#define HMAR_NOALLOC_MAX_ROWS 32768
int hmar_attn_bwd_noalloc(const void* q, const void* k, const void* v, const void* out, const float* lse,
                          const void* dout, void* dq, void* dk, void* dv,
                          int B, int H, int D, int n_scales, const int* side_lens,
                          float softmax_scale, void* stream);

/* Inference step of one scale (Sec. 4.1: no prefix computation or KV cache beyond the previous
 * scale; Sec. 4.2/4.4: every masked refinement sub-step of scale k sees scale k-1 and scale k).
 *   q            : [B,H,n_cur,D]      queries of the current scale, n_cur = side_cur^2
 *   k_prev,v_prev: [B,H,n_prev,D]     cached previous scale, n_prev = side_prev^2;
 *                                     must be NULL iff side_prev == 0 (first scale)
 *   k_cur, v_cur : [B,H,n_cur,D]      the current scale's own keys / values
 *   out          : [B,H,n_cur,D];  lse : [B,H,n_cur] fp32 or NULL.
 * Dense attention of q over (prev followed by cur); no mask inside the window.
 * Windows of at most 128 keys (and 96 queries) run in a kernel of their own: one block per head, K and V
 * of the head in shared memory, warp-level bf16 products; larger ones in the forward kernel's two-segment mode. */
int hmar_attn_scale_step(const void* q, const void* k_prev, const void* v_prev,
                         const void* k_cur, const void* v_cur, void* out, float* lse,
                         int B, int H, int D, int side_prev, int side_cur,
                         float softmax_scale, void* stream);
int hmar_attn_scale_step_f32(const float* q, const float* k_prev, const float* v_prev,
                             const float* k_cur, const float* v_cur, float* out, float* lse,
                             int B, int H, int D, int side_prev, int side_cur,
                             float softmax_scale, void* stream);
/* The same step on tensors whose heads are not packed back to back (Sec. 1 / Sec. 5.2: inference keeps only
 * the previous scale's keys and values, so a sampler holds them in one small ring and must not copy them
 * to concatenate).  Rows are D contiguous elements; head b*H + h of a tensor starts `*_head_stride`
 * elements after head b*H + h - 1 (each at least rows * D and a multiple of 8).  With K and V of the
 * previous and the current scale adjacent in one buffer [B,H,ring_rows,D]: k_cur = k_prev + n_prev * D
 * and kv_prev_head_stride = kv_cur_head_stride = ring_rows * D.  bf16 only; lse stays [B,H,n_cur] dense.
 * Errors as hmar_attn_scale_step; with the plain-kernel debug switch on, only dense strides are accepted
 * (HMAR_ERR_UNSUPPORTED otherwise). */
int hmar_attn_scale_step_strided(const void* q, const void* k_prev, const void* v_prev,
                                 const void* k_cur, const void* v_cur, void* out, float* lse,
                                 int B, int H, int D, int side_prev, int side_cur,
                                 long long q_head_stride, long long kv_prev_head_stride,
                                 long long kv_cur_head_stride, long long out_head_stride,
                                 float softmax_scale, void* stream);

/* The sampler's step next to the attention at inference (Alg. 2, "Multi-scale VQ-VAE Reconstruction", lines
 * 7-8: x~_k = interpolate(lookup(V, r_k), H_K, W_K), x~_{1:k} = x~_{1:k-1} + x~_k) fused with the token
 * selection of a masked refinement sub-step (Sec. 4.2: the positions in the sub-step's mask take the newly
 * generated token, the others keep theirs).  The paper does not name the interpolation; this is bicubic
 * convolution with a = -0.75, half-pixel sample positions and border-clamped indices.
 *   xhat       : [B, C, out_side, out_side] fp32, device, updated in place (+= the interpolated codes)
 *   codebook   : [V, C] fp32, device
 *   tokens_new : [B, side, side] int32 ids, device;  tokens_old : the same shape, or NULL when mask is NULL
 *   mask       : [B, side, side] bytes, nonzero = take tokens_new there; NULL = take tokens_new everywhere
 *   tokens_out : [B, side, side] int32 or NULL; receives the selected map (must not alias the inputs)
 * side <= out_side <= 4096.  Ids outside [0, V) are clamped.  One kernel, asynchronous on `stream`; every
 * element of xhat receives exactly one addition (issued as a reduction to memory), so the result does not
 * depend on scheduling.  No alignment beyond the element types' own is required. */
int hmar_recon_accumulate(float* xhat, const float* codebook, const int* tokens_old, const int* tokens_new,
                          const unsigned char* mask, int* tokens_out, int B, int C, int V, int side, int out_side,
                          void* stream);

/* The other sampler-side step (Sec. 4.1, "Reformulating Next-Scale Prediction to be Markovian": the running
 * reconstruction x~_{1:k-1} is interpolated to the scale's resolution, and the scale is conditioned on that
 * image instead of on all earlier token maps).  The paper does not name the interpolation; this is area
 * interpolation: out(i, j) = the mean of xhat over rows [floor(i * in_side / out_side),
 * ceil((i + 1) * in_side / out_side)) and the like columns.
 *   xhat : [B, C, in_side, in_side] fp32, device (read only);  out : [B, C, out_side, out_side] fp32, device
 * out_side <= in_side <= 4096; the buffers must not overlap.  One kernel (a device-to-device copy when the sizes
 * are equal), asynchronous on `stream`. */
int hmar_recon_downsample(const float* xhat, float* out, int B, int C, int in_side, int out_side, void* stream);

/* Host-side scale-block scheduler (Sec. 4.1: the kernel visits only the live blocks of the mask).
 * Writes the work list of one head for `direction` 0 = forward (tiles of query rows, each with the
 * contiguous key range it must visit) or 1 = backward (tiles of key rows with their query range).
 * Each tile is 6 int32: {row_begin, row_count, partner_begin, partner_end, uniform, cost}; `uniform`
 * is 1 when every row of the tile may see the whole partner range, 0 when rows carry their own
 * bounds (several small scales packed into one tile).  Returns the number of tiles, or a negative
 * hmar_status; writes at most max_tiles entries (pass NULL / 0 to query the count).  Host only. */
int hmar_schedule_tiles(int n_scales, const int* side_lens, int direction,
                        int32_t* tiles, int max_tiles);
/* The same for any mask of the family (see hmar_window). */
int hmar_schedule_tiles_window(int n_scales, const int* side_lens, int window, int direction,
                               int32_t* tiles, int max_tiles);

/* Share, in thousandths, of a head's backward steps (128 key rows x 128 query rows) that belong to full tiles:
 * 128 key rows that all see the tile's whole query range, which the backward kernel processes without mask code.
 * The backward picks its instantiation by it: side lists below 600 run the one that keeps a single, fully
 * masked variant of the softmax-gradient code (smaller code; these lists are bound by instruction fetch), the
 * others the one with three variants.  Returns a negative hmar_status for a bad side list.  Host only. */
int hmar_schedule_bwd_full_tile_share(int n_scales, const int* side_lens, int window);

/* Blocks until the work queued on the current device has finished, then returns the code recorded
 * by the kernels since the last call (HMAR_OK, or HMAR_ERR_DEVICE_TIMEOUT with *detail, if not NULL,
 * telling which wait gave up) and clears it.
 * Every wait inside the tensor-core kernels is bounded (about one second of wall time, which on a GPU shared
 * by time slicing includes the time the context is switched out).  When one runs out, the block gives up,
 * the word latches, and every tensor-core kernel launched on the device afterwards returns at once WITHOUT
 * writing its outputs, while the entry points keep returning HMAR_OK (they never synchronise).  A caller
 * that must know whether its results are valid therefore calls this function after the work it cares
 * about: HMAR_OK means every kernel since the previous call ran to completion. */
int hmar_device_status(int* detail);

/* Self-test of that mechanism (no counterpart in the paper): launches one block that waits, through the
 * kernels' own wait routine with a limit of one millisecond, on a barrier nothing ever arrives on.  The wait
 * gives up and the block returns; the next hmar_device_status() reports HMAR_ERR_DEVICE_TIMEOUT with detail
 * 0xD1A6 and clears it.  Nothing traps or faults; the context stays usable. */
int hmar_selftest_bounded_wait(void* stream);

/* Per-kernel timing for benchmarks.  Between hmar_profile_begin() and hmar_profile_end() every kernel
 * the library launches is bracketed by two CUDA events on its stream.  hmar_profile_end() synchronises
 * the device and writes one line per kernel name, "name launches total_ms\n", into `report`
 * (NUL-terminated, truncated to `capacity`).  Not thread-safe against concurrent entry-point calls. */
void hmar_profile_begin(void);
int hmar_profile_end(char* report, size_t capacity);

/* Debug switch: nonzero routes the bf16 entry points through the plain SIMT kernels (the same ones
 * the _f32 build uses) instead of the tensor-core kernels.  Returns the previous setting. */
int hmar_debug_force_simt(int enable);

/* Number of kernels the library has launched since it was loaded (all entry points, this process). */
long long hmar_launch_count(void);

/* Frees the plan cache on every device.  Safe to call more than once. */
void hmar_shutdown(void);

const char* hmar_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* HMAR_H_ */
