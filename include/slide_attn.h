/*
 * slide_attn.h -- C ABI of the fused Slide Attention forward for NVIDIA B200 (sm_100a).
 *
 * The operation (Slide-Transformer, arXiv 2304.04237):
 *
 *   For every query pixel p = (b, i, j) of a [B, H, W] map and every head h:
 *
 *     Ks[s, c] = sum_t wk[c, s, t] * K0(p + off(t), c)        Sec. 4.2, Eq. 12: depthwise k x k
 *     Vs[s, c] = sum_t wv[c, s, t] * V0(p + off(t), c)        convolution per slot s; wk / wv are
 *                                                             the merged kernels of Sec. 4.3
 *                                                             (fixed shift, Eq. 11, + learned
 *                                                             deformed shift, re-parameterised)
 *     l[s]     = (sum_{c in head h} q[p, c] * Ks[s, c]) / sqrt(head_dim)  (+ bias[h, s])    Eq. 2
 *     a        = softmax over the k*k slots of l                                            Eq. 2
 *     out[p,c] = sum_s a[s] * Vs[s, c]                                                      Eq. 2
 *
 *   r = floor(k/2); slot s = (u+r)*k + (v+r) for the window offset (u, v) in [-r, r]^2
 *   (Eq. 4-9, row-major over (u, v)); tap t = p_*k + q_ for the kernel position (p_, q_) in
 *   [0, k)^2 with off(t) = (p_ - r, q_ - r) (Eq. 12; cross-correlation, no kernel flip).
 *   K0 / V0 read zero outside the map ("[1,1] padding", Fig. 2); padded slots are NOT masked:
 *   they take part in the softmax with key 0 and value 0, as a zero-padded convolution gives.
 *   With wk = wv = the one-hot kernels (w[c, s, t] = 1 iff t == s) the result is plain k x k
 *   local attention (Sec. 3.2 (3)).
 *
 * The k*k-expanded keys and values are never written to device memory: convolution, logits,
 * softmax and aggregation run in one kernel.
 *
 * Tensor layouts (all dense, row-major, no strides):
 *   q, k, v, out : [B][H][W][heads][head_dim], element type = the context's dtype
 *                  (channel c = h*head_dim + e; "channels-last")
 *   wk, wv       : float [C][k*k slot][k*k tap], C = heads*head_dim.  This is the memory of a
 *                  PyTorch-style depthwise weight [C*k*k, 1, k, k] with groups = C and output
 *                  channel c*k*k + s, so a re-parameterised convolution weight can be passed as is.
 *   bias         : float [heads][k*k], or NULL
 *
 * Ownership: the caller owns every tensor.  The library reads/writes them only in stream order
 * within the call that received them and keeps no pointer afterwards.  A context owns a small
 * device workspace (re-laid-out weights, a status word), allocated by slide_attn_create.
 *
 * Errors: every function returns a status code; nothing is thrown or printed; no device code
 * traps.  Arguments are validated on the host before anything is launched.  There is no CPU
 * fallback: on a device that is not sm_100 slide_attn_create returns SLIDE_ATTN_ERR_ARCH.
 *
 * Threading: one context must not be used from two host threads at once, and two forwards on
 * the same context must be ordered on the device (same stream, or events), because they share
 * the context's workspace.  Distinct contexts are independent.  A context belongs to the device
 * that was current when it was created: forward, forward_host and query_status return
 * SLIDE_ATTN_ERR_INVALID_ARG, before launching anything, when another device is current.
 */
#ifndef SLIDE_ATTN_H_
#define SLIDE_ATTN_H_

#ifdef __cplusplus
extern "C" {
#endif

typedef struct slide_attn_ctx slide_attn_ctx;      /* opaque; created and destroyed by the library */

typedef enum {
    SLIDE_ATTN_F32  = 0,    /* q, k, v, out are IEEE float                                        */
    SLIDE_ATTN_BF16 = 1     /* q, k, v, out are bfloat16; arithmetic accumulates in float         */
} slide_attn_dtype;

typedef enum {
    SLIDE_ATTN_OK = 0,
    SLIDE_ATTN_ERR_INVALID_ARG = 1,   /* NULL pointer, non-positive size, unknown enum             */
    SLIDE_ATTN_ERR_UNSUPPORTED = 2,   /* even ksize, ksize > 15, head_dim not a multiple of 8, ...  */
    SLIDE_ATTN_ERR_ALIGNMENT   = 3,   /* a tensor pointer is not 16-byte aligned                   */
    SLIDE_ATTN_ERR_ALLOC       = 4,   /* device or host allocation failed                          */
    SLIDE_ATTN_ERR_CUDA        = 5,   /* a CUDA runtime/driver call failed                         */
    SLIDE_ATTN_ERR_ARCH        = 6,   /* current device is not compute capability 10.x             */
    SLIDE_ATTN_ERR_TIMEOUT     = 7,   /* a bounded device-side wait ran out (see query_status)     */
    SLIDE_ATTN_ERR_TOO_LARGE   = 8,   /* problem exceeds the fixed scratch of forward_noalloc      */
    SLIDE_ATTN_ERR_NOT_FIXED_SHIFT = 9 /* fixed-shift mode was declared but a weight is not one-hot
                                          (reported by query_status; that forward's output is undefined) */
} slide_attn_status;

/* Kernel variants.  AUTO picks the fastest one that supports the context's shape; the others
 * exist for A/B measurements and tests.  All variants compute the same function.  (Values 3, 4 and 7
 * belonged to earlier tensor-core schedules that UMMA_TS replaced; they are not accepted any more.) */
typedef enum {
    SLIDE_ATTN_VARIANT_AUTO    = 0,
    SLIDE_ATTN_VARIANT_DIRECT  = 1,   /* one warp per (pixel, head), global loads, fp32 FMA; any shape */
    SLIDE_ATTN_VARIANT_MMA     = 2,   /* TMA halo tile in shared memory, deformed-shift contraction on
                                         mma.sync tensor cores (bf16 operands, fp32 accumulate); one CTA
                                         per tile and head; bf16, head_dim 32, ksize 3; also what the
                                         allocation-free entry point runs                              */
    SLIDE_ATTN_VARIANT_UMMA_TS = 5,   /* persistent warp-specialised kernel, both contractions on
                                         tcgen05.mma with their A operands (the q.k products, the softmax
                                         weights) held in tensor memory; bf16, head_dim 32, ksize 3: what
                                         AUTO runs there                                               */
    SLIDE_ATTN_VARIANT_STRIP   = 6,   /* DIRECT's arithmetic with transposed weights (one coalesced load
                                         per weight) and 4-8 pixels per warp, operands read from global
                                         memory; fp32 FMA; ksize <= 9, any head_dim, fp32 or bf16        */
    SLIDE_ATTN_VARIANT_TILE    = 8,   /* generic weights on the CUDA cores off a TMA-staged halo tile
                                         in shared memory, 16-byte accesses throughout, convolution
                                         re-associated with the q.k products and the softmax weights;
                                         head_dim 32, ksize <= 9, fp32 or bf16: what AUTO runs for fp32
                                         storage                                                         */
    SLIDE_ATTN_VARIANT_MMA_WIDE = 9   /* large windows with general weights on tensor cores (mma.sync):
                                         TMA-staged halo tile, weights streamed tap by tap from L2 as
                                         register fragments; bf16, head_dim 32, ksize 3 / 5 / 7 / 9: what
                                         AUTO runs for bf16 with ksize >= 5                              */
} slide_attn_variant;

/*
 * Creates a context for one problem shape on the CURRENT CUDA device (Eq. 2 over a k x k window;
 * shapes as in the layout section above).
 *   ctx       [out, host]  receives the context; untouched on error
 *   B, H, W   batch and map size, each >= 1 (H or W smaller than ksize is legal)
 *   heads, head_dim        >= 1; head_dim must be a multiple of 8 and <= 256
 *   ksize     odd, 1..15 (the window offsets u, v range over [-floor(k/2), floor(k/2)], which
 *             is centred only for odd k)
 *   dtype     element type of q, k, v, out
 *   has_bias  non-zero if forward will be given a bias
 * Allocates the context's workspace (cudaMalloc); synchronous.
 */
slide_attn_status slide_attn_create(slide_attn_ctx** ctx,
                                    int B, int H, int W, int heads, int head_dim, int ksize,
                                    slide_attn_dtype dtype, int has_bias);

/*
 * Runs the forward (the five formulas at the top; Eq. 2, Eq. 12, Sec. 4.3) asynchronously on
 * `cuda_stream` (a cudaStream_t; NULL = the legacy default stream).
 *   q, k, v   [in,  DEVICE] [B][H][W][heads][head_dim], ctx dtype, 16-byte aligned
 *   wk, wv    [in,  DEVICE] float [C][k*k][k*k], 16-byte aligned
 *   bias      [in,  DEVICE] float [heads][k*k]; must be non-NULL iff the context has_bias
 *   out       [out, DEVICE] same shape and dtype as q, 16-byte aligned; must not alias an input
 * Does not allocate and does not synchronise; the result is deterministic (bit-identical from
 * run to run for a given variant).  Weight re-layout, where a variant needs it, happens inside
 * this call on the same stream, so wk / wv may change between calls.
 */
slide_attn_status slide_attn_forward(slide_attn_ctx* ctx,
                                     const void* q, const void* k, const void* v,
                                     const float* wk, const float* wv, const float* bias,
                                     void* out, void* cuda_stream);

/*
 * The same forward (Eq. 2, Eq. 12, Sec. 4.3) for HOST buffers of the same layouts: copies q, k,
 * v, wk, wv, bias to device staging buffers owned by the context, runs the forward, copies `out`
 * back and waits until all of that is done.  The images of a batch are independent, so the batch
 * goes through in up to four slices: while one slice is computed on `cuda_stream`, the next one
 * is copied in and the one before is copied out on two copy streams owned by the context (both
 * directions of the host link are then busy at once).  The call starts after the work already in
 * `cuda_stream` and returns with nothing of its own in flight.  Page-locked host buffers are
 * needed for the copies to overlap; pageable ones work too.  The staging buffers, the copy
 * streams and their events are created on the first call and reused afterwards.
 */
slide_attn_status slide_attn_forward_host(slide_attn_ctx* ctx,
                                          const void* q, const void* k, const void* v,
                                          const float* wk, const float* wv, const float* bias,
                                          void* out, void* cuda_stream);

/* Selects the kernel variant used by later forwards.  SLIDE_ATTN_ERR_UNSUPPORTED if the variant
 * cannot run the context's shape or dtype (the previous choice stays). */
slide_attn_status slide_attn_set_variant(slide_attn_ctx* ctx, slide_attn_variant variant);

/* The variant the next forward will run (never AUTO).  *variant [out, host]. */
slide_attn_status slide_attn_get_variant(const slide_attn_ctx* ctx, slide_attn_variant* variant);

/*
 * Fixed-shift mode (Sec. 4.2, Eq. 8-13; the "shift" / depthwise-convolution forms of the method
 * without the deformed shifting module of Sec. 4.3).  With enable != 0 the caller declares that the
 * wk and wv given to later forwards are EXACTLY the one-hot shift kernels of Eq. 11
 * (w[c][s][t] = 1 if t == s, else 0).  Slot s of a pixel then is the key / value at window offset s,
 * and the forward runs a kernel that does 2 k^2 instead of 2 k^4 + 2 k^2 multiply-adds per
 * pixel-channel (head_dim 32, ksize <= 9, both dtypes; SLIDE_ATTN_ERR_UNSUPPORTED otherwise, and the
 * mode stays off).  Every forward in this mode still reads wk and wv once on the device and checks the
 * declaration: if a weight differs, the status word is set and the next slide_attn_query_status
 * returns SLIDE_ATTN_ERR_NOT_FIXED_SHIFT; that forward's output is undefined.  enable == 0 returns to
 * the general kernels.  slide_attn_set_variant has no effect while the mode is on.
 */
slide_attn_status slide_attn_set_fixed_shift(slide_attn_ctx* ctx, int enable);

/*
 * Tells whether wk and wv (DEVICE, float [C][k*k][k*k]) are exactly the one-hot shift kernels of
 * Eq. 11, so that a caller can decide on fixed-shift mode when it loads a model.  Runs a reduction
 * on `cuda_stream` and WAITS for it.  *is_fixed [out, host] = 1 or 0.
 */
slide_attn_status slide_attn_detect_fixed_shift(slide_attn_ctx* ctx, const float* wk, const float* wv,
                                                int* is_fixed, void* cuda_stream);

/* Number of kernels one slide_attn_forward launches with the current variant.  *n [out, host]. */
slide_attn_status slide_attn_launches_per_forward(const slide_attn_ctx* ctx, int* n);

/*
 * Backward pass of the forward above (training through the module, Sec. 4.3 / Fig. 4 (1); the paper
 * prints no backward formulas: these are the derivatives of Eq. 2 with the convolution of Eq. 12
 * inside).  Given dout = d(loss)/d(out), writes the gradients of every input, asynchronously on
 * `cuda_stream`:
 *   q, k, v, wk, wv, bias   [in, DEVICE] exactly what the forward was given
 *   dout                    [in, DEVICE] same shape and dtype as out, 16-byte aligned
 *   dq, dk, dv              [out, DEVICE] same shape and dtype as q; overwritten
 *   dwk, dwv                [out, DEVICE] float [C][k*k][k*k]; overwritten (not accumulated into)
 *   dbias                   [out, DEVICE] float [heads][k*k]; non-NULL iff the context has_bias
 * For the training-time two-path form (fixed shift + learned kernels, merged weights = their sum)
 * dwk / dwv ARE the gradients of the learned kernels.  The attention weights are recomputed, so no
 * forward state is needed.  Supported: head_dim 32, ksize 1 or 3, both dtypes
 * (SLIDE_ATTN_ERR_UNSUPPORTED otherwise).  Arithmetic is fp32; dq, dk, dv are rounded to the dtype
 * once; dwk, dwv, dbias are summed over pixels with floating-point atomics, so their last bits may
 * differ from run to run.  The FIRST backward on a context allocates a scratch buffer of
 * 2 * B*H*W*heads*k*k floats (cudaMalloc, synchronous); later calls allocate nothing.
 */
slide_attn_status slide_attn_backward(slide_attn_ctx* ctx,
                                      const void* q, const void* k, const void* v,
                                      const float* wk, const float* wv, const float* bias,
                                      const void* dout,
                                      void* dq, void* dk, void* dv,
                                      float* dwk, float* dwv, float* dbias,
                                      void* cuda_stream);

/*
 * The dense projections around the attention stage (Eq. 1: q = x W_q, k = x W_k, v = x W_v; Eq. 3:
 * Concat(heads) W_o), as a tensor-core GEMM over the B*H*W tokens of the context's shape:
 *   y_i[token][o] = sum_c x[token][c] * w[i][c][o],  i = 0 .. nmat-1
 *   x            [in, DEVICE]  bf16 [B][H][W][C], C = heads*head_dim, 16-byte aligned
 *   w            [in, DEVICE]  float [nmat][C in][C out], nmat = 1..3 (e.g. W_q, W_k, W_v one after the other)
 *   y0, y1, y2   [out, DEVICE] bf16 [B][H][W][C] each; the first nmat are written, the rest are ignored
 * Weights are rounded to bf16, sums are accumulated in fp32, results rounded to bf16 once.  Asynchronous on
 * `cuda_stream`.  Supported: bf16 contexts with C a multiple of 16, 16 <= C <= 256
 * (SLIDE_ATTN_ERR_UNSUPPORTED otherwise).  Allocates nothing; one kernel launch (two to twelve when C > 128, where
 * the weights of all output columns do not fit shared memory together).
 */
slide_attn_status slide_attn_project(slide_attn_ctx* ctx, const void* x, const float* w, int nmat,
                                     void* y0, void* y1, void* y2, void* cuda_stream);

/*
 * One whole Slide-Attention block (Eq. 1 - 3 with the local attention of Sec. 4 as Eq. 2's attention):
 *   q, k, v = x W_q, x W_k, x W_v      (Eq. 1; slide_attn_project with nmat = 3)
 *   z       = slide_attn_forward(q, k, v, wk, wv, bias)     (channel c of q, k, v = head c / head_dim)
 *   out     = z W_o                    (Eq. 3; slide_attn_project with nmat = 1)
 *   x, out        [in / out, DEVICE] bf16 [B][H][W][C]; out must not alias x
 *   w_qkv         [in, DEVICE] float [3][C in][C out]: W_q, W_k, W_v
 *   w_o           [in, DEVICE] float [C in][C out]
 *   wk, wv, bias  as in slide_attn_forward
 * q, k, v and z live in bf16 in a scratch buffer of the context (4 * B*H*W*C*2 bytes), allocated with
 * cudaMalloc (synchronous) by the first call; they are rounded to bf16 once each.
 * The attention stage runs the context's current variant (or the fixed-shift kernel in fixed-shift mode).
 * Asynchronous on `cuda_stream`; same support as slide_attn_project.
 */
slide_attn_status slide_attn_block_forward(slide_attn_ctx* ctx, const void* x, const float* w_qkv,
                                           const float* w_o, const float* wk, const float* wv,
                                           const float* bias, void* out, void* cuda_stream);

/*
 * Waits for `cuda_stream` and reports the device-side status word: SLIDE_ATTN_OK,
 * SLIDE_ATTN_ERR_TIMEOUT if a kernel gave up on a bounded wait, or SLIDE_ATTN_ERR_NOT_FIXED_SHIFT if a
 * forward in fixed-shift mode met a weight that is not one-hot (the output is then undefined).
 * The word is cleared by this call.
 */
slide_attn_status slide_attn_query_status(slide_attn_ctx* ctx, void* cuda_stream);

/*
 * Forward without a context and without any allocation.  (The paper has no counterpart to this
 * entry point; it computes the same Eq. 2 / Eq. 12 forward as slide_attn_forward.)
 *
 * Who needs it: callers that are not allowed to allocate device memory -- code that runs inside a
 * memory plan with fixed buffers (an inference engine's arena, a plugin), a process whose
 * allocator is frozen after start-up, or a latency-critical loop that cannot afford the implicit
 * device synchronisation of cudaMalloc / cudaFree.  slide_attn_create allocates, so such callers
 * cannot use a context.  Here the scratch memory of the tensor-core variant (re-laid-out weights,
 * status word) is a fixed array inside the library's device image instead; every GPU that loads
 * the library holds it (288.25 KiB) from the moment the driver loads the library's device code on
 * that GPU until the process exits.  This call itself performs no cudaMalloc, cudaFree or other
 * allocating call.
 *
 * Arguments: tensors as for slide_attn_forward (DEVICE pointers, same layouts, 16-byte aligned,
 * bias may be NULL), followed by the shape the context would have carried.
 * Limits: dtype SLIDE_ATTN_BF16, head_dim 32, ksize 3 (else SLIDE_ATTN_ERR_UNSUPPORTED);
 * heads <= 16 (else SLIDE_ATTN_ERR_TOO_LARGE -- the fixed scratch has room for 16 heads).
 *
 * First call on a device: resolves the scratch's device address and configures the kernel.  With
 * CUDA's lazy module loading this is also when the driver may load the library's device code,
 * which takes device memory inside the driver (the scratch array included) and is not legal during
 * stream capture.  So make the first call on each device during start-up, with that device current,
 * outside of any stream capture and before an allocator is frozen.  Later calls on that device make
 * no allocating call of any kind.
 *
 * Sharing: every call on a device uses the same scratch, and the scratch keeps the previous call's
 * contents.  Each call rewrites all of it that it reads and clears the status word first, so
 * back-to-back calls on ONE stream are safe; calls that may overlap on the GPU (different streams
 * without an event between them, or several host threads) race on the scratch and give undefined
 * results.  Device-side time-outs are not reported by this entry point.
 */
slide_attn_status slide_attn_forward_noalloc(const void* q, const void* k, const void* v,
                                             const float* wk, const float* wv, const float* bias,
                                             void* out,
                                             int B, int H, int W, int heads, int head_dim, int ksize,
                                             slide_attn_dtype dtype, void* cuda_stream);

/*
 * Kernel timing for benchmarks (no counterpart in the paper's text; it measures the fused kernel
 * of Eq. 2 / Eq. 12).  After slide_attn_profile_begin every slide_attn_forward on this context
 * records CUDA events on its stream around (a) all kernels of the call and (b) the main fused
 * kernel alone; up to 1024 forwards are kept (later ones overwrite the oldest).
 * slide_attn_profile_end waits for the recorded events and reports the mean durations in
 * milliseconds and the number of forwards averaged, then stops recording.
 *   forward_ms, main_ms, n  [out, host]; any may be NULL.
 * Events cost a few microseconds of host time per forward; leave profiling off otherwise.
 */
slide_attn_status slide_attn_profile_begin(slide_attn_ctx* ctx);
slide_attn_status slide_attn_profile_end(slide_attn_ctx* ctx, double* forward_ms, double* main_ms, int* n);

/* Frees the context and everything it owns.  NULL is accepted.  The caller must make sure no
 * forward of this context is still running. */
slide_attn_status slide_attn_destroy(slide_attn_ctx* ctx);

/* A static, NUL-terminated description of a status code. */
const char* slide_attn_status_string(slide_attn_status status);

#ifdef __cplusplus
}
#endif
#endif  /* SLIDE_ATTN_H_ */
