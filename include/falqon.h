/*
 * falqon.h -- C ABI of the B200 (sm_100a) melded FP8-LoRA linear layer.
 *
 * One linear layer holds its LoRA adapter melded into an FP8 backbone: the E4M3
 * matrix W~' = [W~; A~] of (m + r) rows by n columns, one fp32 scale s_W, and an
 * fp32 DeltaBuffer of m x r that collects the optimizer's changes of B.  The four
 * operations are the quantizer Q_fp8, the melded forward, the backward (input
 * gradient and reformulated adapter gradient) and the row-wise proxy update.
 *
 * Conventions, for every entry point unless it says otherwise
 *  - Layout: all matrices are dense and row-major.  Paper notation W in R^{m x n},
 *    x in R^{n x d} maps to W[m][n] and X[T][n] with T = d tokens; O = Wx is Y[T][m].
 *  - Pointers: everything named "device" is a device pointer to memory the CALLER
 *    owns (including the workspace); the library allocates no device memory, keeps no
 *    hidden per-layer state and frees nothing.  The falqon_layer struct itself is a
 *    HOST struct.  Device pointers must be 16-byte aligned.
 *  - Shapes: n and m must be multiples of 16 (bulk tensor copies need 16-byte row
 *    pitches); r must be a multiple of 8 with 8 <= r <= 256; T >= 1.
 *  - Execution: every call only enqueues work on `stream` and returns; results are
 *    ready once the stream has drained.  Calls that touch the same layer or the same
 *    workspace must be ordered on one stream.  A workspace must have been through
 *    falqon_workspace_init once before its first use.  The kernels are launched with
 *    programmatic stream serialization (each may be scheduled while its predecessor in
 *    the stream still runs and waits on the device for it to finish); a caller's own
 *    kernels placed between two calls are ordinary stream work and need nothing special.
 *    The cast inside falqon_melded_forward / _backward (absmax, grid-wide barrier, cast: one kernel whose CTAs wait
 *    for one another) is launched COOPERATIVELY: the driver starts it only when its whole grid -- one CTA per SM --
 *    can be resident, so work of other streams on the same device delays it but cannot make it wait on CTAs that
 *    never start.  Its barrier counters are balanced even when a wait runs out.  The *_amax calls, the fused casts
 *    and falqon_quantize contain no such barrier.
 *  - Devices: per-device look-ups (symbol addresses, occupancy) are cached for the life of the process; do not keep
 *    using the library on a device after a cudaDeviceReset of it.
 *  - Errors: the return value is a falqon_status.  Bad arguments are detected on the
 *    host before anything is launched (nothing is written).  CUDA launch failures map
 *    to FALQON_ERR_CUDA.  Every device-side wait is bounded; a wait that runs out
 *    records FALQON_ERR_TIMEOUT in a device status word that
 *    falqon_last_device_status() returns.  Nothing traps or aborts.
 *  - Scales follow the reading s = fp8max / amax: quantization multiplies by s,
 *    de-quantization divides, and a product of two quantized operands is rescaled by
 *    1 / (s_a * s_b)  (Eq. quantize, Eq. fp8_matmul of the paper).
 */
#ifndef FALQON_H_
#define FALQON_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FALQON_OK = 0,
  FALQON_ERR_INVALID_ARG = -1,
  FALQON_ERR_UNSUPPORTED = -2,
  FALQON_ERR_WORKSPACE = -3,
  FALQON_ERR_CUDA = -4,
  FALQON_ERR_TIMEOUT = -5
} falqon_status;

typedef enum { FALQON_E4M3 = 0, FALQON_E5M2 = 1 } falqon_fp8;        /* max 448 / max 57344 */
typedef enum { FALQON_BF16 = 0, FALQON_F32 = 1 } falqon_dtype;
typedef enum { FALQON_PER_TENSOR = 0, FALQON_PER_ROW = 1 } falqon_gran;

/* A CUDA stream handle (the same pointer type as cudaStream_t); NULL is the default stream. */
typedef struct CUstream_st *falqon_stream;

/* One melded layer (Alg. 1 of the paper builds it; Eq. A_integ defines W~').  Host struct. */
typedef struct {
  int64_t m;      /* output features (rows of W)                                         */
  int64_t n;      /* input features (columns of W)                                       */
  int64_t r;      /* LoRA rank                                                           */
  uint8_t *wq;    /* device [(m + r)][n] E4M3 codes; rows m..m+r-1 hold A~ = Q(A; s_W)   */
  float *s_w;     /* device [1]: the per-tensor scale of W~, shared by A~ (FALQON_PER_TENSOR, the
                     paper's scheme); or device [m + 1] (FALQON_PER_ROW): s_w[i] = absmax scale of
                     row i of W~, s_w[m] = the one absmax scale of the A~ block                 */
  float *dbuf;    /* device [m][r] fp32 DeltaBuffer                                      */
  int32_t gran;   /* falqon_gran of s_w.  PER_ROW is an extension for heavy-tailed backbones:
                     the forward rescales per output column; backward divides column i of dY by
                     s_w[i] before its E5M2 cast (the row scales lie on dX's contraction axis) and
                     multiplies row i of dB back; the merge weighs DeltaBuffer row i by
                     s_w[i] / s_w[m].  Scales stay frozen after set-up in both modes.          */
  int32_t flags;  /* bit set of falqon_layer_flag; 0 = none                              */
} falqon_layer;

/* Per-layer options (falqon_layer.flags).
 *  FALQON_LAYER_FUSED_CAST  The casts of X (forward) and dY (backward) run inside the producers of the tensor-core
 *      products instead of as passes of their own: the product kernels fetch the bf16 tensor tile by tile, scale and
 *      round it in shared memory, and multiply the codes from there (Alg. 2 lines 5-6 and the cast of Alg. 3's incoming
 *      gradient, Eq. quantize, fused with Eq. o_split's product).  x~ is then never written to memory; g~ is written once,
 *      by the input-gradient product, because the adapter-gradient product reads it as a tensor.  The codes, the
 *      scales and therefore every result are bit for bit those of the un-fused calls.  Only the absmax reduction (one
 *      read of the tensor) remains as a separate pass, and not even that in the *_amax calls.  Applies where the fused
 *      kernel can run -- bf16 inputs; forward: (m + r) a multiple of 16; backward: per-tensor s_w and dX requested -- and
 *      silently falls back to the un-fused path elsewhere.  FALQON_WS_XQ holds no codes after a fused forward.
 *  FALQON_LAYER_EMIT_XQ     With FALQON_LAYER_FUSED_CAST: the fused forward also writes x~ to FALQON_WS_XQ (one extra
 *      write of T*n bytes), for layers that share it through falqon_melded_forward_codes.
 *  FALQON_LAYER_DB_OWN_KERNEL  By default the adapter gradient (Eq. lora_backward_modified) of a call whose dX is
 *      requested is computed inside the launch of the input-gradient product, on the SM pairs that the product's last wave
 *      of tiles leaves idle: one accumulation over all tokens per element, in token order.  With this flag (and always for
 *      calls without dX, and for falqon_melded_backward_update at ranks above 128) dB is a kernel of its own that sums four
 *      token slabs in slab order.  Both are deterministic; they differ in the last bits of dB. */
typedef enum { FALQON_LAYER_FUSED_CAST = 1, FALQON_LAYER_EMIT_XQ = 2, FALQON_LAYER_DB_OWN_KERNEL = 4 } falqon_layer_flag;

/* Names of the regions inside the workspace that hold staged intermediates of the last call
 * (readable by a caller that wants to inspect or reuse them; see falqon_workspace_region). */
typedef enum {
  FALQON_WS_XQ = 0,       /* uint8 [T][n]   E4M3 codes of X       (after falqon_melded_forward)  */
  FALQON_WS_GQ = 1,       /* uint8 [T][m]   E5M2 codes of dY      (after falqon_melded_backward) */
  FALQON_WS_OAQ_T = 2,    /* uint8 [r16][T16] E4M3 codes of O_A, TRANSPOSED; r16 = r rounded up
                             to 16, row pitch T16 = T rounded up to 16 (after backward)          */
  FALQON_WS_SCALES = 3,   /* float [8]: 0 amax(X) 1 s_x 2 amax(dY) 3 s_g 4 amax(O_A) 5 s_OA      */
  FALQON_WS_SCORE = 4     /* float [m] row scores sum_j |DeltaBuffer[i][j]| (after proxy update)  */
} falqon_ws_region;

/* Host, pure.  Bytes of workspace that the calls below need for a layer of this shape with at
 * most T_max tokens.  Returns 0 if the shape is not supported. */
size_t falqon_workspace_bytes(int64_t m, int64_t n, int64_t r, int64_t T_max);

/* Clears the control words at the start of a workspace (8 KB: the counters of the in-kernel grid barrier, of the
 * "last CTA finishes the job" hand-overs and of the merge's row groups).  Call it once after allocating a
 * workspace, before the first falqon_melded_forward / _backward / _proxy_update that uses it, and again after a
 * call reported FALQON_ERR_TIMEOUT.  The calls leave those words cleared, so a workspace that is only ever passed
 * to this library needs it once.  Enqueues a memset on `stream`. */
int falqon_workspace_init(void *ws, size_t ws_bytes, falqon_stream stream);

/* Host, pure.  Byte offset and size of a region inside a workspace laid out for (m, n, r, T_max).
 * Returns FALQON_OK or FALQON_ERR_INVALID_ARG. */
int falqon_workspace_region(int64_t m, int64_t n, int64_t r, int64_t T_max, falqon_ws_region which,
                            size_t *offset, size_t *bytes);

/* Q_fp8 (Eq. quantize): absmax -> scale s = fp8max/amax -> saturating round-to-nearest-even cast.
 *   src        device [rows][cols], bf16 or fp32 (src_dt), dense; cols a multiple of 16
 *   fmt        E4M3 (weights, activations) or E5M2 (gradients)
 *   gran       one scale for the tensor, or one per row
 *   scale_in   device, nullable.  NULL: scale(s) come from the absmax and are written to scale_out.
 *              Non-NULL ([1] or [rows]): cast with these scale(s) -- A~ = Q(gamma*A; s_W), Eq. A_integ.
 *   premul     fp32 factor multiplied in first as its own rounded multiply (gamma = alpha/r); 1.0f = none
 *   dst        device [rows][cols] uint8 codes
 *   scale_out  device [1] or [rows], nullable when scale_in is given
 *   amax_out   device [1] or [rows], nullable
 *   ws         device scratch of at least FALQON_QUANTIZE_WS_BYTES (per-tensor mode with an absmax only);
 *              it needs no initialisation
 * amax == 0 gives scale 1.  NaN inputs are outside the contract. */
#define FALQON_QUANTIZE_WS_BYTES 8192
int falqon_quantize(const void *src, falqon_dtype src_dt, int64_t rows, int64_t cols, falqon_fp8 fmt,
                    falqon_gran gran, const float *scale_in, float premul, uint8_t *dst,
                    float *scale_out, float *amax_out, void *ws, size_t ws_bytes, falqon_stream stream);

/* Melded forward (Alg. 2 lines 5-9; Eq. o_split):  x~, s_x = Q_e4m3(X);
 *   [Y | O_A] = x~ * W~'^T / (s_W * s_x)   accumulated in fp32 on the tensor cores.
 *   X        device [T][n] bf16 or fp32
 *   Y        device [T][m] bf16 or fp32 (y_dt)
 *   OA       device [T][r] fp32: the one activation saved for backward
 *   amax_oa  device [1]: max |O_A|, produced by the same kernel
 *   s_x_out  device [1], nullable
 * Leaves x~ and the scales in the workspace (FALQON_WS_XQ, FALQON_WS_SCALES). */
int falqon_melded_forward(const falqon_layer *L, const void *X, falqon_dtype x_dt, int64_t T, void *Y,
                          falqon_dtype y_dt, float *OA, float *amax_oa, float *s_x_out, void *ws,
                          size_t ws_bytes, falqon_stream stream);

/* max |x| over `count` elements (bf16 or fp32) as an fp32 number in *amax_out (device [1]); ws: device scratch of at least
 * FALQON_QUANTIZE_WS_BYTES.  The first half of Eq. quantize on its own, for callers that hold one shard of a tensor whose
 * scale is shared (token-sharded data parallelism: the shards' maxima are combined before falqon_melded_forward_amax /
 * falqon_melded_backward_amax cast each shard with the common scale). */
int falqon_absmax(const void *src, falqon_dtype src_dt, int64_t count, float *amax_out, void *ws, size_t ws_bytes,
                  falqon_stream stream);

/* falqon_melded_forward for a caller that already knows amax_x = max |X| (device [1], fp32, exactly the maximum of the
 * absolute values of the tensor as stored -- or of a larger tensor of which X is a shard, so that all shards are cast
 * with one scale): the kernel that produced X took it on the way out.  The cast is then a
 * single pass -- no absmax reduction, no grid-wide barrier.  Everything else as falqon_melded_forward. */
int falqon_melded_forward_amax(const falqon_layer *L, const void *X, falqon_dtype x_dt, const float *amax_x, int64_t T,
                               void *Y, falqon_dtype y_dt, float *OA, float *amax_oa, float *s_x_out, void *ws,
                               size_t ws_bytes, falqon_stream stream);

/* The product of the melded forward alone, for inputs that are already quantized: several layers that read the
 * same activations (the q, k and v projections of a block; gate and up) share one x~.
 *   xq   device [T][n] E4M3 codes, e.g. the FALQON_WS_XQ region of the workspace of the layer that ran
 *        falqon_melded_forward on the same X
 *   s_x  device [1], the scale the codes were cast with (entry 1 of that workspace's FALQON_WS_SCALES)
 * Everything else as falqon_melded_forward; this call's workspace holds no x~ afterwards. */
int falqon_melded_forward_codes(const falqon_layer *L, const uint8_t *xq, const float *s_x, int64_t T, void *Y,
                                falqon_dtype y_dt, float *OA, float *amax_oa, void *ws, size_t ws_bytes,
                                falqon_stream stream);

/* Backward (Alg. 3 line 3 with Eq. lora_backward_modified, plus the input gradient the chain rule
 * implies for O = W~ x~ / (s_W s_x)):   g~, s_g = Q_e5m2(dY);   O~_A, s_OA = Q_e4m3(O_A);
 *   dX = g~ * W~ / (s_W * s_g)            (first m rows of W~' only; skipped when dX is NULL)
 *   dB = g~^T * O~_A / (s_g * s_OA)       (fp32 [m][r], overwritten)
 *   dY       device [T][m] bf16 or fp32
 *   OA       device [T][r] fp32 and amax_oa device [1], as the forward produced them
 *   dX       device [T][n] bf16 or fp32 (dx_dt), nullable
 *   s_g_out  device [1], nullable */
int falqon_melded_backward(const falqon_layer *L, const void *dY, falqon_dtype dy_dt, int64_t T,
                           const float *OA, const float *amax_oa, void *dX, falqon_dtype dx_dt, float *dB,
                           float *s_g_out, void *ws, size_t ws_bytes, falqon_stream stream);

/* falqon_melded_backward for a caller that already knows amax_dy = max |dY| (device [1]); per-tensor layers only
 * (FALQON_ERR_UNSUPPORTED for FALQON_PER_ROW, whose cast input is dY divided by the row scales). */
int falqon_melded_backward_amax(const falqon_layer *L, const void *dY, falqon_dtype dy_dt, const float *amax_dy, int64_t T,
                                const float *OA, const float *amax_oa, void *dX, falqon_dtype dx_dt, float *dB,
                                float *s_g_out, void *ws, size_t ws_bytes, falqon_stream stream);

/* falqon_melded_backward for an output gradient that is already quantized: several layers that receive the same gradient
 * (the q, k and v projections of a block whose outputs are summed) share one g~, as falqon_melded_forward_codes shares x~.
 *   gq   device [T][m] E5M2 codes, e.g. the FALQON_WS_GQ region of the workspace of the layer whose
 *        falqon_melded_backward cast the same dY
 *   s_g  device [1], the scale they were cast with (entry 3 of that workspace's FALQON_WS_SCALES)
 * O_A is still cast here (it is the layer's own).  Per-tensor scaled layers only (FALQON_ERR_UNSUPPORTED otherwise: a
 * per-row layer's codes are those of dY divided by its own row scales).  This call's workspace holds no g~ afterwards. */
int falqon_melded_backward_codes(const falqon_layer *L, const uint8_t *gq, const float *s_g, int64_t T, const float *OA,
                                 const float *amax_oa, void *dX, falqon_dtype dx_dt, float *dB, void *ws, size_t ws_bytes,
                                 falqon_stream stream);

/* The second half of falqon_melded_backward as a call of its own (the input-gradient product implied by Alg. 3): after a
 * falqon_melded_backward[_amax] with dX == NULL -- which casts dY and O_A and computes dB -- this call computes
 *   dX = g~ * W~ / (s_W * s_g)
 * from the codes g~ and the scale s_g that call left in the workspace (FALQON_WS_GQ, FALQON_WS_SCALES; same T, same
 * workspace, nothing else run on it in between).  The result is bit for bit the dX of the single call.  For callers
 * that start exchanging dB while dX is still being computed (token-sharded data parallelism: dB is the one tensor
 * that has to be summed over the shards, and nothing needs it before the proxy update). */
int falqon_melded_backward_dx(const falqon_layer *L, int64_t T, void *dX, falqon_dtype dx_dt, void *ws, size_t ws_bytes,
                              falqon_stream stream);

/* Debug hook of the fused casts ("identical FP8 operands"): falqon_melded_forward / _backward for a layer with
 * FALQON_LAYER_FUSED_CAST, in which the product's tiles of output-column block n_block (256 columns each; forward:
 * columns of [Y | O_A], backward: columns of dX) also write the codes they staged in shared memory to FALQON_WS_XQ /
 * FALQON_WS_GQ.  Every column block converts the whole A operand for itself, so running this for each n_block and
 * comparing the region with falqon_quantize (or the oracle's cast) checks every staged tile.  amax (device [1],
 * nullable): max |X| / max |dY| if already known.  Returns FALQON_ERR_UNSUPPORTED where the fused kernel does not
 * apply (see FALQON_LAYER_FUSED_CAST), FALQON_ERR_INVALID_ARG for an n_block outside the product.  In the backward
 * the adapter gradient is computed from the codes this block wrote. */
int falqon_melded_forward_dump(const falqon_layer *L, const void *X, falqon_dtype x_dt, const float *amax_x, int64_t T,
                               void *Y, falqon_dtype y_dt, float *OA, float *amax_oa, float *s_x_out, int32_t n_block,
                               void *ws, size_t ws_bytes, falqon_stream stream);
int falqon_melded_backward_dump(const falqon_layer *L, const void *dY, falqon_dtype dy_dt, const float *amax_dy, int64_t T,
                                const float *OA, const float *amax_oa, void *dX, falqon_dtype dx_dt, float *dB,
                                float *s_g_out, int32_t n_block, void *ws, size_t ws_bytes, falqon_stream stream);

/* Row-wise proxy update (Alg. 3 lines 4-6; Eq. update):
 *   DeltaBuffer <- fma(-lr, dB, DeltaBuffer)          (plain SGD form; skipped when dB is NULL, so a
 *                                                      caller may run its own optimizer on dbuf)
 *   score_i = sum_j |DeltaBuffer[i][j]|               (fp32, j ascending)
 *   idx     = the k rows of largest score, ties to the lowest index, ascending
 *   W~[i][:] <- sat_rne_e4m3( W~[i][:] + DeltaBuffer[i][:] * A~ )  for i in idx, as an fp32 fma chain
 *              over j ascending (s_W cancels because A~ carries it); then DeltaBuffer[i][:] <- 0
 *   idx_out  device [k] int32, nullable.   k == 0: optimizer step and scores only.  k > m: invalid.
 * Mutates L->wq and L->dbuf.  With dB == NULL, lr == 0, k == m and dbuf preset to an initial B this
 * is also the operation that melds that B into the backbone at set-up. */
int falqon_proxy_update(const falqon_layer *L, const float *dB, float lr, int64_t k, int32_t *idx_out,
                        void *ws, size_t ws_bytes, falqon_stream stream);

/* Alg. 3 lines 3-4 in one call: falqon_melded_backward (or, with amax_dy non-NULL, falqon_melded_backward_amax) followed
 * by the plain-SGD step on the DeltaBuffer and the row scores,
 *     DeltaBuffer <- fma(-lr, dB, DeltaBuffer);   score_i = sum_j |DeltaBuffer[i][j]|  (fp32, j ascending),
 * both computed where dB is produced -- in the epilogue of the dB tiles that ride on the input-gradient product's launch
 * (ranks up to 128, dX requested), else in the adapter-gradient kernel's slab-sum phase: either holds whole rows of dB --
 * so the DeltaBuffer and dB are not read again by a pass of their own.  The scores are left in FALQON_WS_SCORE.  Bit for bit the
 * DeltaBuffer and scores that falqon_melded_backward + falqon_proxy_update(dB, lr, k = 0) produce.  Mutates L->dbuf.
 * dB (device [m][r] fp32) is still written.  Follow it with falqon_proxy_update_scored on the same workspace.
 * (Where the kernel's shared memory has no room for the fused step -- ranks near 256 with few token slabs -- the same
 * arithmetic runs as a pass of its own, with the same results.) */
int falqon_melded_backward_update(const falqon_layer *L, const void *dY, falqon_dtype dy_dt, const float *amax_dy, int64_t T,
                                  const float *OA, const float *amax_oa, void *dX, falqon_dtype dx_dt, float *dB, float lr,
                                  float *s_g_out, void *ws, size_t ws_bytes, falqon_stream stream);

/* Alg. 3 lines 5-6 (Eq. update) on their own: row selection and merge, as in falqon_proxy_update, from the row scores
 * that falqon_melded_backward_update left in this workspace (they must be those of the current DeltaBuffer; nothing is
 * recomputed).  k == 0 is a no-op.  The batched form takes host arrays like falqon_proxy_update_batched and is
 * bit-identical to the per-layer calls. */
int falqon_proxy_update_scored(const falqon_layer *L, int64_t k, int32_t *idx_out, void *ws, size_t ws_bytes,
                               falqon_stream stream);
int falqon_proxy_update_scored_batched(const falqon_layer *layers, int32_t count, const int64_t *k, int32_t *const *idx_out,
                                       void *const *ws, const size_t *ws_bytes, falqon_stream stream);

/* falqon_proxy_update for `count` layers in two launches instead of 2 x count (Alg. 3 lines 4-6, Eq. update, for each
 * layer; the paper's layer-wise schedule runs the updates of a block's projections back to back, and one layer's update
 * moves only a few MB, so a single call is bound by launch latency rather than by memory).  All arrays are HOST arrays
 * of `count` entries: layers[i] (each with its own wq / s_w / dbuf), dB[i] (device [m_i][r_i] fp32, or NULL for that
 * layer), k[i], idx_out (NULL, or entries that are device [k_i] int32 or NULL), ws[i] / ws_bytes[i] (each layer's own
 * initialised workspace, as for falqon_proxy_update; two layers must not share one).  The layers may differ in shape,
 * rank, granularity and k.  lr is shared.  The result for every layer is bit-identical to its own
 * falqon_proxy_update call.  Any invalid entry rejects the whole call before anything is launched.  count == 0 is a
 * no-op.  A layer whose k needs more row groups than a workspace has counters for (k > 16384) makes the call fall back
 * to per-layer launches, with the same results. */
int falqon_proxy_update_batched(const falqon_layer *layers, int32_t count, const float *const *dB, float lr,
                                const int64_t *k, int32_t *const *idx_out, void *const *ws, const size_t *ws_bytes,
                                falqon_stream stream);

/* The same update with AdamW as the optimizer -- the one the paper trains with (its Alg. 3 leaves "Optimizer"
 * generic).  exp_avg and exp_avg_sq are device [m][r] fp32 state, zero before step 1, updated in place; they are NOT
 * cleared when a row is merged (only DeltaBuffer rows are).  For every element, in fp32 and in this order:
 *   p = p * (1 - lr*weight_decay);   m = fma(beta1, m, (1-beta1) * g);   v = fma(beta2, v, (1-beta2) * (g*g));
 *   p = fma(-lr / (1 - beta1^step), m / (sqrt(v) / sqrt(1 - beta2^step) + eps), p)
 * where the constants (1 - lr*weight_decay), (1-beta), lr / (1 - beta1^step), sqrt(1 - beta2^step) are evaluated in
 * double from the fp32 hyper-parameters and rounded once to fp32.  step counts from 1.  Everything after the
 * optimizer (scores, top-k, merge, clearing) is as in falqon_proxy_update. */
typedef struct {
  float lr, beta1, beta2, eps, weight_decay;
  int64_t step;
} falqon_adamw;
int falqon_proxy_update_adamw(const falqon_layer *L, const float *dB, float *exp_avg, float *exp_avg_sq,
                              const falqon_adamw *hp, int64_t k, int32_t *idx_out, void *ws, size_t ws_bytes,
                              falqon_stream stream);

/* falqon_proxy_update_adamw for `count` layers in two launches (falqon_proxy_update_batched with AdamW as the optimizer of
 * every layer).  exp_avg[i], exp_avg_sq[i]: device [m_i][r_i] fp32 state of layer i; dB[i] must not be NULL.  The
 * hyper-parameters (and the step count) are shared by the layers.  Bit-identical to the per-layer calls. */
int falqon_proxy_update_batched_adamw(const falqon_layer *layers, int32_t count, const float *const *dB,
                                      float *const *exp_avg, float *const *exp_avg_sq, const falqon_adamw *hp,
                                      const int64_t *k, int32_t *const *idx_out, void *const *ws, const size_t *ws_bytes,
                                      falqon_stream stream);

/* The proxy update for callers that cannot provide a workspace.  The paper has no counterpart: this
 * is the same operation as falqon_proxy_update, with the same arguments minus the workspace, for code
 * that runs as a guest inside another runtime (a framework's custom-op hook, a server's plug-in) whose
 * allocator already owns the device's memory: such a guest has nothing to allocate from, and a
 * cudaMalloc of its own would fail or stall the whole device mid-step.  The scratch (row scores and
 * the selected-row list) is a fixed 128 KB array inside the library image, resident on every GPU that
 * loads the library until the process exits.
 *   - Limits: L->m <= FALQON_STATIC_MAX_ROWS and a per-tensor scaled layer (FALQON_PER_TENSOR); otherwise
 *     FALQON_ERR_UNSUPPORTED and nothing is launched.
 *   - The first call on each device looks up the array's device address (that device must be current);
 *     make that first call outside any stream capture.  Nothing is allocated or freed, ever.
 *   - All calls on a device share the array, which keeps the previous call's contents; nothing needs to
 *     start at zero, but calls whose kernels overlap on the GPU race on it: order them on one stream
 *     or with events.
 *   - The row scores are not exposed (there is no workspace region to read them from). */
#define FALQON_STATIC_MAX_ROWS 16384
int falqon_proxy_update_static(const falqon_layer *L, const float *dB, float lr, int64_t k, int32_t *idx_out,
                               falqon_stream stream);

/* Initialisation of the adapter from the quantization error (Alg. 1 lines 4-5; Eq. q_error, Eq. reform):
 *     Delta W = W - dec(W~) / s_W,      A^ = sqrt(S_r) V_r^T   of the rank-r truncated SVD  Delta W ~ U_r S_r V_r^T
 * (the singular values split evenly between B^ = U_r sqrt(S_r) and A^; only A^ enters the melded layer, B^ is what
 * quantization already did to W).  Computed by a randomized subspace iteration with `power_iters` power steps, fp32,
 * set-up code off the per-step path; its accuracy is that of the method: excellent where the spectrum of Delta W
 * decays, a near-optimal r-dimensional subspace where it is flat (the rows of A^ are then not individually
 * meaningful).  Per-tensor scaled W~ only.
 *   W        device [m][n] bf16 or fp32, the backbone that was quantized
 *   wq, s_w  device [m][n] E4M3 codes and [1] scale from falqon_quantize(W)
 *   omega    device [n][l] fp32, an i.i.d. standard normal test matrix drawn by the caller; l even, r <= l <= 160
 *            (l = r + 16 is a good choice)
 *   A_hat    device [r][n] fp32 out; each row is determined up to its sign
 *   sigma    device [r] fp32 out: the leading singular values of Delta W
 *   scratch  device, falqon_svd_init_scratch_bytes(m, n, l) bytes
 * Returns FALQON_OK, FALQON_ERR_INVALID_ARG, FALQON_ERR_WORKSPACE or FALQON_ERR_CUDA. */
size_t falqon_svd_init_scratch_bytes(int64_t m, int64_t n, int64_t l);
int falqon_svd_init(const void *W, falqon_dtype w_dt, int64_t m, int64_t n, const uint8_t *wq, const float *s_w, int64_t r,
                    const float *omega, int64_t l, int32_t power_iters, float *A_hat, float *sigma, void *scratch,
                    size_t scratch_bytes, falqon_stream stream);

/* The proxy update with a CORRECTLY ROUNDED merge (an extension: the paper does not fix the merge arithmetic, and
 * falqon_proxy_update reads it as an fp32 fma chain).  Steps 1-3 (optimizer, scores, top-k) and the clearing are the
 * same; the merge becomes
 *     W~[i][c] <- sat_rne_e4m3( W~[i][c] + sum_j d'_ij * A~[j][c] )      sum exact, ONE rounding
 * (nearest, ties to the even code, saturating at +-448; a sum that rounds to zero keeps its sign, an exact zero is
 * +0; d'_ij = DeltaBuffer entry, in per-row mode times s_w[i] / s_w[m] as its own fp32 multiply).  The sums are
 * formed on the tensor cores from exact bf16 limbs; an element whose sum lies within the accumulation error bound of
 * a rounding boundary is recomputed in exact integer arithmetic, so the result does not depend on summation order.
 *   scratch        device, falqon_exact_merge_scratch_bytes(m, n, r) bytes, no initialisation needed
 *   sums_out       device [k][n] fp32, nullable: the tensor-core sums before rounding (diagnostics)
 *   fix_count_out  device [1], nullable: number of elements that took the exact path
 * Other arguments and return values as falqon_proxy_update; FALQON_ERR_WORKSPACE also for a scratch that is too
 * small. */
size_t falqon_exact_merge_scratch_bytes(int64_t m, int64_t n, int64_t r);
int falqon_proxy_update_exact(const falqon_layer *L, const float *dB, float lr, int64_t k, int32_t *idx_out, void *ws,
                              size_t ws_bytes, void *scratch, size_t scratch_bytes, float *sums_out,
                              uint32_t *fix_count_out, falqon_stream stream);

/* The "update A" variant (the paper's appendix ablation with a trainable A; an extension: the melded scheme freezes A):
 *     dL/dA = B^T dL/dO x^T
 * evaluated in the layer's FP8 scheme and applied, after the backward of the same step, in this order:
 *     B~, s_B = Q_e4m3(B)                    per tensor; B: device [m][r] fp32, the caller's record of the adapter's B
 *                                            (the melded scheme keeps none: whatever the caller accumulates)
 *     P = g~ B~ / (s_g s_B)                  [T][r] fp32, g~ and s_g as the backward left them in the workspace
 *     P~, s_P = Q_e4m3(P)                    per tensor
 *     dA = P~^T x~ / (s_P s_x)               [r][n] fp32 (kept transposed, [n][r], in the scratch)
 *     A_master <- fma(-lr, dA, A_master)     device [r][n] fp32, the master copy of A, in place (fold gamma into lr)
 *     A~ <- Q_e4m3(gamma * A_master; s_W)    over rows m .. m+r-1 of L->wq (Eq. A_integ)
 * Rows of W~ merged earlier keep the products with the A~ of their time.  Per-tensor scaled layers only.
 *   xq, s_x   device [T][n] E4M3 codes of the step's X and their scale [1]: a copy the caller kept from the forward
 *             (FALQON_WS_XQ / entry 1 of FALQON_WS_SCALES; the backward reuses that workspace region for g~)
 *   ws        the layer's workspace, holding g~ and s_g of falqon_melded_backward for the same T
 *   scratch   device, falqon_update_a_scratch_bytes(m, n, r, T) bytes, no initialisation needed; afterwards its
 *             regions (falqon_update_a_region) hold the intermediates: FALQON_UA_SCALARS float [4] = amax(B), s_B,
 *             amax(P), s_P; FALQON_UA_BQ_T uint8 [r16][m] codes of B transposed; FALQON_UA_P float [T][r];
 *             FALQON_UA_PQ_T uint8 [r16][T16] codes of P transposed; FALQON_UA_DA_T float [n][r] = dA transposed.
 * Returns FALQON_OK, _INVALID_ARG, _UNSUPPORTED (per-row layer), _WORKSPACE or _CUDA. */
typedef enum { FALQON_UA_SCALARS = 0, FALQON_UA_BQ_T = 1, FALQON_UA_P = 2, FALQON_UA_PQ_T = 3, FALQON_UA_DA_T = 4 } falqon_ua_region;
size_t falqon_update_a_scratch_bytes(int64_t m, int64_t n, int64_t r, int64_t T);
int falqon_update_a_region(int64_t m, int64_t n, int64_t r, int64_t T, falqon_ua_region which, size_t *offset, size_t *bytes);
int falqon_update_a(const falqon_layer *L, const uint8_t *xq, const float *s_x, const float *B, float *A_master, float gamma,
                    float lr, int64_t T, void *ws, size_t ws_bytes, void *scratch, size_t scratch_bytes, falqon_stream stream);

/* falqon_proxy_update_exact for `count` layers: the optimizer steps, scores and selections in one launch and the correctly
 * rounded merges of all layers in three (row preparation, tensor-core sums with the guard-band rounding, exact
 * recomputation of the flagged elements).  Host arrays as in falqon_proxy_update_batched, plus one scratch per layer
 * (falqon_exact_merge_scratch_bytes; two layers must not share one).  Bit-identical to the per-layer
 * falqon_proxy_update_exact calls.
 *   a_prepared  0: the bf16 copy of each layer's A~ rows and its column maxima are rebuilt in this call (two more
 *               launches per layer).  Non-zero: falqon_exact_merge_prepare was run on every layer's scratch and the A~
 *               rows have not changed since (the proxy update never changes them; falqon_update_a does).
 * When to prefer it over the fp32 chain of falqon_proxy_update_batched is a matter of definition first (the two round
 * differently: the chain after every fma, this once) and of size second: the chain costs k n r fp32 fmas, this a
 * tensor-core product plus fixed launches. */
int falqon_exact_merge_prepare(const falqon_layer *L, void *scratch, size_t scratch_bytes, falqon_stream stream);
int falqon_proxy_update_batched_exact(const falqon_layer *layers, int32_t count, const float *const *dB, float lr,
                                      const int64_t *k, int32_t *const *idx_out, void *const *ws, const size_t *ws_bytes,
                                      void *const *scratch, const size_t *scratch_bytes, int32_t a_prepared,
                                      falqon_stream stream);

/* Synchronizes `stream`, then returns and clears the device status word of the current device:
 * FALQON_OK, FALQON_ERR_TIMEOUT (a bounded device-side wait ran out; results of that call are
 * undefined) or FALQON_ERR_CUDA (the synchronize itself failed). */
int falqon_last_device_status(falqon_stream stream);

/* Self-test of the bounded device-side waits: launches one small CTA that waits on a barrier nobody ever signals.  The
 * wait gives up after limit_ms (1..1000) milliseconds, records FALQON_ERR_TIMEOUT in the device status word and the
 * kernel returns; nothing traps, and every later call works as usual.  falqon_last_device_status then returns
 * FALQON_ERR_TIMEOUT once.  (Every wait inside the library's kernels uses the same helper, with a limit of 2 s.) */
int falqon_selftest_wait_timeout(uint32_t limit_ms, falqon_stream stream);

/* Measurement aid (no counterpart in the paper): the ceiling of this GPU's FP8 tensor pipe.  One launch in which every
 * SM pair issues kblocks x 4 of the 256 x 256 x 32 E4M3 MMAs that the forward and input-gradient products issue, on
 * operand tiles that stay in shared memory (random_fill 0: zeros; 1: uniformly random codes drawn from `seed`; 2: the
 * codes of a bell-shaped variable under absmax scaling, as quantized activations are; the data decide the power drawn
 * and with it the clock).  Asynchronous on `stream`; the caller times a sequence of
 * launches with events.  *flops_out (host, nullable) receives the floating-point operations of one launch.
 * sink: device [4 * falqon_tensor_ceiling_ctas()] fp32 or NULL; receives partial sums of the accumulators (all zero
 * for zero operands).  1 <= kblocks <= 2^20.  A wait that runs out sets the device status word.
 * load_src (device, nullable; load_bytes a multiple of 16384, at least 32768): when given, every CTA also streams
 * 2 x 16 KB per k-block from that buffer into its operand slots through a 6-slot producer/consumer ring, i.e. the MMAs
 * now wait for operand traffic from L2 as those of a real 256 x 256 tile pipeline do (a buffer that fits L2 stays
 * there); the MMAs then multiply whatever the buffer holds, and the sums in `sink` follow from it.
 * bytes_per_kblock: what one CTA fetches per k-block (four MMAs): 0 or 32768 for the traffic of 256 x 256 tiles, down to
 * 16384 (a multiple of 16) to model tiles that share more of their operands. */
int falqon_tensor_ceiling_ctas(void);
int falqon_tensor_ceiling(int64_t kblocks, uint32_t seed, int32_t random_fill, float *sink, double *flops_out,
                          const void *load_src, size_t load_bytes, int32_t bytes_per_kblock, falqon_stream stream);

/* Stages that the optional timing hook can bracket with CUDA events (bit i of the mask = stage i). */
typedef enum {
  FALQON_STAGE_QUANT_X = 0,   /* absmax + cast of X            (S1) */
  FALQON_STAGE_GEMM_FWD = 1,  /* melded forward product        (S2) */
  FALQON_STAGE_QUANT_DY = 2,  /* absmax + cast of dY, with the cast of O_A riding along (S3, S5a) */
  FALQON_STAGE_QUANT_OA = 3,  /* unused: the cast of O_A runs inside stage 2 */
  FALQON_STAGE_GEMM_DX = 4,   /* input-gradient product        (S4) */
  FALQON_STAGE_GEMM_DB = 5,   /* adapter-gradient product with the slab sum (S5b) */
  FALQON_STAGE_REDUCE_DB = 6, /* unused: the slab sum runs inside stage 5 */
  FALQON_STAGE_SGD_SCORE = 7, /* optimizer step, row scores and row selection (S6, S7) */
  FALQON_STAGE_TOPK = 8,      /* unused: the row selection runs inside stage 7 (falqon_proxy_update_static, where it is
                                 a kernel of its own, is not bracketed by the timing hook) */
  FALQON_STAGE_MERGE = 9      /* merge + requantize + clear    (S8) */
} falqon_stage;

/* Timing hook for benchmarks (the paper reports the same forward / backward / quantization
 * breakdown).  Host only; not thread safe; off by default.  falqon_profile_start makes the calls
 * above record a pair of CUDA events, on their stream, around each stage whose bit is set in
 * stage_mask, for at most max_records stages (later ones are not recorded).  The events are host
 * objects owned by the library; no device memory is allocated.  falqon_profile_stop waits for the
 * recorded events, writes the elapsed milliseconds and the stage id of each record, in call order,
 * to the two HOST arrays (capacity entries each), releases the events and returns the number of
 * records written (>= 0) or a negative falqon_status. */
int falqon_profile_start(int max_records, unsigned stage_mask);
int falqon_profile_stop(float *ms_out, int *stage_out, int capacity);

/* Host, pure.  Number of kernels the named call launches for this shape (for launch accounting).  The forward and
 * backward of a layer with FALQON_LAYER_FUSED_CAST are named "falqon_melded_forward:fused" / "falqon_melded_backward:fused",
 * a backward whose dB is a kernel of its own (see FALQON_LAYER_DB_OWN_KERNEL) "falqon_melded_backward:own_db". */
int falqon_launch_count(const char *entry_point, int64_t m, int64_t n, int64_t r, int64_t T, int64_t k);

#ifdef __cplusplus
}
#endif
#endif /* FALQON_H_ */
