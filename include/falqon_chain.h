/* Element-wise bf16 operations of the stand-in decoder chain that the 32-layer stack benchmark runs between
 * the melded linear layers (residual sums, the q/k/v mixing stand-in, RMS normalisation, the SiLU-gated MLP and
 * their gradients).
 * Harness code: none of this is part of the paper's method, which is the linear layer alone (falqon.h).
 * Every tensor is a dense device array of `count` bf16 values, 16-byte aligned, count a multiple of 8;
 * arithmetic is fp32, results rounded to nearest even.  Calls are asynchronous on `stream` and return
 * FALQON_OK, FALQON_ERR_INVALID_ARG or FALQON_ERR_CUDA.
 * amax_out arguments (device [1] fp32, nullable): the kernel raises the word to the largest |value| it stored (an
 * atomic max on the bit pattern, so the word must hold 0, or any lower bound >= 0, beforehand).  A melded layer that
 * consumes the tensor can then skip its own absmax pass (falqon_melded_forward_amax / _backward_amax). */
#ifndef FALQON_CHAIN_H
#define FALQON_CHAIN_H

#include "falqon.h"

#ifdef __cplusplus
extern "C" {
#endif

/* out = bf16(sa*a + sb*b + sc*c + sd*d), accumulated left to right with fma; b, c, d may be NULL (skipped).
 * out may alias any input. */
int falqon_chain_combine(void *out, const void *a, float sa, const void *b, float sb, const void *c, float sc,
                         const void *d, float sd, int64_t count, float *amax_out, falqon_stream stream);

/* z = bf16(silu(g) * u), silu(x) = x / (1 + exp(-x)). */
int falqon_chain_silu_mul(void *z, const void *g, const void *u, int64_t count, float *amax_out, falqon_stream stream);

/* Gradient of the above: with s = 1 / (1 + exp(-g)):  du = dz * g * s,  dg = dz * u * s * (1 + g * (1 - s)).
 * dg may alias g or dz, du may alias u. */
int falqon_chain_silu_mul_grad(void *dg, void *du, const void *g, const void *u, const void *dz, int64_t count,
                               float *amax_dg, float *amax_du, falqon_stream stream);

/* Per-row RMS normalisation without a gain: y[t][:] = bf16(x[t][:] * inv_rms[t]), inv_rms[t] = 1 / sqrt(mean(x[t][:]^2) + eps).
 * x, y: [rows][cols] bf16, cols a multiple of 8 and at most 16384; inv_rms: device [rows] fp32, kept for the gradient. */
int falqon_chain_rmsnorm(void *y, float *inv_rms, const void *x, int64_t rows, int64_t cols, float eps,
                         float *amax_out, falqon_stream stream);

/* Gradient of the above: with xh = x * inv_rms:  dx = inv_rms * (dy - xh * mean(dy * xh)), one row at a time. */
int falqon_chain_rmsnorm_grad(void *dx, const void *dy, const void *x, const float *inv_rms, int64_t rows,
                              int64_t cols, falqon_stream stream);

/* falqon_chain_combine (two inputs) followed by falqon_chain_rmsnorm of its result, in one pass: sum_out = bf16(sa*a + sb*b)
 * is stored, y = rmsnorm(sum_out) with inv_rms kept.  Bit for bit the two calls; saves writing the sum and reading it back. */
int falqon_chain_combine_rmsnorm(void *sum_out, void *y, float *inv_rms, const void *a, float sa, const void *b, float sb,
                                 int64_t rows, int64_t cols, float eps, float *amax_out, falqon_stream stream);

/* Three calls in one pass: dy = bf16(dy_a + dy_b (+ dy_c, nullable));  g = falqon_chain_rmsnorm_grad(dy, x, inv_rms);
 * out = bf16(s_res * res + g).  Bit for bit the three calls.  out may alias dy_a, dy_b, dy_c or res. */
int falqon_chain_rmsnorm_grad_combine(void *out, const void *dy_a, const void *dy_b, const void *dy_c, const void *x,
                                      const float *inv_rms, const void *res, float s_res, int64_t rows, int64_t cols,
                                      float *amax_out, falqon_stream stream);

/* ---- Quantizing forms: the chain operation AND the per-tensor cast of its result (Eq. quantize: s = fp8max / absmax,
 * saturating round to nearest even) in one launch, so that the tensor a melded layer consumes never takes a separate
 * quantize pass: the codes go straight to falqon_melded_forward_codes / falqon_melded_backward_codes.  Bit for bit:
 * codes and *scale_out are those of falqon_quantize applied to the bf16 tensor the plain call would have stored.
 *   codes      device [count] bytes, 16-byte aligned (count = rows * cols for the row-wise calls)
 *   scale_out  device [1] fp32
 *   fmt        FALQON_E4M3 (a forward input) or FALQON_E5M2 (an output gradient)
 *   out16      device [count] bf16, 16-byte aligned.  keep16 != 0: receives the bf16 result as the plain call stores it.
 *              keep16 == 0: working space -- the part of the tensor that does not fit in the SMs' shared memory between
 *              the two phases of the kernel passes through it; its contents afterwards are unspecified.
 *              It may be one of the inputs (every position is read before it is written).
 *   scratch    FALQON_CHAIN_SCRATCH_BYTES device bytes, 16-byte aligned, zero before the first call and left zero by every
 *              call; calls that may run at the same time need scratch of their own.
 * The kernel holds a grid-wide barrier (the absmax of the whole tensor precedes the first code), so the launch is
 * cooperative with one CTA per SM; the barrier's wait is bounded and a wait that runs out is reported by
 * falqon_last_device_status (the codes are then incomplete). */
#define FALQON_CHAIN_SCRATCH_BYTES 4096

int falqon_chain_combine_quantize(void *codes, float *scale_out, int fmt, void *out16, int keep16, const void *a, float sa,
                                  const void *b, float sb, const void *c, float sc, const void *d, float sd, int64_t count,
                                  void *scratch, falqon_stream stream);

int falqon_chain_silu_mul_quantize(void *codes, float *scale_out, int fmt, void *out16, int keep16, const void *g, const void *u,
                                   int64_t count, void *scratch, falqon_stream stream);

/* Two results, each with its own codes, scale and bf16 buffer (index 0 of the scratch's partial maxima serves dg, 1 du). */
int falqon_chain_silu_mul_grad_quantize(void *codes_dg, void *codes_du, float *scale_dg, float *scale_du, int fmt, void *dg16,
                                        void *du16, int keep16, const void *g, const void *u, const void *dz, int64_t count,
                                        void *scratch, falqon_stream stream);

/* y = rmsnorm(x) with x = a (b == NULL and sum_out == NULL; sa, sb ignored) or x = bf16(sa*a + sb*b), which is stored to
 * sum_out (falqon_chain_combine_rmsnorm).  inv_rms as in falqon_chain_rmsnorm; y16 plays the part of out16. */
int falqon_chain_rmsnorm_quantize(void *codes, float *scale_out, int fmt, void *y16, int keep16, float *inv_rms, void *sum_out,
                                  const void *a, float sa, const void *b, float sb, int64_t rows, int64_t cols, float eps,
                                  void *scratch, falqon_stream stream);

/* falqon_chain_rmsnorm_grad_combine whose result is stored to out (always: the chain needs it again) and cast. */
int falqon_chain_rmsnorm_grad_combine_quantize(void *codes, float *scale_out, int fmt, void *out, const void *dy_a,
                                               const void *dy_b, const void *dy_c, const void *x, const float *inv_rms,
                                               const void *res, float s_res, int64_t rows, int64_t cols, void *scratch,
                                               falqon_stream stream);

#ifdef __cplusplus
}
#endif
#endif
