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

#ifdef __cplusplus
}
#endif
#endif
