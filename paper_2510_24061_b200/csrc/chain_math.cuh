// Per-vector and per-row arithmetic of the stand-in decoder chain (include/falqon_chain.h), shared by the plain chain
// kernels and by their quantizing forms so that both produce the same bf16 values bit for bit.  A vector is eight
// bf16 values (16 bytes); arithmetic is fp32, results rounded to nearest even.
#pragma once

#include <cstdint>

#include "ptx.cuh"

namespace falqon {

__device__ __forceinline__ void unpack8(const uint4& q, float (&x)[8]) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    x[2 * i] = __uint_as_float(w[i] << 16);
    x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint4 pack8(const float (&x)[8]) {
  return make_uint4(pack2(x[0], x[1]), pack2(x[2], x[3]), pack2(x[4], x[5]), pack2(x[6], x[7]));
}

// Largest |bf16| bit pattern (15 bits) among the two halves of each word.
__device__ __forceinline__ uint32_t max_abs_bf16(const uint4& q, uint32_t m) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) m = max(m, max(w[i] & 0x7FFFu, (w[i] >> 16) & 0x7FFFu));
  return m;
}

__device__ __forceinline__ float sigmoidf(float x) { return 1.0f / (1.0f + expf(-x)); }

// bf16(sa*a + sb*b + sc*c + sd*d), left to right with fma; has_b / has_c / has_d say which terms exist.
__device__ __forceinline__ uint4 combine8(const uint4& a, float sa, const uint4& b, float sb, bool has_b, const uint4& c, float sc,
                                          bool has_c, const uint4& d, float sd, bool has_d) {
  float x[8], y[8], acc[8];
  unpack8(a, x);
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = __fmul_rn(sa, x[i]);
  if (has_b) {
    unpack8(b, y);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = __fmaf_rn(sb, y[i], acc[i]);
  }
  if (has_c) {
    unpack8(c, y);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = __fmaf_rn(sc, y[i], acc[i]);
  }
  if (has_d) {
    unpack8(d, y);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = __fmaf_rn(sd, y[i], acc[i]);
  }
  return pack8(acc);
}

// bf16(silu(g) * u)
__device__ __forceinline__ uint4 silu_mul8(const uint4& g, const uint4& u) {
  float x[8], y[8], o[8];
  unpack8(g, x);
  unpack8(u, y);
#pragma unroll
  for (int i = 0; i < 8; ++i) o[i] = x[i] * sigmoidf(x[i]) * y[i];
  return pack8(o);
}

// Gradient of the above: du = dz * g * s, dg = dz * u * s * (1 + g * (1 - s)), s = sigmoid(g).
__device__ __forceinline__ void silu_mul_grad8(const uint4& g, const uint4& u, const uint4& dz, uint4& qg, uint4& qu) {
  float x[8], y[8], t[8], og[8], ou[8];
  unpack8(g, x);
  unpack8(u, y);
  unpack8(dz, t);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float s = sigmoidf(x[i]);
    ou[i] = t[i] * x[i] * s;
    og[i] = t[i] * y[i] * s * (1.0f + x[i] * (1.0f - s));
  }
  qg = pack8(og);
  qu = pack8(ou);
}

// ---- row-wise operations: a group of 128 threads works on one row, a thread keeping its vectors (column vectors
// tid, tid + 128, ..., up to kMaxVec <= kNormMaxVec of them: the caller picks kMaxVec >= vec_per_row / 128) in registers
// between the reduction and the scaling.
constexpr int kNormThreads = 128;
constexpr int kNormMaxVec = 16;   // cols <= 128 * 16 * 8 = 16384

// The 128 threads of a group: tid in [0, 128), a hardware barrier of their own (0 = the CTA-wide one, for CTAs that
// are one group) and four floats of shared memory.
struct RowGroup {
  int tid;
  int bar;
  float* red;
};
__device__ __forceinline__ void group_sync(const RowGroup& g) {
  asm volatile("bar.sync %0, %1;" ::"r"(g.bar), "n"(kNormThreads) : "memory");
}
__device__ __forceinline__ float group_sum(float v, const RowGroup& g) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  if ((g.tid & 31) == 0) g.red[g.tid >> 5] = v;
  group_sync(g);
  const float total = (g.red[0] + g.red[1]) + (g.red[2] + g.red[3]);
  group_sync(g);
  return total;
}

// One row of y = x * inv_rms(x), optionally with x = bf16(sa * a + sb * b) formed (and stored through put_sum) first.
// put_y(v, q) / put_sum(v, q) receive column vector v of the row.  Returns the row's 1 / rms.
template <int kMaxVec, bool kCombine, class PutSum, class PutY>
__device__ __forceinline__ float rmsnorm_row(const uint4* a, float sa, const uint4* b, float sb, int vec_per_row, float inv_cols,
                                             float eps, const RowGroup& g, PutSum put_sum, PutY put_y) {
  uint4 raw[kMaxVec];
  float ss = 0.0f;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int v = g.tid + i * kNormThreads;
    if (v < vec_per_row) {
      if (kCombine) {
        float fa[8], fb[8], acc[8];
        unpack8(ld_stream(a + v), fa);
        unpack8(ld_stream(b + v), fb);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = __fmaf_rn(sb, fb[e], __fmul_rn(sa, fa[e]));
        raw[i] = pack8(acc);
        put_sum(v, raw[i]);
      } else {
        raw[i] = ld_stream(a + v);
      }
      float f[8];
      unpack8(raw[i], f);
#pragma unroll
      for (int e = 0; e < 8; ++e) ss = __fmaf_rn(f[e], f[e], ss);
    }
  }
  const float inv = rsqrtf(group_sum(ss, g) * inv_cols + eps);
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int v = g.tid + i * kNormThreads;
    if (v < vec_per_row) {
      float f[8];
      unpack8(raw[i], f);
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] *= inv;
      put_y(v, pack8(f));
    }
  }
  return inv;
}

// One row of out = bf16(s_res * res + grad) with grad = bf16(inv * (dy - x * inv * mean(dy * x * inv))) and
// dy = bf16(dy_a + dy_b (+ dy_c)); kCombine false: out = grad of dy_a alone (dy_b, dy_c, res unused).
template <int kMaxVec, bool kCombine, class Put>
__device__ __forceinline__ void rmsnorm_grad_row(const uint4* dy_a, const uint4* dy_b, const uint4* dy_c, const uint4* x, float inv,
                                                 const uint4* res, float s_res, int vec_per_row, float inv_cols, const RowGroup& g,
                                                 Put put) {
  uint4 rx[kMaxVec], rdy[kMaxVec];
  float dot = 0.0f;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int v = g.tid + i * kNormThreads;
    if (v < vec_per_row) {
      rx[i] = ld_stream(x + v);
      if (kCombine) {
        float fa[8], fb[8], acc[8];
        unpack8(ld_stream(dy_a + v), fa);
        unpack8(ld_stream(dy_b + v), fb);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = __fmaf_rn(1.0f, fb[e], __fmul_rn(1.0f, fa[e]));
        if (dy_c != nullptr) {
          unpack8(ld_stream(dy_c + v), fb);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[e] = __fmaf_rn(1.0f, fb[e], acc[e]);
        }
        rdy[i] = pack8(acc);
      } else {
        rdy[i] = ld_stream(dy_a + v);
      }
      float fx[8], fd[8];
      unpack8(rx[i], fx);
      unpack8(rdy[i], fd);
#pragma unroll
      for (int e = 0; e < 8; ++e) dot = __fmaf_rn(fd[e], fx[e] * inv, dot);
    }
  }
  const float mean = group_sum(dot, g) * inv_cols;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int v = g.tid + i * kNormThreads;
    if (v < vec_per_row) {
      float fx[8], fd[8], o[8];
      unpack8(rx[i], fx);
      unpack8(rdy[i], fd);
#pragma unroll
      for (int e = 0; e < 8; ++e) o[e] = inv * (fd[e] - fx[e] * inv * mean);
      if (kCombine) {
        float fr[8], gr[8];
        unpack8(pack8(o), gr);                     // the gradient as a kernel of its own would have stored it
        unpack8(ld_stream(res + v), fr);
#pragma unroll
        for (int e = 0; e < 8; ++e) o[e] = __fmaf_rn(1.0f, gr[e], __fmul_rn(s_res, fr[e]));
      }
      put(v, pack8(o));
    }
  }
}

}  // namespace falqon
