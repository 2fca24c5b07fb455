// Element-wise bf16 kernels of the stand-in decoder chain (see include/falqon_chain.h): harness code for the
// 32-layer stack benchmark, HBM-bound, 16-byte loads and stores, eight elements per thread and iteration.
#include "../../include/falqon_chain.h"
#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

constexpr int kChainThreads = 256;

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
// Raises *amax (the fp32 bit pattern of a non-negative value) to the CTA's largest |bf16| with one atomic per CTA.
__device__ __forceinline__ void publish_amax(uint32_t m, float* amax) {
  __shared__ uint32_t s_max;
  if (threadIdx.x == 0) s_max = 0u;
  __syncthreads();
  m = __reduce_max_sync(0xFFFFFFFFu, m);
  if ((threadIdx.x & 31) == 0 && m != 0u) atomicMax(&s_max, m);
  __syncthreads();
  if (threadIdx.x == 0 && s_max != 0u) atomicMax(reinterpret_cast<unsigned int*>(amax), s_max << 16);
}

__global__ void __launch_bounds__(kChainThreads) combine_kernel(uint4* out, const uint4* a, float sa, const uint4* b, float sb,
                                                                const uint4* c, float sc, const uint4* d, float sd,
                                                                int64_t nvec, float* amax) {
  pdl_trigger();
  pdl_wait();
  uint32_t mx = 0;
  for (int64_t v = blockIdx.x * (int64_t)kChainThreads + threadIdx.x; v < nvec; v += (int64_t)gridDim.x * kChainThreads) {
    float x[8], y[8], acc[8];
    unpack8(ld_stream(a + v), x);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = __fmul_rn(sa, x[i]);
    if (b != nullptr) {
      unpack8(ld_stream(b + v), y);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = __fmaf_rn(sb, y[i], acc[i]);
    }
    if (c != nullptr) {
      unpack8(ld_stream(c + v), y);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = __fmaf_rn(sc, y[i], acc[i]);
    }
    if (d != nullptr) {
      unpack8(ld_stream(d + v), y);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = __fmaf_rn(sd, y[i], acc[i]);
    }
    const uint4 o = pack8(acc);
    out[v] = o;
    mx = max_abs_bf16(o, mx);
  }
  if (amax != nullptr) publish_amax(mx, amax);
}

__device__ __forceinline__ float sigmoidf(float x) { return 1.0f / (1.0f + expf(-x)); }

__global__ void __launch_bounds__(kChainThreads) silu_mul_kernel(uint4* z, const uint4* g, const uint4* u, int64_t nvec,
                                                                 float* amax) {
  pdl_trigger();
  pdl_wait();
  uint32_t mx = 0;
  for (int64_t v = blockIdx.x * (int64_t)kChainThreads + threadIdx.x; v < nvec; v += (int64_t)gridDim.x * kChainThreads) {
    float x[8], y[8], o[8];
    unpack8(ld_stream(g + v), x);
    unpack8(ld_stream(u + v), y);
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i] = x[i] * sigmoidf(x[i]) * y[i];
    const uint4 q = pack8(o);
    z[v] = q;
    mx = max_abs_bf16(q, mx);
  }
  if (amax != nullptr) publish_amax(mx, amax);
}

__global__ void __launch_bounds__(kChainThreads) silu_mul_grad_kernel(uint4* dg, uint4* du, const uint4* g, const uint4* u,
                                                                      const uint4* dz, int64_t nvec, float* amax_dg,
                                                                      float* amax_du) {
  pdl_trigger();
  pdl_wait();
  uint32_t mg = 0, mu = 0;
  for (int64_t v = blockIdx.x * (int64_t)kChainThreads + threadIdx.x; v < nvec; v += (int64_t)gridDim.x * kChainThreads) {
    float x[8], y[8], t[8], og[8], ou[8];
    unpack8(ld_stream(g + v), x);
    unpack8(ld_stream(u + v), y);
    unpack8(ld_stream(dz + v), t);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float s = sigmoidf(x[i]);
      ou[i] = t[i] * x[i] * s;
      og[i] = t[i] * y[i] * s * (1.0f + x[i] * (1.0f - s));
    }
    const uint4 qg = pack8(og), qu = pack8(ou);
    dg[v] = qg;
    du[v] = qu;
    mg = max_abs_bf16(qg, mg);
    mu = max_abs_bf16(qu, mu);
  }
  if (amax_dg != nullptr) publish_amax(mg, amax_dg);
  if (amax_du != nullptr) publish_amax(mu, amax_du);
}

// One CTA of 128 threads per row; a thread keeps its elements (up to 16 vectors of 8) in registers between the
// reduction and the scaling.
constexpr int kNormThreads = 128;
constexpr int kNormMaxVec = 16;   // cols <= 128 * 16 * 8 = 16384

__device__ __forceinline__ float block_sum_128(float v, float* red /* [4] */) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  const float total = (red[0] + red[1]) + (red[2] + red[3]);
  __syncthreads();
  return total;
}

__global__ void __launch_bounds__(kNormThreads) rmsnorm_kernel(uint4* y, float* inv_rms, const uint4* x, int vec_per_row,
                                                               float inv_cols, float eps, float* amax) {
  __shared__ float red[4];
  pdl_trigger();
  pdl_wait();
  const uint4* xr = x + static_cast<int64_t>(blockIdx.x) * vec_per_row;
  uint4* yr = y + static_cast<int64_t>(blockIdx.x) * vec_per_row;
  uint4 raw[kNormMaxVec];
  float ss = 0.0f;
#pragma unroll
  for (int i = 0; i < kNormMaxVec; ++i) {
    const int v = threadIdx.x + i * kNormThreads;
    if (v < vec_per_row) {
      raw[i] = ld_stream(xr + v);
      float f[8];
      unpack8(raw[i], f);
#pragma unroll
      for (int e = 0; e < 8; ++e) ss = __fmaf_rn(f[e], f[e], ss);
    }
  }
  const float inv = rsqrtf(block_sum_128(ss, red) * inv_cols + eps);
  if (threadIdx.x == 0) inv_rms[blockIdx.x] = inv;
  uint32_t mx = 0;
#pragma unroll
  for (int i = 0; i < kNormMaxVec; ++i) {
    const int v = threadIdx.x + i * kNormThreads;
    if (v < vec_per_row) {
      float f[8];
      unpack8(raw[i], f);
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] *= inv;
      const uint4 o = pack8(f);
      yr[v] = o;
      mx = max_abs_bf16(o, mx);
    }
  }
  if (amax != nullptr) publish_amax(mx, amax);
}

__global__ void __launch_bounds__(kNormThreads) rmsnorm_grad_kernel(uint4* dx, const uint4* dy, const uint4* x,
                                                                    const float* inv_rms, int vec_per_row, float inv_cols) {
  __shared__ float red[4];
  pdl_trigger();
  pdl_wait();
  const int64_t base = static_cast<int64_t>(blockIdx.x) * vec_per_row;
  const float inv = ld_stream(inv_rms + blockIdx.x);
  uint4 rx[kNormMaxVec], rdy[kNormMaxVec];
  float dot = 0.0f;
#pragma unroll
  for (int i = 0; i < kNormMaxVec; ++i) {
    const int v = threadIdx.x + i * kNormThreads;
    if (v < vec_per_row) {
      rx[i] = ld_stream(x + base + v);
      rdy[i] = ld_stream(dy + base + v);
      float fx[8], fd[8];
      unpack8(rx[i], fx);
      unpack8(rdy[i], fd);
#pragma unroll
      for (int e = 0; e < 8; ++e) dot = __fmaf_rn(fd[e], fx[e] * inv, dot);
    }
  }
  const float mean = block_sum_128(dot, red) * inv_cols;
#pragma unroll
  for (int i = 0; i < kNormMaxVec; ++i) {
    const int v = threadIdx.x + i * kNormThreads;
    if (v < vec_per_row) {
      float fx[8], fd[8], o[8];
      unpack8(rx[i], fx);
      unpack8(rdy[i], fd);
#pragma unroll
      for (int e = 0; e < 8; ++e) o[e] = inv * (fd[e] - fx[e] * inv * mean);
      dx[base + v] = pack8(o);
    }
  }
}

// sum = bf16(sa * a + sb * b), stored, and the RMS normalisation of that stored (rounded) sum, in one pass over the row:
// the results are bit for bit those of combine_kernel followed by rmsnorm_kernel, without writing the sum and reading it back.
__global__ void __launch_bounds__(kNormThreads) combine_rmsnorm_kernel(uint4* sum_out, uint4* y, float* inv_rms, const uint4* a,
                                                                       float sa, const uint4* b, float sb, int vec_per_row,
                                                                       float inv_cols, float eps, float* amax) {
  __shared__ float red[4];
  pdl_trigger();
  pdl_wait();
  const int64_t base = static_cast<int64_t>(blockIdx.x) * vec_per_row;
  uint4 raw[kNormMaxVec];
  float ss = 0.0f;
#pragma unroll
  for (int i = 0; i < kNormMaxVec; ++i) {
    const int v = threadIdx.x + i * kNormThreads;
    if (v < vec_per_row) {
      float fa[8], fb[8], acc[8];
      unpack8(ld_stream(a + base + v), fa);
      unpack8(ld_stream(b + base + v), fb);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = __fmaf_rn(sb, fb[e], __fmul_rn(sa, fa[e]));
      raw[i] = pack8(acc);
      sum_out[base + v] = raw[i];
      float f[8];
      unpack8(raw[i], f);
#pragma unroll
      for (int e = 0; e < 8; ++e) ss = __fmaf_rn(f[e], f[e], ss);
    }
  }
  const float inv = rsqrtf(block_sum_128(ss, red) * inv_cols + eps);
  if (threadIdx.x == 0) inv_rms[blockIdx.x] = inv;
  uint32_t mx = 0;
#pragma unroll
  for (int i = 0; i < kNormMaxVec; ++i) {
    const int v = threadIdx.x + i * kNormThreads;
    if (v < vec_per_row) {
      float f[8];
      unpack8(raw[i], f);
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] *= inv;
      const uint4 o = pack8(f);
      y[base + v] = o;
      mx = max_abs_bf16(o, mx);
    }
  }
  if (amax != nullptr) publish_amax(mx, amax);
}

// out = bf16(s_res * res + g) with g = rmsnorm_grad(dy, x, inv_rms) and dy = bf16(dy_a + dy_b (+ dy_c)), in one pass over
// the row: bit for bit combine_kernel, rmsnorm_grad_kernel, combine_kernel in a row (the two intermediates are rounded to
// bf16 in registers exactly as they would be in memory).
__global__ void __launch_bounds__(kNormThreads) rmsnorm_grad_combine_kernel(uint4* out, const uint4* dy_a, const uint4* dy_b,
                                                                            const uint4* dy_c, const uint4* x,
                                                                            const float* inv_rms, const uint4* res, float s_res,
                                                                            int vec_per_row, float inv_cols, float* amax) {
  __shared__ float red[4];
  pdl_trigger();
  pdl_wait();
  const int64_t base = static_cast<int64_t>(blockIdx.x) * vec_per_row;
  const float inv = ld_stream(inv_rms + blockIdx.x);
  uint4 rx[kNormMaxVec], rdy[kNormMaxVec];
  float dot = 0.0f;
#pragma unroll
  for (int i = 0; i < kNormMaxVec; ++i) {
    const int v = threadIdx.x + i * kNormThreads;
    if (v < vec_per_row) {
      float fa[8], fb[8], acc[8];
      rx[i] = ld_stream(x + base + v);
      unpack8(ld_stream(dy_a + base + v), fa);
      unpack8(ld_stream(dy_b + base + v), fb);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = __fmaf_rn(1.0f, fb[e], __fmul_rn(1.0f, fa[e]));
      if (dy_c != nullptr) {
        unpack8(ld_stream(dy_c + base + v), fb);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = __fmaf_rn(1.0f, fb[e], acc[e]);
      }
      rdy[i] = pack8(acc);
      float fx[8], fd[8];
      unpack8(rx[i], fx);
      unpack8(rdy[i], fd);
#pragma unroll
      for (int e = 0; e < 8; ++e) dot = __fmaf_rn(fd[e], fx[e] * inv, dot);
    }
  }
  const float mean = block_sum_128(dot, red) * inv_cols;
  uint32_t mx = 0;
#pragma unroll
  for (int i = 0; i < kNormMaxVec; ++i) {
    const int v = threadIdx.x + i * kNormThreads;
    if (v < vec_per_row) {
      float fx[8], fd[8], o[8], fr[8], g[8];
      unpack8(rx[i], fx);
      unpack8(rdy[i], fd);
#pragma unroll
      for (int e = 0; e < 8; ++e) o[e] = inv * (fd[e] - fx[e] * inv * mean);
      unpack8(pack8(o), g);                       // the gradient as the separate kernel would have stored it
      unpack8(ld_stream(res + base + v), fr);
#pragma unroll
      for (int e = 0; e < 8; ++e) o[e] = __fmaf_rn(1.0f, g[e], __fmul_rn(s_res, fr[e]));
      const uint4 q = pack8(o);
      out[base + v] = q;
      mx = max_abs_bf16(q, mx);
    }
  }
  if (amax != nullptr) publish_amax(mx, amax);
}

inline bool ok16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
inline unsigned chain_grid(int64_t nvec) {
  int64_t blocks = (nvec + kChainThreads - 1) / kChainThreads;
  const int64_t cap = static_cast<int64_t>(sm_count()) * 8;
  if (blocks > cap) blocks = cap;
  return static_cast<unsigned>(blocks < 1 ? 1 : blocks);
}

}  // namespace
}  // namespace falqon

using namespace falqon;

extern "C" {

int falqon_chain_combine(void* out, const void* a, float sa, const void* b, float sb, const void* c, float sc, const void* d,
                         float sd, int64_t count, float* amax_out, falqon_stream stream) {
  if (out == nullptr || a == nullptr || count < 8 || count % 8 || !ok16(out) || !ok16(a) || !ok16(b) || !ok16(c) || !ok16(d))
    return FALQON_ERR_INVALID_ARG;
  const int64_t nvec = count / 8;
  cudaError_t e = launch_pdl(combine_kernel, dim3(chain_grid(nvec)), dim3(kChainThreads), 0, static_cast<cudaStream_t>(stream), 1,
                             static_cast<uint4*>(out), static_cast<const uint4*>(a), sa, static_cast<const uint4*>(b), sb,
                             static_cast<const uint4*>(c), sc, static_cast<const uint4*>(d), sd, nvec, amax_out);
  return e == cudaSuccess ? FALQON_OK : FALQON_ERR_CUDA;
}

int falqon_chain_silu_mul(void* z, const void* g, const void* u, int64_t count, float* amax_out, falqon_stream stream) {
  if (z == nullptr || g == nullptr || u == nullptr || count < 8 || count % 8 || !ok16(z) || !ok16(g) || !ok16(u))
    return FALQON_ERR_INVALID_ARG;
  const int64_t nvec = count / 8;
  cudaError_t e = launch_pdl(silu_mul_kernel, dim3(chain_grid(nvec)), dim3(kChainThreads), 0, static_cast<cudaStream_t>(stream), 1,
                             static_cast<uint4*>(z), static_cast<const uint4*>(g), static_cast<const uint4*>(u), nvec, amax_out);
  return e == cudaSuccess ? FALQON_OK : FALQON_ERR_CUDA;
}

int falqon_chain_silu_mul_grad(void* dg, void* du, const void* g, const void* u, const void* dz, int64_t count,
                               float* amax_dg, float* amax_du, falqon_stream stream) {
  if (dg == nullptr || du == nullptr || g == nullptr || u == nullptr || dz == nullptr || count < 8 || count % 8 || !ok16(dg) ||
      !ok16(du) || !ok16(g) || !ok16(u) || !ok16(dz))
    return FALQON_ERR_INVALID_ARG;
  const int64_t nvec = count / 8;
  cudaError_t e = launch_pdl(silu_mul_grad_kernel, dim3(chain_grid(nvec)), dim3(kChainThreads), 0,
                             static_cast<cudaStream_t>(stream), 1, static_cast<uint4*>(dg), static_cast<uint4*>(du),
                             static_cast<const uint4*>(g), static_cast<const uint4*>(u), static_cast<const uint4*>(dz), nvec,
                             amax_dg, amax_du);
  return e == cudaSuccess ? FALQON_OK : FALQON_ERR_CUDA;
}

int falqon_chain_rmsnorm(void* y, float* inv_rms, const void* x, int64_t rows, int64_t cols, float eps, float* amax_out,
                         falqon_stream stream) {
  if (y == nullptr || inv_rms == nullptr || x == nullptr || rows < 1 || rows > (1ll << 30) || cols < 8 || cols % 8 ||
      cols > kNormThreads * kNormMaxVec * 8 || !ok16(y) || !ok16(x) || !(eps >= 0.0f))
    return FALQON_ERR_INVALID_ARG;
  cudaError_t e = launch_pdl(rmsnorm_kernel, dim3(static_cast<unsigned>(rows)), dim3(kNormThreads), 0,
                             static_cast<cudaStream_t>(stream), 1, static_cast<uint4*>(y), inv_rms, static_cast<const uint4*>(x),
                             static_cast<int>(cols / 8), 1.0f / static_cast<float>(cols), eps, amax_out);
  return e == cudaSuccess ? FALQON_OK : FALQON_ERR_CUDA;
}

int falqon_chain_rmsnorm_grad(void* dx, const void* dy, const void* x, const float* inv_rms, int64_t rows, int64_t cols,
                              falqon_stream stream) {
  if (dx == nullptr || dy == nullptr || x == nullptr || inv_rms == nullptr || rows < 1 || rows > (1ll << 30) || cols < 8 ||
      cols % 8 || cols > kNormThreads * kNormMaxVec * 8 || !ok16(dx) || !ok16(dy) || !ok16(x))
    return FALQON_ERR_INVALID_ARG;
  cudaError_t e = launch_pdl(rmsnorm_grad_kernel, dim3(static_cast<unsigned>(rows)), dim3(kNormThreads), 0,
                             static_cast<cudaStream_t>(stream), 1, static_cast<uint4*>(dx), static_cast<const uint4*>(dy),
                             static_cast<const uint4*>(x), inv_rms, static_cast<int>(cols / 8), 1.0f / static_cast<float>(cols));
  return e == cudaSuccess ? FALQON_OK : FALQON_ERR_CUDA;
}

int falqon_chain_combine_rmsnorm(void* sum_out, void* y, float* inv_rms, const void* a, float sa, const void* b, float sb,
                                 int64_t rows, int64_t cols, float eps, float* amax_out, falqon_stream stream) {
  if (sum_out == nullptr || y == nullptr || inv_rms == nullptr || a == nullptr || b == nullptr || rows < 1 || rows > (1ll << 30) ||
      cols < 8 || cols % 8 || cols > kNormThreads * kNormMaxVec * 8 || !ok16(sum_out) || !ok16(y) || !ok16(a) || !ok16(b) ||
      !(eps >= 0.0f))
    return FALQON_ERR_INVALID_ARG;
  cudaError_t e = launch_pdl(combine_rmsnorm_kernel, dim3(static_cast<unsigned>(rows)), dim3(kNormThreads), 0,
                             static_cast<cudaStream_t>(stream), 1, static_cast<uint4*>(sum_out), static_cast<uint4*>(y), inv_rms,
                             static_cast<const uint4*>(a), sa, static_cast<const uint4*>(b), sb, static_cast<int>(cols / 8),
                             1.0f / static_cast<float>(cols), eps, amax_out);
  return e == cudaSuccess ? FALQON_OK : FALQON_ERR_CUDA;
}

int falqon_chain_rmsnorm_grad_combine(void* out, const void* dy_a, const void* dy_b, const void* dy_c, const void* x,
                                      const float* inv_rms, const void* res, float s_res, int64_t rows, int64_t cols,
                                      float* amax_out, falqon_stream stream) {
  if (out == nullptr || dy_a == nullptr || dy_b == nullptr || x == nullptr || inv_rms == nullptr || res == nullptr || rows < 1 ||
      rows > (1ll << 30) || cols < 8 || cols % 8 || cols > kNormThreads * kNormMaxVec * 8 || !ok16(out) || !ok16(dy_a) ||
      !ok16(dy_b) || !ok16(dy_c) || !ok16(x) || !ok16(res))
    return FALQON_ERR_INVALID_ARG;
  cudaError_t e = launch_pdl(rmsnorm_grad_combine_kernel, dim3(static_cast<unsigned>(rows)), dim3(kNormThreads), 0,
                             static_cast<cudaStream_t>(stream), 1, static_cast<uint4*>(out), static_cast<const uint4*>(dy_a),
                             static_cast<const uint4*>(dy_b), static_cast<const uint4*>(dy_c), static_cast<const uint4*>(x), inv_rms,
                             static_cast<const uint4*>(res), s_res, static_cast<int>(cols / 8), 1.0f / static_cast<float>(cols),
                             amax_out);
  return e == cudaSuccess ? FALQON_OK : FALQON_ERR_CUDA;
}

}  // extern "C"
