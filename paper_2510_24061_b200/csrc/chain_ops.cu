// Element-wise bf16 kernels of the stand-in decoder chain (see include/falqon_chain.h): harness code for the
// 32-layer stack benchmark, HBM-bound, 16-byte loads and stores, eight elements per thread and iteration.
#include "../../include/falqon_chain.h"
#include "chain_math.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

constexpr int kChainThreads = 256;

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
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  for (int64_t v = blockIdx.x * (int64_t)kChainThreads + threadIdx.x; v < nvec; v += (int64_t)gridDim.x * kChainThreads) {
    const uint4 o = combine8(ld_stream(a + v), sa, b != nullptr ? ld_stream(b + v) : zero, sb, b != nullptr,
                             c != nullptr ? ld_stream(c + v) : zero, sc, c != nullptr, d != nullptr ? ld_stream(d + v) : zero, sd,
                             d != nullptr);
    out[v] = o;
    mx = max_abs_bf16(o, mx);
  }
  if (amax != nullptr) publish_amax(mx, amax);
}

__global__ void __launch_bounds__(kChainThreads) silu_mul_kernel(uint4* z, const uint4* g, const uint4* u, int64_t nvec,
                                                                 float* amax) {
  pdl_trigger();
  pdl_wait();
  uint32_t mx = 0;
  for (int64_t v = blockIdx.x * (int64_t)kChainThreads + threadIdx.x; v < nvec; v += (int64_t)gridDim.x * kChainThreads) {
    const uint4 q = silu_mul8(ld_stream(g + v), ld_stream(u + v));
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
    uint4 qg, qu;
    silu_mul_grad8(ld_stream(g + v), ld_stream(u + v), ld_stream(dz + v), qg, qu);
    dg[v] = qg;
    du[v] = qu;
    mg = max_abs_bf16(qg, mg);
    mu = max_abs_bf16(qu, mu);
  }
  if (amax_dg != nullptr) publish_amax(mg, amax_dg);
  if (amax_du != nullptr) publish_amax(mu, amax_du);
}

// The row-wise kernels: one CTA of 128 threads per row (the row arithmetic is in chain_math.cuh).  kMaxVec: vectors a thread
// holds; rows of up to 4096 values take the 4-vector form (a third of the registers, twice the resident warps).
template <int kMaxVec>
__global__ void __launch_bounds__(kNormThreads) rmsnorm_kernel(uint4* y, float* inv_rms, const uint4* x, int vec_per_row,
                                                               float inv_cols, float eps, float* amax) {
  __shared__ float red[4];
  pdl_trigger();
  pdl_wait();
  const int64_t base = static_cast<int64_t>(blockIdx.x) * vec_per_row;
  const RowGroup grp{static_cast<int>(threadIdx.x), 0, red};
  uint32_t mx = 0;
  const float inv = rmsnorm_row<kMaxVec, false>(x + base, 0.0f, nullptr, 0.0f, vec_per_row, inv_cols, eps, grp, [](int, const uint4&) {},
                                       [&](int v, const uint4& o) {
                                         y[base + v] = o;
                                         mx = max_abs_bf16(o, mx);
                                       });
  if (threadIdx.x == 0) inv_rms[blockIdx.x] = inv;
  if (amax != nullptr) publish_amax(mx, amax);
}

template <int kMaxVec>
__global__ void __launch_bounds__(kNormThreads) rmsnorm_grad_kernel(uint4* dx, const uint4* dy, const uint4* x,
                                                                    const float* inv_rms, int vec_per_row, float inv_cols) {
  __shared__ float red[4];
  pdl_trigger();
  pdl_wait();
  const int64_t base = static_cast<int64_t>(blockIdx.x) * vec_per_row;
  const RowGroup grp{static_cast<int>(threadIdx.x), 0, red};
  rmsnorm_grad_row<kMaxVec, false>(dy + base, nullptr, nullptr, x + base, ld_stream(inv_rms + blockIdx.x), nullptr, 0.0f, vec_per_row,
                          inv_cols, grp, [&](int v, const uint4& o) { dx[base + v] = o; });
}

// sum = bf16(sa * a + sb * b), stored, and the RMS normalisation of that stored (rounded) sum, in one pass over the row:
// the results are bit for bit those of combine_kernel followed by rmsnorm_kernel, without writing the sum and reading it back.
template <int kMaxVec>
__global__ void __launch_bounds__(kNormThreads) combine_rmsnorm_kernel(uint4* sum_out, uint4* y, float* inv_rms, const uint4* a,
                                                                       float sa, const uint4* b, float sb, int vec_per_row,
                                                                       float inv_cols, float eps, float* amax) {
  __shared__ float red[4];
  pdl_trigger();
  pdl_wait();
  const int64_t base = static_cast<int64_t>(blockIdx.x) * vec_per_row;
  const RowGroup grp{static_cast<int>(threadIdx.x), 0, red};
  uint32_t mx = 0;
  const float inv = rmsnorm_row<kMaxVec, true>(a + base, sa, b + base, sb, vec_per_row, inv_cols, eps, grp,
                                      [&](int v, const uint4& s) { sum_out[base + v] = s; },
                                      [&](int v, const uint4& o) {
                                        y[base + v] = o;
                                        mx = max_abs_bf16(o, mx);
                                      });
  if (threadIdx.x == 0) inv_rms[blockIdx.x] = inv;
  if (amax != nullptr) publish_amax(mx, amax);
}

// out = bf16(s_res * res + g) with g = rmsnorm_grad(dy, x, inv_rms) and dy = bf16(dy_a + dy_b (+ dy_c)), in one pass over
// the row: bit for bit combine_kernel, rmsnorm_grad_kernel, combine_kernel in a row (the two intermediates are rounded to
// bf16 in registers exactly as they would be in memory).
template <int kMaxVec>
__global__ void __launch_bounds__(kNormThreads) rmsnorm_grad_combine_kernel(uint4* out, const uint4* dy_a, const uint4* dy_b,
                                                                            const uint4* dy_c, const uint4* x,
                                                                            const float* inv_rms, const uint4* res, float s_res,
                                                                            int vec_per_row, float inv_cols, float* amax) {
  __shared__ float red[4];
  pdl_trigger();
  pdl_wait();
  const int64_t base = static_cast<int64_t>(blockIdx.x) * vec_per_row;
  const RowGroup grp{static_cast<int>(threadIdx.x), 0, red};
  uint32_t mx = 0;
  rmsnorm_grad_row<kMaxVec, true>(dy_a + base, dy_b + base, dy_c != nullptr ? dy_c + base : nullptr, x + base,
                         ld_stream(inv_rms + blockIdx.x), res + base, s_res, vec_per_row, inv_cols, grp,
                         [&](int v, const uint4& q) {
                           out[base + v] = q;
                           mx = max_abs_bf16(q, mx);
                         });
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
  const bool narrow = cols <= 4 * kNormThreads * 8;
  cudaError_t e = narrow ? launch_pdl(rmsnorm_kernel<4>, dim3(static_cast<unsigned>(rows)), dim3(kNormThreads), 0,
                             static_cast<cudaStream_t>(stream), 1, static_cast<uint4*>(y), inv_rms, static_cast<const uint4*>(x),
                             static_cast<int>(cols / 8), 1.0f / static_cast<float>(cols), eps, amax_out)
                         : launch_pdl(rmsnorm_kernel<kNormMaxVec>, dim3(static_cast<unsigned>(rows)), dim3(kNormThreads), 0,
                             static_cast<cudaStream_t>(stream), 1, static_cast<uint4*>(y), inv_rms, static_cast<const uint4*>(x),
                             static_cast<int>(cols / 8), 1.0f / static_cast<float>(cols), eps, amax_out);
  return e == cudaSuccess ? FALQON_OK : FALQON_ERR_CUDA;
}

int falqon_chain_rmsnorm_grad(void* dx, const void* dy, const void* x, const float* inv_rms, int64_t rows, int64_t cols,
                              falqon_stream stream) {
  if (dx == nullptr || dy == nullptr || x == nullptr || inv_rms == nullptr || rows < 1 || rows > (1ll << 30) || cols < 8 ||
      cols % 8 || cols > kNormThreads * kNormMaxVec * 8 || !ok16(dx) || !ok16(dy) || !ok16(x))
    return FALQON_ERR_INVALID_ARG;
  const bool narrow = cols <= 4 * kNormThreads * 8;
  cudaError_t e = narrow ? launch_pdl(rmsnorm_grad_kernel<4>, dim3(static_cast<unsigned>(rows)), dim3(kNormThreads), 0,
                             static_cast<cudaStream_t>(stream), 1, static_cast<uint4*>(dx), static_cast<const uint4*>(dy),
                             static_cast<const uint4*>(x), inv_rms, static_cast<int>(cols / 8), 1.0f / static_cast<float>(cols))
                         : launch_pdl(rmsnorm_grad_kernel<kNormMaxVec>, dim3(static_cast<unsigned>(rows)), dim3(kNormThreads), 0,
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
  const bool narrow = cols <= 4 * kNormThreads * 8;
  cudaError_t e = narrow ? launch_pdl(combine_rmsnorm_kernel<4>, dim3(static_cast<unsigned>(rows)), dim3(kNormThreads), 0,
                             static_cast<cudaStream_t>(stream), 1, static_cast<uint4*>(sum_out), static_cast<uint4*>(y), inv_rms,
                             static_cast<const uint4*>(a), sa, static_cast<const uint4*>(b), sb, static_cast<int>(cols / 8),
                             1.0f / static_cast<float>(cols), eps, amax_out)
                         : launch_pdl(combine_rmsnorm_kernel<kNormMaxVec>, dim3(static_cast<unsigned>(rows)), dim3(kNormThreads), 0,
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
  const bool narrow = cols <= 4 * kNormThreads * 8;
  cudaError_t e = narrow ? launch_pdl(rmsnorm_grad_combine_kernel<4>, dim3(static_cast<unsigned>(rows)), dim3(kNormThreads), 0,
                             static_cast<cudaStream_t>(stream), 1, static_cast<uint4*>(out), static_cast<const uint4*>(dy_a),
                             static_cast<const uint4*>(dy_b), static_cast<const uint4*>(dy_c), static_cast<const uint4*>(x), inv_rms,
                             static_cast<const uint4*>(res), s_res, static_cast<int>(cols / 8), 1.0f / static_cast<float>(cols),
                             amax_out)
                         : launch_pdl(rmsnorm_grad_combine_kernel<kNormMaxVec>, dim3(static_cast<unsigned>(rows)), dim3(kNormThreads), 0,
                             static_cast<cudaStream_t>(stream), 1, static_cast<uint4*>(out), static_cast<const uint4*>(dy_a),
                             static_cast<const uint4*>(dy_b), static_cast<const uint4*>(dy_c), static_cast<const uint4*>(x), inv_rms,
                             static_cast<const uint4*>(res), s_res, static_cast<int>(cols / 8), 1.0f / static_cast<float>(cols),
                             amax_out);
  return e == cudaSuccess ? FALQON_OK : FALQON_ERR_CUDA;
}

}  // extern "C"
