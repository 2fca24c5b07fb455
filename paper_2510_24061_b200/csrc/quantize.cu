// Q_fp8 kernels (Eq. quantize of the paper): absmax reduction, scale = fp8max / amax, saturating
// round-to-nearest-even cast to E4M3 / E5M2.  HBM-bound: 128-bit loads and stores, warp-shuffle
// reductions, one atomicMax per CTA on the bit pattern of |x| (max is order-free, so the result is
// bit-exact whatever the schedule).
#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxBlocks = 148 * 8;

__device__ __forceinline__ float fp8_max(int fmt) { return fmt == kE4M3 ? 448.0f : 57344.0f; }

// scale = fp8max / amax as one IEEE fp32 division; amax == 0 -> 1; an infinite quotient -> FLT_MAX.
__device__ __forceinline__ float scale_from_amax(float amax, int fmt) {
  if (!(amax > 0.0f)) return 1.0f;
  float s = __fdiv_rn(fp8_max(fmt), amax);
  if (isinf(s)) s = 3.402823466e+38f;
  return s;
}

// Loads 16 consecutive elements as fp32 (element index must be a multiple of 16).
template <int kDt>
__device__ __forceinline__ void load16(const void* src, int64_t elem, float (&v)[16]) {
  if (kDt == kBF16) {
    const uint4* p = reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(src) + elem);
    uint4 a = __ldg(p), b = __ldg(p + 1);
    const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  } else {
    const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(src) + elem);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float4 f = __ldg(p + i);
      v[4 * i] = f.x; v[4 * i + 1] = f.y; v[4 * i + 2] = f.z; v[4 * i + 3] = f.w;
    }
  }
}

template <int kDt>
__device__ __forceinline__ float load1(const void* src, int64_t elem) {
  if (kDt == kBF16) return __uint_as_float(static_cast<uint32_t>(static_cast<const uint16_t*>(src)[elem]) << 16);
  return static_cast<const float*>(src)[elem];
}

__device__ __forceinline__ uint32_t abs_bits(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

template <int kFmt>
__device__ __forceinline__ uint4 cast16(const float (&v)[16], float premul, bool use_premul, float s) {
  float t[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    float x = v[i];
    if (use_premul) x = __fmul_rn(premul, x);  // its own rounded multiply
    t[i] = __fmul_rn(x, s);
  }
  uint4 o;
  o.x = cvt_fp8x4<kFmt>(t[0], t[1], t[2], t[3]);
  o.y = cvt_fp8x4<kFmt>(t[4], t[5], t[6], t[7]);
  o.z = cvt_fp8x4<kFmt>(t[8], t[9], t[10], t[11]);
  o.w = cvt_fp8x4<kFmt>(t[12], t[13], t[14], t[15]);
  return o;
}

__device__ __forceinline__ uint32_t block_max_u32(uint32_t v, uint32_t* smem /* >= 32 words */) {
  v = __reduce_max_sync(0xFFFFFFFFu, v);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) smem[warp] = v;
  __syncthreads();
  const int nwarps = (blockDim.x + 31) >> 5;
  uint32_t w = (threadIdx.x < nwarps) ? smem[threadIdx.x] : 0u;
  if (warp == 0) w = __reduce_max_sync(0xFFFFFFFFu, w);
  if (threadIdx.x == 0) smem[0] = w;
  __syncthreads();
  const uint32_t out = smem[0];
  __syncthreads();
  return out;
}

// ---- pass 1: running max of |premul * x| into *amax_bits (must be 0 on entry)
template <int kDt>
__global__ void __launch_bounds__(kThreads) absmax_kernel(const void* __restrict__ src, int64_t count, float premul,
                                                          bool use_premul, uint32_t* __restrict__ amax_bits) {
  __shared__ uint32_t red[32];
  const int64_t nvec = count / 16;
  uint32_t m = 0;
  for (int64_t v = blockIdx.x * (int64_t)kThreads + threadIdx.x; v < nvec; v += (int64_t)gridDim.x * kThreads) {
    float x[16];
    load16<kDt>(src, v * 16, x);
#pragma unroll
    for (int i = 0; i < 16; ++i) m = max(m, abs_bits(use_premul ? __fmul_rn(premul, x[i]) : x[i]));
  }
  if (blockIdx.x == 0) {  // ragged tail (count not a multiple of 16)
    for (int64_t e = nvec * 16 + threadIdx.x; e < count; e += kThreads) {
      const float x = load1<kDt>(src, e);
      m = max(m, abs_bits(use_premul ? __fmul_rn(premul, x) : x));
    }
  }
  m = block_max_u32(m, red);
  if (threadIdx.x == 0 && m != 0) atomicMax(amax_bits, m);
}

// ---- pass 2: cast with one scale for the whole tensor
template <int kDt, int kFmt>
__global__ void __launch_bounds__(kThreads) cast_kernel(const void* __restrict__ src, int64_t count, float premul,
                                                        bool use_premul, const float* __restrict__ amax_or_scale,
                                                        bool from_amax, uint8_t* __restrict__ dst,
                                                        float* __restrict__ scale_out, float* __restrict__ amax_out) {
  const float in = *amax_or_scale;
  const float s = from_amax ? scale_from_amax(in, kFmt) : in;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    if (scale_out) *scale_out = s;
    if (amax_out && from_amax) *amax_out = in;
  }
  const int64_t nvec = count / 16;
  for (int64_t v = blockIdx.x * (int64_t)kThreads + threadIdx.x; v < nvec; v += (int64_t)gridDim.x * kThreads) {
    float x[16];
    load16<kDt>(src, v * 16, x);
    reinterpret_cast<uint4*>(dst)[v] = cast16<kFmt>(x, premul, use_premul, s);
  }
  if (blockIdx.x == 0) {
    for (int64_t e = nvec * 16 + threadIdx.x; e < count; e += kThreads) {
      float x = load1<kDt>(src, e);
      if (use_premul) x = __fmul_rn(premul, x);
      dst[e] = static_cast<uint8_t>(cvt_fp8x2<kFmt>(__fmul_rn(x, s), 0.0f) & 0xFF);
    }
  }
}

// ---- per-row scaling: one CTA per row, the row is read twice (second time from L1/L2)
template <int kDt, int kFmt>
__global__ void __launch_bounds__(kThreads) quantize_rows_kernel(const void* __restrict__ src, int64_t cols, float premul,
                                                                 bool use_premul, const float* __restrict__ scale_in,
                                                                 uint8_t* __restrict__ dst, float* __restrict__ scale_out,
                                                                 float* __restrict__ amax_out) {
  __shared__ uint32_t red[32];
  const int64_t row = blockIdx.x;
  const int64_t base = row * cols;
  const int64_t nvec = cols / 16;
  float s;
  if (scale_in == nullptr || amax_out != nullptr) {
    uint32_t m = 0;
    for (int64_t v = threadIdx.x; v < nvec; v += kThreads) {
      float x[16];
      load16<kDt>(src, base + v * 16, x);
#pragma unroll
      for (int i = 0; i < 16; ++i) m = max(m, abs_bits(use_premul ? __fmul_rn(premul, x[i]) : x[i]));
    }
    m = block_max_u32(m, red);
    const float amax = __uint_as_float(m);
    if (threadIdx.x == 0 && amax_out) amax_out[row] = amax;
    s = scale_in ? scale_in[row] : scale_from_amax(amax, kFmt);
  } else {
    s = scale_in[row];
  }
  if (threadIdx.x == 0 && scale_out) scale_out[row] = s;
  for (int64_t v = threadIdx.x; v < nvec; v += kThreads) {
    float x[16];
    load16<kDt>(src, base + v * 16, x);
    reinterpret_cast<uint4*>(dst + base)[v] = cast16<kFmt>(x, premul, use_premul, s);
  }
}

// ---- O_A [T][r] fp32 -> E4M3 codes, transposed to [r][ldt] so the dB product reads it K-major
constexpr int kOaTileT = 64;
__global__ void __launch_bounds__(256) quantize_oa_transposed_kernel(const float* __restrict__ oa,
                                                                     const float* __restrict__ amax_oa, int64_t T, int r,
                                                                     int64_t ldt, uint8_t* __restrict__ oaq_t,
                                                                     float* __restrict__ s_oa_out) {
  __shared__ uint8_t tile[256][kOaTileT + 16];
  const float s = scale_from_amax(*amax_oa, kE4M3);
  if (blockIdx.x == 0 && threadIdx.x == 0 && s_oa_out) *s_oa_out = s;
  const int64_t t0 = (int64_t)blockIdx.x * kOaTileT;
  const int tcount = static_cast<int>(min((int64_t)kOaTileT, T - t0));
  for (int e = threadIdx.x; e < tcount * r; e += blockDim.x) {
    const int tl = e / r, j = e - tl * r;
    const float x = oa[(t0 + tl) * r + j];
    tile[j][tl] = static_cast<uint8_t>(cvt_fp8x2<kE4M3>(__fmul_rn(x, s), 0.0f) & 0xFF);
  }
  __syncthreads();
  for (int e = threadIdx.x; e < r * kOaTileT; e += blockDim.x) {
    const int j = e / kOaTileT, tl = e - j * kOaTileT;
    if (tl < tcount) oaq_t[(int64_t)j * ldt + t0 + tl] = tile[j][tl];
  }
}

inline int grid_for(int64_t nvec) {
  int64_t blocks = (nvec + kThreads - 1) / kThreads;
  if (blocks < 1) blocks = 1;
  if (blocks > kMaxBlocks) blocks = kMaxBlocks;
  return static_cast<int>(blocks);
}

}  // namespace

cudaError_t launch_absmax(const void* src, int src_dt, int64_t count, float premul, uint32_t* amax_bits,
                          cudaStream_t stream) {
  cudaError_t e = cudaMemsetAsync(amax_bits, 0, sizeof(uint32_t), stream);
  if (e != cudaSuccess) return e;
  const int grid = grid_for(count / 16);
  const bool use_premul = premul != 1.0f;
  if (src_dt == kBF16) absmax_kernel<kBF16><<<grid, kThreads, 0, stream>>>(src, count, premul, use_premul, amax_bits);
  else absmax_kernel<kF32><<<grid, kThreads, 0, stream>>>(src, count, premul, use_premul, amax_bits);
  return cudaGetLastError();
}

cudaError_t launch_cast_per_tensor(const void* src, int src_dt, int64_t count, int fmt, float premul,
                                   const float* amax_or_scale, bool from_amax, uint8_t* dst, float* scale_out,
                                   float* amax_out, cudaStream_t stream) {
  const int grid = grid_for(count / 16);
  const bool up = premul != 1.0f;
#define FALQON_CAST(DT, FMT) \
  cast_kernel<DT, FMT><<<grid, kThreads, 0, stream>>>(src, count, premul, up, amax_or_scale, from_amax, dst, scale_out, amax_out)
  if (src_dt == kBF16) { if (fmt == kE4M3) FALQON_CAST(kBF16, kE4M3); else FALQON_CAST(kBF16, kE5M2); }
  else { if (fmt == kE4M3) FALQON_CAST(kF32, kE4M3); else FALQON_CAST(kF32, kE5M2); }
#undef FALQON_CAST
  return cudaGetLastError();
}

cudaError_t launch_quantize_per_row(const void* src, int src_dt, int64_t rows, int64_t cols, int fmt, float premul,
                                    const float* scale_in, uint8_t* dst, float* scale_out, float* amax_out,
                                    cudaStream_t stream) {
  const bool up = premul != 1.0f;
  const int grid = static_cast<int>(rows);
#define FALQON_ROWS(DT, FMT) \
  quantize_rows_kernel<DT, FMT><<<grid, kThreads, 0, stream>>>(src, cols, premul, up, scale_in, dst, scale_out, amax_out)
  if (src_dt == kBF16) { if (fmt == kE4M3) FALQON_ROWS(kBF16, kE4M3); else FALQON_ROWS(kBF16, kE5M2); }
  else { if (fmt == kE4M3) FALQON_ROWS(kF32, kE4M3); else FALQON_ROWS(kF32, kE5M2); }
#undef FALQON_ROWS
  return cudaGetLastError();
}

cudaError_t launch_quantize_oa_transposed(const float* oa, const float* amax_oa, int64_t T, int64_t r, int64_t r16,
                                          int64_t ldt, uint8_t* oaq_t, float* s_oa_out, cudaStream_t stream) {
  (void)r16;
  const int grid = static_cast<int>((T + kOaTileT - 1) / kOaTileT);
  quantize_oa_transposed_kernel<<<grid, 256, 0, stream>>>(oa, amax_oa, T, static_cast<int>(r), ldt, oaq_t, s_oa_out);
  return cudaGetLastError();
}

}  // namespace falqon
