// Q_fp8 kernels (Eq. quantize of the paper): absmax reduction, scale = fp8max / amax, saturating
// round-to-nearest-even cast to E4M3 / E5M2.  HBM-bound: 128-bit loads and stores, warp-shuffle
// reductions, one partial maximum per CTA on the bit pattern of |x| (max is order-free, so the result
// is bit-exact whatever the schedule; nothing has to be cleared between calls).
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

// ---- pass 1: max of |premul * x| per CTA, written to partial[blockIdx.x] (no atomics, nothing to
// clear beforehand; the consumer takes the max over the gridDim.x partials)
template <int kDt>
__global__ void __launch_bounds__(kThreads) absmax_kernel(const void* __restrict__ src, int64_t count, float premul,
                                                          bool use_premul, uint32_t* __restrict__ partial) {
  __shared__ uint32_t red[32];
  pdl_trigger();
  pdl_wait();
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
  if (threadIdx.x == 0) partial[blockIdx.x] = m;
}

// ---- pass 2: cast with one scale for the whole tensor.  nparts > 0: the scale comes from the max of
// the absmax partials; nparts == 0: *scale_in is used as given.
struct CastOutputs {
  float* scale_out;    // nullable: receives the scale
  float* scale_out2;   // nullable: second copy of the scale (the caller's own output pointer)
  float* amax_out;     // nullable: receives the absmax (only when it was computed)
  float* clear_word;   // nullable: set to 0 (the next kernel accumulates a max into it)
};
template <int kDt, int kFmt>
__global__ void __launch_bounds__(kThreads) cast_kernel(const void* __restrict__ src, int64_t count, float premul,
                                                        bool use_premul, const uint32_t* __restrict__ partial, int nparts,
                                                        const float* __restrict__ scale_in, uint8_t* __restrict__ dst,
                                                        CastOutputs out) {
  __shared__ uint32_t red[32];
  pdl_trigger();
  pdl_wait();
  float s, amax = 0.0f;
  if (nparts > 0) {
    uint32_t mb = 0;
    for (int i = threadIdx.x; i < nparts; i += kThreads) mb = max(mb, partial[i]);
    amax = __uint_as_float(block_max_u32(mb, red));
    s = scale_from_amax(amax, kFmt);
  } else {
    s = *scale_in;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    if (out.scale_out) *out.scale_out = s;
    if (out.scale_out2) *out.scale_out2 = s;
    if (out.amax_out && nparts > 0) *out.amax_out = amax;
    if (out.clear_word) *out.clear_word = 0.0f;
  }
  // walk the tensor from its end: the absmax pass read it front to back, so its tail is what is still in L2
  const int64_t nvec = count / 16;
  for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < nvec; i += (int64_t)gridDim.x * kThreads) {
    const int64_t v = nvec - 1 - i;
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
  pdl_trigger();
  pdl_wait();
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

// ---- O_A [T][r] fp32 -> E4M3 codes, transposed to [r][ldt] so the dB product reads it K-major.
// A CTA converts 32 tokens x r: float4 loads along r, byte transposition through shared memory,
// 16-byte stores along the tokens.
constexpr int kOaTileT = 32;
__global__ void __launch_bounds__(256) quantize_oa_transposed_kernel(const float* __restrict__ oa,
                                                                     const float* __restrict__ amax_oa, int64_t T, int r,
                                                                     int64_t ldt, uint8_t* __restrict__ oaq_t,
                                                                     float* __restrict__ s_oa_out,
                                                                     float* __restrict__ amax_copy) {
  __shared__ __align__(16) uint8_t tile[256][kOaTileT + 16];
  pdl_trigger();
  pdl_wait();
  const float amax = *amax_oa;
  const float s = scale_from_amax(amax, kE4M3);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    if (s_oa_out) *s_oa_out = s;
    if (amax_copy) *amax_copy = amax;
  }
  const int64_t t0 = (int64_t)blockIdx.x * kOaTileT;
  const int tcount = static_cast<int>(min((int64_t)kOaTileT, T - t0));
  const int r4 = r >> 2;                       // r is a multiple of 8
  const int tx = threadIdx.x % r4, ty = threadIdx.x / r4;
  const int rows_per_pass = blockDim.x / r4;
  if (ty < rows_per_pass) {
    for (int tl = ty; tl < kOaTileT; tl += rows_per_pass) {
      uint32_t codes = 0;
      if (tl < tcount) {
        const float4 x = __ldg(reinterpret_cast<const float4*>(oa + (t0 + tl) * r) + tx);
        codes = cvt_fp8x4<kE4M3>(__fmul_rn(x.x, s), __fmul_rn(x.y, s), __fmul_rn(x.z, s), __fmul_rn(x.w, s));
      }
      tile[4 * tx + 0][tl] = static_cast<uint8_t>(codes);
      tile[4 * tx + 1][tl] = static_cast<uint8_t>(codes >> 8);
      tile[4 * tx + 2][tl] = static_cast<uint8_t>(codes >> 16);
      tile[4 * tx + 3][tl] = static_cast<uint8_t>(codes >> 24);
    }
  }
  __syncthreads();
  // each row j of the tile is 32 bytes = two 16-byte stores (tokens beyond T are zero codes and land in
  // the padding of the row pitch, which is a multiple of 16, or are skipped at the very end)
  for (int e = threadIdx.x; e < r * 2; e += blockDim.x) {
    const int j = e >> 1, half = e & 1;
    if (t0 + half * 16 < ldt)
      *reinterpret_cast<uint4*>(oaq_t + (int64_t)j * ldt + t0 + half * 16) = *reinterpret_cast<const uint4*>(&tile[j][half * 16]);
  }
}

inline int grid_for(int64_t nvec) {
  int64_t blocks = (nvec + kThreads - 1) / kThreads;
  if (blocks < 1) blocks = 1;
  if (blocks > kMaxBlocks) blocks = kMaxBlocks;
  return static_cast<int>(blocks);
}

}  // namespace

int absmax_grid(int64_t count) { return grid_for(count / 16); }

cudaError_t launch_absmax(const void* src, int src_dt, int64_t count, float premul, uint32_t* partial, int* nparts,
                          cudaStream_t stream) {
  const int grid = absmax_grid(count);
  *nparts = grid;
  const bool use_premul = premul != 1.0f;
  if (src_dt == kBF16)
    return launch_pdl(absmax_kernel<kBF16>, dim3(grid), dim3(kThreads), 0, stream, 1, src, count, premul, use_premul, partial);
  return launch_pdl(absmax_kernel<kF32>, dim3(grid), dim3(kThreads), 0, stream, 1, src, count, premul, use_premul, partial);
}

cudaError_t launch_cast_per_tensor(const void* src, int src_dt, int64_t count, int fmt, float premul,
                                   const uint32_t* partial, int nparts, const float* scale_in, uint8_t* dst,
                                   float* scale_out, float* scale_out2, float* amax_out, float* clear_word,
                                   cudaStream_t stream) {
  const int grid = grid_for(count / 16);
  const bool up = premul != 1.0f;
  const CastOutputs out{scale_out, scale_out2, amax_out, clear_word};
#define FALQON_CAST(DT, FMT) \
  return launch_pdl(cast_kernel<DT, FMT>, dim3(grid), dim3(kThreads), 0, stream, 1, src, count, premul, up, partial, nparts, \
                    scale_in, dst, out)
  if (src_dt == kBF16) { if (fmt == kE4M3) FALQON_CAST(kBF16, kE4M3); else FALQON_CAST(kBF16, kE5M2); }
  else { if (fmt == kE4M3) FALQON_CAST(kF32, kE4M3); else FALQON_CAST(kF32, kE5M2); }
#undef FALQON_CAST
}

cudaError_t launch_quantize_per_row(const void* src, int src_dt, int64_t rows, int64_t cols, int fmt, float premul,
                                    const float* scale_in, uint8_t* dst, float* scale_out, float* amax_out,
                                    cudaStream_t stream) {
  const bool up = premul != 1.0f;
  const int grid = static_cast<int>(rows);
#define FALQON_ROWS(DT, FMT) \
  return launch_pdl(quantize_rows_kernel<DT, FMT>, dim3(grid), dim3(kThreads), 0, stream, 1, src, cols, premul, up, \
                    scale_in, dst, scale_out, amax_out)
  if (src_dt == kBF16) { if (fmt == kE4M3) FALQON_ROWS(kBF16, kE4M3); else FALQON_ROWS(kBF16, kE5M2); }
  else { if (fmt == kE4M3) FALQON_ROWS(kF32, kE4M3); else FALQON_ROWS(kF32, kE5M2); }
#undef FALQON_ROWS
}

cudaError_t launch_quantize_oa_transposed(const float* oa, const float* amax_oa, int64_t T, int64_t r, int64_t r16,
                                          int64_t ldt, uint8_t* oaq_t, float* s_oa_out, float* amax_copy,
                                          cudaStream_t stream) {
  (void)r16;
  const int grid = static_cast<int>((T + kOaTileT - 1) / kOaTileT);
  return launch_pdl(quantize_oa_transposed_kernel, dim3(grid), dim3(256), 0, stream, 1, oa, amax_oa, T, static_cast<int>(r),
                    ldt, oaq_t, s_oa_out, amax_copy);
}

}  // namespace falqon
