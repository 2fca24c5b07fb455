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
    uint4 a = ld_stream(p), b = ld_stream(p + 1);
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
      float4 f = ld_stream(p + i);
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
__global__ void __launch_bounds__(kThreads) absmax_kernel(const void* src, int64_t count, float premul,
                                                          bool use_premul, uint32_t* partial) {
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
__global__ void __launch_bounds__(kThreads) cast_kernel(const void* src, int64_t count, float premul,
                                                        bool use_premul, const uint32_t* partial, int nparts,
                                                        const float* scale_in, uint8_t* dst,
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

// ---- fused per-tensor quantizer: absmax, a grid-wide barrier, then the cast, in ONE kernel.
// All CTAs are co-resident (the host sizes the grid from the occupancy), so a CTA can wait for the others.
// Each thread keeps the first kCache 16-element vectors it read in registers, so for tensors up to
// grid x 256 x kCache x 16 elements the cast never touches memory again; what does not fit is re-read, most
// recent first (that is what L2 still holds).  The barrier is two counters in the caller's workspace that
// start at zero and are put back to zero by the last CTA to leave, and its wait is bounded.
struct GridSync {
  unsigned int arrive;
  unsigned int depart;
};

__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

template <int kDt> struct RawVec;
template <> struct RawVec<kBF16> { uint4 a, b; };              // 16 bf16
template <> struct RawVec<kF32> { float4 a, b, c, d; };        // 16 fp32

template <int kDt>
__device__ __forceinline__ RawVec<kDt> load_raw(const void* src, int64_t elem);
template <>
__device__ __forceinline__ RawVec<kBF16> load_raw<kBF16>(const void* src, int64_t elem) {
  const uint4* p = reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(src) + elem);
  RawVec<kBF16> r; r.a = ld_stream(p); r.b = ld_stream(p + 1); return r;
}
template <>
__device__ __forceinline__ RawVec<kF32> load_raw<kF32>(const void* src, int64_t elem) {
  const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(src) + elem);
  RawVec<kF32> r; r.a = ld_stream(p); r.b = ld_stream(p + 1); r.c = ld_stream(p + 2); r.d = ld_stream(p + 3); return r;
}
__device__ __forceinline__ void unpack_raw(const RawVec<kBF16>& r, float (&v)[16]) {
  const uint32_t w[8] = {r.a.x, r.a.y, r.a.z, r.a.w, r.b.x, r.b.y, r.b.z, r.b.w};
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ void unpack_raw(const RawVec<kF32>& r, float (&v)[16]) {
  v[0] = r.a.x; v[1] = r.a.y; v[2] = r.a.z; v[3] = r.a.w; v[4] = r.b.x; v[5] = r.b.y; v[6] = r.b.z; v[7] = r.b.w;
  v[8] = r.c.x; v[9] = r.c.y; v[10] = r.c.z; v[11] = r.c.w; v[12] = r.d.x; v[13] = r.d.y; v[14] = r.d.z; v[15] = r.d.w;
}

// Multiplies the 16 values of one vector by the per-column factors col_mul[col .. col+15] (each its own
// rounded multiply); a vector never straddles a row because the row length is a multiple of 16.
__device__ __forceinline__ void apply_col_mul(float (&x)[16], const float* col_mul, int64_t elem, int cols) {
  const int col = static_cast<int>(elem % cols);
  const float4* p = reinterpret_cast<const float4*>(col_mul + col);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float4 f = ld_stream(p + i);
    x[4 * i] = __fmul_rn(x[4 * i], f.x); x[4 * i + 1] = __fmul_rn(x[4 * i + 1], f.y);
    x[4 * i + 2] = __fmul_rn(x[4 * i + 2], f.z); x[4 * i + 3] = __fmul_rn(x[4 * i + 3], f.w);
  }
}

// kColMul: every column c of the [rows][cols] tensor is first multiplied by col_mul[c] (the output gradient
// of a layer whose backbone rows carry their own scales: col_mul[c] = 1 / s_w[c]).
template <int kDt, int kFmt, bool kColMul>
__global__ void __launch_bounds__(kThreads) quantize_fused_kernel(const void* src, int64_t count,
                                                                  uint8_t* dst, uint32_t* partial,
                                                                  GridSync* sync, CastOutputs out,
                                                                  int* status,
                                                                  const float* col_mul, int cols) {
  constexpr int kCache = (kDt == kBF16) ? 4 : 2;
  __shared__ uint32_t red[32];
  __shared__ int s_ok;
  pdl_trigger();
  pdl_wait();
  const int64_t nvec = count / 16;
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  const int64_t first = blockIdx.x * (int64_t)kThreads + threadIdx.x;
  RawVec<kDt> cache[kCache];
  uint32_t m = 0;
  float x[16];
#pragma unroll
  for (int i = 0; i < kCache; ++i) {
    const int64_t v = first + i * stride;
    if (v < nvec) cache[i] = load_raw<kDt>(src, v * 16);
  }
#pragma unroll
  for (int i = 0; i < kCache; ++i) {
    const int64_t v = first + i * stride;
    if (v < nvec) {
      unpack_raw(cache[i], x);
      if (kColMul) apply_col_mul(x, col_mul, v * 16, cols);
#pragma unroll
      for (int e = 0; e < 16; ++e) m = max(m, abs_bits(x[e]));
    }
  }
  int64_t v_last = first + (int64_t)(kCache - 1) * stride;   // last vector index visited by this thread
  for (int64_t v = first + (int64_t)kCache * stride; v < nvec; v += stride) {
    load16<kDt>(src, v * 16, x);
    if (kColMul) apply_col_mul(x, col_mul, v * 16, cols);
#pragma unroll
    for (int e = 0; e < 16; ++e) m = max(m, abs_bits(x[e]));
    v_last = v;
  }
  if (blockIdx.x == 0) {  // ragged tail (count not a multiple of 16)
    for (int64_t e = nvec * 16 + threadIdx.x; e < count; e += kThreads) m = max(m, abs_bits(load1<kDt>(src, e)));
  }
  m = block_max_u32(m, red);
  // ---- grid barrier
  if (threadIdx.x == 0) {
    partial[blockIdx.x] = m;
    __threadfence();
    atomicAdd(&sync->arrive, 1u);
    int ok = 1;
    if (ld_acquire_gpu(&sync->arrive) < gridDim.x) {
      const uint64_t t0 = global_timer_ns();
      for (;;) {
        if (ld_acquire_gpu(&sync->arrive) >= gridDim.x) break;
        __nanosleep(40);
        if (global_timer_ns() - t0 > kWaitLimitNs) { ok = 0; atomicExch(status, kStatusTimeout); break; }
      }
    }
    s_ok = ok;
  }
  __syncthreads();
  if (s_ok) {
    uint32_t mb = 0;
    for (int i = threadIdx.x; i < (int)gridDim.x; i += kThreads) mb = max(mb, __ldcg(partial + i));
    const float amax = __uint_as_float(block_max_u32(mb, red));
    const float s = scale_from_amax(amax, kFmt);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      if (out.scale_out) *out.scale_out = s;
      if (out.scale_out2) *out.scale_out2 = s;
      if (out.amax_out) *out.amax_out = amax;
      if (out.clear_word) *out.clear_word = 0.0f;
    }
    // streamed part, most recent first
    for (int64_t v = v_last; v >= first + (int64_t)kCache * stride; v -= stride) {
      load16<kDt>(src, v * 16, x);
      if (kColMul) apply_col_mul(x, col_mul, v * 16, cols);
      reinterpret_cast<uint4*>(dst)[v] = cast16<kFmt>(x, 1.0f, false, s);
    }
#pragma unroll
    for (int i = kCache - 1; i >= 0; --i) {
      const int64_t v = first + i * stride;
      if (v < nvec) {
        unpack_raw(cache[i], x);
        if (kColMul) apply_col_mul(x, col_mul, v * 16, cols);
        reinterpret_cast<uint4*>(dst)[v] = cast16<kFmt>(x, 1.0f, false, s);
      }
    }
    if (blockIdx.x == 0) {
      for (int64_t e = nvec * 16 + threadIdx.x; e < count; e += kThreads)
        dst[e] = static_cast<uint8_t>(cvt_fp8x2<kFmt>(__fmul_rn(load1<kDt>(src, e), s), 0.0f) & 0xFF);
    }
  }
  // ---- leave: the last CTA puts the counters back to zero for the next call
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int prev = atomicAdd(&sync->depart, 1u);
    if (prev == gridDim.x - 1) {
      sync->arrive = 0u;
      sync->depart = 0u;
      __threadfence();
    }
  }
}

// ---- per-row-scaled backbone: small tables derived from the row scales s_w[0..m] (s_w[m] = scale of the A~ block)
//   mode 0: out[i] = 1 / s_w[i], i < m                      (column factors of dY before its E5M2 cast)
//   mode 1: out[c] = 1 / (s_w[min(c, m)] * s_x), c < m + r  (column factors of the forward epilogue); zero beyond
__global__ void __launch_bounds__(256) scale_table_kernel(int mode, const float* s_w, int m, int r,
                                                          const float* s_x, float* out, int padded) {
  pdl_trigger();
  pdl_wait();
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= padded) return;
  if (mode == 0) out[c] = c < m ? __fdiv_rn(1.0f, s_w[c]) : 0.0f;
  else out[c] = c < m + r ? __fdiv_rn(1.0f, __fmul_rn(s_w[c < m ? c : m], *s_x)) : 0.0f;
}

// ---- per-row scaling: one CTA per row, the row is read twice (second time from L1/L2)
template <int kDt, int kFmt>
__global__ void __launch_bounds__(kThreads) quantize_rows_kernel(const void* src, int64_t cols, float premul,
                                                                 bool use_premul, const float* scale_in,
                                                                 uint8_t* dst, float* scale_out,
                                                                 float* amax_out) {
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
__global__ void __launch_bounds__(256) quantize_oa_transposed_kernel(const float* oa,
                                                                     const float* amax_oa, int64_t T, int r,
                                                                     int64_t ldt, uint8_t* oaq_t,
                                                                     float* s_oa_out,
                                                                     float* amax_copy) {
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
        const float4 x = ld_stream(reinterpret_cast<const float4*>(oa + (t0 + tl) * r) + tx);
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

template <int kDt, int kFmt, bool kColMul>
cudaError_t launch_fused_variant(const void* src, int64_t count, uint8_t* dst, uint32_t* partial, void* sync,
                                 const CastOutputs& out, int* status, const float* col_mul, int cols, cudaStream_t stream) {
  static int blocks_per_sm = 0;
  if (blocks_per_sm == 0) {
    int b = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, quantize_fused_kernel<kDt, kFmt, kColMul>, kThreads, 0);
    if (e != cudaSuccess) return e;
    blocks_per_sm = b < 1 ? 1 : b;
  }
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int64_t grid = (count / 16 + kThreads - 1) / kThreads;
  const int64_t resident = static_cast<int64_t>(blocks_per_sm) * sms;
  if (grid > resident) grid = resident;
  if (grid > kMaxAbsmaxParts) grid = kMaxAbsmaxParts;
  if (grid < 1) grid = 1;
  return launch_pdl(quantize_fused_kernel<kDt, kFmt, kColMul>, dim3(static_cast<unsigned>(grid)), dim3(kThreads), 0, stream,
                    1, src, count, dst, partial, static_cast<GridSync*>(sync), out, status, col_mul, cols);
}

cudaError_t launch_quantize_fused(const void* src, int src_dt, int64_t count, int fmt, uint8_t* dst, uint32_t* partial,
                                  void* sync, float* scale_out, float* scale_out2, float* amax_out, float* clear_word,
                                  int* status, const float* col_mul, int cols, cudaStream_t stream) {
  const CastOutputs out{scale_out, scale_out2, amax_out, clear_word};
#define FALQON_FUSED(DT, FMT)                                                                                              \
  do {                                                                                                                     \
    if (col_mul != nullptr)                                                                                                \
      return launch_fused_variant<DT, FMT, true>(src, count, dst, partial, sync, out, status, col_mul, cols, stream);       \
    return launch_fused_variant<DT, FMT, false>(src, count, dst, partial, sync, out, status, nullptr, 0, stream);           \
  } while (0)
  if (src_dt == kBF16) {
    if (fmt == kE4M3) FALQON_FUSED(kBF16, kE4M3);
    FALQON_FUSED(kBF16, kE5M2);
  }
  if (fmt == kE4M3) FALQON_FUSED(kF32, kE4M3);
  FALQON_FUSED(kF32, kE5M2);
#undef FALQON_FUSED
}

cudaError_t launch_scale_table(int mode, const float* s_w, int64_t m, int64_t r, const float* s_x, float* out, int64_t padded,
                               cudaStream_t stream) {
  const int grid = static_cast<int>((padded + 255) / 256);
  return launch_pdl(scale_table_kernel, dim3(grid), dim3(256), 0, stream, 1, mode, s_w, static_cast<int>(m),
                    static_cast<int>(r), s_x, out, static_cast<int>(padded));
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
