// Q_fp8 kernels (Eq. quantize of the paper): absmax reduction, scale = fp8max / amax, saturating
// round-to-nearest-even cast to E4M3 / E5M2.  HBM-bound: 128-bit loads and stores, warp-shuffle
// reductions, one partial maximum per CTA on the bit pattern of |x| (max is order-free, so the result
// is bit-exact whatever the schedule; nothing has to be cleared between calls).
#include "grid_sync.cuh"
#include "internal.h"
#include "oa_cast.cuh"
#include "ptx.cuh"

namespace falqon {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxBlocks = 148 * 8;

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

// ---- the max over the partials of pass 1, as a number of its own (for callers that combine it with the absmax of other
// shards of the same tensor before the cast)
__global__ void __launch_bounds__(kThreads) absmax_finalize_kernel(const uint32_t* partial, int nparts, float* amax_out) {
  __shared__ uint32_t red[32];
  pdl_trigger();
  pdl_wait();
  uint32_t mb = 0;
  for (int i = threadIdx.x; i < nparts; i += kThreads) mb = max(mb, partial[i]);
  mb = block_max_u32(mb, red);
  if (threadIdx.x == 0) *amax_out = __uint_as_float(mb);
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

// ---- the scale of Eq. quantize on its own, for the products that cast their A operand themselves: from the partial
// maxima of absmax_kernel (nparts > 0) or from an absmax the caller already has (*amax_in), with the same side outputs
// as the cast kernels.  One CTA.
__global__ void __launch_bounds__(kThreads) scale_prep_kernel(const uint32_t* partial, int nparts, const float* amax_in, int fmt,
                                                              CastOutputs out) {
  __shared__ uint32_t red[32];
  pdl_trigger();
  pdl_wait();
  float amax;
  if (nparts > 0) {
    uint32_t mb = 0;
    for (int i = threadIdx.x; i < nparts; i += kThreads) mb = max(mb, ld_stream(partial + i));
    amax = __uint_as_float(block_max_u32(mb, red));
  } else {
    amax = ld_stream(amax_in);
  }
  if (threadIdx.x == 0) {
    const float s = scale_from_amax(amax, fmt);
    if (out.scale_out) *out.scale_out = s;
    if (out.scale_out2) *out.scale_out2 = s;
    if (out.amax_out) *out.amax_out = amax;
    if (out.clear_word) *out.clear_word = 0.0f;
  }
}

// ---- fused per-tensor quantizer: absmax, a grid-wide barrier, then the cast, in ONE kernel, with the tensor held
// in shared memory across the barrier.  All CTAs are co-resident (one per SM; the host sizes the grid from the
// occupancy), so a CTA can wait for the others; the wait is bounded.  Each CTA streams its 56 KB chunks (chunk c belongs to CTA c mod grid;
// every chunk costs a barrier wait and a CTA-wide synchronisation, so few large chunks beat many small ones: 14 x 16 KB
// was 10 % slower)
// through a ring of kStagedSlots bulk-copy targets, so up to 224 KB per SM are in flight or resident without
// costing a register.  After the barrier the chunks still in the ring (the last kStagedSlots of the CTA) are cast
// straight from shared memory; earlier ones are fetched again, most recent first (what L2 still holds), into the
// slots as they free up.  Tensors up to 148 x 224 KB are read from memory exactly once.
constexpr int kStagedThreads = 512;
constexpr int kChunkBytes = 57344;
constexpr int kStagedSlots = 4;

template <int kDt> struct Unit { static constexpr int kElems = kDt == kBF16 ? 8 : 4; };

// The elements of one 16-byte unit as fp32, times their column factors when kColMul.
template <int kDt, bool kColMul>
__device__ __forceinline__ void unit_values(const uint4& q, const float* col_mul, const float* table, int col,
                                            float (&x)[Unit<kDt>::kElems]) {
  if (kDt == kBF16) {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(w[i] << 16);
      x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  } else {
    x[0] = __uint_as_float(q.x); x[1] = __uint_as_float(q.y); x[2] = __uint_as_float(q.z); x[3] = __uint_as_float(q.w);
  }
  if (kColMul) {   // the factors come from the CTA's shared-memory copy when there is one
    const float4* f = reinterpret_cast<const float4*>((table != nullptr ? table : col_mul) + col);
#pragma unroll
    for (int i = 0; i < Unit<kDt>::kElems / 4; ++i) {
      const float4 c = table != nullptr ? f[i] : ld_stream(f + i);
      x[4 * i] = __fmul_rn(x[4 * i], c.x); x[4 * i + 1] = __fmul_rn(x[4 * i + 1], c.y);
      x[4 * i + 2] = __fmul_rn(x[4 * i + 2], c.z); x[4 * i + 3] = __fmul_rn(x[4 * i + 3], c.w);
    }
  }
}

// x mod cols for x < cols + 8192 (a column offset inside one chunk): a compare and a subtract for the wide rows of
// real layers, a division only for narrow ones.
__device__ __forceinline__ uint32_t wrap_col(uint32_t x, uint32_t cols) {
  if (cols >= static_cast<uint32_t>(kChunkBytes / 2)) return x >= cols ? x - cols : x;
  return x % cols;
}

// Casts the elements of one 16-byte unit (element index e of the tensor) and stores their codes.
template <int kDt, int kFmt, bool kColMul>
__device__ __forceinline__ void cast_unit(const uint4& q, int64_t e, int col, const float* col_mul, const float* table, float sc,
                                          uint8_t* dst) {
  constexpr int kUnit = Unit<kDt>::kElems;
  float x[kUnit];
  unit_values<kDt, kColMul>(q, col_mul, table, col, x);
#pragma unroll
  for (int k = 0; k < kUnit; ++k) x[k] = __fmul_rn(x[k], sc);
  if (kDt == kBF16) {
    uint2 o;
    o.x = cvt_fp8x4<kFmt>(x[0], x[1], x[2], x[3]);
    o.y = cvt_fp8x4<kFmt>(x[kUnit - 4], x[kUnit - 3], x[kUnit - 2], x[kUnit - 1]);
    *reinterpret_cast<uint2*>(dst + e) = o;
  } else {
    *reinterpret_cast<uint32_t*>(dst + e) = cvt_fp8x4<kFmt>(x[0], x[1], x[2], x[3]);
  }
}

// The column-scaled cast of one 16-byte unit of bf16 values with packed multiplies: fl(fl(x * c) * s), each half of
// a mul.rn.f32x2 being an ordinary rounded product.  f: the unit's eight column factors in shared memory (16-byte aligned).
template <int kFmt>
__device__ __forceinline__ uint2 cast_unit_colmul_packed(const uint4& q, const float* f, uint64_t s2) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
  const ulonglong2 c01 = *reinterpret_cast<const ulonglong2*>(f);
  const ulonglong2 c23 = *reinterpret_cast<const ulonglong2*>(f + 4);
  const uint64_t c[4] = {c01.x, c01.y, c23.x, c23.y};
  float x[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint64_t v = pack_f32x2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
    asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(v) : "l"(c[i]));
    asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(v) : "l"(s2));
    unpack_f32x2(v, x[2 * i], x[2 * i + 1]);
  }
  uint2 o;
  o.x = cvt_fp8x4<kFmt>(x[0], x[1], x[2], x[3]);
  o.y = cvt_fp8x4<kFmt>(x[4], x[5], x[6], x[7]);
  return o;
}

template <int kDt, int kFmt, bool kColMul>
__global__ void __launch_bounds__(kStagedThreads, 1)
quantize_staged_kernel(const void* src, int64_t count, uint8_t* dst, uint32_t* partial, GridSync* sync, CastOutputs out,
                       int* status, const float* col_mul, int cols, OaCastJob oa_job, int slots, int table_floats,
                       int rows_per_chunk) {
  constexpr int kEsize = kDt == kBF16 ? 2 : 4;
  constexpr int kUnit = Unit<kDt>::kElems;
  // Row-aligned mode of the column-scaled form (rows_per_chunk > 0; bf16 input, the factors in shared memory): a chunk is
  // a whole number of rows, so unit u of EVERY chunk belongs to columns 8 (u mod cols/8) ..., and a thread, which always
  // takes the units tid, tid + 512, ..., always sees the same columns.  The absmax pass then needs no multiply at all:
  // fl(|x| c) is monotone in |x| for c > 0, so max_t |fl(x[t][i] c_i)| = fl(max_t |x[t][i]| c_i) -- the thread keeps the
  // largest |bf16| pattern per column position (packed 16-bit maxima) and applies the factors once, after the last chunk.
  const bool row_mode = kColMul && kDt == kBF16 && rows_per_chunk > 0;
  const int64_t kChunkElems = row_mode ? static_cast<int64_t>(rows_per_chunk) * cols : kChunkBytes / kEsize;
  constexpr int kRowUnits = kChunkBytes / 16 / kStagedThreads;   // units per thread and chunk in row-aligned mode (7)
  // dynamic shared memory: [table_floats column factors, padded to whole chunks][slots x 16 KB ring]
  extern __shared__ __align__(128) uint8_t staged_smem[];
  // (only the column-scaled form has a table; without one the ring is the whole array and its size a constant)
  const float* table = kColMul && table_floats > 0 ? reinterpret_cast<const float*>(staged_smem) : nullptr;
  uint8_t* stage = kColMul ? staged_smem + (static_cast<size_t>(table_floats) * 4 + kChunkBytes - 1) / kChunkBytes * kChunkBytes
                           : staged_smem;
  const int nslots = kColMul ? slots : kStagedSlots;
  __shared__ __align__(8) uint64_t bars[kStagedSlots];
  __shared__ uint32_t red[32];
  __shared__ int s_ok;
  const int tid = threadIdx.x;
  if (tid == 0) {
    for (int s = 0; s < nslots; ++s) mbar_init(smem_u32(&bars[s]), 1);
    mbar_fence_init();
  }
  pdl_trigger();
  __syncthreads();
  pdl_wait();
  if (kColMul && table_floats > 0) {   // the column factors, once per CTA (they are read twice per element otherwise)
    float* tw = reinterpret_cast<float*>(staged_smem);
    for (int c = tid; c < table_floats; c += kStagedThreads) tw[c] = ld_stream(col_mul + c);
    __syncthreads();
  }

  // (row-aligned mode: count is a whole number of rows of a multiple of 8 values, every chunk a multiple of 16 bytes)
  const int64_t bulk_elems = row_mode ? count : (count / 16) * 16;   // the rest (fewer than 16 elements) goes element by element
  const int64_t n_chunks = (bulk_elems + kChunkElems - 1) / kChunkElems;
  const int grid = static_cast<int>(gridDim.x);
  const int n_my = blockIdx.x < n_chunks ? static_cast<int>((n_chunks - blockIdx.x + grid - 1) / grid) : 0;
  auto chunk_of = [&](int i) -> int64_t { return blockIdx.x + static_cast<int64_t>(i) * grid; };
  auto chunk_elems = [&](int64_t c) -> int {
    const int64_t rem = bulk_elems - c * kChunkElems;
    return static_cast<int>(rem < kChunkElems ? rem : kChunkElems);
  };
  const uint64_t evict_first = l2_policy_evict_first();
  auto issue = [&](int i) {   // one thread: fetch the CTA's i-th chunk into slot i mod nslots
    const int s = i % nslots;
    const int64_t c = chunk_of(i);
    const uint32_t bytes = static_cast<uint32_t>(chunk_elems(c)) * kEsize;   // a multiple of 32
    const uint32_t bar = smem_u32(&bars[s]);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier reads of the slot come first
    mbar_expect_tx(bar, bytes);
    // a chunk that will still be in the ring when the cast pass starts is read from memory exactly once: it need not
    // stay in L2 (and should not displace what is there); an earlier chunk will be fetched again and should
    if (i + nslots >= n_my)
      bulk_load_1d_hint(smem_u32(stage + s * kChunkBytes), static_cast<const uint8_t*>(src) + c * kChunkElems * kEsize, bytes, bar, evict_first);
    else
      bulk_load_1d(smem_u32(stage + s * kChunkBytes), static_cast<const uint8_t*>(src) + c * kChunkElems * kEsize, bytes, bar);
  };

  // ---- pass 1: absmax
  if (tid == 0)
    for (int i = 0; i < n_my && i < nslots; ++i) issue(i);
  uint32_t phase_bits = 0;   // bit s: parity of the next completion of slot s
  uint32_t m = 0;
  bool failed = false;
  // row-aligned mode: the first column of each of this thread's units (the same in every chunk), and the running
  // maxima of |bf16| per column position, two to a word
  int my_col[kRowUnits];
  uint32_t colmax[kRowUnits][4];
  if (row_mode) {
    const int upr = cols / kUnit;
#pragma unroll
    for (int j = 0; j < kRowUnits; ++j) {
      my_col[j] = ((tid + j * kStagedThreads) % upr) * kUnit;
#pragma unroll
      for (int w = 0; w < 4; ++w) colmax[j][w] = 0u;
    }
  }
  // (the slot index is stepped along with i: an integer division per chunk costs as much as a third of the chunk's work)
  for (int i = 0, s = 0; i < n_my; ++i, s = s + 1 == nslots ? 0 : s + 1) {
    const bool ok = mbar_wait(smem_u32(&bars[s]), (phase_bits >> s) & 1u, status);
    phase_bits ^= 1u << s;
    const int64_t e0 = chunk_of(i) * kChunkElems;
    const int units = chunk_elems(chunk_of(i)) / kUnit;
    const uint4* sp = reinterpret_cast<const uint4*>(stage + s * kChunkBytes);
    if (row_mode) {
#pragma unroll
      for (int j = 0; j < kRowUnits; ++j) {
        const int u = tid + j * kStagedThreads;
        if (u < units) {
          const uint4 q = sp[u];
          const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
          for (int k = 0; k < 4; ++k)
            asm("max.u16x2 %0, %0, %1;" : "+r"(colmax[j][k]) : "r"(w[k] & 0x7FFF7FFFu));
        }
      }
    } else {
      const uint32_t col0 = kColMul ? static_cast<uint32_t>(e0 % cols) : 0u;   // one 64-bit modulo per chunk, 32-bit ones per unit
      for (int u = tid; u < units; u += kStagedThreads) {
        float x[kUnit];
        unit_values<kDt, kColMul>(sp[u], col_mul, table, kColMul ? static_cast<int>(wrap_col(col0 + static_cast<uint32_t>(u) * kUnit, static_cast<uint32_t>(cols))) : 0, x);
#pragma unroll
        for (int e = 0; e < kUnit; ++e) m = max(m, abs_bits(x[e]));
      }
    }
    if (!__syncthreads_and(ok)) { failed = true; break; }   // block-uniform; also: the slot is free again
    if (tid == 0 && i + nslots < n_my) issue(i + nslots);
  }
  if (row_mode) {   // the factors, once per column position this thread has seen
#pragma unroll
    for (int j = 0; j < kRowUnits; ++j) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t pair = colmax[j][k];
        if (pair != 0u) {
          const float* f = table + my_col[j] + 2 * k;
          m = max(m, abs_bits(__fmul_rn(__uint_as_float(pair << 16), f[0])));
          m = max(m, abs_bits(__fmul_rn(__uint_as_float(pair & 0xFFFF0000u), f[1])));
        }
      }
    }
  }
  if (blockIdx.x == 0) {   // ragged tail
    for (int64_t e = bulk_elems + tid; e < count; e += kStagedThreads) {
      float x = load1<kDt>(src, e);
      if (kColMul) x = __fmul_rn(x, ld_stream(col_mul + static_cast<int>(e % cols)));
      m = max(m, abs_bits(x));
    }
  }
  m = block_max_u32(m, red);
  // the rider runs here, on warps that would otherwise idle while thread 0 waits at the grid barrier: this CTA's
  // bulk copies have landed, so the rider's loads do not queue behind them
  if (oa_job.oa != nullptr && tid >= kStagedThreads / 2)   // the upper half of the CTA's warps
    cast_oa_transposed(oa_job, (tid >> 5) - kStagedThreads / 64, kStagedThreads / 64);
  // ---- grid barrier.  Every CTA arrives and (below) departs, whatever happened to it, so that the two counters are
  // back at zero once the whole grid has run: a wait that ran out is reported through the status word and does not
  // leave the workspace unusable for the next call.
  if (tid == 0) {
    int ok = failed ? 0 : 1;
    if (!ok) atomicExch(status, kStatusTimeout);
    partial[blockIdx.x] = m;
    __threadfence();
    atomicAdd(&sync->arrive, 1u);
    if (ok) {
      if (ld_acquire_gpu(&sync->arrive) < gridDim.x) {
        const uint64_t t0 = global_timer_ns();
        for (;;) {
          if (ld_acquire_gpu(&sync->arrive) >= gridDim.x) break;
          __nanosleep(40);
          if (global_timer_ns() - t0 > kWaitLimitNs) { ok = 0; atomicExch(status, kStatusTimeout); break; }
        }
      }
    }
    s_ok = ok;
  }
  __syncthreads();
  if (s_ok) {
    uint32_t mb = 0;
    for (int i = tid; i < grid; i += kStagedThreads) mb = max(mb, __ldcg(partial + i));
    const float amax = __uint_as_float(block_max_u32(mb, red));
    const float sc = scale_from_amax(amax, kFmt);
    if (blockIdx.x == 0 && tid == 0) {
      if (out.scale_out) *out.scale_out = sc;
      if (out.scale_out2) *out.scale_out2 = sc;
      if (out.amax_out) *out.amax_out = amax;
      if (out.clear_word) *out.clear_word = 0.0f;
    }
    // ---- pass 2: cast, most recent chunk first
    for (int t = 0, s = n_my > 0 ? (n_my - 1) % nslots : 0; t < n_my; ++t, s = (s == 0 ? nslots : s) - 1) {
      const int i = n_my - 1 - t;
      bool ok = true;
      if (t >= nslots) {   // this chunk had left the ring and was fetched again
        ok = mbar_wait(smem_u32(&bars[s]), (phase_bits >> s) & 1u, status);
        phase_bits ^= 1u << s;
      }
      const int64_t e0 = chunk_of(i) * kChunkElems;
      const uint32_t col0 = kColMul && !row_mode ? static_cast<uint32_t>(e0 % cols) : 0u;
      const uint32_t ucols = kColMul ? static_cast<uint32_t>(cols) : 1u;
      const int units = chunk_elems(chunk_of(i)) / kUnit;
      const uint4* sp = reinterpret_cast<const uint4*>(stage + s * kChunkBytes);
      if (row_mode) {   // the thread's columns are known; two packed multiplies per pair of values
        const uint64_t s2 = pack_f32x2(sc, sc);
#pragma unroll
        for (int j = 0; j < kRowUnits; ++j) {
          const int u = tid + j * kStagedThreads;
          if (u < units)
            *reinterpret_cast<uint2*>(dst + e0 + static_cast<int64_t>(u) * kUnit) = cast_unit_colmul_packed<kFmt>(sp[u], table + my_col[j], s2);
        }
      }
      // two units per thread and iteration (a full chunk is exactly one iteration): both shared-memory loads are
      // issued before either conversion chain starts
      for (int u = tid; !row_mode && u < units; u += 2 * kStagedThreads) {
        const int u1 = u + kStagedThreads;
        const bool has1 = u1 < units;
        const uint4 q0 = sp[u];
        const uint4 q1 = has1 ? sp[u1] : make_uint4(0u, 0u, 0u, 0u);
        cast_unit<kDt, kFmt, kColMul>(q0, e0 + static_cast<int64_t>(u) * kUnit,
                                      kColMul ? static_cast<int>(wrap_col(col0 + static_cast<uint32_t>(u) * kUnit, ucols)) : 0, col_mul, table, sc, dst);
        if (has1)
          cast_unit<kDt, kFmt, kColMul>(q1, e0 + static_cast<int64_t>(u1) * kUnit,
                                        kColMul ? static_cast<int>(wrap_col(col0 + static_cast<uint32_t>(u1) * kUnit, ucols)) : 0, col_mul, table, sc, dst);
      }
      if (t + nslots < n_my) {
        if (!__syncthreads_and(ok)) { failed = true; break; }
        if (tid == 0) issue(i - nslots);
      }
    }
    if (blockIdx.x == 0) {
      for (int64_t e = bulk_elems + tid; e < count; e += kStagedThreads) {
        float x = load1<kDt>(src, e);
        if (kColMul) x = __fmul_rn(x, ld_stream(col_mul + static_cast<int>(e % cols)));
        dst[e] = static_cast<uint8_t>(cvt_fp8x2<kFmt>(__fmul_rn(x, sc), 0.0f) & 0xFF);
      }
    }
  }
  // ---- leave: the last CTA puts the counters back to zero for the next call
  if (failed) {   // copies may still be in flight towards this CTA's shared memory: give them time to land
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) { }
  }
  __syncthreads();
  if (tid == 0) {
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

cudaError_t launch_absmax_value(const void* src, int src_dt, int64_t count, uint32_t* partial, float* amax_out,
                                cudaStream_t stream) {
  int nparts = 0;
  cudaError_t e = launch_absmax(src, src_dt, count, 1.0f, partial, &nparts, stream);
  if (e != cudaSuccess) return e;
  return launch_pdl(absmax_finalize_kernel, dim3(1), dim3(kThreads), 0, stream, 1, static_cast<const uint32_t*>(partial), nparts,
                    amax_out);
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

cudaError_t launch_scale_prep(const uint32_t* partial, int nparts, const float* amax_in, int fmt, float* scale_out,
                              float* scale_out2, float* amax_out, float* clear_word, cudaStream_t stream) {
  const CastOutputs out{scale_out, scale_out2, amax_out, clear_word};
  return launch_pdl(scale_prep_kernel, dim3(1), dim3(kThreads), 0, stream, 1, partial, nparts, amax_in, fmt, out);
}

// The O_A cast as a kernel of its own (for a backward whose output-gradient absmax is already known, so that no fused
// quantizer launch exists for it to ride on).
__global__ void __launch_bounds__(256) oa_cast_kernel(OaCastJob job) {
  pdl_trigger();
  pdl_wait();
  cast_oa_transposed(job, threadIdx.x >> 5, blockDim.x >> 5);
}

template <int kDt, int kFmt, bool kColMul>
cudaError_t launch_staged_variant(const void* src, int64_t count, uint8_t* dst, uint32_t* partial, void* sync,
                                  const CastOutputs& out, int* status, const float* col_mul, int cols, const OaCastJob& oa_job,
                                  cudaStream_t stream) {
  constexpr size_t kSmem = static_cast<size_t>(kStagedSlots) * kChunkBytes;
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(quantize_staged_kernel<kDt, kFmt, kColMul>, static_cast<int>(kSmem), configured);
    if (ec != cudaSuccess) return ec;
  }
  // the kernel's grid barrier needs every CTA resident: the grid is sized from the occupancy of the current device
  // (looked up once per device) and the launch is cooperative, so the driver holds it until the whole grid fits
  static std::atomic<int> blocks_per_sm_of[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  int blocks_per_sm = blocks_per_sm_of[dev].load();
  if (blocks_per_sm == 0) {
    const cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_per_sm, quantize_staged_kernel<kDt, kFmt, kColMul>,
                                                                        kStagedThreads, kSmem);
    if (e != cudaSuccess) return e;
    if (blocks_per_sm < 1) return cudaErrorLaunchOutOfResources;
    blocks_per_sm_of[dev].store(blocks_per_sm);
  }
  const int sms = sm_count();
  // per-row mode: the column factors live in shared memory too when they fit beside at least 128 KB of ring slots
  int table_floats = 0, slots = kStagedSlots, rows_per_chunk = 0;
  if (kColMul) {
    const int table_chunks = static_cast<int>((static_cast<int64_t>(cols) * 4 + kChunkBytes - 1) / kChunkBytes);
    if (table_chunks <= kStagedSlots - (128 * 1024) / kChunkBytes) { table_floats = cols; slots = kStagedSlots - table_chunks; }
    // ... and the chunks are whole rows (the kernel's row-aligned mode) when a row of bf16 fits a chunk
    if (kDt == kBF16 && table_floats > 0 && cols % 8 == 0 && count % cols == 0 && static_cast<int64_t>(cols) * 2 <= kChunkBytes)
      rows_per_chunk = static_cast<int>(kChunkBytes / (static_cast<int64_t>(cols) * 2));
  }
  const int64_t chunk_elems = rows_per_chunk > 0 ? static_cast<int64_t>(rows_per_chunk) * cols : kChunkBytes / (kDt == kBF16 ? 2 : 4);
  int64_t grid = ((rows_per_chunk > 0 ? count : count / 16 * 16) + chunk_elems - 1) / chunk_elems;
  const int64_t resident = static_cast<int64_t>(blocks_per_sm) * sms;   // all CTAs must be resident together
  if (grid > resident) grid = resident;
  if (grid > kMaxAbsmaxParts) grid = kMaxAbsmaxParts;
  if (grid < 1) grid = 1;
  return launch_pdl(quantize_staged_kernel<kDt, kFmt, kColMul>, dim3(static_cast<unsigned>(grid)), dim3(kStagedThreads), kSmem,
                    stream, -1 /* cooperative */, src, count, dst, partial, static_cast<GridSync*>(sync), out, status, col_mul, cols,
                    oa_job, slots, table_floats, rows_per_chunk);
}

cudaError_t launch_quantize_fused(const void* src, int src_dt, int64_t count, int fmt, uint8_t* dst, uint32_t* partial,
                                  void* sync, float* scale_out, float* scale_out2, float* amax_out, float* clear_word,
                                  int* status, const float* col_mul, int cols, const OaCastJob* oa_cast, cudaStream_t stream) {
  const CastOutputs out{scale_out, scale_out2, amax_out, clear_word};
  const OaCastJob oa_job = oa_cast != nullptr ? *oa_cast : OaCastJob{};
#define FALQON_FUSED(DT, FMT)                                                                                              \
  do {                                                                                                                     \
    if (col_mul != nullptr)                                                                                                \
      return launch_staged_variant<DT, FMT, true>(src, count, dst, partial, sync, out, status, col_mul, cols, oa_job, stream); \
    return launch_staged_variant<DT, FMT, false>(src, count, dst, partial, sync, out, status, nullptr, 0, oa_job, stream); \
  } while (0)
  if (src_dt == kBF16) {
    if (fmt == kE4M3) FALQON_FUSED(kBF16, kE4M3);
    FALQON_FUSED(kBF16, kE5M2);
  }
  if (fmt == kE4M3) FALQON_FUSED(kF32, kE4M3);
  FALQON_FUSED(kF32, kE5M2);
#undef FALQON_FUSED
}

cudaError_t launch_oa_cast(const OaCastJob& job, cudaStream_t stream) {
  // one warp converts a tile of 32 tokens; the tensor is small (T x r fp32), so the kernel is as long as its slowest warp:
  // few warps per CTA spread the tiles over the whole chip (4096 tokens: 128 tiles on 128 SMs instead of 16)
  const long long tiles = (job.T + 31) / 32;
  const int warps = tiles >= 148 * 8 * 4 ? 8 : tiles >= 148 * 4 ? 2 : 1;
  long long grid = (tiles + warps - 1) / warps;
  if (grid > 148 * 8) grid = 148 * 8;
  return launch_pdl(oa_cast_kernel, dim3(static_cast<unsigned>(grid)), dim3(32 * warps), 0, stream, 1, job);
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

}  // namespace falqon
