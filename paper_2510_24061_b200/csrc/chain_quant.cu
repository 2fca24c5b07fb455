// Quantizing forms of the chain kernels (include/falqon_chain.h): the bf16 operation that produces a melded layer's
// input (or its output gradient) and the per-tensor cast of Eq. quantize of that tensor, in ONE launch -- the cast
// fused into the epilogue of the kernel that produces the tensor, so that no separate quantize pass reads it back.
//
// Per-tensor absmax scaling needs the whole tensor before the first code can be written, so the kernel has two
// phases around a grid-wide barrier (cooperative launch, one CTA per SM, bounded wait):
//   phase 1  every CTA computes its contiguous share of the result, rounds it to bf16 exactly as the plain kernel
//            would store it, keeps it in its 224 KB of shared memory (148 x 224 KB = 33.9 MB: a [4096][4096] tensor
//            stays on chip) and tracks max |value|; what does not fit goes to the caller's bf16 buffer;
//   barrier  partial maxima -> absmax -> scale = fp8max / absmax (the same arithmetic as the quantizer);
//   phase 2  the kept values are multiplied by the scale, rounded and saturated to FP8 and stored as codes; the part that
//            went to memory is read back (from L2 where it still is).
// Codes and scale are bit for bit those of falqon_quantize applied to the plain kernel's output.
#include "../../include/falqon_chain.h"
#include "chain_math.cuh"
#include "grid_sync.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

constexpr int kCqThreads = 512;      // row-wise producers on wide rows: four groups of 128 threads (the registers hold the row)
constexpr int kCqWideThreads = 1024;  // element-wise producers and rows of up to 4096 values: more warps hide the arithmetic
                                      // behind the loads
constexpr int kCqStageBytes = 224 * 1024;
constexpr int kCqStageVecs = kCqStageBytes / 16;   // 14336 vectors of eight bf16 = 28 rows of 4096
constexpr int kCqMaxGrid = 256;                    // partial maxima per output in the scratch
static_assert(8 + 2 * kCqMaxGrid * 4 <= FALQON_CHAIN_SCRATCH_BYTES, "scratch layout");

struct CqScratch {
  GridSync sync;
  uint32_t partial[2][kCqMaxGrid];   // fp32 bit patterns of the CTAs' max |value|, per output
};

template <int kOutputs>
struct CqTail {
  uint8_t* codes[kOutputs];
  uint4* out16[kOutputs];
  float* scale_out[kOutputs];
  CqScratch* scratch;
  int* status;
  int keep16;
};

template <int kThreads>
__device__ __forceinline__ uint32_t cta_max_u32(uint32_t v, uint32_t* red /* >= 32 words */) {
  v = __reduce_max_sync(0xFFFFFFFFu, v);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) red[warp] = v;
  __syncthreads();
  uint32_t w = threadIdx.x < kThreads / 32 ? red[threadIdx.x] : 0u;
  if (warp == 0) w = __reduce_max_sync(0xFFFFFFFFu, w);
  if (threadIdx.x == 0) red[0] = w;
  __syncthreads();
  const uint32_t out = red[0];
  __syncthreads();
  return out;
}

// A CTA's contiguous share of `units` (vectors or rows).
__device__ __forceinline__ void share_of(int64_t units, int64_t& first, int64_t& n) {
  const int64_t per = (units + gridDim.x - 1) / gridDim.x;
  first = per * blockIdx.x;
  n = units - first;
  if (n > per) n = per;
  if (n < 0) n = 0;
}

// ---- producers.  produce(put) computes the CTA's share; put(which, li, o) takes vector li (local index) of output `which`.
struct CombineOp {
  static constexpr int kThreads = kCqWideThreads;
  static constexpr int kOutputs = 1;
  const uint4 *a, *b, *c, *d;
  float sa, sb, sc, sd;
  int64_t nvec;
  __device__ __forceinline__ void range(int64_t& first, int64_t& n) const { share_of(nvec, first, n); }
  template <class Put>
  __device__ __forceinline__ void produce(int64_t first, int64_t n, float (*)[4], Put put) const {
    constexpr int kU = 2;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    for (int64_t li0 = threadIdx.x; li0 < n; li0 += kThreads * kU) {
      uint4 ra[kU], rb[kU], rc[kU], rd[kU];
#pragma unroll
      for (int u = 0; u < kU; ++u) {
        const int64_t li = li0 + u * kThreads;
        ra[u] = rb[u] = rc[u] = rd[u] = zero;
        if (li < n) {
          ra[u] = ld_stream(a + first + li);
          if (b != nullptr) rb[u] = ld_stream(b + first + li);
          if (c != nullptr) rc[u] = ld_stream(c + first + li);
          if (d != nullptr) rd[u] = ld_stream(d + first + li);
        }
      }
#pragma unroll
      for (int u = 0; u < kU; ++u) {
        const int64_t li = li0 + u * kThreads;
        if (li < n) put(0, li, combine8(ra[u], sa, rb[u], sb, b != nullptr, rc[u], sc, c != nullptr, rd[u], sd, d != nullptr));
      }
    }
  }
};

struct SiluMulOp {
  static constexpr int kThreads = kCqWideThreads;
  static constexpr int kOutputs = 1;
  const uint4 *g, *u;
  int64_t nvec;
  __device__ __forceinline__ void range(int64_t& first, int64_t& n) const { share_of(nvec, first, n); }
  template <class Put>
  __device__ __forceinline__ void produce(int64_t first, int64_t n, float (*)[4], Put put) const {
    constexpr int kU = 2;
    // the inputs are read once here: marked evict-first, they do not push the part of the result that waits in L2 for
    // phase 2 out to memory
    const uint64_t once = l2_policy_evict_first();
    for (int64_t li0 = threadIdx.x; li0 < n; li0 += kThreads * kU) {
      uint4 rg[kU], ru[kU];
#pragma unroll
      for (int k = 0; k < kU; ++k) {
        const int64_t li = li0 + k * kThreads;
        if (li < n) {
          rg[k] = ld_global_hint(g + first + li, once);
          ru[k] = ld_global_hint(u + first + li, once);
        }
      }
#pragma unroll
      for (int k = 0; k < kU; ++k) {
        const int64_t li = li0 + k * kThreads;
        if (li < n) put(0, li, silu_mul8(rg[k], ru[k]));
      }
    }
  }
};

struct SiluMulGradOp {
  static constexpr int kThreads = kCqWideThreads;
  static constexpr int kOutputs = 2;   // 0: dg, 1: du
  const uint4 *g, *u, *dz;
  int64_t nvec;
  __device__ __forceinline__ void range(int64_t& first, int64_t& n) const { share_of(nvec, first, n); }
  template <class Put>
  __device__ __forceinline__ void produce(int64_t first, int64_t n, float (*)[4], Put put) const {
    constexpr int kU = 2;
    for (int64_t li0 = threadIdx.x; li0 < n; li0 += kThreads * kU) {
      uint4 rg[kU], ru[kU], rz[kU];
#pragma unroll
      for (int k = 0; k < kU; ++k) {
        const int64_t li = li0 + k * kThreads;
        if (li < n) {
          rg[k] = ld_stream(g + first + li);
          ru[k] = ld_stream(u + first + li);
          rz[k] = ld_stream(dz + first + li);
        }
      }
#pragma unroll
      for (int k = 0; k < kU; ++k) {
        const int64_t li = li0 + k * kThreads;
        if (li < n) {
          uint4 qg, qu;
          silu_mul_grad8(rg[k], ru[k], rz[k], qg, qu);
          put(0, li, qg);
          put(1, li, qu);
        }
      }
    }
  }
};

// Row-wise producers: the CTA owns whole rows; its four groups of 128 threads take them in turn.
template <bool kCombine, int kMaxVec>
struct RmsnormOp {
  static constexpr int kThreads = kMaxVec <= 4 ? kCqWideThreads : kCqThreads;
  static constexpr int kOutputs = 1;
  const uint4 *a, *b;
  float sa, sb;
  uint4* sum_out;
  float* inv_rms;
  int64_t rows;
  int vec_per_row;
  float inv_cols, eps;
  __device__ __forceinline__ void range(int64_t& first, int64_t& n) const {
    share_of(rows, first, n);
    first *= vec_per_row;
    n *= vec_per_row;
  }
  template <class Put>
  __device__ __forceinline__ void produce(int64_t first, int64_t n, float (*gred)[4], Put put) const {
    const int grp = threadIdx.x >> 7;
    const RowGroup g{static_cast<int>(threadIdx.x & 127), 1 + grp, gred[grp]};
    const int nrows = static_cast<int>(n / vec_per_row);
    for (int lr = grp; lr < nrows; lr += kThreads / kNormThreads) {
      const int64_t base = first + static_cast<int64_t>(lr) * vec_per_row;
      const int64_t lbase = static_cast<int64_t>(lr) * vec_per_row;
      const float inv = rmsnorm_row<kMaxVec, kCombine>(a + base, sa, kCombine ? b + base : nullptr, sb, vec_per_row, inv_cols, eps, g,
                                              [&](int v, const uint4& s) { sum_out[base + v] = s; },
                                              [&](int v, const uint4& o) { put(0, lbase + v, o); });
      if (g.tid == 0) inv_rms[base / vec_per_row] = inv;
    }
  }
};

template <int kMaxVec>
struct RmsnormGradCombineOp {
  static constexpr int kThreads = kMaxVec <= 4 ? kCqWideThreads : kCqThreads;
  static constexpr int kOutputs = 1;
  const uint4 *dy_a, *dy_b, *dy_c, *x, *res;
  const float* inv_rms;
  float s_res;
  int64_t rows;
  int vec_per_row;
  float inv_cols;
  __device__ __forceinline__ void range(int64_t& first, int64_t& n) const {
    share_of(rows, first, n);
    first *= vec_per_row;
    n *= vec_per_row;
  }
  template <class Put>
  __device__ __forceinline__ void produce(int64_t first, int64_t n, float (*gred)[4], Put put) const {
    const int grp = threadIdx.x >> 7;
    const RowGroup g{static_cast<int>(threadIdx.x & 127), 1 + grp, gred[grp]};
    const int nrows = static_cast<int>(n / vec_per_row);
    for (int lr = grp; lr < nrows; lr += kThreads / kNormThreads) {
      const int64_t base = first + static_cast<int64_t>(lr) * vec_per_row;
      const int64_t lbase = static_cast<int64_t>(lr) * vec_per_row;
      rmsnorm_grad_row<kMaxVec, true>(dy_a + base, dy_b + base, dy_c != nullptr ? dy_c + base : nullptr, x + base,
                             ld_stream(inv_rms + base / vec_per_row), res + base, s_res, vec_per_row, inv_cols, g,
                             [&](int v, const uint4& o) { put(0, lbase + v, o); });
    }
  }
};

template <int kFmt>
__device__ __forceinline__ uint2 cast_vec(const uint4& q, float sc) {
  float x[8];
  unpack8(q, x);
#pragma unroll
  for (int i = 0; i < 8; ++i) x[i] = __fmul_rn(x[i], sc);
  uint2 o;
  o.x = cvt_fp8x4<kFmt>(x[0], x[1], x[2], x[3]);
  o.y = cvt_fp8x4<kFmt>(x[4], x[5], x[6], x[7]);
  return o;
}

template <class Op, int kFmt>
__global__ void __launch_bounds__(Op::kThreads, 1) chain_quant_kernel(const Op op, const CqTail<Op::kOutputs> tail) {
  constexpr int kOut = Op::kOutputs;
  constexpr int kThreads = Op::kThreads;
  constexpr int kCap = kCqStageVecs / kOut;   // vectors of each output that stay in shared memory
  extern __shared__ __align__(128) uint8_t cq_smem[];
  uint4* stage = reinterpret_cast<uint4*>(cq_smem);
  __shared__ uint32_t red[32];
  __shared__ float gred[kCqWideThreads / kNormThreads][4];
  __shared__ int s_ok;
  pdl_trigger();
  pdl_wait();
  const int tid = threadIdx.x;
  int64_t first, n;
  op.range(first, n);

  // ---- phase 1
  uint32_t mx[kOut];
#pragma unroll
  for (int w = 0; w < kOut; ++w) mx[w] = 0u;
  const bool keep16 = tail.keep16 != 0;
  op.produce(first, n, gred, [&](int which, int64_t li, const uint4& o) {
    if (li < kCap) stage[which * kCap + li] = o;
    if (li >= kCap || keep16) tail.out16[which][first + li] = o;
    mx[which] = max_abs_bf16(o, mx[which]);
  });
#pragma unroll
  for (int w = 0; w < kOut; ++w) {
    const uint32_t m = cta_max_u32<kThreads>(mx[w], red);
    if (tid == 0) tail.scratch->partial[w][blockIdx.x] = m << 16;
  }
  // ---- grid barrier (the CTA-wide barriers above ordered every thread's stores before thread 0's arrival)
  if (tid == 0) s_ok = grid_arrive_and_wait(&tail.scratch->sync, tail.status, false) ? 1 : 0;
  __syncthreads();
  if (s_ok) {
    // ---- phase 2
#pragma unroll
    for (int w = 0; w < kOut; ++w) {
      uint32_t mb = 0;
      for (int i = tid; i < static_cast<int>(gridDim.x); i += kThreads) mb = max(mb, __ldcg(&tail.scratch->partial[w][i]));
      const float amax = __uint_as_float(cta_max_u32<kThreads>(mb, red));
      const float sc = scale_from_amax(amax, kFmt);
      if (blockIdx.x == 0 && tid == 0) *tail.scale_out[w] = sc;
      uint2* dst = reinterpret_cast<uint2*>(tail.codes[w]) + first;
      const uint4* kept = stage + w * kCap;
      const uint4* spilled = tail.out16[w] + first;
      const uint64_t once = l2_policy_evict_first();   // the passed-through part is dead once it has been read back
      const int64_t n_kept = n < kCap ? n : kCap;
      constexpr int kU = 4;
      for (int64_t li0 = tid; li0 < n_kept; li0 += kThreads * kU) {
        uint4 q[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
          const int64_t li = li0 + u * kThreads;
          if (li < n_kept) q[u] = kept[li];
        }
#pragma unroll
        for (int u = 0; u < kU; ++u) {
          const int64_t li = li0 + u * kThreads;
          if (li < n_kept) dst[li] = cast_vec<kFmt>(q[u], sc);
        }
      }
      for (int64_t li0 = kCap + tid; li0 < n; li0 += kThreads * kU) {
        uint4 q[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
          const int64_t li = li0 + u * kThreads;
          if (li < n) q[u] = ld_global_hint(spilled + li, once);
        }
#pragma unroll
        for (int u = 0; u < kU; ++u) {
          const int64_t li = li0 + u * kThreads;
          if (li < n) dst[li] = cast_vec<kFmt>(q[u], sc);
        }
      }
    }
  }
  __syncthreads();
  if (tid == 0) grid_depart(&tail.scratch->sync);
}

inline bool ok16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

template <class Op, int kFmt>
cudaError_t launch_variant(const Op& op, const CqTail<Op::kOutputs>& tail, int64_t units, cudaStream_t stream) {
  static DeviceMask configured{0};
  const cudaError_t ec = set_max_dynamic_smem(chain_quant_kernel<Op, kFmt>, kCqStageBytes, configured);
  if (ec != cudaSuccess) return ec;
  // one CTA per SM (the shared-memory stage fills it), all resident: the launch is cooperative
  int64_t grid = sm_count();
  if (grid > kCqMaxGrid) grid = kCqMaxGrid;
  if (grid > units) grid = units;
  if (grid < 1) grid = 1;
  return launch_pdl(chain_quant_kernel<Op, kFmt>, dim3(static_cast<unsigned>(grid)), dim3(Op::kThreads), kCqStageBytes, stream,
                    -1 /* cooperative */, op, tail);
}

template <class Op>
int launch_op(const Op& op, CqTail<Op::kOutputs> tail, int fmt, int64_t units, falqon_stream stream) {
  tail.status = device_status_ptr();
  if (tail.status == nullptr) return FALQON_ERR_CUDA;
  const cudaError_t e = fmt == FALQON_E4M3 ? launch_variant<Op, kE4M3>(op, tail, units, static_cast<cudaStream_t>(stream))
                                           : launch_variant<Op, kE5M2>(op, tail, units, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? FALQON_OK : FALQON_ERR_CUDA;
}

inline bool tail_ok(const void* codes, const void* scale_out, const void* out16, const void* scratch, int fmt) {
  return codes != nullptr && scale_out != nullptr && out16 != nullptr && scratch != nullptr && ok16(codes) && ok16(out16) &&
         ok16(scratch) && (fmt == FALQON_E4M3 || fmt == FALQON_E5M2);
}
inline bool row_shape_ok(int64_t rows, int64_t cols) {
  return rows >= 1 && rows <= (1ll << 30) && cols >= 8 && cols % 8 == 0 && cols <= kNormThreads * kNormMaxVec * 8;
}

}  // namespace
}  // namespace falqon

using namespace falqon;

extern "C" {

int falqon_chain_combine_quantize(void* codes, float* scale_out, int fmt, void* out16, int keep16, const void* a, float sa,
                                  const void* b, float sb, const void* c, float sc, const void* d, float sd, int64_t count,
                                  void* scratch, falqon_stream stream) {
  if (!tail_ok(codes, scale_out, out16, scratch, fmt) || a == nullptr || count < 8 || count % 8 || !ok16(a) || !ok16(b) || !ok16(c) ||
      !ok16(d))
    return FALQON_ERR_INVALID_ARG;
  const CombineOp op{static_cast<const uint4*>(a), static_cast<const uint4*>(b), static_cast<const uint4*>(c),
                     static_cast<const uint4*>(d), sa, sb, sc, sd, count / 8};
  CqTail<1> tail{{static_cast<uint8_t*>(codes)}, {static_cast<uint4*>(out16)}, {scale_out}, static_cast<CqScratch*>(scratch), nullptr,
                 keep16};
  return launch_op(op, tail, fmt, (count / 8 + kCqWideThreads - 1) / kCqWideThreads, stream);
}

int falqon_chain_silu_mul_quantize(void* codes, float* scale_out, int fmt, void* out16, int keep16, const void* g, const void* u,
                                   int64_t count, void* scratch, falqon_stream stream) {
  if (!tail_ok(codes, scale_out, out16, scratch, fmt) || g == nullptr || u == nullptr || count < 8 || count % 8 || !ok16(g) || !ok16(u))
    return FALQON_ERR_INVALID_ARG;
  const SiluMulOp op{static_cast<const uint4*>(g), static_cast<const uint4*>(u), count / 8};
  CqTail<1> tail{{static_cast<uint8_t*>(codes)}, {static_cast<uint4*>(out16)}, {scale_out}, static_cast<CqScratch*>(scratch), nullptr,
                 keep16};
  return launch_op(op, tail, fmt, (count / 8 + kCqWideThreads - 1) / kCqWideThreads, stream);
}

int falqon_chain_silu_mul_grad_quantize(void* codes_dg, void* codes_du, float* scale_dg, float* scale_du, int fmt, void* dg16,
                                        void* du16, int keep16, const void* g, const void* u, const void* dz, int64_t count,
                                        void* scratch, falqon_stream stream) {
  if (!tail_ok(codes_dg, scale_dg, dg16, scratch, fmt) || !tail_ok(codes_du, scale_du, du16, scratch, fmt) || g == nullptr ||
      u == nullptr || dz == nullptr || count < 8 || count % 8 || !ok16(g) || !ok16(u) || !ok16(dz))
    return FALQON_ERR_INVALID_ARG;
  const SiluMulGradOp op{static_cast<const uint4*>(g), static_cast<const uint4*>(u), static_cast<const uint4*>(dz), count / 8};
  CqTail<2> tail{{static_cast<uint8_t*>(codes_dg), static_cast<uint8_t*>(codes_du)},
                 {static_cast<uint4*>(dg16), static_cast<uint4*>(du16)},
                 {scale_dg, scale_du},
                 static_cast<CqScratch*>(scratch),
                 nullptr,
                 keep16};
  return launch_op(op, tail, fmt, (count / 8 + kCqWideThreads - 1) / kCqWideThreads, stream);
}

int falqon_chain_rmsnorm_quantize(void* codes, float* scale_out, int fmt, void* y16, int keep16, float* inv_rms, void* sum_out,
                                  const void* a, float sa, const void* b, float sb, int64_t rows, int64_t cols, float eps,
                                  void* scratch, falqon_stream stream) {
  if (!tail_ok(codes, scale_out, y16, scratch, fmt) || inv_rms == nullptr || a == nullptr || !row_shape_ok(rows, cols) || !ok16(a) ||
      !ok16(b) || !ok16(sum_out) || (b == nullptr) != (sum_out == nullptr) || !(eps >= 0.0f))
    return FALQON_ERR_INVALID_ARG;
  CqTail<1> tail{{static_cast<uint8_t*>(codes)}, {static_cast<uint4*>(y16)}, {scale_out}, static_cast<CqScratch*>(scratch), nullptr,
                 keep16};
  const int vpr = static_cast<int>(cols / 8);
  const float inv_cols = 1.0f / static_cast<float>(cols);
  // (rows of up to 4096 values need four vectors per thread; wider ones take the 16-vector form, which is slower)
#define FALQON_NORM_OP(COMBINE, MAXVEC)                                                                              \
  do {                                                                                                               \
    const RmsnormOp<COMBINE, MAXVEC> op{static_cast<const uint4*>(a), static_cast<const uint4*>(b), sa, sb,          \
                                        static_cast<uint4*>(sum_out), inv_rms, rows, vpr, inv_cols, eps};            \
    return launch_op(op, tail, fmt, rows, stream);                                                                   \
  } while (0)
  if (b != nullptr) {
    if (vpr <= 4 * kNormThreads) FALQON_NORM_OP(true, 4);
    FALQON_NORM_OP(true, kNormMaxVec);
  }
  if (vpr <= 4 * kNormThreads) FALQON_NORM_OP(false, 4);
  FALQON_NORM_OP(false, kNormMaxVec);
#undef FALQON_NORM_OP
}

int falqon_chain_rmsnorm_grad_combine_quantize(void* codes, float* scale_out, int fmt, void* out, const void* dy_a, const void* dy_b,
                                               const void* dy_c, const void* x, const float* inv_rms, const void* res, float s_res,
                                               int64_t rows, int64_t cols, void* scratch, falqon_stream stream) {
  if (!tail_ok(codes, scale_out, out, scratch, fmt) || dy_a == nullptr || dy_b == nullptr || x == nullptr || inv_rms == nullptr ||
      res == nullptr || !row_shape_ok(rows, cols) || !ok16(dy_a) || !ok16(dy_b) || !ok16(dy_c) || !ok16(x) || !ok16(res))
    return FALQON_ERR_INVALID_ARG;
  CqTail<1> tail{{static_cast<uint8_t*>(codes)}, {static_cast<uint4*>(out)}, {scale_out}, static_cast<CqScratch*>(scratch), nullptr, 1};
  const int vpr = static_cast<int>(cols / 8);
#define FALQON_GRAD_OP(MAXVEC)                                                                                        \
  do {                                                                                                                \
    const RmsnormGradCombineOp<MAXVEC> op{static_cast<const uint4*>(dy_a), static_cast<const uint4*>(dy_b),          \
                                          static_cast<const uint4*>(dy_c), static_cast<const uint4*>(x),              \
                                          static_cast<const uint4*>(res), inv_rms, s_res, rows, vpr,                 \
                                          1.0f / static_cast<float>(cols)};                                          \
    return launch_op(op, tail, fmt, rows, stream);                                                                   \
  } while (0)
  if (vpr <= 4 * kNormThreads) FALQON_GRAD_OP(4);
  FALQON_GRAD_OP(kNormMaxVec);
#undef FALQON_GRAD_OP
}

}  // extern "C"
