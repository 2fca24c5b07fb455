// Correctly rounded merge on the tensor cores (an extension of S8 beyond the paper's text):
//   W~[i][c] <- sat_rne_e4m3( W~[i][c] + sum_j d'_ij * A~[j][c] ),  the sum exact, ONE rounding
// for the selected rows i (d'_ij = DeltaBuffer entry, times the row coefficient as its own fp32 multiply in per-row
// mode).  The fp32 fma chain of the plain merge costs k n r dependent ALU operations; here the bulk of the work is
// a bf16 product with fp32 accumulation, and exactness comes from a guard band plus an exact fallback:
//   1. every d' is split EXACTLY into three bf16 limbs (8 + 8 + 8 significand bits), every A~ value is exactly a
//      bf16, so all products are exact in fp32 and only the accumulation rounds;
//   2. the accumulated sum S differs from the exact sum by at most eps = kappa * (|w| + (sum_j |d'_ij|) * max_j |A~[j][c]|);
//   3. if round(S - eps) and round(S + eps) give the same E4M3 code, that code is the correctly rounded result
//      (rounding is monotone); otherwise the element is flagged in a bit mask and keeps its old code for now;
//   4. a second kernel recomputes the flagged elements exactly (the sum held as a big integer in units of 2^-158)
//      and rounds once: nearest, ties to the even code, saturating, a sum that rounds to zero keeps its sign.
// Rows with an entry too small for a bf16 limb (below 2^-100) get eps = inf, i.e. all their elements go to step 4.
#include <cuda.h>

#include <cmath>

#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

constexpr int kXThreads = 320;              // warp 0 TMA, warp 1 MMA, warps 2..9 epilogue
constexpr int kXBlockM = 128;
constexpr int kXBlockKBytes = 128;          // 64 bf16 per 128-byte swizzle row
constexpr int kXUmmaKBytes = 32;            // K = 16 bf16 per tcgen05.mma kind::f16
constexpr uint32_t kXATile = kXBlockM * kXBlockKBytes;
constexpr int kXStages = 3;                 // the K loop is 3 to 12 blocks long; 96 KB per CTA leaves room for two CTAs per SM

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ uint16_t trunc_bf16_bits(float x) { return static_cast<uint16_t>(__float_as_uint(x) >> 16); }
__device__ __forceinline__ float bf16_bits_value(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

// ---- step 0a: A~ [r][n] E4M3 -> a_t [n][r_pad] bf16 (exact; a thread converts the pair (j, j+1) of one column),
// then amax_c[c] = max_j |A~[j][c]| from the finished rows of a_t
__global__ void __launch_bounds__(256) exact_prep_a_kernel(const uint8_t* aq, int64_t n, int r, int r_pad, uint16_t* a_t) {
  pdl_trigger();
  pdl_wait();
  const int64_t c = blockIdx.x * 256ll + threadIdx.x;
  const int j = 2 * static_cast<int>(blockIdx.y);
  if (c >= n) return;
  uint32_t pair = 0;
  if (j < r) pair |= static_cast<uint32_t>(ld_stream(aq + static_cast<int64_t>(j) * n + c));
  if (j + 1 < r) pair |= static_cast<uint32_t>(ld_stream(aq + static_cast<int64_t>(j + 1) * n + c)) << 8;
  const float2 v = e4m3x2_to_float2(pair);
  *reinterpret_cast<uint32_t*>(a_t + c * r_pad + j) = static_cast<uint32_t>(trunc_bf16_bits(v.x)) |
                                                      (static_cast<uint32_t>(trunc_bf16_bits(v.y)) << 16);   // exact: 4 significand bits
}

__global__ void __launch_bounds__(256) exact_amax_a_kernel(const uint16_t* a_t, int64_t n, int r_pad, float* amax_c) {
  pdl_trigger();
  pdl_wait();
  const int64_t c = blockIdx.x * 256ll + threadIdx.x;
  if (c >= n) return;
  const uint4* row = reinterpret_cast<const uint4*>(a_t + c * r_pad);
  uint32_t m2 = 0;   // the maximum of |bf16| bit patterns, both halves at once is not possible: keep two maxima
  uint32_t lo_max = 0, hi_max = 0;
  for (int v = 0; v < r_pad / 8; ++v) {
    const uint4 q = ld_stream(row + v);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      lo_max = max(lo_max, w[e] & 0x7FFFu);
      hi_max = max(hi_max, (w[e] >> 16) & 0x7FFFu);
    }
  }
  m2 = max(lo_max, hi_max);
  amax_c[c] = __uint_as_float(m2 << 16);
}

// ---- step 0b: the selected DeltaBuffer rows -> d' (fp32 copy for the exact fallback), three exact bf16 limbs
// (the A operand, [k][3 r_pad]), sum_j |d'_j| for the guard band; the DeltaBuffer rows are cleared here.
// One warp per selected row, eight rows per CTA.
// Several layers per launch: the CTAs of all layers are laid end to end (cta_begin), as in the batched score kernel.
constexpr int kXBatchMax = kProxyBatchMax;
struct PrepRowsLayer {
  float* dbuf;
  const int32_t* sel_idx;
  const float* row_scales;
  uint16_t* limbs;
  float* dprime;
  float* sprime;
  long long m;
  int k, r, r_pad, cta_begin;
};
struct PrepRowsBatch {
  PrepRowsLayer layer[kXBatchMax];
  int count;
};
__global__ void __launch_bounds__(256) exact_prep_rows_kernel(const __grid_constant__ PrepRowsBatch args) {
  pdl_trigger();
  pdl_wait();
  int l = 0;
#pragma unroll 1
  for (int i = 1; i < args.count; ++i) l = static_cast<int>(blockIdx.x) >= args.layer[i].cta_begin ? i : l;
  const PrepRowsLayer& a = args.layer[l];
  float* dbuf = a.dbuf;
  const int32_t* sel_idx = a.sel_idx;
  const float* row_scales = a.row_scales;
  uint16_t* limbs = a.limbs;
  float* dprime = a.dprime;
  float* sprime = a.sprime;
  const long long m = a.m;
  const int k = a.k, r = a.r, r_pad = a.r_pad;
  const int lane = threadIdx.x & 31;
  const int q = (static_cast<int>(blockIdx.x) - a.cta_begin) * 8 + (threadIdx.x >> 5);
  if (q >= k) return;
  const int row = ld_stream(sel_idx + q);
  float coef = 1.0f;
  if (row_scales != nullptr) coef = __fdiv_rn(ld_stream(row_scales + row), ld_stream(row_scales + m));
  float* src = dbuf + static_cast<int64_t>(row) * r;
  uint16_t* a_row = limbs + static_cast<int64_t>(q) * (3 * r_pad);
  float* d_row = dprime + static_cast<int64_t>(q) * r_pad;
  float asum = 0.0f;
  bool tiny = false;
  float dv[8];                       // r_pad <= 256: at most eight entries per lane, all loads issued together
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int j = lane + 32 * u;
    dv[u] = j < r ? ld_stream(src + j) : 0.0f;
  }
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int j = lane + 32 * u;
    if (j >= r_pad) break;
    float d = dv[u];
    if (j < r) {
      src[j] = 0.0f;
      if (row_scales != nullptr) d = __fmul_rn(d, coef);
    }
    const uint16_t hi = trunc_bf16_bits(d);
    const float r1 = d - bf16_bits_value(hi);          // exact: the low 16 significand bits
    const uint16_t mid = trunc_bf16_bits(r1);
    const float r2 = r1 - bf16_bits_value(mid);        // exact: the low 8 significand bits, a bf16 value
    a_row[j] = hi;
    a_row[r_pad + j] = mid;
    a_row[2 * r_pad + j] = trunc_bf16_bits(r2);
    d_row[j] = d;
    asum += fabsf(d);
    tiny = tiny || (d != 0.0f && fabsf(d) < 7.888609052210118e-31f);   // 2^-100: a limb could underflow
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) asum += __shfl_xor_sync(0xFFFFFFFFu, asum, o);
  tiny = __any_sync(0xFFFFFFFFu, tiny);
  if (lane == 0) sprime[q] = tiny ? INFINITY : asum * 1.0001f;   // a little slack for this sum's own rounding
}

struct XParams {
  int k, n, r_pad, block_n;
  int m_tiles, n_tiles, kblocks_total, kblocks_wrap;
  uint32_t idesc, tmem_cols;
  float kappa;
  uint8_t* wq;              // [m + r][n]
  const int32_t* sel_idx;   // [k]
  const float* sprime;      // [k]
  const float* amax_c;      // [n padded to 32]
  uint32_t* flags;          // [k][words_per_row]
  int words_per_row;
  float* sums_out;          // nullable [k][n]: the accumulated sums, for diagnostics
};
// The layers of one launch: per layer its two tensor maps and parameters; the tiles of all layers are laid end to end
// (tile_begin), every layer with the same tile width, so the shared-memory stages and barriers serve them all.
struct XBatch {
  CUtensorMap ta[kXBatchMax];
  CUtensorMap tb[kXBatchMax];
  XParams p[kXBatchMax];
  int tile_begin[kXBatchMax + 1];
  int count, block_n;
  uint32_t tmem_cols;
  int* status;
};
__device__ __forceinline__ int xbatch_layer(const XBatch& b, int tile) {
  int l = 0;
#pragma unroll 1
  for (int i = 1; i < b.count; ++i) l = tile >= b.tile_begin[i] ? i : l;
  return l;
}

// ---- steps 1-3: S = limbs x a_t^T on the tensor cores (K-major bf16 operands, fp32 accumulators in TMEM), then the
// guard-band rounding in the epilogue (the heavy part: two CTAs per SM give it sixteen warps).  Persistent CTAs walk
// 128 x block_n tiles (block_n <= 128); the B operand's k
// coordinate wraps every r_pad elements (the three limb blocks of A meet the same A~ block).
__global__ void __launch_bounds__(kXThreads, 2)
merge_exact_kernel(const __grid_constant__ XBatch args) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t smem_base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - raw_addr);

  const uint32_t b_tile = static_cast<uint32_t>(args.block_n) * kXBlockKBytes;
  const uint32_t stage_bytes = kXATile + b_tile;
  constexpr int S = kXStages;
  const uint32_t bars = smem_base + S * stage_bytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (S + s); };
  auto tmem_full_bar = [&](int a) { return bars + 8u * (2 * S + a); };
  auto tmem_empty_bar = [&](int a) { return bars + 8u * (2 * S + 2 + a); };
  const uint32_t slot_off = S * stage_bytes + 8u * (2 * S + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + slot_off);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  constexpr uint32_t kEpiWarps = 8;

  if (threadIdx.x == 0) {
    for (int i = 0; i < args.count; ++i) {
      prefetch_tensor_map(&args.ta[i]);
      prefetch_tensor_map(&args.tb[i]);
    }
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tmem_full_bar(a), 1); mbar_init(tmem_empty_bar(a), kEpiWarps); }
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_base + slot_off, args.tmem_cols);
    tmem_relinquish();
  }
  pdl_trigger();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();

  const int total_tiles = args.tile_begin[args.count];
  const uint32_t acc_cols = static_cast<uint32_t>(args.block_n);
  int* const status = args.status;
  bool aborted = false;

  if (warp == 0) {
    int stage = 0;
    uint32_t phase = 0;
    for (int gtile = blockIdx.x; gtile < total_tiles && !aborted; gtile += gridDim.x) {
      const int l = xbatch_layer(args, gtile);
      const XParams& p = args.p[l];
      const int tile = gtile - args.tile_begin[l];
      const int n_idx = tile / p.m_tiles, m_idx = tile - n_idx * p.m_tiles;
      for (int kb = 0; kb < p.kblocks_total; ++kb) {
        if (!mbar_wait_warp(empty_bar(stage), phase ^ 1u, status)) { aborted = true; break; }
        if (elect_one()) {
          const uint32_t fb = full_bar(stage);
          mbar_expect_tx(fb, stage_bytes);
          const uint32_t a_dst = smem_base + stage * stage_bytes;
          tma_load_2d(a_dst, &args.ta[l], fb, kb * kXBlockKBytes, m_idx * kXBlockM);
          tma_load_2d(a_dst + kXATile, &args.tb[l], fb, (kb % p.kblocks_wrap) * kXBlockKBytes, n_idx * p.block_n);
        }
        __syncwarp();
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    int stage = 0, acc = 0;
    uint32_t phase = 0, acc_phase = 0;
    const uint64_t a_desc0 = make_smem_desc(smem_base, 16, 1024);
    const uint64_t b_desc0 = make_smem_desc(smem_base + kXATile, 16, 1024);
    constexpr uint32_t kStep = kXUmmaKBytes >> 4;
    for (int gtile = blockIdx.x; gtile < total_tiles && !aborted; gtile += gridDim.x) {
      const XParams& p = args.p[xbatch_layer(args, gtile)];
      if (!mbar_wait_warp(tmem_empty_bar(acc), acc_phase ^ 1u, status)) { aborted = true; break; }
      tc_fence_after_sync();
      const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc) * acc_cols;
      for (int kb = 0; kb < p.kblocks_total; ++kb) {
        if (!mbar_wait_warp(full_bar(stage), phase, status)) { aborted = true; break; }
        tc_fence_after_sync();
        const uint32_t stage_off = (static_cast<uint32_t>(stage) * stage_bytes) >> 4;
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < kXBlockKBytes / kXUmmaKBytes; ++k)
            umma_bf16(d_tmem, a_desc0 + stage_off + k * kStep, b_desc0 + stage_off + k * kStep, p.idesc,
                      (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit(empty_bar(stage));
        }
        __syncwarp();
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
      if (aborted) break;
      if (elect_one()) umma_commit(tmem_full_bar(acc));
      __syncwarp();
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
  } else {
    // ------------------------------------------------------------ epilogue: guard-band rounding
    const int quad = warp & 3;
    const int col_half = (warp - 2) >> 2;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int gtile = blockIdx.x; gtile < total_tiles && !aborted; gtile += gridDim.x) {
      const int l = xbatch_layer(args, gtile);
      const XParams& p = args.p[l];
      const int tile = gtile - args.tile_begin[l];
      const int n_idx = tile / p.m_tiles, m_idx = tile - n_idx * p.m_tiles;
      if (!mbar_wait(tmem_full_bar(acc), acc_phase, status)) { aborted = true; break; }
      tc_fence_after_sync();
      const int q = m_idx * kXBlockM + quad * 32 + lane;
      const bool row_ok = q < p.k;
      const int64_t wrow = row_ok ? static_cast<int64_t>(ld_stream(p.sel_idx + q)) * p.n : 0;
      const float ksp = row_ok ? __fmul_rn(p.kappa * 1.0001f, ld_stream(p.sprime + q)) : 0.0f;   // kappa sum|d'|, rounded up a little
      const uint32_t t_row = tmem_base + static_cast<uint32_t>(acc) * acc_cols + (static_cast<uint32_t>(quad * 32) << 16);
      const int half = max(32, p.block_n / 2);                  // block_n is 32, 64, 128 or 256
      const int c_begin = col_half ? half : 0, c_end = col_half ? p.block_n : min(half, p.block_n);
      // per chunk of 32 columns a thread needs 32 bytes of old codes from its own backbone row and the 32 column
      // maxima (one per lane, handed round by shuffles); the loads of chunk i + 1 are issued before chunk i is computed
      uint4 w_next[2] = {make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)};
      float am_next = 0.0f;
      auto fetch = [&](int cl) {
        const int c0 = n_idx * p.block_n + cl;
        if (cl >= c_end || c0 >= p.n) return;
        am_next = ld_stream(p.amax_c + c0 + lane);
        if (row_ok) {
          w_next[0] = ld_stream(reinterpret_cast<const uint4*>(p.wq + wrow + c0));
          if (p.n - c0 > 16) w_next[1] = ld_stream(reinterpret_cast<const uint4*>(p.wq + wrow + c0) + 1);
        }
      };
      fetch(c_begin);
      for (int cl = c_begin; cl < c_end; cl += 32) {
        const int c0 = n_idx * p.block_n + cl;                  // a multiple of 32
        if (c0 >= p.n) break;                                   // warp-uniform
        uint32_t v[32];
        tmem_ld_32x32b_x32(t_row + static_cast<uint32_t>(cl), v);
        const uint4 wcodes[2] = {w_next[0], w_next[1]};
        const float am_lane = am_next;
        fetch(cl + 32);
        tmem_ld_wait();
        const int valid = min(32, p.n - c0);                    // n is a multiple of 16: 16 or 32
        const uint32_t win[8] = {wcodes[0].x, wcodes[0].y, wcodes[0].z, wcodes[0].w, wcodes[1].x, wcodes[1].y, wcodes[1].z, wcodes[1].w};
        uint32_t wout[8];
        uint32_t flag = 0;
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const float2 w01 = e4m3x2_to_float2(win[g]), w23 = e4m3x2_to_float2(win[g] >> 16);
          const float wv[4] = {w01.x, w01.y, w23.x, w23.y};
          uint32_t word = 0;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float am = __shfl_sync(0xFFFFFFFFu, am_lane, 4 * g + e);
            const float s = __fadd_rn(__uint_as_float(v[4 * g + e]), wv[e]);
            const float eps = __fmaf_rn(ksp, am, __fmul_rn(p.kappa, fabsf(wv[e])));
            const uint32_t both = cvt_fp8x2<kE4M3>(__fsub_rn(s, eps), __fadd_rn(s, eps));   // low byte, high byte
            const uint32_t lo = both & 0xFFu, hi = (both >> 8) & 0xFFu;
            const uint32_t old_code = (win[g] >> (8 * e)) & 0xFFu;
            const bool sure = lo == hi && (lo & 0x7Fu) != 0x7Fu;     // (a NaN code only if eps was inf or NaN)
            word |= (sure ? lo : old_code) << (8 * e);
            if (!sure && 4 * g + e < valid) flag |= 1u << (4 * g + e);
            if (p.sums_out != nullptr && row_ok && 4 * g + e < valid)
              p.sums_out[static_cast<int64_t>(q) * p.n + c0 + 4 * g + e] = s;
          }
          wout[g] = word;
        }
        if (!row_ok) continue;
        *reinterpret_cast<uint4*>(p.wq + wrow + c0) = make_uint4(wout[0], wout[1], wout[2], wout[3]);
        if (valid > 16) *(reinterpret_cast<uint4*>(p.wq + wrow + c0) + 1) = make_uint4(wout[4], wout[5], wout[6], wout[7]);
        p.flags[static_cast<int64_t>(q) * p.words_per_row + (c0 >> 5)] = flag;
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(tmem_empty_bar(acc));
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
  }

  if (aborted) {
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) { }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, args.tmem_cols);
  }
}

// ---- step 4: the flagged elements, exactly.  Every term is an integer multiple of 2^-158 (fp32: 2^-149, E4M3: 2^-9);
// the sum is a big integer in that unit, radix-2^32 digits in 64-bit bins (a carry pass at the end), rounded once.
struct ExactSumDev {
  static constexpr int kBins = 12;
  long long bin[kBins];
  __device__ void clear() {
#pragma unroll
    for (int i = 0; i < kBins; ++i) bin[i] = 0;
  }
  __device__ void add_shifted(long long p, int shift) {
    const int k = shift >> 5, t = shift & 31;
    const __int128 v = static_cast<__int128>(p) << t;
    bin[k] += static_cast<long long>(static_cast<unsigned long long>(static_cast<unsigned __int128>(v) & 0xFFFFFFFFu));
    bin[k + 1] += static_cast<long long>(static_cast<unsigned long long>((static_cast<unsigned __int128>(v) >> 32) & 0xFFFFFFFFu));
    bin[k + 2] += static_cast<long long>(v >> 64);
  }
  __device__ void add_product(float d, int a_int) {
    const uint32_t b = __float_as_uint(d);
    const int ef = static_cast<int>((b >> 23) & 0xFF);
    const long long frac = static_cast<long long>(b & 0x7FFFFFu);
    long long mant = ef == 0 ? frac : (frac | 0x800000ll);
    const int e = ef == 0 ? -149 : ef - 150;
    if (b >> 31) mant = -mant;
    if (mant == 0 || a_int == 0) return;
    add_shifted(mant * static_cast<long long>(a_int), e + 149);
  }
  __device__ uint32_t round_to_e4m3() const {
    long long d[kBins];
    long long carry = 0;
    for (int i = 0; i < kBins; ++i) {
      const long long t = bin[i] + carry;
      d[i] = t & 0xFFFFFFFFll;
      carry = t >> 32;
    }
    const bool negative = carry < 0;
    if (negative) {
      long long c = 1;
      for (int i = 0; i < kBins; ++i) { const long long t = (~d[i] & 0xFFFFFFFFll) + c; d[i] = t & 0xFFFFFFFFll; c = t >> 32; }
    }
    int top = -1;
    for (int i = kBins - 1; i >= 0; --i)
      if (d[i] != 0) { top = i * 32 + 31 - __clz(static_cast<int>(static_cast<uint32_t>(d[i]))); break; }
    if (top < 0) return 0u;
    auto bit_at = [&](int pos) -> int { return pos < 0 ? 0 : static_cast<int>((d[pos >> 5] >> (pos & 31)) & 1); };
    const int q = max(149, top - 3);
    int Q = 0;
    for (int pos = top; pos >= q; --pos) Q = (Q << 1) | bit_at(pos);
    const int half = bit_at(q - 1);
    bool sticky = false;
    for (int pos = q - 2; pos >= 0 && !sticky; --pos) sticky = bit_at(pos) != 0;
    if (half && (sticky || (Q & 1))) ++Q;
    // Q * 2^(q - 158) with Q <= 16 is exact in fp32 whenever it is at most 448; beyond that it saturates anyway
    const float mag = q - 158 > 10 ? 1.0e9f : ldexpf(static_cast<float>(Q), q - 158);
    const uint32_t code = cvt_fp8x2<kE4M3>(mag, 0.0f) & 0xFFu;       // representable (or saturating): no rounding here
    return negative ? (code | 0x80u) : code;
  }
};

__device__ __forceinline__ int e4m3_times_512(uint32_t code) {
  const float2 v = e4m3x2_to_float2(code & 0xFFu);
  return __float2int_rn(v.x * 512.0f);
}

// One element, exactly, by a whole warp: the lanes split the r terms, their partial sums (plain integer bins) are added
// across the warp, lane 0 rounds.  Kept out of line: the scan below should stay light, almost no word has a bit set.
__device__ __noinline__ uint32_t exact_element_warp(uint32_t w_code, const float* d, const uint8_t* a_col, int64_t n, int r) {
  const int lane = threadIdx.x & 31;
  ExactSumDev acc;
  acc.clear();
  for (int j = lane; j < r; j += 32)
    acc.add_product(ld_stream(d + j), e4m3_times_512(ld_stream(a_col + static_cast<int64_t>(j) * n)));
  if (lane == 0) {
    const long long w_int = e4m3_times_512(w_code);
    if (w_int != 0) acc.add_shifted(w_int, 149);
  }
#pragma unroll
  for (int b = 0; b < ExactSumDev::kBins; ++b) {
    long long v = acc.bin[b];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);   // at most 8 x 32 terms of < 2^33 each per bin
    acc.bin[b] = v;
  }
  return acc.round_to_e4m3();     // every lane holds the full sum and computes the same code
}

// A warp scans 32 flag words at a time (one per lane); for every set bit all its lanes recompute that element.
struct FixLayer {
  uint8_t* wq;
  const uint8_t* aq;
  const int32_t* sel_idx;
  const float* dprime;
  const uint32_t* flags;
  unsigned int* fix_count;     // nullable
  long long total_words, n;
  int r, r_pad, words_per_row, cta_begin, ctas;
};
struct FixBatch {
  FixLayer layer[kXBatchMax];
  int count;
};
__global__ void __launch_bounds__(256) exact_fix_kernel(const __grid_constant__ FixBatch args) {
  pdl_trigger();
  pdl_wait();
  int l = 0;
#pragma unroll 1
  for (int i = 1; i < args.count; ++i) l = static_cast<int>(blockIdx.x) >= args.layer[i].cta_begin ? i : l;
  const FixLayer& a = args.layer[l];
  uint8_t* wq = a.wq;
  const uint8_t* aq = a.aq;
  const int32_t* sel_idx = a.sel_idx;
  const float* dprime = a.dprime;
  const uint32_t* flags = a.flags;
  unsigned int* fix_count = a.fix_count;
  const int64_t total_words = a.total_words, n = a.n;
  const int r = a.r, r_pad = a.r_pad, words_per_row = a.words_per_row;
  const int cta = static_cast<int>(blockIdx.x) - a.cta_begin;
  const int lane = threadIdx.x & 31;
  unsigned int fixed = 0;
  const int64_t warps = static_cast<int64_t>(a.ctas) * 8;
  for (int64_t base = (cta * 8ll + (threadIdx.x >> 5)) * 32; base < total_words; base += warps * 32) {
    const int64_t wi = base + lane;
    const uint32_t mine = wi < total_words ? ld_stream(flags + wi) : 0u;
    uint32_t pending = __ballot_sync(0xFFFFFFFFu, mine != 0);
    while (pending != 0) {                                     // warp-uniform
      const int src_lane = __ffs(pending) - 1;
      pending &= pending - 1;
      uint32_t word = __shfl_sync(0xFFFFFFFFu, mine, src_lane);
      const int64_t w_idx = base + src_lane;
      const int q = static_cast<int>(w_idx / words_per_row);
      const int64_t c0 = (w_idx - static_cast<int64_t>(q) * words_per_row) * 32;
      const int64_t wrow = static_cast<int64_t>(ld_stream(sel_idx + q)) * n;
      while (word != 0) {
        const int bit = __ffs(word) - 1;
        word &= word - 1;
        const int64_t c = c0 + bit;
        const uint32_t code = exact_element_warp(wq[wrow + c], dprime + static_cast<int64_t>(q) * r_pad, aq + c, n, r);
        if (lane == 0) { wq[wrow + c] = static_cast<uint8_t>(code); ++fixed; }
      }
    }
  }
  if (fix_count != nullptr && fixed != 0) atomicAdd(fix_count, fixed);
}

}  // namespace

size_t exact_merge_scratch_bytes(int64_t m, int64_t n, int64_t r) {
  const int64_t r_pad = round_up(r, 64);
  size_t b = 0;
  b += round_up(n * r_pad * 2, 1024);                          // a_t
  b += round_up(round_up(n, 32) * 4, 1024);                    // amax_c
  b += round_up(m * 3 * r_pad * 2, 1024);                      // limbs
  b += round_up(m * r_pad * 4, 1024);                          // dprime
  b += round_up(m * 4, 1024);                                  // sprime
  b += round_up(m * ((n + 31) / 32) * 4, 1024);                // flags
  b += 1024;                                                   // counter of exactly recomputed elements
  return b;
}

namespace {
struct ExactScratch {
  uint16_t* a_t; float* amax_c; uint16_t* limbs; float* dprime; float* sprime; uint32_t* flags; unsigned int* counter;
};
ExactScratch carve_scratch(void* scratch, int64_t m, int64_t n, int64_t r_pad) {
  uint8_t* base = static_cast<uint8_t*>(scratch);
  size_t off = 0;
  ExactScratch x;
  x.a_t = reinterpret_cast<uint16_t*>(base + off); off += round_up(n * r_pad * 2, 1024);
  x.amax_c = reinterpret_cast<float*>(base + off); off += round_up(round_up(n, 32) * 4, 1024);
  x.limbs = reinterpret_cast<uint16_t*>(base + off); off += round_up(m * 3 * r_pad * 2, 1024);
  x.dprime = reinterpret_cast<float*>(base + off); off += round_up(m * r_pad * 4, 1024);
  x.sprime = reinterpret_cast<float*>(base + off); off += round_up(m * 4, 1024);
  x.flags = reinterpret_cast<uint32_t*>(base + off); off += round_up(m * ((n + 31) / 32) * 4, 1024);
  x.counter = reinterpret_cast<unsigned int*>(base + off);
  return x;
}
}  // namespace

// Step 0a on its own: the bf16 copy of A~ (transposed) and its column maxima depend only on the A~ rows of the backbone,
// which the proxy update never changes, so a caller may prepare them once per layer.
cudaError_t launch_exact_merge_prepare(const uint8_t* wq, int64_t m, int64_t n, int64_t r, void* scratch, cudaStream_t stream) {
  const int64_t r_pad = round_up(r, 64);
  const ExactScratch x = carve_scratch(scratch, m, n, r_pad);
  const uint8_t* aq = wq + m * n;
  cudaError_t e = launch_pdl(exact_prep_a_kernel, dim3(static_cast<unsigned>((n + 255) / 256), static_cast<unsigned>(r_pad / 2)),
                             dim3(256), 0, stream, 1, aq, n, static_cast<int>(r), static_cast<int>(r_pad), x.a_t);
  if (e != cudaSuccess) return e;
  return launch_pdl(exact_amax_a_kernel, dim3(static_cast<unsigned>((n + 255) / 256)), dim3(256), 0, stream, 1,
                    static_cast<const uint16_t*>(x.a_t), n, static_cast<int>(r_pad), x.amax_c);
}

// Steps 0b-4 for up to kProxyBatchMax layers in three launches (row preparation, tensor-core sums with the guard-band
// rounding, exact recomputation of the flagged elements).  a_prepared: step 0a was run on every layer's scratch
// (launch_exact_merge_prepare) and the A~ rows have not changed since; otherwise it runs here, two launches per layer.
cudaError_t launch_merge_exact_batched(const ExactMergeLayer* layers, int count, bool a_prepared, int* status, cudaStream_t stream) {
  if (count < 1 || count > kXBatchMax) return cudaErrorInvalidValue;
  PrepRowsBatch pb{};
  XBatch xb{};
  FixBatch fb{};
  ExactScratch xs[kXBatchMax];
  int64_t r_pad[kXBatchMax];
  int active = 0, prep_ctas = 0;
  for (int i = 0; i < count; ++i) {
    const ExactMergeLayer& L = layers[i];
    if (L.k == 0) continue;
    if (L.k < 1 || L.k > L.m || L.r < 8 || L.r > 256 || L.n % 16) return cudaErrorInvalidValue;
    r_pad[active] = round_up(L.r, 64);
    xs[active] = carve_scratch(L.scratch, L.m, L.n, r_pad[active]);
    if (!a_prepared) {
      const cudaError_t e = launch_exact_merge_prepare(L.wq, L.m, L.n, L.r, L.scratch, stream);
      if (e != cudaSuccess) return e;
    }
    PrepRowsLayer& a = pb.layer[active];
    a.dbuf = L.dbuf; a.sel_idx = L.sel_idx; a.row_scales = L.row_scales; a.limbs = xs[active].limbs; a.dprime = xs[active].dprime;
    a.sprime = xs[active].sprime; a.m = L.m; a.k = static_cast<int>(L.k); a.r = static_cast<int>(L.r);
    a.r_pad = static_cast<int>(r_pad[active]); a.cta_begin = prep_ctas;
    prep_ctas += static_cast<int>((L.k + 7) / 8);
    ++active;
  }
  if (active == 0) return cudaSuccess;
  pb.count = active;
  cudaError_t e = launch_pdl(exact_prep_rows_kernel, dim3(static_cast<unsigned>(prep_ctas)), dim3(256), 0, stream, 1, pb);
  if (e != cudaSuccess) return e;

  // one tile width for the whole launch: narrower tiles when there would be too few of them for two CTAs per SM
  int block_n = 128;
  auto tiles_at = [&](int bn) {
    int64_t t = 0;
    for (int i = 0; i < count; ++i)
      if (layers[i].k > 0) t += ((layers[i].k + kXBlockM - 1) / kXBlockM) * ((layers[i].n + bn - 1) / bn);
    return t;
  };
  while (block_n > 32 && tiles_at(block_n) < 2 * sm_count()) block_n >>= 1;
  xb.count = active; xb.block_n = block_n; xb.tmem_cols = static_cast<uint32_t>(2 * block_n); xb.status = status;
  int tiles = 0, fix_ctas = 0, a = 0;
  for (int i = 0; i < count; ++i) {
    const ExactMergeLayer& L = layers[i];
    if (L.k == 0) continue;
    XParams& p = xb.p[a];
    p.k = static_cast<int>(L.k); p.n = static_cast<int>(L.n); p.r_pad = static_cast<int>(r_pad[a]);
    p.m_tiles = static_cast<int>((L.k + kXBlockM - 1) / kXBlockM);
    p.block_n = block_n;
    p.n_tiles = static_cast<int>((L.n + block_n - 1) / block_n);
    p.kblocks_wrap = static_cast<int>(r_pad[a] * 2 / kXBlockKBytes);
    p.kblocks_total = 3 * p.kblocks_wrap;
    // instruction descriptor: fp32 accumulate, A and B bf16 K-major, N = block_n, M = 128
    p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(block_n >> 3) << 17) |
              (static_cast<uint32_t>(kXBlockM >> 4) << 24);
    p.tmem_cols = xb.tmem_cols;
    // accumulation error: 3 r_pad exact products summed in fp32 in an unknown order, each partial sum bounded by
    // T = |w| + sum|d'| max|a|: (N - 1) 2^-24 T for round-to-nearest adds; taken with a factor 2 (2^-23 per add) for adds
    // that truncate, plus the final add of w.  Measured on B200: the sums use 0.2-0.7 % of this band.
    p.kappa = 1.02f * static_cast<float>(3 * r_pad[a] + 8) * 1.1920928955078125e-07f;   // 2^-23
    p.wq = L.wq; p.sel_idx = L.sel_idx; p.sprime = xs[a].sprime; p.amax_c = xs[a].amax_c; p.flags = xs[a].flags;
    p.words_per_row = static_cast<int>((L.n + 31) / 32);
    p.sums_out = L.sums_out;
    if (!make_tensor_map(&xb.ta[a], reinterpret_cast<const uint8_t*>(xs[a].limbs), L.k, 3 * r_pad[a] * 2, 3 * r_pad[a] * 2,
                         kXBlockKBytes, kXBlockM))
      return cudaErrorInvalidValue;
    if (!make_tensor_map(&xb.tb[a], reinterpret_cast<const uint8_t*>(xs[a].a_t), L.n, r_pad[a] * 2, r_pad[a] * 2, kXBlockKBytes,
                         static_cast<uint32_t>(block_n)))
      return cudaErrorInvalidValue;
    xb.tile_begin[a] = tiles;
    tiles += p.m_tiles * p.n_tiles;
    FixLayer& f = fb.layer[a];
    f.wq = L.wq; f.aq = L.wq + L.m * L.n; f.sel_idx = L.sel_idx; f.dprime = xs[a].dprime; f.flags = xs[a].flags;
    f.fix_count = L.fix_count_out != nullptr ? xs[a].counter : nullptr;
    f.total_words = L.k * p.words_per_row; f.n = L.n; f.r = static_cast<int>(L.r); f.r_pad = static_cast<int>(r_pad[a]);
    f.words_per_row = p.words_per_row; f.cta_begin = fix_ctas;
    int64_t fg = (f.total_words + 255) / 256;
    const int64_t cap = static_cast<int64_t>(sm_count()) * 8 / active;
    if (fg > cap) fg = cap > 0 ? cap : 1;
    f.ctas = static_cast<int>(fg);
    fix_ctas += f.ctas;
    if (L.fix_count_out != nullptr) {
      e = cudaMemsetAsync(xs[a].counter, 0, sizeof(unsigned int), stream);
      if (e != cudaSuccess) return e;
    }
    ++a;
  }
  xb.tile_begin[active] = tiles;
  fb.count = active;
  const size_t smem = static_cast<size_t>(kXStages) * (kXATile + static_cast<size_t>(block_n) * kXBlockKBytes) + 256 + 1024;
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(merge_exact_kernel, 227 * 1024, configured);
    if (ec != cudaSuccess) return ec;
  }
  int grid = 2 * sm_count();
  if (tiles < grid) grid = tiles;
  e = launch_pdl(merge_exact_kernel, dim3(static_cast<unsigned>(grid)), dim3(kXThreads), smem, stream, 1, xb);
  if (e != cudaSuccess) return e;
  e = launch_pdl(exact_fix_kernel, dim3(static_cast<unsigned>(fix_ctas)), dim3(256), 0, stream, 1, fb);
  if (e != cudaSuccess) return e;
  a = 0;
  for (int i = 0; i < count; ++i) {
    if (layers[i].k == 0) continue;
    if (layers[i].fix_count_out != nullptr) {
      e = cudaMemcpyAsync(layers[i].fix_count_out, xs[a].counter, sizeof(unsigned int), cudaMemcpyDeviceToDevice, stream);
      if (e != cudaSuccess) return e;
    }
    ++a;
  }
  return cudaSuccess;
}

cudaError_t launch_merge_exact(uint8_t* wq, float* dbuf, const int32_t* sel_idx, int64_t k, int64_t m, int64_t n, int64_t r,
                               const float* row_scales, void* scratch, float* sums_out, unsigned int* fix_count_out, int* status,
                               cudaStream_t stream) {
  if (k < 1 || k > m || r < 8 || r > 256 || n % 16) return cudaErrorInvalidValue;
  const ExactMergeLayer one{wq, dbuf, sel_idx, row_scales, scratch, sums_out, fix_count_out, m, n, r, k};
  return launch_merge_exact_batched(&one, 1, false, status, stream);
}

}  // namespace falqon
