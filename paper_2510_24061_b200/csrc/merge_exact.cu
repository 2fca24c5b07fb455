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
__global__ void __launch_bounds__(256) exact_prep_rows_kernel(float* dbuf, const int32_t* sel_idx, int k, int r, int r_pad,
                                                              const float* row_scales, int64_t m, uint16_t* limbs,
                                                              float* dprime, float* sprime) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int q = blockIdx.x * 8 + (threadIdx.x >> 5);
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
  int* status;
};

// ---- steps 1-3: S = limbs x a_t^T on the tensor cores (K-major bf16 operands, fp32 accumulators in TMEM), then the
// guard-band rounding in the epilogue (the heavy part: two CTAs per SM give it sixteen warps).  Persistent CTAs walk
// 128 x block_n tiles (block_n <= 128); the B operand's k
// coordinate wraps every r_pad elements (the three limb blocks of A meet the same A~ block).
__global__ void __launch_bounds__(kXThreads, 2)
merge_exact_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const XParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t smem_base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - raw_addr);

  const uint32_t b_tile = static_cast<uint32_t>(p.block_n) * kXBlockKBytes;
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
    prefetch_tensor_map(&tmap_a);
    prefetch_tensor_map(&tmap_b);
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tmem_full_bar(a), 1); mbar_init(tmem_empty_bar(a), kEpiWarps); }
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_base + slot_off, p.tmem_cols);
    tmem_relinquish();
  }
  pdl_trigger();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();

  const int total_tiles = p.m_tiles * p.n_tiles;
  const uint32_t acc_cols = static_cast<uint32_t>(p.block_n);
  bool aborted = false;

  if (warp == 0) {
    int stage = 0;
    uint32_t phase = 0;
    for (int tile = blockIdx.x; tile < total_tiles && !aborted; tile += gridDim.x) {
      const int n_idx = tile / p.m_tiles, m_idx = tile - n_idx * p.m_tiles;
      for (int kb = 0; kb < p.kblocks_total; ++kb) {
        if (!mbar_wait_warp(empty_bar(stage), phase ^ 1u, p.status)) { aborted = true; break; }
        if (elect_one()) {
          const uint32_t fb = full_bar(stage);
          mbar_expect_tx(fb, stage_bytes);
          const uint32_t a_dst = smem_base + stage * stage_bytes;
          tma_load_2d(a_dst, &tmap_a, fb, kb * kXBlockKBytes, m_idx * kXBlockM);
          tma_load_2d(a_dst + kXATile, &tmap_b, fb, (kb % p.kblocks_wrap) * kXBlockKBytes, n_idx * p.block_n);
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
    for (int tile = blockIdx.x; tile < total_tiles && !aborted; tile += gridDim.x) {
      if (!mbar_wait_warp(tmem_empty_bar(acc), acc_phase ^ 1u, p.status)) { aborted = true; break; }
      tc_fence_after_sync();
      const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc) * acc_cols;
      for (int kb = 0; kb < p.kblocks_total; ++kb) {
        if (!mbar_wait_warp(full_bar(stage), phase, p.status)) { aborted = true; break; }
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
    for (int tile = blockIdx.x; tile < total_tiles && !aborted; tile += gridDim.x) {
      const int n_idx = tile / p.m_tiles, m_idx = tile - n_idx * p.m_tiles;
      if (!mbar_wait(tmem_full_bar(acc), acc_phase, p.status)) { aborted = true; break; }
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
    tmem_dealloc(tmem_base, p.tmem_cols);
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
__global__ void __launch_bounds__(256) exact_fix_kernel(uint8_t* wq, const uint8_t* aq, const int32_t* sel_idx,
                                                        const float* dprime, const uint32_t* flags, int64_t total_words, int64_t n,
                                                        int r, int r_pad, int words_per_row, unsigned int* fix_count) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  unsigned int fixed = 0;
  const int64_t warps = static_cast<int64_t>(gridDim.x) * 8;
  for (int64_t base = (blockIdx.x * 8ll + (threadIdx.x >> 5)) * 32; base < total_words; base += warps * 32) {
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

cudaError_t launch_merge_exact(uint8_t* wq, float* dbuf, const int32_t* sel_idx, int64_t k, int64_t m, int64_t n, int64_t r,
                               const float* row_scales, void* scratch, float* sums_out, unsigned int* fix_count_out, int* status,
                               cudaStream_t stream) {
  if (k < 1 || k > m || r < 8 || r > 256 || n % 16) return cudaErrorInvalidValue;
  const int64_t r_pad = round_up(r, 64);
  uint8_t* base = static_cast<uint8_t*>(scratch);
  size_t off = 0;
  uint16_t* a_t = reinterpret_cast<uint16_t*>(base + off); off += round_up(n * r_pad * 2, 1024);
  float* amax_c = reinterpret_cast<float*>(base + off); off += round_up(round_up(n, 32) * 4, 1024);
  uint16_t* limbs = reinterpret_cast<uint16_t*>(base + off); off += round_up(m * 3 * r_pad * 2, 1024);
  float* dprime = reinterpret_cast<float*>(base + off); off += round_up(m * r_pad * 4, 1024);
  float* sprime = reinterpret_cast<float*>(base + off); off += round_up(m * 4, 1024);
  uint32_t* flags = reinterpret_cast<uint32_t*>(base + off); off += round_up(m * ((n + 31) / 32) * 4, 1024);
  unsigned int* counter = reinterpret_cast<unsigned int*>(base + off);
  const uint8_t* aq = wq + m * n;

  cudaError_t e = launch_pdl(exact_prep_a_kernel, dim3(static_cast<unsigned>((n + 255) / 256), static_cast<unsigned>(r_pad / 2)),
                             dim3(256), 0, stream, 1, aq, n, static_cast<int>(r), static_cast<int>(r_pad), a_t);
  if (e != cudaSuccess) return e;
  e = launch_pdl(exact_amax_a_kernel, dim3(static_cast<unsigned>((n + 255) / 256)), dim3(256), 0, stream, 1,
                 static_cast<const uint16_t*>(a_t), n, static_cast<int>(r_pad), amax_c);
  if (e != cudaSuccess) return e;
  e = launch_pdl(exact_prep_rows_kernel, dim3(static_cast<unsigned>((k + 7) / 8)), dim3(256), 0, stream, 1, dbuf, sel_idx,
                 static_cast<int>(k), static_cast<int>(r), static_cast<int>(r_pad), row_scales, m, limbs, dprime, sprime);
  if (e != cudaSuccess) return e;

  XParams p{};
  p.k = static_cast<int>(k); p.n = static_cast<int>(n); p.r_pad = static_cast<int>(r_pad);
  p.m_tiles = static_cast<int>((k + kXBlockM - 1) / kXBlockM);
  int block_n = 128;   // narrower tiles when there would be too few of them for two CTAs per SM
  while (block_n > 32 && static_cast<int64_t>(p.m_tiles) * ((n + block_n - 1) / block_n) < 2 * sm_count()) block_n >>= 1;
  p.block_n = block_n;
  p.n_tiles = static_cast<int>((n + block_n - 1) / block_n);
  p.kblocks_wrap = static_cast<int>(r_pad * 2 / kXBlockKBytes);
  p.kblocks_total = 3 * p.kblocks_wrap;
  // instruction descriptor: fp32 accumulate, A and B bf16 K-major, N = block_n, M = 128
  p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(block_n >> 3) << 17) |
            (static_cast<uint32_t>(kXBlockM >> 4) << 24);
  p.tmem_cols = static_cast<uint32_t>(2 * block_n);
  // accumulation error: 3 r_pad exact products summed in fp32 in an unknown order, each partial sum bounded by
  // T = |w| + sum|d'| max|a|: (N - 1) 2^-24 T for round-to-nearest adds; taken with a factor 2 (2^-23 per add) for adds
  // that truncate, plus the final add of w.  Measured on B200: the sums use 0.2-0.7 % of this band.
  p.kappa = 1.02f * static_cast<float>(3 * r_pad + 8) * 1.1920928955078125e-07f;   // 2^-23
  p.wq = wq; p.sel_idx = sel_idx; p.sprime = sprime; p.amax_c = amax_c; p.flags = flags;
  p.words_per_row = static_cast<int>((n + 31) / 32);
  p.sums_out = sums_out; p.status = status;
  CUtensorMap ta, tb;
  if (!make_tensor_map(&ta, reinterpret_cast<const uint8_t*>(limbs), k, 3 * r_pad * 2, 3 * r_pad * 2, kXBlockKBytes, kXBlockM))
    return cudaErrorInvalidValue;
  if (!make_tensor_map(&tb, reinterpret_cast<const uint8_t*>(a_t), n, r_pad * 2, r_pad * 2, kXBlockKBytes,
                       static_cast<uint32_t>(block_n)))
    return cudaErrorInvalidValue;
  const size_t smem = static_cast<size_t>(kXStages) * (kXATile + static_cast<size_t>(block_n) * kXBlockKBytes) + 256 + 1024;
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(merge_exact_kernel, 227 * 1024, configured);
    if (ec != cudaSuccess) return ec;
  }
  int grid = 2 * sm_count();
  const int64_t tiles = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
  if (tiles < grid) grid = static_cast<int>(tiles);
  e = launch_pdl(merge_exact_kernel, dim3(static_cast<unsigned>(grid)), dim3(kXThreads), smem, stream, 1, ta, tb, p);
  if (e != cudaSuccess) return e;
  if (fix_count_out != nullptr) {
    e = cudaMemsetAsync(counter, 0, sizeof(unsigned int), stream);
    if (e != cudaSuccess) return e;
  }
  const int64_t words = k * p.words_per_row;
  int64_t fgrid = (words + 255) / 256;
  if (fgrid > static_cast<int64_t>(sm_count()) * 8) fgrid = static_cast<int64_t>(sm_count()) * 8;
  e = launch_pdl(exact_fix_kernel, dim3(static_cast<unsigned>(fgrid)), dim3(256), 0, stream, 1, wq, aq, sel_idx, dprime, flags,
                 words, n, static_cast<int>(r), static_cast<int>(r_pad), p.words_per_row,
                 fix_count_out != nullptr ? counter : nullptr);
  if (e != cudaSuccess) return e;
  if (fix_count_out != nullptr)
    e = cudaMemcpyAsync(fix_count_out, counter, sizeof(unsigned int), cudaMemcpyDeviceToDevice, stream);
  return e;
}

}  // namespace falqon
