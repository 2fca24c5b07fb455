// CPU oracle for the melded FP8-LoRA linear layer.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
// method computes, written from the paper; the CUDA library never includes,
// links or calls it, and it includes nothing of the CUDA path.  Only the test
// suite, the smoke check and the benchmark's CPU-baseline leg may load it.
//
// Conventions (paper notation -> row-major arrays):
//   W  in R^{m x n}  -> W[m][n]      x in R^{n x d} -> X[T][n]  (T = d tokens)
//   O = W x          -> Y[T][m]      W' = [W~; A~]  -> Wq[(m+r)][n], E4M3 codes
//   O_A = A x        -> OA[T][r]     DeltaBuffer    -> dbuf[m][r], fp32
//
// Arithmetic rules: FP8 encode/decode are done on bit patterns in software;
// every contraction is accumulated in double; steps whose result feeds a
// bit-exact stage (scales, optimizer step, row scores, merge chain) are done
// in explicit fp32 operations in a fixed order.  Build with
// -O2 -ffp-contract=off so the compiler fuses nothing.
//
// Parity pins live in tests/test_oracle_*.py; the whole-step result on
// realistic data is "parity unpinned" in absolute terms (the paper prints no
// worked numbers) and is pinned only through invariants and exact cases.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum { FMT_E4M3 = 0, FMT_E5M2 = 1 };
enum { DT_BF16 = 0, DT_F32 = 1 };
enum { GRAN_TENSOR = 0, GRAN_ROW = 1 };

struct Fp8Format {
  int mant_bits;   // explicit mantissa bits
  int bias;        // exponent bias
  uint8_t max_code;  // code of the largest finite magnitude
  float max_value;   // its value: 448 (E4M3) or 57344 (E5M2), Eq. (quantize)
};

inline Fp8Format format_of(int fmt) {
  // E4M3 is the variant whose largest finite value is 448 (no infinities, one
  // NaN mantissa pattern); E5M2 is the IEEE-like one with largest finite 57344.
  if (fmt == FMT_E4M3) return Fp8Format{3, 7, 0x7E, 448.0f};
  return Fp8Format{2, 15, 0x7B, 57344.0f};
}

inline uint32_t bits_of(float v) { uint32_t u; std::memcpy(&u, &v, 4); return u; }
inline float float_of(uint32_t u) { float v; std::memcpy(&v, &u, 4); return v; }

// Exact value of an FP8 code.
double fp8_decode(uint8_t code, int fmt) {
  const Fp8Format f = format_of(fmt);
  const int sign = code >> 7;
  const int expo = (code & 0x7F) >> f.mant_bits;
  const int mant = code & ((1 << f.mant_bits) - 1);
  const int expo_all_ones = (1 << (7 - f.mant_bits)) - 1;
  double mag;
  if (fmt == FMT_E4M3) {
    if (expo == expo_all_ones && mant == 7) return std::numeric_limits<double>::quiet_NaN();
  } else {
    if (expo == expo_all_ones) {
      if (mant != 0) return std::numeric_limits<double>::quiet_NaN();
      return sign ? -std::numeric_limits<double>::infinity() : std::numeric_limits<double>::infinity();
    }
  }
  if (expo == 0) {
    mag = std::ldexp((double)mant, 1 - f.bias - f.mant_bits);            // subnormal
  } else {
    mag = std::ldexp((double)((1 << f.mant_bits) + mant), expo - f.bias - f.mant_bits);
  }
  return sign ? -mag : mag;
}

// Round-to-nearest-even, saturating conversion of an fp32 value to an FP8 code.
// Finite values beyond the largest finite magnitude (and infinities) give that
// magnitude; gradual underflow and the sign of zero are kept; NaN gives 0x7F.
uint8_t fp8_encode(float v, int fmt) {
  const Fp8Format f = format_of(fmt);
  const uint32_t u = bits_of(v);
  const uint8_t sign = (uint8_t)((u >> 31) << 7);
  const uint32_t a = u & 0x7FFFFFFFu;
  if (a > 0x7F800000u) return 0x7F;                       // NaN
  if (a > bits_of(f.max_value)) return sign | f.max_code;  // saturate (covers +-inf)
  if (a == 0) return sign;
  int e = (int)(a >> 23) - 127;                           // unbiased fp32 exponent
  uint64_t mant = a & 0x7FFFFFu;
  if ((a >> 23) == 0) e = -126; else mant |= (1u << 23);  // value = mant * 2^(e-23)
  const int emin = 1 - f.bias;                            // exponent of the smallest normal
  const int eq = std::max(e, emin);                       // binade the result is rounded in
  const int shift = (eq - f.mant_bits) - (e - 23);        // low bits to drop, > 0
  uint64_t q;
  if (shift > 40) {
    q = 0;
  } else {
    const uint64_t half = 1ull << (shift - 1);
    const uint64_t rem = mant & ((1ull << shift) - 1);
    q = mant >> shift;
    if (rem > half || (rem == half && (q & 1))) q += 1;  // nearest, ties to even
  }
  // q counts quanta 2^(eq - mant_bits).  In the subnormal binade the code is q
  // itself (q == 2^mant_bits is the smallest normal); in a normal binade q lies
  // in [2^mant_bits, 2^(mant_bits+1)] and a carry moves to the next exponent.
  uint32_t code = (uint32_t)((eq - emin) << f.mant_bits) + (uint32_t)q;
  if (code > f.max_code) code = f.max_code;
  return sign | (uint8_t)code;
}

inline float bf16_to_f32(uint16_t h) { return float_of((uint32_t)h << 16); }

inline uint16_t f32_to_bf16(float v) {  // round to nearest even (finite inputs)
  uint32_t u = bits_of(v);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x40);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

inline float load_elem(const void* src, int dt, int64_t i) {
  if (dt == DT_BF16) return bf16_to_f32(((const uint16_t*)src)[i]);
  return ((const float*)src)[i];
}

// s = fpmax / amax in one fp32 division.  The paper prints the scale as
// amax/fpmax but multiplies by it to quantize and divides to dequantize
// (Eq. quantize, Eq. fp8_matmul, Alg. 1, Alg. 2), so fpmax/amax is the only
// consistent reading.  amax == 0 gives s = 1; an infinite quotient is clamped.
inline float scale_from_amax(float amax, int fmt) {
  if (!(amax > 0.0f)) return 1.0f;
  float s = format_of(fmt).max_value / amax;
  if (std::isinf(s)) s = std::numeric_limits<float>::max();
  return s;
}

// ---- exact merge arithmetic (the correctly rounded variant of the merge, an extension beyond the paper's text):
// every E4M3 value is an integer multiple of 2^-9 and every fp32 value an integer multiple of 2^-149, so each term
// DeltaBuffer * A~ and the backbone code itself are integer multiples of 2^-158.  The sum is held exactly as a big
// integer in that unit (radix 2^32 digits in 64-bit bins, so hundreds of terms can be added before a carry pass),
// and rounded ONCE to E4M3: nearest, ties to the even code, saturating at +-448; a sum that rounds to zero keeps
// its sign, an exact zero is +0.
struct ExactSum {
  static constexpr int kBins = 12;       // 384 bits: 2^-158 .. beyond 2^127 * 2^18
  int64_t bin[kBins];
  ExactSum() { for (int i = 0; i < kBins; ++i) bin[i] = 0; }
  // adds p * 2^shift (in units of 2^-158); |p| < 2^62, shift >= 0
  void add_shifted(int64_t p, int shift) {
    const int k = shift >> 5, t = shift & 31;
    const __int128 v = (__int128)p << t;
    bin[k] += (int64_t)(uint64_t)((unsigned __int128)v & 0xFFFFFFFFu);
    bin[k + 1] += (int64_t)(uint64_t)(((unsigned __int128)v >> 32) & 0xFFFFFFFFu);
    bin[k + 2] += (int64_t)(v >> 64);    // arithmetic shift: carries the sign
  }
  // d * (a_int * 2^-9) for an fp32 d (finite) and an E4M3 value a_int * 2^-9
  void add_product(float d, int32_t a_int) {
    uint32_t b;
    std::memcpy(&b, &d, 4);
    const int ef = (int)((b >> 23) & 0xFF);
    const int64_t frac = (int64_t)(b & 0x7FFFFFu);
    int64_t mant = ef == 0 ? frac : (frac | 0x800000);
    const int e = ef == 0 ? -149 : ef - 150;          // d = +-mant * 2^e
    if (b >> 31) mant = -mant;
    if (mant == 0 || a_int == 0) return;
    add_shifted(mant * (int64_t)a_int, e + 149);      // unit 2^-158 = 2^(e-9) / 2^(e+149)
  }
  void add_code_value(int32_t w_int) { if (w_int) add_shifted((int64_t)w_int, 149); }   // w_int * 2^-9
  uint8_t round_to_e4m3() const {
    int64_t d[kBins];
    int64_t carry = 0;
    for (int i = 0; i < kBins; ++i) {                 // normalise to digits in [0, 2^32), sign in the last carry
      const int64_t t = bin[i] + carry;
      d[i] = t & 0xFFFFFFFFll;
      carry = t >> 32;                                 // arithmetic shift: floor division
    }
    const bool negative = carry < 0;                   // value = digits - 2^(32 kBins) when negative
    if (negative) {                                    // magnitude = two's complement
      int64_t c = 1;
      for (int i = 0; i < kBins; ++i) { const int64_t t = (~d[i] & 0xFFFFFFFFll) + c; d[i] = t & 0xFFFFFFFFll; c = t >> 32; }
    }
    int top = -1;                                      // index of the highest set bit of the magnitude
    for (int i = kBins - 1; i >= 0 && top < 0; --i)
      if (d[i]) for (int bit = 31; bit >= 0; --bit) if ((d[i] >> bit) & 1) { top = i * 32 + bit; break; }
    if (top < 0) return 0x00;                          // exact zero: +0
    auto bit_at = [&](int pos) -> int { return pos < 0 ? 0 : (int)((d[pos >> 5] >> (pos & 31)) & 1); };
    // quantum 2^q: 2^-9 (bit 149 of the unit) up to and including the binade [2^-6, 2^-5), then three bits below the top
    const int q = std::max(149, top - 3);
    int Q = 0;
    for (int pos = top; pos >= q; --pos) Q = (Q << 1) | bit_at(pos);
    const int half = bit_at(q - 1);
    bool sticky = false;
    for (int pos = q - 2; pos >= 0 && !sticky; --pos) sticky = bit_at(pos) != 0;
    if (half && (sticky || (Q & 1))) ++Q;
    double mag = std::ldexp((double)Q, q - 158);
    if (mag > 448.0) mag = 448.0;
    const uint8_t code = fp8_encode((float)mag, FMT_E4M3);     // exactly representable: no further rounding
    return negative ? (uint8_t)(code | 0x80) : code;
  }
};

struct DecodeTable {
  double v[256];
  explicit DecodeTable(int fmt) { for (int c = 0; c < 256; ++c) v[c] = fp8_decode((uint8_t)c, fmt); }
};

}  // namespace

extern "C" {

double orc_fp8_decode(uint8_t code, int fmt) { return fp8_decode(code, fmt); }
uint8_t orc_fp8_encode(float v, int fmt) { return fp8_encode(v, fmt); }

void orc_fp8_encode_array(const float* src, int64_t count, int fmt, uint8_t* dst) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) dst[i] = fp8_encode(src[i], fmt);
}

void orc_fp8_decode_array(const uint8_t* src, int64_t count, int fmt, double* dst) {
  for (int64_t i = 0; i < count; ++i) dst[i] = fp8_decode(src[i], fmt);
}

uint16_t orc_f32_to_bf16(float v) { return f32_to_bf16(v); }

// Q_fp8 (Eq. quantize): amax -> scale -> saturating round-to-nearest-even cast.
//   src        [rows][cols] bf16 (as uint16) or fp32, dense
//   gran       per tensor (one scale) or per row (rows scales)
//   scale_in   null: absmax scaling, scale(s) written to scale_out;
//              non-null: cast with the given scale(s) (A~ = Q(gamma*A; s_W), Eq. A_integ)
//   premul     fp32 factor applied first as its own rounded multiply (gamma = alpha/r); 1 skips it
//   amax_out   nullable; receives max|premul*x| per tensor / per row
int orc_quantize(const void* src, int src_dt, int64_t rows, int64_t cols, int fmt, int gran,
                 const float* scale_in, float premul, uint8_t* dst, float* scale_out, float* amax_out) {
  if (rows < 0 || cols < 0) return -1;
  const int64_t groups = (gran == GRAN_ROW) ? rows : 1;
  const int64_t group_len = (gran == GRAN_ROW) ? cols : rows * cols;
  for (int64_t g = 0; g < groups; ++g) {
    const int64_t base = g * group_len;
    float amax = 0.0f;
    for (int64_t i = 0; i < group_len; ++i) {
      float x = load_elem(src, src_dt, base + i);
      if (premul != 1.0f) x = premul * x;
      amax = std::max(amax, std::fabs(x));
    }
    const float s = scale_in ? scale_in[g] : scale_from_amax(amax, fmt);
    if (scale_out) scale_out[g] = s;
    if (amax_out) amax_out[g] = amax;
    for (int64_t i = 0; i < group_len; ++i) {
      float x = load_elem(src, src_dt, base + i);
      if (premul != 1.0f) x = premul * x;     // rounded fp32 product
      dst[base + i] = fp8_encode(x * s, fmt);  // second rounded fp32 product, then the cast
    }
  }
  return 0;
}

// Q_fp8 of dY in the per-row-scaled-backbone mode: column i of dY is first multiplied by 1 / s_w[i] (one fp32
// reciprocal, one rounded fp32 multiply), then the tensor is quantized per tensor as in orc_quantize.
int orc_quantize_colscaled(const void* src, int src_dt, int64_t rows, int64_t cols, int fmt, const float* col_div,
                           uint8_t* dst, float* scale_out, float* amax_out) {
  std::vector<float> inv((size_t)cols);
  for (int64_t c = 0; c < cols; ++c) inv[c] = 1.0f / col_div[c];
  float amax = 0.0f;
  for (int64_t t = 0; t < rows; ++t)
    for (int64_t c = 0; c < cols; ++c) amax = std::max(amax, std::fabs(load_elem(src, src_dt, t * cols + c) * inv[c]));
  const float s = scale_from_amax(amax, fmt);
  if (scale_out) *scale_out = s;
  if (amax_out) *amax_out = amax;
  for (int64_t t = 0; t < rows; ++t)
    for (int64_t c = 0; c < cols; ++c) {
      const float x = load_elem(src, src_dt, t * cols + c) * inv[c];
      dst[t * cols + c] = fp8_encode(x * s, fmt);
    }
  return 0;
}

// Melded forward GEMM (Eq. o_split, Alg. 2): O_merged = W~' x~ / (s_W s_x).
// Computes the outputs for tokens tsel[0..nt) x merged features fsel[0..nf)
// (feature index i < m is O, i >= m is O_A); a null selection means "all".
//   out[a*nf + b] = sum_c dec(xq[t_a][c]) * dec(wq[i_b][c]) / ((double)s_w * (double)s_x)
// Scales: per tensor, s_w[0] serves every row (the paper's scheme).  Per row (an extension for
// heavy-tailed backbones): s_w[i] is the scale of row i < m and s_w[m] the one scale of the A~ block.
int orc_forward_gemm(const uint8_t* xq, float s_x, const uint8_t* wq, const float* s_w, int gran,
                     int64_t T, int64_t m, int64_t n, int64_t r,
                     const int64_t* tsel, int64_t nt, const int64_t* fsel, int64_t nf, double* out) {
  const DecodeTable e4(FMT_E4M3);
  if (!tsel) nt = T;
  if (!fsel) nf = m + r;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t a = 0; a < nt; ++a) {
    for (int64_t b = 0; b < nf; ++b) {
      const int64_t t = tsel ? tsel[a] : a;
      const int64_t i = fsel ? fsel[b] : b;
      const uint8_t* xr = xq + t * n;
      const uint8_t* wr = wq + i * n;
      double acc = 0.0;
      for (int64_t c = 0; c < n; ++c) acc += e4.v[xr[c]] * e4.v[wr[c]];
      const float sw = (gran == GRAN_ROW) ? s_w[i < m ? i : m] : s_w[0];
      out[a * nf + b] = acc / ((double)sw * (double)s_x);
    }
  }
  return 0;
}

// Full forward of one layer on already-quantized activations: splits O_merged
// into Y[T][m] (double) and the saved O_A[T][r] (rounded once to fp32), and
// reports amax(O_A) over the fp32 values.
int orc_forward(const uint8_t* xq, float s_x, const uint8_t* wq, const float* s_w, int gran,
                int64_t T, int64_t m, int64_t n, int64_t r, double* Y, float* OA, float* amax_oa) {
  std::vector<double> merged((size_t)T * (size_t)(m + r));
  orc_forward_gemm(xq, s_x, wq, s_w, gran, T, m, n, r, nullptr, 0, nullptr, 0, merged.data());
  float amax = 0.0f;
  for (int64_t t = 0; t < T; ++t) {
    for (int64_t i = 0; i < m; ++i) Y[t * m + i] = merged[t * (m + r) + i];
    for (int64_t j = 0; j < r; ++j) {
      const float v = (float)merged[t * (m + r) + m + j];
      OA[t * r + j] = v;
      amax = std::max(amax, std::fabs(v));
    }
  }
  if (amax_oa) *amax_oa = amax;
  return 0;
}

// Input gradient (backprop through O = W~ x~ / (s_W s_x) with E5M2 output
// gradients; only the first m rows of W~' carry gradient to x):
//   dX[t][c] = sum_{i<m} dec5(gq[t][i]) * dec4(wq[i][c]) / ((double)s_w * (double)s_g)
// for tokens tsel x input channels csel (null = all).
// Per-row scales sit on the contraction axis here, so in that mode they were divided out of dY before its
// E5M2 cast (see orc_quantize_colscaled) and only s_g remains: dX = sum_i dec5(gq) dec4(wq) / s_g.
int orc_dx_gemm(const uint8_t* gq, float s_g, const uint8_t* wq, const float* s_w, int gran,
                int64_t T, int64_t m, int64_t n,
                const int64_t* tsel, int64_t nt, const int64_t* csel, int64_t nc, double* out) {
  const DecodeTable e4(FMT_E4M3), e5(FMT_E5M2);
  if (!tsel) nt = T;
  if (!csel) nc = n;
  const double d = (gran == GRAN_ROW) ? (double)s_g : (double)s_w[0] * (double)s_g;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t a = 0; a < nt; ++a) {
    for (int64_t b = 0; b < nc; ++b) {
      const int64_t t = tsel ? tsel[a] : a;
      const int64_t c = csel ? csel[b] : b;
      double acc = 0.0;
      for (int64_t i = 0; i < m; ++i) acc += e5.v[gq[t * m + i]] * e4.v[wq[i * n + c]];
      out[a * nc + b] = acc / d;
    }
  }
  return 0;
}

// Reformulated adapter gradient (Eq. lora_backward_modified, Alg. 3 line 3):
//   dB[i][j] = sum_t dec5(gq[t][i]) * dec4(oaq[t][j]) / ((double)s_g * (double)s_oa)
// for rows isel (null = all m rows), all r columns.  row_scale (nullable): in the per-row mode gq carries
// dY / s_w[i], so row i of the result is multiplied back by s_w[i].
int orc_db_gemm(const uint8_t* gq, float s_g, const uint8_t* oaq, float s_oa, const float* row_scale,
                int64_t T, int64_t m, int64_t r, const int64_t* isel, int64_t ni, double* out) {
  const DecodeTable e4(FMT_E4M3), e5(FMT_E5M2);
  if (!isel) ni = m;
  const double d = (double)s_g * (double)s_oa;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t a = 0; a < ni; ++a) {
    for (int64_t j = 0; j < r; ++j) {
      const int64_t i = isel ? isel[a] : a;
      double acc = 0.0;
      for (int64_t t = 0; t < T; ++t) acc += e5.v[gq[t * m + i]] * e4.v[oaq[t * r + j]];
      out[a * r + j] = row_scale ? (acc / d) * (double)row_scale[i] : acc / d;
    }
  }
  return 0;
}

// Row-wise proxy update (Alg. 3 lines 4-6, Eq. update), per-tensor scale.
//   1. optimizer (plain SGD form): dbuf = fma(-lr, dB, dbuf)            (skipped when dB is null)
//   2. score_i = ((|d_i0| + |d_i1|) + |d_i2|) + ...   fp32, ascending j
//   3. idx = the k rows with the largest score, ties to the lowest index, returned ascending
//   4. for each selected row i, column c:  v = dec(W~[i][c]);  v = fma(dbuf[i][j], dec(A~[j][c]), v), j ascending;
//      W~[i][c] = encode_e4m3(v)  -- the scale s_W cancels because A~ carries it (Eq. A_integ)
//   5. the merged rows of dbuf are cleared (their change now lives in W~)
// score_out (nullable) receives all m scores; idx_out (nullable) the k indices.
// row_scales (nullable, m+1 entries): per-row mode.  The merge then works in row i's own scaled domain, where
// A~ (scaled by s_w[m]) enters with the coefficient c_i = s_w[i] / s_w[m] (one fp32 division), applied to the
// DeltaBuffer entry as its own rounded multiply before the chain.
static int proxy_update_impl(uint8_t* wq, float* dbuf, const float* dB, float lr, const float* row_scales,
                             int64_t m, int64_t n, int64_t r, int64_t k, int32_t* idx_out, float* score_out,
                             bool exact_merge) {
  if (k < 0 || k > m) return -1;
  const DecodeTable e4(FMT_E4M3);
  if (dB) {
    const float neg_lr = -lr;
    for (int64_t e = 0; e < m * r; ++e) dbuf[e] = std::fmaf(neg_lr, dB[e], dbuf[e]);
  }
  std::vector<float> score((size_t)m);
  for (int64_t i = 0; i < m; ++i) {
    float s = 0.0f;
    for (int64_t j = 0; j < r; ++j) s = s + std::fabs(dbuf[i * r + j]);
    score[i] = s;
  }
  if (score_out) std::copy(score.begin(), score.end(), score_out);
  std::vector<int64_t> order((size_t)m);
  std::iota(order.begin(), order.end(), (int64_t)0);
  std::stable_sort(order.begin(), order.end(),
                   [&](int64_t a, int64_t b) { return score[a] > score[b]; });  // stable: equal scores keep index order
  std::vector<int64_t> sel(order.begin(), order.begin() + k);
  std::sort(sel.begin(), sel.end());
  const uint8_t* aq = wq + m * n;  // rows m..m+r-1 of W~' are A~
#pragma omp parallel for schedule(static)
  for (int64_t s = 0; s < k; ++s) {
    const int64_t i = sel[s];
    const float coef = row_scales ? row_scales[i] / row_scales[m] : 1.0f;
    for (int64_t c = 0; c < n; ++c) {
      if (exact_merge) {   // one rounding of the exact sum (the coefficient is still its own rounded fp32 multiply)
        ExactSum acc;
        acc.add_code_value((int32_t)std::lrint(e4.v[wq[i * n + c]] * 512.0));
        for (int64_t j = 0; j < r; ++j) {
          const float d = row_scales ? dbuf[i * r + j] * coef : dbuf[i * r + j];
          acc.add_product(d, (int32_t)std::lrint(e4.v[aq[j * n + c]] * 512.0));
        }
        wq[i * n + c] = acc.round_to_e4m3();
        continue;
      }
      float v = (float)e4.v[wq[i * n + c]];
      for (int64_t j = 0; j < r; ++j) {
        const float d = row_scales ? dbuf[i * r + j] * coef : dbuf[i * r + j];
        v = std::fmaf(d, (float)e4.v[aq[j * n + c]], v);
      }
      wq[i * n + c] = fp8_encode(v, FMT_E4M3);
    }
  }
  for (int64_t s = 0; s < k; ++s) {
    for (int64_t j = 0; j < r; ++j) dbuf[sel[s] * r + j] = 0.0f;
    if (idx_out) idx_out[s] = (int32_t)sel[s];
  }
  return 0;
}

int orc_proxy_update(uint8_t* wq, float* dbuf, const float* dB, float lr, const float* row_scales,
                     int64_t m, int64_t n, int64_t r, int64_t k, int32_t* idx_out, float* score_out) {
  return proxy_update_impl(wq, dbuf, dB, lr, row_scales, m, n, r, k, idx_out, score_out, false);
}

// The same update with the correctly rounded merge: W~[i][c] <- sat_rne_e4m3(W~[i][c] + sum_j d'_ij * A~[j][c]) where
// the sum is exact and rounded once (d'_ij = DeltaBuffer entry, times the row coefficient as its own fp32 multiply
// in per-row mode).  Steps 1-3 and 5 are unchanged.
int orc_proxy_update_exact(uint8_t* wq, float* dbuf, const float* dB, float lr, const float* row_scales,
                           int64_t m, int64_t n, int64_t r, int64_t k, int32_t* idx_out, float* score_out) {
  return proxy_update_impl(wq, dbuf, dB, lr, row_scales, m, n, r, k, idx_out, score_out, true);
}

// One exactly rounded dot product, for pins: code of sat_rne_e4m3(dec(w) + sum_j d[j] * dec(a[j])).
uint8_t orc_exact_merge_element(uint8_t w, const float* d, const uint8_t* a, int64_t r) {
  const DecodeTable e4(FMT_E4M3);
  ExactSum acc;
  acc.add_code_value((int32_t)std::lrint(e4.v[w] * 512.0));
  for (int64_t j = 0; j < r; ++j) acc.add_product(d[j], (int32_t)std::lrint(e4.v[a[j]] * 512.0));
  return acc.round_to_e4m3();
}

// AdamW on the DeltaBuffer (the optimizer the paper trains with; Alg. 3 line 4 leaves "Optimizer" generic).
// One step t >= 1 for every element, all in fp32 in this order (decoupled weight decay first):
//   p  = p * decay                          decay     = (float)(1 - lr*wd)
//   m  = fma(beta1, m, (1-beta1) * g)
//   v  = fma(beta2, v, (1-beta2) * (g*g))
//   p  = fma(-step_size, m / (sqrt(v) / sqrt_bc2 + eps), p)
//                                           step_size = (float)(lr / (1 - beta1^t)),  sqrt_bc2 = (float)sqrt(1 - beta2^t)
// The three derived constants are evaluated in double and rounded once to fp32.
void orc_adamw_constants(float lr, float beta1, float beta2, float weight_decay, int64_t step, float* decay,
                         float* one_minus_b1, float* one_minus_b2, float* step_size, float* sqrt_bc2) {
  *decay = (float)(1.0 - (double)lr * (double)weight_decay);
  *one_minus_b1 = (float)(1.0 - (double)beta1);
  *one_minus_b2 = (float)(1.0 - (double)beta2);
  *step_size = (float)((double)lr / (1.0 - std::pow((double)beta1, (double)step)));
  *sqrt_bc2 = (float)std::sqrt(1.0 - std::pow((double)beta2, (double)step));
}

int orc_adamw_step(float* p, const float* g, float* exp_avg, float* exp_avg_sq, int64_t count, float lr, float beta1,
                   float beta2, float eps, float weight_decay, int64_t step) {
  if (step < 1) return -1;
  float decay, omb1, omb2, step_size, sqrt_bc2;
  orc_adamw_constants(lr, beta1, beta2, weight_decay, step, &decay, &omb1, &omb2, &step_size, &sqrt_bc2);
  for (int64_t e = 0; e < count; ++e) {
    const float gi = g[e];
    const float p1 = p[e] * decay;
    const float m1 = std::fmaf(beta1, exp_avg[e], omb1 * gi);
    const float g2 = gi * gi;
    const float v1 = std::fmaf(beta2, exp_avg_sq[e], omb2 * g2);
    const float denom = std::sqrt(v1) / sqrt_bc2 + eps;
    p[e] = std::fmaf(-step_size, m1 / denom, p1);
    exp_avg[e] = m1;
    exp_avg_sq[e] = v1;
  }
  return 0;
}

// ---- "update A" variant (the paper's ablation with a trainable A: dL/dA = B^T dL/dO x^T).
// A plain product of two matrices of FP8 codes, both stored with the contraction index innermost, in double:
//   out[i][j] = sum_k dec_a(a[i][k]) * dec_b(b[j][k]) / (s_a * s_b)
int orc_codes_gemm(const uint8_t* a, int fmt_a, float s_a, const uint8_t* b, int fmt_b, float s_b, int64_t M, int64_t N,
                   int64_t K, double* out) {
  if (M < 0 || N < 0 || K < 0) return -1;
  const DecodeTable ta(fmt_a), tb(fmt_b);
  const double d = (double)s_a * (double)s_b;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t i = 0; i < M; ++i) {
    for (int64_t j = 0; j < N; ++j) {
      double acc = 0.0;
      for (int64_t k = 0; k < K; ++k) acc += ta.v[a[i * K + k]] * tb.v[b[j * K + k]];
      out[i * N + j] = acc / d;
    }
  }
  return 0;
}

// Plain SGD on an fp32 tensor: p[e] = fma(-lr, g[e], p[e]), one rounding per element.
int orc_sgd_step(float* p, const float* g, float lr, int64_t count) {
  for (int64_t e = 0; e < count; ++e) p[e] = std::fmaf(-lr, g[e], p[e]);
  return 0;
}

int orc_num_threads(void) {
  int nthreads = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp single
    nthreads = omp_get_num_threads();
  }
#endif
  return nthreads;
}

}  // extern "C"
