// Initialisation of the adapter from the quantization error (Alg. 1 lines 4-5; Eq. q_error, Eq. reform):
//   Delta W = W - dec(W~) / s_W,   (B^, A^) = rank-r truncated SVD of Delta W,   A^ = sqrt(S_r) V_r^T
// as a randomized subspace iteration (set-up code, off the per-step path; fp32 on the ordinary ALUs):
//   Y = E Omega;  orth(Y);  q times { Z = E^T Y; orth(Z); Y = E Z; orth(Y) };
//   C = E^T Y  (so C^T = Y^T E, l x n);  C^T C = Q Lambda Q^T;  sigma_i = sqrt(lambda_i);
//   A^_i = (C q_i)^T / sqrt(sigma_i)     (= sqrt(sigma_i) times the i-th right singular vector)
// Omega (n x l Gaussian, l = r + oversampling) is an INPUT: the caller draws it, so that a test can hand the same
// numbers to an independent implementation.  orth = Cholesky-QR applied three times, the first time with a shifted
// Gram matrix (a rapidly decaying spectrum makes the plain Gram matrix indefinite in fp32).  The l x l factorisations
// (Cholesky + triangular inverse, cyclic Jacobi eigen-decomposition) run in one CTA each, in shared memory.
#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

// ---- E = W - dec(W~) / s_W
template <int kDt>
__global__ void __launch_bounds__(256) svd_residual_kernel(const void* w, const uint8_t* wq, const float* s_w, int64_t count,
                                                           float* e) {
  pdl_trigger();
  pdl_wait();
  const float s = ld_stream(s_w);
  for (int64_t i = (blockIdx.x * 256ll + threadIdx.x) * 4; i < count; i += static_cast<int64_t>(gridDim.x) * 1024) {
    const uint32_t codes = ld_stream(reinterpret_cast<const uint32_t*>(wq + i));
    const float2 d01 = e4m3x2_to_float2(codes), d23 = e4m3x2_to_float2(codes >> 16);
    float wv[4];
    if (kDt == kBF16) {
      const uint2 raw = ld_stream(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(w) + i));
      wv[0] = __uint_as_float(raw.x << 16); wv[1] = __uint_as_float(raw.x & 0xFFFF0000u);
      wv[2] = __uint_as_float(raw.y << 16); wv[3] = __uint_as_float(raw.y & 0xFFFF0000u);
    } else {
      const float4 raw = ld_stream(reinterpret_cast<const float4*>(static_cast<const float*>(w) + i));
      wv[0] = raw.x; wv[1] = raw.y; wv[2] = raw.z; wv[3] = raw.w;
    }
    float4 out;
    out.x = wv[0] - __fdiv_rn(d01.x, s); out.y = wv[1] - __fdiv_rn(d01.y, s);
    out.z = wv[2] - __fdiv_rn(d23.x, s); out.w = wv[3] - __fdiv_rn(d23.y, s);
    *reinterpret_cast<float4*>(e + i) = out;
  }
}

// ---- C[M][N] = sum_k A(row, k) B[k][col];  A(row, k) = a[row * ars + k * aks] (so A may be a transposed view)
struct MulArgs {
  const float* a; long long ars, aks;
  const float* b; long long ldb;
  float* c; long long ldc;
  int M, N, K;
};
__global__ void __launch_bounds__(256) svd_mul_kernel(MulArgs g) {
  __shared__ float As[16][65];
  __shared__ float Bs[16][64];
  pdl_trigger();
  pdl_wait();
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < g.K; k0 += 16) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int e = tid + 256 * i;
      int row, kk;
      if (g.aks == 1) { row = e >> 4; kk = e & 15; } else { row = e & 63; kk = e >> 6; }   // contiguous along the unit stride
      const bool ok = m0 + row < g.M && k0 + kk < g.K;
      As[kk][row] = ok ? ld_stream(g.a + (m0 + row) * g.ars + (k0 + kk) * g.aks) : 0.0f;
      const int bk = e >> 6, bc = e & 63;
      const bool okb = k0 + bk < g.K && n0 + bc < g.N;
      Bs[bk][bc] = okb ? ld_stream(g.b + (k0 + bk) * g.ldb + n0 + bc) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { av[i] = As[kk][ty * 4 + i]; bv[i] = Bs[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (m0 + ty * 4 + i < g.M && n0 + tx * 4 + j < g.N) g.c[(m0 + ty * 4 + i) * g.ldc + n0 + tx * 4 + j] = acc[i][j];
}

// ---- one CTA: G (l x l, symmetric positive semi-definite) -> Rinv = R^-1 with G + shift I = R^T R, R upper triangular;
// shift = shift_rel x the largest diagonal entry (0 for a well-conditioned G).  A pivot that still comes out
// non-positive is replaced by the shift (or a tiny number): that column is then merely rescaled, not orthogonalised.
__global__ void __launch_bounds__(256) svd_chol_inv_kernel(const float* gmat, int l, float shift_rel, float* rinv) {
  extern __shared__ float sm[];
  float* R = sm;             // [l][l]
  float* X = sm + l * l;     // [l][l]
  pdl_trigger();
  pdl_wait();
  const int tid = threadIdx.x;
  __shared__ float s_shift;
  for (int e = tid; e < l * l; e += 256) { R[e] = ld_stream(gmat + e); X[e] = 0.0f; }
  __syncthreads();
  if (tid == 0) {
    float dmax = 0.0f;
    for (int i = 0; i < l; ++i) dmax = fmaxf(dmax, R[i * l + i]);
    s_shift = shift_rel * dmax;
  }
  __syncthreads();
  const float shift = s_shift;
  for (int i = tid; i < l; i += 256) R[i * l + i] += shift;
  __syncthreads();
  for (int k = 0; k < l; ++k) {     // right-looking Cholesky on the upper triangle
    float d = R[k * l + k];
    if (!(d > 0.0f)) d = fmaxf(shift, 1e-30f);
    const float inv = rsqrtf(d);
    __syncthreads();
    if (tid == 0) R[k * l + k] = d;
    __syncthreads();
    for (int j = k + tid; j < l; j += 256) R[k * l + j] *= inv;
    __syncthreads();
    for (int e = tid; e < (l - k - 1) * (l - k - 1); e += 256) {
      const int i = k + 1 + e / (l - k - 1), j = k + 1 + e % (l - k - 1);
      if (j >= i) R[i * l + j] -= R[k * l + i] * R[k * l + j];
    }
    __syncthreads();
  }
  // X = R^-1 (upper triangular), one column per thread by back substitution
  for (int j = tid; j < l; j += 256) {
    for (int i = j; i >= 0; --i) {
      float s = (i == j) ? 1.0f : 0.0f;
      for (int t = i + 1; t <= j; ++t) s -= R[i * l + t] * X[t * l + j];
      X[i * l + j] = s / R[i * l + i];
    }
  }
  __syncthreads();
  for (int e = tid; e < l * l; e += 256) rinv[e] = X[e];
}

// ---- one CTA: symmetric G (l x l, l even) -> eigenvalues (descending) and eigenvectors (columns of Q, same order)
// by cyclic Jacobi with a round-robin ordering: each step rotates l/2 disjoint index pairs at once.
__global__ void __launch_bounds__(256) svd_jacobi_kernel(const float* gmat, int l, int sweeps, float* lambda, float* q) {
  extern __shared__ float sm[];
  float* A = sm;                 // [l][l]
  float* V = sm + l * l;         // [l][l]
  __shared__ float cs[256], sn[256];
  __shared__ int pp[256], qq[256];
  __shared__ int order[512];
  pdl_trigger();
  pdl_wait();
  const int tid = threadIdx.x, half = l / 2;
  for (int e = tid; e < l * l; e += 256) { A[e] = ld_stream(gmat + e); V[e] = (e / l == e % l) ? 1.0f : 0.0f; }
  __syncthreads();
  for (int sweep = 0; sweep < sweeps; ++sweep) {
    for (int step = 0; step < l - 1; ++step) {
      if (tid < half) {   // round-robin tournament: player l-1 stays, the others rotate
        int a = (tid == 0) ? l - 1 : (step + tid) % (l - 1);
        int b = (step + l - 1 - tid) % (l - 1);
        const int p = min(a, b), r2 = max(a, b);
        const float app = A[p * l + p], aqq = A[r2 * l + r2], apq = A[p * l + r2];
        float c = 1.0f, s = 0.0f;
        if (fabsf(apq) > 1e-30f) {
          const float tau = (aqq - app) / (2.0f * apq);
          const float t = (tau >= 0.0f ? 1.0f : -1.0f) / (fabsf(tau) + sqrtf(1.0f + tau * tau));
          c = rsqrtf(1.0f + t * t);
          s = t * c;
        }
        cs[tid] = c; sn[tid] = s; pp[tid] = p; qq[tid] = r2;
      }
      __syncthreads();
      for (int e = tid; e < half * l; e += 256) {      // rows: A <- J^T A
        const int pr = e / l, j = e % l, p = pp[pr], r2 = qq[pr];
        const float c = cs[pr], s = sn[pr], ap = A[p * l + j], aq = A[r2 * l + j];
        A[p * l + j] = c * ap - s * aq;
        A[r2 * l + j] = s * ap + c * aq;
      }
      __syncthreads();
      for (int e = tid; e < half * l; e += 256) {      // columns: A <- A J, V <- V J
        const int pr = e / l, i = e % l, p = pp[pr], r2 = qq[pr];
        const float c = cs[pr], s = sn[pr];
        const float ap = A[i * l + p], aq = A[i * l + r2];
        A[i * l + p] = c * ap - s * aq;
        A[i * l + r2] = s * ap + c * aq;
        const float vp = V[i * l + p], vq = V[i * l + r2];
        V[i * l + p] = c * vp - s * vq;
        V[i * l + r2] = s * vp + c * vq;
      }
      __syncthreads();
    }
  }
  if (tid == 0) {   // order the eigenvalues, largest first (l is a few hundred at most)
    for (int i = 0; i < l; ++i) order[i] = i;
    for (int i = 0; i < l; ++i) {
      int best = i;
      for (int j = i + 1; j < l; ++j)
        if (A[order[j] * l + order[j]] > A[order[best] * l + order[best]]) best = j;
      const int t = order[i]; order[i] = order[best]; order[best] = t;
    }
  }
  __syncthreads();
  for (int e = tid; e < l * l; e += 256) q[e] = V[(e / l) * l + order[e % l]];
  for (int i = tid; i < l; i += 256) lambda[i] = A[order[i] * l + order[i]];
}

// ---- A^[i][c] = (sum_j C[c][j] Q[j][i]) / sqrt(sigma_i), sigma_i = sqrt(lambda_i), i < r
__global__ void __launch_bounds__(256) svd_finish_kernel(const float* cmat, const float* q, const float* lambda, int64_t n, int l,
                                                         int r, float* a_hat, float* sigma) {
  pdl_trigger();
  pdl_wait();
  const int64_t c = blockIdx.x * 256ll + threadIdx.x;
  const int i = blockIdx.y;
  const float sg = sqrtf(fmaxf(ld_stream(lambda + i), 0.0f));
  if (c == 0) sigma[i] = sg;
  if (c >= n) return;
  float acc = 0.0f;
  for (int j = 0; j < l; ++j) acc = fmaf(ld_stream(cmat + c * l + j), ld_stream(q + j * l + i), acc);
  a_hat[static_cast<int64_t>(i) * n + c] = sg > 0.0f ? acc * rsqrtf(sg) : 0.0f;
}

cudaError_t mul(const float* a, long long ars, long long aks, const float* b, long long ldb, float* c, long long ldc, int M, int N,
                int K, cudaStream_t stream) {
  const MulArgs g{a, ars, aks, b, ldb, c, ldc, M, N, K};
  return launch_pdl(svd_mul_kernel, dim3((N + 63) / 64, (M + 63) / 64), dim3(256), 0, stream, 1, g);
}

}  // namespace

size_t svd_init_scratch_bytes(int64_t m, int64_t n, int64_t l) {
  const int64_t big = m > n ? m : n;
  return static_cast<size_t>(round_up(m * n * 4, 1024) + 3 * round_up(big * l * 4, 1024) + 4 * round_up(l * l * 4, 1024));
}

cudaError_t launch_svd_init(const void* w, int w_dt, int64_t m, int64_t n, const uint8_t* wq, const float* s_w, int64_t r,
                            const float* omega, int64_t l, int power_iters, float* a_hat, float* sigma, void* scratch,
                            cudaStream_t stream) {
  if (l < r || l % 2 || l > 160 || r < 1 || (m * n) % 4) return cudaErrorInvalidValue;
  uint8_t* base = static_cast<uint8_t*>(scratch);
  const int64_t big = m > n ? m : n;
  float* E = reinterpret_cast<float*>(base); base += round_up(m * n * 4, 1024);
  float* P0 = reinterpret_cast<float*>(base); base += round_up(big * l * 4, 1024);
  float* P1 = reinterpret_cast<float*>(base); base += round_up(big * l * 4, 1024);
  float* P2 = reinterpret_cast<float*>(base); base += round_up(big * l * 4, 1024);
  float* G = reinterpret_cast<float*>(base); base += round_up(l * l * 4, 1024);
  float* Rinv = reinterpret_cast<float*>(base); base += round_up(l * l * 4, 1024);
  float* Q = reinterpret_cast<float*>(base); base += round_up(l * l * 4, 1024);
  float* lam = reinterpret_cast<float*>(base);
  const int L = static_cast<int>(l), M = static_cast<int>(m), N = static_cast<int>(n);
  const size_t small_smem = static_cast<size_t>(2) * l * l * sizeof(float);
  static DeviceMask configured_chol{0}, configured_jacobi{0};
  {
    cudaError_t ec = set_max_dynamic_smem(svd_chol_inv_kernel, 210 * 1024, configured_chol);
    if (ec == cudaSuccess) ec = set_max_dynamic_smem(svd_jacobi_kernel, 210 * 1024, configured_jacobi);
    if (ec != cudaSuccess) return ec;
  }
#define SVD_TRY(expr) do { cudaError_t e__ = (expr); if (e__ != cudaSuccess) return e__; } while (0)
  int64_t blocks = (m * n / 4 + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (w_dt == kBF16)
    SVD_TRY(launch_pdl(svd_residual_kernel<kBF16>, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, stream, 1, w, wq, s_w, m * n, E));
  else
    SVD_TRY(launch_pdl(svd_residual_kernel<kF32>, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, stream, 1, w, wq, s_w, m * n, E));
  // orth(X [rows][l]) in place (through a second buffer): Cholesky-QR three times, the first with a shift
  auto orth = [&](float*& x, float*& tmp, int rows) -> cudaError_t {
    for (int pass = 0; pass < 3; ++pass) {
      SVD_TRY(mul(x, 1, l, x, l, G, l, L, L, rows, stream));                       // G = X^T X
      SVD_TRY(launch_pdl(svd_chol_inv_kernel, dim3(1), dim3(256), small_smem, stream, 1, static_cast<const float*>(G), L,
                         pass == 0 ? 1.0e-5f : 0.0f, Rinv));
      SVD_TRY(mul(x, l, 1, Rinv, l, tmp, l, rows, L, L, stream));                  // X <- X R^-1
      float* t = x; x = tmp; tmp = t;
    }
    return cudaSuccess;
  };
  float* Y = P0; float* Z = P1; float* T = P2;
  SVD_TRY(mul(E, n, 1, omega, l, Y, l, M, L, N, stream));                           // Y = E Omega
  SVD_TRY(orth(Y, T, M));
  for (int it = 0; it < power_iters; ++it) {
    SVD_TRY(mul(E, 1, n, Y, l, Z, l, N, L, M, stream));                             // Z = E^T Y
    SVD_TRY(orth(Z, T, N));
    SVD_TRY(mul(E, n, 1, Z, l, Y, l, M, L, N, stream));                             // Y = E Z
    SVD_TRY(orth(Y, T, M));
  }
  SVD_TRY(mul(E, 1, n, Y, l, Z, l, N, L, M, stream));                               // C = E^T Y  (n x l)
  SVD_TRY(mul(Z, 1, l, Z, l, G, l, L, L, N, stream));                               // G = C^T C
  SVD_TRY(launch_pdl(svd_jacobi_kernel, dim3(1), dim3(256), small_smem, stream, 1, static_cast<const float*>(G), L, 12, lam, Q));
  SVD_TRY(launch_pdl(svd_finish_kernel, dim3(static_cast<unsigned>((n + 255) / 256), static_cast<unsigned>(r)), dim3(256), 0, stream,
                     1, static_cast<const float*>(Z), static_cast<const float*>(Q), static_cast<const float*>(lam), n, L,
                     static_cast<int>(r), a_hat, sigma));
#undef SVD_TRY
  return cudaSuccess;
}

}  // namespace falqon
