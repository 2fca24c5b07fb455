// The "update A" variant (the paper's appendix ablation with a trainable A):  dL/dA = B^T dL/dO x^T, evaluated in the
// layer's FP8 scheme and followed by a plain SGD step on an fp32 master copy of A and the re-creation of the A~ rows of
// the melded backbone (Eq. A_integ).  Composed from the library's own kernels -- per-tensor casts (written transposed,
// as the O_A cast is), the tensor-core product for P = dY B, the adapter-gradient kernel for dA^T = x~^T P~ -- plus one
// small kernel for the transposed fma step.  The paper shows this variant is slower and no better; it is not on the
// default path.
#include "../../include/falqon.h"
#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

__global__ void __launch_bounds__(256) sgd_step_transposed_kernel(float* p, const float* g_t, float neg_lr, int rows, int cols) {
  pdl_trigger();
  pdl_wait();
  // a 32 x 32 tile of p per iteration, the gradient read through shared memory so that both sides are coalesced
  __shared__ float tile[32][33];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
  const int col_tiles = (cols + 31) / 32, row_tiles = (rows + 31) / 32;
  for (int t = blockIdx.x; t < col_tiles * row_tiles; t += gridDim.x) {
    const int c0 = (t / row_tiles) * 32, j0 = (t % row_tiles) * 32;
    for (int i = ty; i < 32; i += 8) {          // g_t[c0 + i][j0 + tx]
      const int c = c0 + i, j = j0 + tx;
      tile[i][tx] = (c < cols && j < rows) ? ld_stream(g_t + static_cast<long long>(c) * rows + j) : 0.0f;
    }
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {          // p[j0 + i][c0 + tx]
      const int j = j0 + i, c = c0 + tx;
      if (j < rows && c < cols) {
        float* dst = p + static_cast<long long>(j) * cols + c;
        *dst = __fmaf_rn(neg_lr, tile[tx][i], *dst);
      }
    }
    __syncthreads();
  }
}

struct UaLayout {
  size_t scalars, bq_t, p, pq_t, da_t, total;
  size_t bq_t_bytes, p_bytes, pq_t_bytes, da_t_bytes;
  int64_t r16, t16;
};
constexpr size_t kUaHeaderBytes = 8192;     // floats 0 amax(B) 1 s_B 2 amax(P) 3 s_P; absmax partials from byte 1024
constexpr size_t kUaPartialsOffset = 1024;
static_assert(kUaPartialsOffset + kMaxAbsmaxParts * sizeof(uint32_t) <= kUaHeaderBytes, "header too small");

bool ua_layout(int64_t m, int64_t n, int64_t r, int64_t T, UaLayout* u) {
  if (m < 16 || n < 16 || m % 16 || n % 16 || r < 8 || r > 256 || r % 8 || T < 1 || m >= (1ll << 30) || n >= (1ll << 30) ||
      T >= (1ll << 30))
    return false;
  u->r16 = round_up(r, 16);
  u->t16 = round_up(T, 16);
  u->bq_t_bytes = static_cast<size_t>(u->r16) * m;
  u->p_bytes = static_cast<size_t>(T) * r * sizeof(float);
  u->pq_t_bytes = static_cast<size_t>(u->r16) * u->t16;
  u->da_t_bytes = static_cast<size_t>(n) * r * sizeof(float);
  size_t off = 0;
  u->scalars = off; off += kUaHeaderBytes;
  u->bq_t = off; off += round_up(u->bq_t_bytes, 1024);
  u->p = off; off += round_up(u->p_bytes, 1024);
  u->pq_t = off; off += round_up(u->pq_t_bytes, 1024);
  u->da_t = off; off += round_up(u->da_t_bytes, 1024);
  u->total = off;
  return true;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace

cudaError_t launch_sgd_step_transposed(float* p, const float* g_t, float lr, int64_t rows, int64_t cols, cudaStream_t stream) {
  const int64_t tiles = ((rows + 31) / 32) * ((cols + 31) / 32);
  const int grid = static_cast<int>(tiles < 148 * 8 ? tiles : 148 * 8);
  return launch_pdl(sgd_step_transposed_kernel, dim3(grid), dim3(256), 0, stream, 1, p, g_t, -lr, static_cast<int>(rows),
                    static_cast<int>(cols));
}

}  // namespace falqon

using namespace falqon;

extern "C" {

size_t falqon_update_a_scratch_bytes(int64_t m, int64_t n, int64_t r, int64_t T) {
  UaLayout u;
  return ua_layout(m, n, r, T, &u) ? u.total : 0;
}

int falqon_update_a_region(int64_t m, int64_t n, int64_t r, int64_t T, falqon_ua_region which, size_t* offset, size_t* bytes) {
  UaLayout u;
  if (offset == nullptr || bytes == nullptr || !ua_layout(m, n, r, T, &u)) return FALQON_ERR_INVALID_ARG;
  switch (which) {
    case FALQON_UA_SCALARS: *offset = u.scalars; *bytes = 4 * sizeof(float); break;
    case FALQON_UA_BQ_T: *offset = u.bq_t; *bytes = u.bq_t_bytes; break;
    case FALQON_UA_P: *offset = u.p; *bytes = u.p_bytes; break;
    case FALQON_UA_PQ_T: *offset = u.pq_t; *bytes = u.pq_t_bytes; break;
    case FALQON_UA_DA_T: *offset = u.da_t; *bytes = u.da_t_bytes; break;
    default: return FALQON_ERR_INVALID_ARG;
  }
  return FALQON_OK;
}

int falqon_update_a(const falqon_layer* L, const uint8_t* xq, const float* s_x, const float* B, float* A_master, float gamma,
                    float lr, int64_t T, void* ws, size_t ws_bytes, void* scratch, size_t scratch_bytes, falqon_stream stream) {
  if (L == nullptr || L->wq == nullptr || L->s_w == nullptr || xq == nullptr || s_x == nullptr || B == nullptr ||
      A_master == nullptr || !aligned16(L->wq) || !aligned16(xq) || !aligned16(B) || !aligned16(A_master) || !(gamma == gamma) ||
      !(lr == lr) || (L->flags & ~(FALQON_LAYER_FUSED_CAST | FALQON_LAYER_EMIT_XQ)) != 0)
    return FALQON_ERR_INVALID_ARG;
  if (L->gran != FALQON_PER_TENSOR) return FALQON_ERR_UNSUPPORTED;
  UaLayout u;
  if (!ua_layout(L->m, L->n, L->r, T, &u)) return FALQON_ERR_INVALID_ARG;
  const size_t ws_need = falqon_workspace_bytes(L->m, L->n, L->r, T);
  if (ws == nullptr || !aligned16(ws) || ws_need == 0 || ws_bytes < ws_need) return FALQON_ERR_WORKSPACE;
  if (scratch == nullptr || !aligned16(scratch) || scratch_bytes < u.total) return FALQON_ERR_WORKSPACE;
  size_t gq_off = 0, gq_bytes = 0, sc_off = 0, sc_bytes = 0;
  if (falqon_workspace_region(L->m, L->n, L->r, T, FALQON_WS_GQ, &gq_off, &gq_bytes) != FALQON_OK ||
      falqon_workspace_region(L->m, L->n, L->r, T, FALQON_WS_SCALES, &sc_off, &sc_bytes) != FALQON_OK)
    return FALQON_ERR_INVALID_ARG;
  int* status = device_status_ptr();
  if (status == nullptr) return FALQON_ERR_CUDA;
#define FALQON_UA_CUDA(expr) do { if ((expr) != cudaSuccess) return FALQON_ERR_CUDA; } while (0)
  const int64_t m = L->m, n = L->n, r = L->r;
  uint8_t* sbase = static_cast<uint8_t*>(scratch);
  float* scal = reinterpret_cast<float*>(sbase + u.scalars);
  uint32_t* partial = reinterpret_cast<uint32_t*>(sbase + kUaPartialsOffset);
  uint8_t* bq_t = sbase + u.bq_t;
  float* P = reinterpret_cast<float*>(sbase + u.p);
  uint8_t* pq_t = sbase + u.pq_t;
  float* da_t = reinterpret_cast<float*>(sbase + u.da_t);
  const uint8_t* gq = static_cast<const uint8_t*>(ws) + gq_off;
  const float* s_g = reinterpret_cast<const float*>(static_cast<const uint8_t*>(ws) + sc_off) + 3;

  // B~^T, s_B = Q_e4m3(B): the absmax, then the cast written transposed ([r][m]: the contraction index m innermost)
  FALQON_UA_CUDA(launch_absmax_value(B, kF32, m * r, partial, scal + 0, stream));
  const OaCastJob cast_b{B, scal + 0, m, static_cast<int>(r), m, bq_t, scal + 1, nullptr};
  FALQON_UA_CUDA(launch_oa_cast(cast_b, stream));
  // P = g~ B~ / (s_g s_B), [T][r] fp32, with max |P| from the epilogue
  FALQON_UA_CUDA(cudaMemsetAsync(scal + 2, 0, sizeof(float), stream));
  {
    GemmProblem g{};
    g.M = T; g.N = r; g.K = m;
    g.a = gq; g.lda = m; g.a_fmt = kE5M2;
    g.b = bq_t; g.ldb = m; g.b_mn_major = false; g.b_fmt = kE4M3;
    g.block_n = static_cast<int>(u.r16);
    g.c0 = nullptr; g.ldc0 = 0; g.c0_dt = kF32; g.n_split = 0;
    g.c1 = P; g.ldc1 = r; g.amax1_bits = reinterpret_cast<uint32_t*>(scal + 2);
    g.scale_a = s_g; g.scale_b = scal + 1;
    g.status = status;
    FALQON_UA_CUDA(launch_gemm_fp8(g, stream));
  }
  // P~^T, s_P = Q_e4m3(P), transposed ([r][T16]: the contraction index T innermost)
  const OaCastJob cast_p{P, scal + 2, T, static_cast<int>(r), u.t16, pq_t, scal + 3, nullptr};
  FALQON_UA_CUDA(launch_oa_cast(cast_p, stream));
  // dA^T = x~^T P~ / (s_x s_P), [n][r] fp32: the adapter-gradient kernel with x~ in the place of g~
  {
    DbFusedProblem d{};
    d.m = n; d.r = r; d.T = T;
    d.gq = xq; d.g_is_e4m3 = true; d.oaq_t = pq_t; d.ldt = u.t16; d.s_oa = scal + 3; d.s_g = s_x;
    d.dB = da_t; d.status = status;
    FALQON_UA_CUDA(launch_db_fused(d, stream));
  }
  // A <- fma(-lr, dA, A) on the master copy, then A~ = Q_e4m3(gamma A; s_W) over rows m .. m + r - 1 of the backbone
  FALQON_UA_CUDA(launch_sgd_step_transposed(A_master, da_t, lr, r, n, stream));
  FALQON_UA_CUDA(launch_cast_per_tensor(A_master, kF32, r * n, kE4M3, gamma, nullptr, 0, L->s_w, L->wq + m * n, nullptr, nullptr,
                                        nullptr, nullptr, stream));
#undef FALQON_UA_CUDA
  return FALQON_OK;
}

}  // extern "C"
