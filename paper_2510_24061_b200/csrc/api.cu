// The C ABI of libfalqon (see include/falqon.h): argument validation, workspace layout, and the
// sequence of kernel launches behind each entry point.  No device memory is allocated here.
#include <cstring>

#include "../../include/falqon.h"
#include "internal.h"

namespace falqon {
namespace {

__device__ int g_status_word;  // written by kernels whose bounded waits run out

int* status_ptr() {   // of the current device; host threads may race here: every racer looks up and stores the same address
  static std::atomic<int*> ptrs[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  int* cached = ptrs[dev].load(std::memory_order_acquire);
  if (cached == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
    cached = static_cast<int*>(p);
    ptrs[dev].store(cached, std::memory_order_release);
  }
  return cached;
}

}  // namespace
int* device_status_ptr() { return status_ptr(); }
namespace {

struct WorkspaceLayout {
  size_t scales, act8, oaq_t, score, sel_idx, inv_sw, col_scale, total;
  size_t act8_bytes, oaq_t_bytes, score_bytes, sel_idx_bytes, inv_sw_bytes, col_scale_bytes;
  int64_t inv_sw_len, col_scale_len;   // table lengths, padded to a multiple of 32 (+32) so vector reads stay inside
  int64_t r16, t16;
};

constexpr size_t kHeaderBytes = 8192;     // scales at 0, absmax partials at kPartialsOffset
constexpr size_t kPartialsOffset = 1024;
constexpr size_t kSyncOffset = 256;       // counters of the in-kernel barriers: zero between calls (falqon_workspace_init)
constexpr size_t kDoneOffset = 320;       // last-CTA counter of the fused optimizer/score/selection kernel
constexpr size_t kGroupCountersOffset = 6144;   // row-group counters of the merge (2 KB: up to 512 groups of 32 rows)
constexpr size_t kMaxMergeGroups = (kHeaderBytes - kGroupCountersOffset) / sizeof(unsigned int);
constexpr size_t kInitBytes = kHeaderBytes;  // what falqon_workspace_init clears
static_assert(kPartialsOffset + kMaxAbsmaxParts * sizeof(uint32_t) <= kHeaderBytes, "header too small");

bool shape_ok(int64_t m, int64_t n, int64_t r) {
  return m >= 16 && n >= 16 && m % 16 == 0 && n % 16 == 0 && r >= 8 && r <= 256 && r % 8 == 0 &&
         m < (1ll << 30) && n < (1ll << 30);
}

bool make_layout(int64_t m, int64_t n, int64_t r, int64_t T, WorkspaceLayout* w) {
  if (!shape_ok(m, n, r) || T < 1 || T >= (1ll << 30)) return false;
  w->r16 = round_up(r, 16);
  w->t16 = round_up(T, 16);
  w->act8_bytes = static_cast<size_t>(T) * static_cast<size_t>(m > n ? m : n);
  w->oaq_t_bytes = static_cast<size_t>(w->r16) * static_cast<size_t>(w->t16);
  w->score_bytes = static_cast<size_t>(m) * sizeof(float);
  w->sel_idx_bytes = static_cast<size_t>(m) * sizeof(int32_t);
  w->inv_sw_len = round_up(m, 32) + 32;
  w->col_scale_len = round_up(m + r, 32) + 32;
  w->inv_sw_bytes = static_cast<size_t>(w->inv_sw_len) * sizeof(float);
  w->col_scale_bytes = static_cast<size_t>(w->col_scale_len) * sizeof(float);
  size_t off = 0;
  w->scales = off; off += kHeaderBytes;
  w->score = off; off += round_up(w->score_bytes, 1024);      // token-independent regions first, so the
  w->sel_idx = off; off += round_up(w->sel_idx_bytes, 1024);  // proxy update finds them for any T_max
  w->inv_sw = off; off += round_up(w->inv_sw_bytes, 1024);        // per-row mode: 1/s_w[i]
  w->col_scale = off; off += round_up(w->col_scale_bytes, 1024);  // per-row mode: 1/(s_w[c] s_x)
  w->act8 = off; off += round_up(w->act8_bytes, 1024);
  w->oaq_t = off; off += round_up(w->oaq_t_bytes, 1024);
  w->total = off;
  return true;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
inline bool dtype_ok(int dt) { return dt == FALQON_BF16 || dt == FALQON_F32; }

bool layer_ok(const falqon_layer* L) {
  return L != nullptr && shape_ok(L->m, L->n, L->r) && L->wq != nullptr && L->s_w != nullptr && L->dbuf != nullptr &&
         aligned16(L->wq) && aligned16(L->dbuf) && (L->gran == FALQON_PER_TENSOR || L->gran == FALQON_PER_ROW) &&
         (L->flags & ~(FALQON_LAYER_FUSED_CAST | FALQON_LAYER_EMIT_XQ | FALQON_LAYER_DB_OWN_KERNEL)) == 0;
}

#define FALQON_CUDA(expr)                                   \
  do {                                                      \
    cudaError_t e__ = (expr);                               \
    if (e__ != cudaSuccess) return FALQON_ERR_CUDA;         \
  } while (0)

// ---- optional per-stage timing (host-side CUDA events owned by the library; off by default)
struct ProfileState {
  bool active = false;
  unsigned mask = 0;
  int capacity = 0, used = 0;
  cudaEvent_t* start = nullptr;
  cudaEvent_t* stop = nullptr;
  int* kind = nullptr;
};
ProfileState g_prof;

struct StageTimer {
  int slot = -1;
  cudaStream_t stream;
  StageTimer(int kind, cudaStream_t s) : stream(s) {
    if (g_prof.active && ((g_prof.mask >> kind) & 1u) && g_prof.used < g_prof.capacity) {
      slot = g_prof.used++;
      g_prof.kind[slot] = kind;
      cudaEventRecord(g_prof.start[slot], stream);
    }
  }
  ~StageTimer() {
    if (slot >= 0) cudaEventRecord(g_prof.stop[slot], stream);
  }
};

// S2: [Y | O_A] = x~ W~'^T / (s_W s_x), amax(O_A) from the epilogue (which accumulates into *amax_oa: zero beforehand)
int forward_product(const falqon_layer* L, const uint8_t* xq, const float* s_x, int64_t T, void* Y, int y_dt, float* OA,
                    float* amax_oa, uint8_t* base, const WorkspaceLayout& w, int* status, cudaStream_t stream,
                    const FusedOperand* fused = nullptr) {
  const int64_t m = L->m, n = L->n, r = L->r;
  const bool per_row = L->gran == FALQON_PER_ROW;
  float* col_scale = reinterpret_cast<float*>(base + w.col_scale);
  if (per_row)   // epilogue factors 1 / (s_w[column] * s_x); s_w[m] serves the O_A columns
    FALQON_CUDA(launch_scale_table(1, L->s_w, m, r, s_x, col_scale, w.col_scale_len, stream));
  GemmProblem g{};
  g.M = T; g.N = m + r; g.K = n;
  g.a = xq; g.lda = n; g.a_fmt = kE4M3;
  g.b = L->wq; g.ldb = n; g.b_mn_major = false; g.b_fmt = kE4M3;
  g.block_n = 256;
  g.c0 = Y; g.ldc0 = m; g.c0_dt = y_dt; g.n_split = m;
  g.c1 = OA; g.ldc1 = r; g.amax1_bits = reinterpret_cast<uint32_t*>(amax_oa);
  g.scale_a = per_row ? nullptr : s_x; g.scale_b = per_row ? nullptr : L->s_w;
  g.col_scale = per_row ? col_scale : nullptr;
  g.status = status;
  StageTimer timer(FALQON_STAGE_GEMM_FWD, stream);
  if (fused != nullptr) FALQON_CUDA(launch_gemm_fp8_fused(g, *fused, stream));
  else FALQON_CUDA(launch_gemm_fp8(g, stream));
  return FALQON_OK;
}

// The product shapes of a layer that the fused kernel takes (see FALQON_LAYER_FUSED_CAST).
bool fused_forward_ok(const falqon_layer* L, int x_dt) {
  return (L->flags & FALQON_LAYER_FUSED_CAST) != 0 && x_dt == FALQON_BF16 && (L->m + L->r) % 16 == 0;
}
bool fused_backward_ok(const falqon_layer* L, int dy_dt, const void* dX) {
  return (L->flags & FALQON_LAYER_FUSED_CAST) != 0 && dy_dt == FALQON_BF16 && L->gran == FALQON_PER_TENSOR && dX != nullptr;
}

}  // namespace
}  // namespace falqon

using namespace falqon;

extern "C" {

size_t falqon_workspace_bytes(int64_t m, int64_t n, int64_t r, int64_t T_max) {
  WorkspaceLayout w;
  if (!make_layout(m, n, r, T_max, &w)) return 0;
  return w.total;
}

int falqon_workspace_region(int64_t m, int64_t n, int64_t r, int64_t T_max, falqon_ws_region which, size_t* offset,
                            size_t* bytes) {
  WorkspaceLayout w;
  if (offset == nullptr || bytes == nullptr || !make_layout(m, n, r, T_max, &w)) return FALQON_ERR_INVALID_ARG;
  switch (which) {
    case FALQON_WS_XQ: *offset = w.act8; *bytes = static_cast<size_t>(T_max) * n; break;
    case FALQON_WS_GQ: *offset = w.act8; *bytes = static_cast<size_t>(T_max) * m; break;
    case FALQON_WS_OAQ_T: *offset = w.oaq_t; *bytes = w.oaq_t_bytes; break;
    case FALQON_WS_SCALES: *offset = w.scales; *bytes = 8 * sizeof(float); break;
    case FALQON_WS_SCORE: *offset = w.score; *bytes = w.score_bytes; break;
    default: return FALQON_ERR_INVALID_ARG;
  }
  return FALQON_OK;
}

int falqon_quantize(const void* src, falqon_dtype src_dt, int64_t rows, int64_t cols, falqon_fp8 fmt, falqon_gran gran,
                    const float* scale_in, float premul, uint8_t* dst, float* scale_out, float* amax_out, void* ws,
                    size_t ws_bytes, falqon_stream stream) {
  if (src == nullptr || dst == nullptr || rows < 1 || cols < 16 || cols % 16 != 0 || !dtype_ok(src_dt) ||
      (fmt != FALQON_E4M3 && fmt != FALQON_E5M2) || (gran != FALQON_PER_TENSOR && gran != FALQON_PER_ROW) ||
      !aligned16(src) || !aligned16(dst) || !(premul == premul) || rows * cols >= (1ll << 40))
    return FALQON_ERR_INVALID_ARG;
  if (scale_in == nullptr && scale_out == nullptr) return FALQON_ERR_INVALID_ARG;
  if (gran == FALQON_PER_ROW) {
    if (rows >= (1ll << 31)) return FALQON_ERR_INVALID_ARG;
    FALQON_CUDA(launch_quantize_per_row(src, src_dt, rows, cols, fmt, premul, scale_in, dst, scale_out, amax_out, stream));
    return FALQON_OK;
  }
  const int64_t count = rows * cols;
  int nparts = 0;
  if (scale_in != nullptr && amax_out == nullptr) {
    FALQON_CUDA(launch_cast_per_tensor(src, src_dt, count, fmt, premul, nullptr, 0, scale_in, dst, scale_out, nullptr,
                                       nullptr, nullptr, stream));
    return FALQON_OK;
  }
  if (ws == nullptr || ws_bytes < FALQON_QUANTIZE_WS_BYTES || !aligned16(ws)) return FALQON_ERR_WORKSPACE;
  uint32_t* partial = static_cast<uint32_t*>(ws);
  FALQON_CUDA(launch_absmax(src, src_dt, count, premul, partial, &nparts, stream));
  if (scale_in != nullptr) {
    // given scale, but the caller also wants the absmax: a cast from the partials yields it; then the real cast
    FALQON_CUDA(launch_cast_per_tensor(src, src_dt, count, fmt, premul, partial, nparts, nullptr, dst, nullptr, nullptr,
                                       amax_out, nullptr, stream));
    FALQON_CUDA(launch_cast_per_tensor(src, src_dt, count, fmt, premul, nullptr, 0, scale_in, dst, scale_out, nullptr,
                                       nullptr, nullptr, stream));
    return FALQON_OK;
  }
  FALQON_CUDA(launch_cast_per_tensor(src, src_dt, count, fmt, premul, partial, nparts, nullptr, dst, scale_out, nullptr,
                                     amax_out, nullptr, stream));
  return FALQON_OK;
}

int falqon_absmax(const void* src, falqon_dtype src_dt, int64_t count, float* amax_out, void* ws, size_t ws_bytes,
                  falqon_stream stream) {
  if (src == nullptr || amax_out == nullptr || count < 1 || count >= (1ll << 40) || !dtype_ok(src_dt) || !aligned16(src))
    return FALQON_ERR_INVALID_ARG;
  if (ws == nullptr || ws_bytes < FALQON_QUANTIZE_WS_BYTES || !aligned16(ws)) return FALQON_ERR_WORKSPACE;
  FALQON_CUDA(launch_absmax_value(src, src_dt, count, static_cast<uint32_t*>(ws), amax_out, stream));
  return FALQON_OK;
}

int falqon_workspace_init(void* ws, size_t ws_bytes, falqon_stream stream) {
  if (ws == nullptr || !aligned16(ws) || ws_bytes < kInitBytes) return FALQON_ERR_WORKSPACE;
  FALQON_CUDA(cudaMemsetAsync(ws, 0, kInitBytes, stream));
  return FALQON_OK;
}

namespace {
// amax_x (nullable, device [1]): the caller already knows max |X| (the kernel that produced X took it), so the cast is a
// single pass with no reduction and no grid barrier.
// dump_block >= 0: the debug hook (fused path required; that column block writes its staged codes to FALQON_WS_XQ).
int forward_impl(const falqon_layer* L, const void* X, falqon_dtype x_dt, const float* amax_x, int64_t T, void* Y,
                 falqon_dtype y_dt, float* OA, float* amax_oa, float* s_x_out, void* ws, size_t ws_bytes, falqon_stream stream,
                 int dump_block = -1) {
  if (!layer_ok(L) || X == nullptr || Y == nullptr || OA == nullptr || amax_oa == nullptr || T < 1 || !dtype_ok(x_dt) ||
      !dtype_ok(y_dt) || !aligned16(X) || !aligned16(Y) || !aligned16(OA))
    return FALQON_ERR_INVALID_ARG;
  if (dump_block >= 0) {
    if (!fused_forward_ok(L, x_dt)) return FALQON_ERR_UNSUPPORTED;
    if (dump_block >= (L->m + L->r + 255) / 256) return FALQON_ERR_INVALID_ARG;
  }
  WorkspaceLayout w;
  if (!make_layout(L->m, L->n, L->r, T, &w)) return FALQON_ERR_INVALID_ARG;
  if (ws == nullptr || !aligned16(ws) || ws_bytes < w.total) return FALQON_ERR_WORKSPACE;
  int* status = status_ptr();
  if (status == nullptr) return FALQON_ERR_CUDA;
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* scales = reinterpret_cast<float*>(base + w.scales);
  uint8_t* xq = base + w.act8;
  const int64_t n = L->n;

  uint32_t* partial = reinterpret_cast<uint32_t*>(base + w.scales + kPartialsOffset);
  if (fused_forward_ok(L, x_dt)) {
    // S1 + S2 in one product: only the scale is prepared here (from an absmax pass over X when it is not known)
    {
      StageTimer timer(FALQON_STAGE_QUANT_X, stream);
      int nparts = 0;
      if (amax_x == nullptr) FALQON_CUDA(launch_absmax(X, x_dt, T * n, 1.0f, partial, &nparts, stream));
      FALQON_CUDA(launch_scale_prep(partial, nparts, amax_x, kE4M3, scales + 1, s_x_out, scales + 0, amax_oa, stream));
    }
    const bool emit = dump_block >= 0 || (L->flags & FALQON_LAYER_EMIT_XQ) != 0;
    const FusedOperand f{X, n, scales + 1, emit ? xq : nullptr, n, dump_block >= 0 ? dump_block : 0};
    return forward_product(L, nullptr, scales + 1, T, Y, y_dt, OA, amax_oa, base, w, status, stream, &f);
  }
  // S1: x~, s_x = Q_e4m3(X); the cast also clears amax(O_A), which the product's epilogue accumulates
  {
    StageTimer timer(FALQON_STAGE_QUANT_X, stream);
    if (amax_x != nullptr) {
      FALQON_CUDA(launch_cast_per_tensor(X, x_dt, T * n, kE4M3, 1.0f, reinterpret_cast<const uint32_t*>(amax_x), 1, nullptr, xq,
                                         scales + 1, s_x_out, scales + 0, amax_oa, stream));
    } else {
      FALQON_CUDA(launch_quantize_fused(X, x_dt, T * n, kE4M3, xq, partial, base + w.scales + kSyncOffset, scales + 1, s_x_out,
                                        scales + 0, amax_oa, status, nullptr, 0, nullptr, stream));
    }
  }
  return forward_product(L, xq, scales + 1, T, Y, y_dt, OA, amax_oa, base, w, status, stream);
}
}  // namespace

int falqon_melded_forward(const falqon_layer* L, const void* X, falqon_dtype x_dt, int64_t T, void* Y, falqon_dtype y_dt,
                          float* OA, float* amax_oa, float* s_x_out, void* ws, size_t ws_bytes, falqon_stream stream) {
  return forward_impl(L, X, x_dt, nullptr, T, Y, y_dt, OA, amax_oa, s_x_out, ws, ws_bytes, stream);
}

int falqon_melded_forward_amax(const falqon_layer* L, const void* X, falqon_dtype x_dt, const float* amax_x, int64_t T, void* Y,
                               falqon_dtype y_dt, float* OA, float* amax_oa, float* s_x_out, void* ws, size_t ws_bytes,
                               falqon_stream stream) {
  if (amax_x == nullptr) return FALQON_ERR_INVALID_ARG;
  return forward_impl(L, X, x_dt, amax_x, T, Y, y_dt, OA, amax_oa, s_x_out, ws, ws_bytes, stream);
}

int falqon_melded_forward_dump(const falqon_layer* L, const void* X, falqon_dtype x_dt, const float* amax_x, int64_t T, void* Y,
                               falqon_dtype y_dt, float* OA, float* amax_oa, float* s_x_out, int32_t n_block, void* ws,
                               size_t ws_bytes, falqon_stream stream) {
  if (n_block < 0) return FALQON_ERR_INVALID_ARG;
  return forward_impl(L, X, x_dt, amax_x, T, Y, y_dt, OA, amax_oa, s_x_out, ws, ws_bytes, stream, n_block);
}

int falqon_melded_forward_codes(const falqon_layer* L, const uint8_t* xq, const float* s_x, int64_t T, void* Y,
                                falqon_dtype y_dt, float* OA, float* amax_oa, void* ws, size_t ws_bytes, falqon_stream stream) {
  if (!layer_ok(L) || xq == nullptr || s_x == nullptr || Y == nullptr || OA == nullptr || amax_oa == nullptr || T < 1 ||
      !dtype_ok(y_dt) || !aligned16(xq) || !aligned16(Y) || !aligned16(OA))
    return FALQON_ERR_INVALID_ARG;
  WorkspaceLayout w;
  if (!make_layout(L->m, L->n, L->r, T, &w)) return FALQON_ERR_INVALID_ARG;
  if (ws == nullptr || !aligned16(ws) || ws_bytes < w.total) return FALQON_ERR_WORKSPACE;
  int* status = status_ptr();
  if (status == nullptr) return FALQON_ERR_CUDA;
  FALQON_CUDA(cudaMemsetAsync(amax_oa, 0, sizeof(float), stream));   // the product's epilogue accumulates a max into it
  return forward_product(L, xq, s_x, T, Y, y_dt, OA, amax_oa, static_cast<uint8_t*>(ws), w, status, stream);
}

namespace {
// amax_dy (nullable, device [1]; per-tensor layers only): max |dY| is already known, see forward_impl.
// sgd_lr (nullable, host): also run Alg. 3 line 4 in its plain-SGD form and the row scores (into the workspace's score region),
// inside the dB kernel where its shared memory has the room, else as the separate pass.
// S5b and S4 of one backward: dB (d) and, when dX is wanted, the input-gradient product (g).  Where the product runs on
// CTA pairs, dB rides on the product's launch (the pairs its last wave leaves idle), with the optimizer step and the row
// scores if d asks for them; otherwise -- no dX, a fused optimizer step at a rank above 128, FALQON_LAYER_DB_OWN_KERNEL -- dB
// is a kernel of its own, launched first (g~ was written a moment ago and is still in L2).
// oa_todo (nullable): the cast of O_A (S5a) has not run yet (no output-gradient quantizer launch carried it): it rides on
// the product's launch too where dB does, and is a small kernel of its own otherwise.  sync: 8 bytes, zero between launches.
int launch_db_and_dx(const falqon_layer* L, DbFusedProblem& d, GemmProblem* g, const OaCastJob* oa_todo, void* sync,
                     cudaStream_t stream) {
  const bool ride = g != nullptr && (L->flags & FALQON_LAYER_DB_OWN_KERNEL) == 0 && gemm_db_rider_supported(*g, d);
  if (oa_todo != nullptr && !ride) {
    StageTimer timer(FALQON_STAGE_QUANT_DY, stream);   // only S5a is left of this stage
    FALQON_CUDA(launch_oa_cast(*oa_todo, stream));
  }
  if (!ride) {
    StageTimer timer(FALQON_STAGE_GEMM_DB, stream);
    FALQON_CUDA(launch_db_fused(d, stream));
  }
  if (g != nullptr) {
    g->db_rider = ride ? &d : nullptr;
    g->oa_rider = ride ? oa_todo : nullptr;
    g->oa_sync = sync;
    StageTimer timer(FALQON_STAGE_GEMM_DX, stream);
    FALQON_CUDA(launch_gemm_fp8(*g, stream));
  }
  return FALQON_OK;
}

int backward_impl(const falqon_layer* L, const void* dY, falqon_dtype dy_dt, const float* amax_dy, int64_t T, const float* OA,
                  const float* amax_oa, void* dX, falqon_dtype dx_dt, float* dB, float* s_g_out, void* ws, size_t ws_bytes,
                  falqon_stream stream, int dump_block = -1, const float* sgd_lr = nullptr) {
  if (!layer_ok(L) || dY == nullptr || OA == nullptr || amax_oa == nullptr || dB == nullptr || T < 1 || !dtype_ok(dy_dt) ||
      !dtype_ok(dx_dt) || !aligned16(dY) || !aligned16(OA) || !aligned16(dB) || (dX != nullptr && !aligned16(dX)))
    return FALQON_ERR_INVALID_ARG;
  if (dump_block >= 0) {
    if (!fused_backward_ok(L, dy_dt, dX)) return FALQON_ERR_UNSUPPORTED;
    if (dump_block >= (L->n + 255) / 256) return FALQON_ERR_INVALID_ARG;
  }
  WorkspaceLayout w;
  if (!make_layout(L->m, L->n, L->r, T, &w)) return FALQON_ERR_INVALID_ARG;
  if (ws == nullptr || !aligned16(ws) || ws_bytes < w.total) return FALQON_ERR_WORKSPACE;
  int* status = status_ptr();
  if (status == nullptr) return FALQON_ERR_CUDA;
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* scales = reinterpret_cast<float*>(base + w.scales);
  uint8_t* gq = base + w.act8;
  uint8_t* oaq_t = base + w.oaq_t;
  const int64_t m = L->m, n = L->n, r = L->r;

  uint32_t* partial = reinterpret_cast<uint32_t*>(base + w.scales + kPartialsOffset);
  if (fused_backward_ok(L, dy_dt, dX)) {
    // S3 inside S4's producer: the input-gradient product casts dY tile by tile and its first column block also writes
    // g~, which S5b (run after it here) reads as a tensor
    {
      StageTimer timer(FALQON_STAGE_QUANT_DY, stream);
      int nparts = 0;
      if (amax_dy == nullptr) FALQON_CUDA(launch_absmax(dY, dy_dt, T * m, 1.0f, partial, &nparts, stream));
      FALQON_CUDA(launch_scale_prep(partial, nparts, amax_dy, kE5M2, scales + 3, s_g_out, scales + 2, nullptr, stream));
      const OaCastJob oa_cast{OA, amax_oa, T, static_cast<int>(r), w.t16, oaq_t, scales + 5, scales + 4};
      FALQON_CUDA(launch_oa_cast(oa_cast, stream));
    }
    {
      GemmProblem g{};
      g.M = T; g.N = n; g.K = m;
      g.a = nullptr; g.lda = m; g.a_fmt = kE5M2;
      g.b = L->wq; g.ldb = n; g.b_mn_major = true; g.b_fmt = kE4M3;
      g.block_n = 256;
      g.c0 = dX; g.ldc0 = n; g.c0_dt = dx_dt; g.n_split = n;
      g.scale_a = scales + 3; g.scale_b = L->s_w;
      g.status = status;
      const FusedOperand f{dY, m, scales + 3, gq, m, dump_block >= 0 ? dump_block : 0};
      StageTimer timer(FALQON_STAGE_GEMM_DX, stream);
      FALQON_CUDA(launch_gemm_fp8_fused(g, f, stream));
    }
    DbFusedProblem d{};
    d.m = m; d.r = r; d.T = T;
    d.gq = gq; d.oaq_t = oaq_t; d.ldt = w.t16; d.s_oa = scales + 5;
    d.s_g = scales + 3; d.row_mul = nullptr; d.dB = dB; d.status = status;
    const bool fuse_update = sgd_lr != nullptr && db_fused_update_fits(m, r, T);
    if (fuse_update) { d.dbuf = L->dbuf; d.score = reinterpret_cast<float*>(base + w.score); d.neg_lr = -*sgd_lr; }
    {
      StageTimer timer(FALQON_STAGE_GEMM_DB, stream);
      FALQON_CUDA(launch_db_fused(d, stream));
    }
    if (sgd_lr != nullptr && !fuse_update) {
      StageTimer timer(FALQON_STAGE_SGD_SCORE, stream);
      FALQON_CUDA(launch_sgd_score(L->dbuf, dB, *sgd_lr, m, r, reinterpret_cast<float*>(base + w.score), stream));
    }
    return FALQON_OK;
  }
  // S3: g~, s_g = Q_e5m2(dY)
  const bool per_row = L->gran == FALQON_PER_ROW;
  float* inv_sw = reinterpret_cast<float*>(base + w.inv_sw);
  if (per_row)   // the row scales lie on dX's contraction axis: divide them out of dY before its cast
    FALQON_CUDA(launch_scale_table(0, L->s_w, m, r, nullptr, inv_sw, w.inv_sw_len, stream));
  // S5a rides along: O~_A = Q_e4m3(O_A) with s_OA from the forward's amax, written transposed for the dB product
  const OaCastJob oa_cast{OA, amax_oa, T, static_cast<int>(r), w.t16, oaq_t, scales + 5, scales + 4};
  const OaCastJob* oa_todo = amax_dy != nullptr ? &oa_cast : nullptr;   // not carried by the quantizer launch below
  void* sync_words = base + w.scales + kSyncOffset;
  {
    StageTimer timer(FALQON_STAGE_QUANT_DY, stream);
    if (amax_dy != nullptr) {   // single-pass cast: no grid barrier for the O_A cast to ride on; it goes with dB / dX below
      FALQON_CUDA(launch_cast_per_tensor(dY, dy_dt, T * m, kE5M2, 1.0f, reinterpret_cast<const uint32_t*>(amax_dy), 1, nullptr, gq,
                                         scales + 3, s_g_out, scales + 2, nullptr, stream));
    } else {
      FALQON_CUDA(launch_quantize_fused(dY, dy_dt, T * m, kE5M2, gq, partial, sync_words, scales + 3, s_g_out,
                                        scales + 2, nullptr, status, per_row ? inv_sw : nullptr, static_cast<int>(m), &oa_cast,
                                        stream));
    }
  }
  // S5b: dB = g~^T O~_A / (s_g s_OA), and S4 (neither needs the other): dB rides on S4's launch where it can, and is a
  // kernel of its own (token slabs, slab sum in slab order across a thread-block cluster) before S4 where it cannot.
  {
    DbFusedProblem d{};
    d.m = m; d.r = r; d.T = T;
    d.gq = gq; d.oaq_t = oaq_t; d.ldt = w.t16; d.s_oa = scales + 5;
    d.s_g = scales + 3; d.row_mul = per_row ? L->s_w : nullptr; d.dB = dB; d.status = status;
    const bool fuse_update = sgd_lr != nullptr && db_fused_update_fits(m, r, T);
    if (fuse_update) { d.dbuf = L->dbuf; d.score = reinterpret_cast<float*>(base + w.score); d.neg_lr = -*sgd_lr; }
    // S4: dX = g~ W~ / (s_W s_g)   (contraction over the m output channels; W~ read MN-major)
    GemmProblem g{};
    g.M = T; g.N = n; g.K = m;
    g.a = gq; g.lda = m; g.a_fmt = kE5M2;
    g.b = L->wq; g.ldb = n; g.b_mn_major = true; g.b_fmt = kE4M3;
    g.block_n = 256;
    g.c0 = dX; g.ldc0 = n; g.c0_dt = dx_dt; g.n_split = n;
    g.c1 = nullptr; g.ldc1 = 0; g.amax1_bits = nullptr;
    g.scale_a = scales + 3; g.scale_b = per_row ? nullptr : L->s_w;
    g.col_scale = nullptr;
    g.status = status;
    // with a separate optimizer pass the pass must follow dB: it keeps dB in a kernel of its own, before the product
    const bool own_db = sgd_lr != nullptr && !fuse_update;
    if (own_db) {
      if (oa_todo != nullptr) {
        StageTimer timer(FALQON_STAGE_QUANT_DY, stream);
        FALQON_CUDA(launch_oa_cast(*oa_todo, stream));
      }
      {
        StageTimer timer(FALQON_STAGE_GEMM_DB, stream);
        FALQON_CUDA(launch_db_fused(d, stream));
      }
      {
        StageTimer timer(FALQON_STAGE_SGD_SCORE, stream);
        FALQON_CUDA(launch_sgd_score(L->dbuf, dB, *sgd_lr, m, r, reinterpret_cast<float*>(base + w.score), stream));
      }
      if (dX != nullptr) {
        StageTimer timer(FALQON_STAGE_GEMM_DX, stream);
        FALQON_CUDA(launch_gemm_fp8(g, stream));
      }
    } else {
      const int rc = launch_db_and_dx(L, d, dX != nullptr ? &g : nullptr, oa_todo, sync_words, stream);
      if (rc != FALQON_OK) return rc;
    }
  }
  return FALQON_OK;
}
}  // namespace

int falqon_melded_backward(const falqon_layer* L, const void* dY, falqon_dtype dy_dt, int64_t T, const float* OA,
                           const float* amax_oa, void* dX, falqon_dtype dx_dt, float* dB, float* s_g_out, void* ws,
                           size_t ws_bytes, falqon_stream stream) {
  return backward_impl(L, dY, dy_dt, nullptr, T, OA, amax_oa, dX, dx_dt, dB, s_g_out, ws, ws_bytes, stream);
}

int falqon_melded_backward_update(const falqon_layer* L, const void* dY, falqon_dtype dy_dt, const float* amax_dy, int64_t T,
                                  const float* OA, const float* amax_oa, void* dX, falqon_dtype dx_dt, float* dB, float lr,
                                  float* s_g_out, void* ws, size_t ws_bytes, falqon_stream stream) {
  if (!(lr == lr)) return FALQON_ERR_INVALID_ARG;
  if (amax_dy != nullptr && L != nullptr && L->gran == FALQON_PER_ROW) return FALQON_ERR_UNSUPPORTED;
  return backward_impl(L, dY, dy_dt, amax_dy, T, OA, amax_oa, dX, dx_dt, dB, s_g_out, ws, ws_bytes, stream, -1, &lr);
}

int falqon_melded_backward_codes(const falqon_layer* L, const uint8_t* gq, const float* s_g, int64_t T, const float* OA,
                                 const float* amax_oa, void* dX, falqon_dtype dx_dt, float* dB, void* ws, size_t ws_bytes,
                                 falqon_stream stream) {
  if (!layer_ok(L) || gq == nullptr || s_g == nullptr || OA == nullptr || amax_oa == nullptr || dB == nullptr || T < 1 ||
      !dtype_ok(dx_dt) || !aligned16(gq) || !aligned16(OA) || !aligned16(dB) || (dX != nullptr && !aligned16(dX)))
    return FALQON_ERR_INVALID_ARG;
  if (L->gran == FALQON_PER_ROW) return FALQON_ERR_UNSUPPORTED;   // there the codes are those of dY / s_w[column]: the layer's own
  WorkspaceLayout w;
  if (!make_layout(L->m, L->n, L->r, T, &w)) return FALQON_ERR_INVALID_ARG;
  if (ws == nullptr || !aligned16(ws) || ws_bytes < w.total) return FALQON_ERR_WORKSPACE;
  int* status = status_ptr();
  if (status == nullptr) return FALQON_ERR_CUDA;
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* scales = reinterpret_cast<float*>(base + w.scales);
  uint8_t* oaq_t = base + w.oaq_t;
  const int64_t m = L->m, n = L->n, r = L->r;
  const OaCastJob oa_cast{OA, amax_oa, T, static_cast<int>(r), w.t16, oaq_t, scales + 5, scales + 4};   // S5a: still to do
  DbFusedProblem d{};
  d.m = m; d.r = r; d.T = T;
  d.gq = gq; d.oaq_t = oaq_t; d.ldt = w.t16; d.s_oa = scales + 5; d.s_g = s_g; d.dB = dB; d.status = status;
  GemmProblem g{};
  g.M = T; g.N = n; g.K = m;
  g.a = gq; g.lda = m; g.a_fmt = kE5M2;
  g.b = L->wq; g.ldb = n; g.b_mn_major = true; g.b_fmt = kE4M3;
  g.block_n = 256;
  g.c0 = dX; g.ldc0 = n; g.c0_dt = dx_dt; g.n_split = n;
  g.scale_a = s_g; g.scale_b = L->s_w;
  g.status = status;
  return launch_db_and_dx(L, d, dX != nullptr ? &g : nullptr, &oa_cast, base + w.scales + kSyncOffset, stream);
}

int falqon_melded_backward_dx(const falqon_layer* L, int64_t T, void* dX, falqon_dtype dx_dt, void* ws, size_t ws_bytes,
                              falqon_stream stream) {
  if (!layer_ok(L) || dX == nullptr || T < 1 || !dtype_ok(dx_dt) || !aligned16(dX)) return FALQON_ERR_INVALID_ARG;
  WorkspaceLayout w;
  if (!make_layout(L->m, L->n, L->r, T, &w)) return FALQON_ERR_INVALID_ARG;
  if (ws == nullptr || !aligned16(ws) || ws_bytes < w.total) return FALQON_ERR_WORKSPACE;
  int* status = status_ptr();
  if (status == nullptr) return FALQON_ERR_CUDA;
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* scales = reinterpret_cast<float*>(base + w.scales);
  // S4 on the codes and the scale that the backward call before it left in the workspace
  GemmProblem g{};
  g.M = T; g.N = L->n; g.K = L->m;
  g.a = base + w.act8; g.lda = L->m; g.a_fmt = kE5M2;
  g.b = L->wq; g.ldb = L->n; g.b_mn_major = true; g.b_fmt = kE4M3;
  g.block_n = 256;
  g.c0 = dX; g.ldc0 = L->n; g.c0_dt = dx_dt; g.n_split = L->n;
  g.scale_a = scales + 3; g.scale_b = L->gran == FALQON_PER_ROW ? nullptr : L->s_w;
  g.status = status;
  StageTimer timer(FALQON_STAGE_GEMM_DX, stream);
  FALQON_CUDA(launch_gemm_fp8(g, stream));
  return FALQON_OK;
}

int falqon_melded_backward_dump(const falqon_layer* L, const void* dY, falqon_dtype dy_dt, const float* amax_dy, int64_t T,
                                const float* OA, const float* amax_oa, void* dX, falqon_dtype dx_dt, float* dB, float* s_g_out,
                                int32_t n_block, void* ws, size_t ws_bytes, falqon_stream stream) {
  if (n_block < 0) return FALQON_ERR_INVALID_ARG;
  return backward_impl(L, dY, dy_dt, amax_dy, T, OA, amax_oa, dX, dx_dt, dB, s_g_out, ws, ws_bytes, stream, n_block);
}

int falqon_melded_backward_amax(const falqon_layer* L, const void* dY, falqon_dtype dy_dt, const float* amax_dy, int64_t T,
                                const float* OA, const float* amax_oa, void* dX, falqon_dtype dx_dt, float* dB, float* s_g_out,
                                void* ws, size_t ws_bytes, falqon_stream stream) {
  if (amax_dy == nullptr) return FALQON_ERR_INVALID_ARG;
  if (L != nullptr && L->gran == FALQON_PER_ROW) return FALQON_ERR_UNSUPPORTED;   // the cast input is dY / s_w[column] there
  return backward_impl(L, dY, dy_dt, amax_dy, T, OA, amax_oa, dX, dx_dt, dB, s_g_out, ws, ws_bytes, stream);
}

namespace {
// Shared tail of the two proxy-update entry points.  adamw == nullptr: plain SGD with `lr` (or no optimizer when dB is null).
// exact != nullptr: the merge runs in its correctly rounded form with the caller's scratch.
struct ExactMergeArgs {
  void* scratch;
  float* sums_out;
  unsigned int* fix_count_out;
};
int proxy_update_impl(const falqon_layer* L, const float* dB, float lr, const falqon_adamw* adamw, float* exp_avg,
                      float* exp_avg_sq, int64_t k, int32_t* idx_out, void* ws, size_t ws_bytes, falqon_stream stream,
                      const ExactMergeArgs* exact = nullptr, bool scored = false) {
  if (!layer_ok(L) || k < 0 || k > L->m || !(lr == lr) || (dB != nullptr && !aligned16(dB)))
    return FALQON_ERR_INVALID_ARG;
  WorkspaceLayout w;
  if (!make_layout(L->m, L->n, L->r, 1, &w)) return FALQON_ERR_INVALID_ARG;  // score / index regions do not depend on T
  if (ws == nullptr || !aligned16(ws) || ws_bytes < w.total) return FALQON_ERR_WORKSPACE;
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* score = reinterpret_cast<float*>(base + w.score);
  int32_t* sel = reinterpret_cast<int32_t*>(base + w.sel_idx);
  const int64_t m = L->m, n = L->n, r = L->r;
  unsigned int* done_counter = reinterpret_cast<unsigned int*>(base + w.scales + kDoneOffset);
  unsigned int* group_counters = reinterpret_cast<unsigned int*>(base + w.scales + kGroupCountersOffset);
  const bool fused_merge = static_cast<size_t>(merge_group_count(k)) <= kMaxMergeGroups;
  {
    StageTimer timer(FALQON_STAGE_SGD_SCORE, stream);   // optimizer step, scores and (k > 0) the selection: one kernel
    if (scored) {    // the scores of the current DeltaBuffer are in the workspace already: selection only
      if (k > 0) FALQON_CUDA(launch_topk(score, m, k, sel, idx_out, stream));
    } else if (adamw != nullptr) {
      FALQON_CUDA(launch_adamw_score_topk(L->dbuf, dB, exp_avg, exp_avg_sq, adamw->lr, adamw->beta1, adamw->beta2, adamw->eps,
                                          adamw->weight_decay, adamw->step, m, r, k, score, sel, idx_out, done_counter, stream));
    } else {
      FALQON_CUDA(launch_sgd_score_topk(L->dbuf, dB, lr, m, r, k, score, sel, idx_out, done_counter, stream));
    }
  }
  if (k > 0) {
    StageTimer timer(FALQON_STAGE_MERGE, stream);
    const float* row_scales = L->gran == FALQON_PER_ROW ? L->s_w : nullptr;
    if (exact != nullptr) {
      int* status = status_ptr();
      if (status == nullptr) return FALQON_ERR_CUDA;
      FALQON_CUDA(launch_merge_exact(L->wq, L->dbuf, sel, k, m, n, r, row_scales, exact->scratch, exact->sums_out,
                                     exact->fix_count_out, status, stream));
    } else if (fused_merge) {
      FALQON_CUDA(launch_merge_rows_fused(L->wq, L->dbuf, sel, k, m, n, r, group_counters, row_scales, stream));
    } else if (row_scales == nullptr) {
      FALQON_CUDA(launch_merge_rows(L->wq, L->dbuf, sel, k, m, n, r, stream));
    } else {   // more row groups than counters: merge without the fused clearing, then clear
      FALQON_CUDA(launch_merge_rows_fused(L->wq, L->dbuf, sel, k, m, n, r, nullptr, row_scales, stream));
      FALQON_CUDA(launch_zero_rows(L->dbuf, sel, k, r, stream));
    }
  }
  return FALQON_OK;
}
}  // namespace

int falqon_proxy_update(const falqon_layer* L, const float* dB, float lr, int64_t k, int32_t* idx_out, void* ws,
                        size_t ws_bytes, falqon_stream stream) {
  return proxy_update_impl(L, dB, lr, nullptr, nullptr, nullptr, k, idx_out, ws, ws_bytes, stream);
}

int falqon_proxy_update_scored(const falqon_layer* L, int64_t k, int32_t* idx_out, void* ws, size_t ws_bytes,
                               falqon_stream stream) {
  return proxy_update_impl(L, nullptr, 0.0f, nullptr, nullptr, nullptr, k, idx_out, ws, ws_bytes, stream, nullptr, true);
}

namespace {
bool adamw_ok(const falqon_adamw* hp) {
  return hp != nullptr && hp->step >= 1 && hp->lr == hp->lr && hp->beta1 >= 0.0f && hp->beta1 < 1.0f && hp->beta2 >= 0.0f &&
         hp->beta2 < 1.0f && hp->eps >= 0.0f && hp->weight_decay == hp->weight_decay;
}

// hp == null: plain SGD with lr.  hp != null: AdamW on every layer (dB, exp_avg, exp_avg_sq all required).
int proxy_update_batched_impl(const falqon_layer* layers, int32_t count, const float* const* dB, float lr, const falqon_adamw* hp,
                              float* const* exp_avg, float* const* exp_avg_sq, const int64_t* k, int32_t* const* idx_out,
                              void* const* ws, const size_t* ws_bytes, falqon_stream stream, bool scored = false) {
  if (count < 0 || !(lr == lr)) return FALQON_ERR_INVALID_ARG;
  if (count == 0) return FALQON_OK;
  if (layers == nullptr || (dB == nullptr && !scored) || k == nullptr || ws == nullptr || ws_bytes == nullptr) return FALQON_ERR_INVALID_ARG;
  if (hp != nullptr && (exp_avg == nullptr || exp_avg_sq == nullptr)) return FALQON_ERR_INVALID_ARG;
  bool fused = true;
  for (int32_t i = 0; i < count; ++i) {
    const falqon_layer* L = &layers[i];
    if (!layer_ok(L) || k[i] < 0 || k[i] > L->m || (!scored && dB[i] != nullptr && !aligned16(dB[i]))) return FALQON_ERR_INVALID_ARG;
    if (hp != nullptr && (dB[i] == nullptr || exp_avg[i] == nullptr || exp_avg_sq[i] == nullptr || !aligned16(exp_avg[i]) ||
                          !aligned16(exp_avg_sq[i])))
      return FALQON_ERR_INVALID_ARG;
    WorkspaceLayout w;
    if (!make_layout(L->m, L->n, L->r, 1, &w)) return FALQON_ERR_INVALID_ARG;
    if (ws[i] == nullptr || !aligned16(ws[i]) || ws_bytes[i] < w.total) return FALQON_ERR_WORKSPACE;
    for (int32_t j = 0; j < i; ++j)
      if (ws[j] == ws[i] || layers[j].wq == L->wq || layers[j].dbuf == L->dbuf) return FALQON_ERR_INVALID_ARG;
    if (static_cast<size_t>(merge_group_count(k[i])) > kMaxMergeGroups) fused = false;
  }
  if (!fused) {
    for (int32_t i = 0; i < count; ++i) {
      const int rc = proxy_update_impl(&layers[i], scored ? nullptr : dB[i], lr, hp, hp != nullptr ? exp_avg[i] : nullptr,
                                       hp != nullptr ? exp_avg_sq[i] : nullptr, k[i], idx_out != nullptr ? idx_out[i] : nullptr,
                                       ws[i], ws_bytes[i], stream, nullptr, scored);
      if (rc != FALQON_OK) return rc;
    }
    return FALQON_OK;
  }
  AdamwHyper hyper{};
  if (hp != nullptr) hyper = AdamwHyper{hp->lr, hp->beta1, hp->beta2, hp->eps, hp->weight_decay, hp->step};
  const AdamwHyper* adamw = hp != nullptr ? &hyper : nullptr;
  for (int32_t first = 0; first < count; first += kProxyBatchMax) {
    const int chunk = count - first < kProxyBatchMax ? count - first : kProxyBatchMax;
    ProxyBatchLayer b[kProxyBatchMax];
    bool any_merge = false;
    for (int c = 0; c < chunk; ++c) {
      const int32_t i = first + c;
      const falqon_layer* L = &layers[i];
      WorkspaceLayout w;
      make_layout(L->m, L->n, L->r, 1, &w);
      uint8_t* base = static_cast<uint8_t*>(ws[i]);
      b[c].wq = L->wq;
      b[c].dbuf = L->dbuf;
      b[c].dB = scored ? nullptr : dB[i];
      b[c].scored = scored;
      b[c].exp_avg = hp != nullptr ? exp_avg[i] : nullptr;
      b[c].exp_avg_sq = hp != nullptr ? exp_avg_sq[i] : nullptr;
      b[c].row_scales = L->gran == FALQON_PER_ROW ? L->s_w : nullptr;
      b[c].score = reinterpret_cast<float*>(base + w.score);
      b[c].sel_idx = reinterpret_cast<int32_t*>(base + w.sel_idx);
      b[c].idx_out = idx_out != nullptr ? idx_out[i] : nullptr;
      b[c].done_counter = reinterpret_cast<unsigned int*>(base + w.scales + kDoneOffset);
      b[c].group_counters = reinterpret_cast<unsigned int*>(base + w.scales + kGroupCountersOffset);
      b[c].m = L->m; b[c].n = L->n; b[c].r = L->r; b[c].k = k[i];
      any_merge = any_merge || k[i] > 0;
    }
    {
      StageTimer timer(FALQON_STAGE_SGD_SCORE, stream);
      FALQON_CUDA(launch_proxy_update_batched(b, chunk, lr, adamw, 0, stream));
    }
    if (any_merge) {
      StageTimer timer(FALQON_STAGE_MERGE, stream);
      FALQON_CUDA(launch_proxy_update_batched(b, chunk, lr, adamw, 1, stream));
    }
  }
  return FALQON_OK;
}

}  // namespace

int falqon_proxy_update_batched(const falqon_layer* layers, int32_t count, const float* const* dB, float lr, const int64_t* k,
                                int32_t* const* idx_out, void* const* ws, const size_t* ws_bytes, falqon_stream stream) {
  return proxy_update_batched_impl(layers, count, dB, lr, nullptr, nullptr, nullptr, k, idx_out, ws, ws_bytes, stream);
}

int falqon_proxy_update_scored_batched(const falqon_layer* layers, int32_t count, const int64_t* k, int32_t* const* idx_out,
                                       void* const* ws, const size_t* ws_bytes, falqon_stream stream) {
  return proxy_update_batched_impl(layers, count, nullptr, 0.0f, nullptr, nullptr, nullptr, k, idx_out, ws, ws_bytes, stream, true);
}

int falqon_proxy_update_batched_adamw(const falqon_layer* layers, int32_t count, const float* const* dB, float* const* exp_avg,
                                      float* const* exp_avg_sq, const falqon_adamw* hp, const int64_t* k, int32_t* const* idx_out,
                                      void* const* ws, const size_t* ws_bytes, falqon_stream stream) {
  if (!adamw_ok(hp)) return FALQON_ERR_INVALID_ARG;
  return proxy_update_batched_impl(layers, count, dB, hp->lr, hp, exp_avg, exp_avg_sq, k, idx_out, ws, ws_bytes, stream);
}

int falqon_proxy_update_adamw(const falqon_layer* L, const float* dB, float* exp_avg, float* exp_avg_sq,
                              const falqon_adamw* hp, int64_t k, int32_t* idx_out, void* ws, size_t ws_bytes,
                              falqon_stream stream) {
  if (hp == nullptr || dB == nullptr || exp_avg == nullptr || exp_avg_sq == nullptr || !aligned16(exp_avg) ||
      !aligned16(exp_avg_sq) || hp->step < 1 || !(hp->lr == hp->lr) || !(hp->beta1 >= 0.0f && hp->beta1 < 1.0f) ||
      !(hp->beta2 >= 0.0f && hp->beta2 < 1.0f) || !(hp->eps >= 0.0f) || !(hp->weight_decay == hp->weight_decay))
    return FALQON_ERR_INVALID_ARG;
  return proxy_update_impl(L, dB, hp->lr, hp, exp_avg, exp_avg_sq, k, idx_out, ws, ws_bytes, stream);
}

size_t falqon_exact_merge_scratch_bytes(int64_t m, int64_t n, int64_t r) {
  if (!shape_ok(m, n, r)) return 0;
  return exact_merge_scratch_bytes(m, n, r);
}

int falqon_proxy_update_exact(const falqon_layer* L, const float* dB, float lr, int64_t k, int32_t* idx_out, void* ws,
                              size_t ws_bytes, void* scratch, size_t scratch_bytes, float* sums_out, uint32_t* fix_count_out,
                              falqon_stream stream) {
  if (!layer_ok(L)) return FALQON_ERR_INVALID_ARG;
  if (scratch == nullptr || !aligned16(scratch) || scratch_bytes < exact_merge_scratch_bytes(L->m, L->n, L->r))
    return FALQON_ERR_WORKSPACE;
  if (sums_out != nullptr && !aligned16(sums_out)) return FALQON_ERR_INVALID_ARG;
  const ExactMergeArgs exact{scratch, sums_out, fix_count_out};
  return proxy_update_impl(L, dB, lr, nullptr, nullptr, nullptr, k, idx_out, ws, ws_bytes, stream, &exact);
}

int falqon_exact_merge_prepare(const falqon_layer* L, void* scratch, size_t scratch_bytes, falqon_stream stream) {
  if (!layer_ok(L)) return FALQON_ERR_INVALID_ARG;
  if (scratch == nullptr || !aligned16(scratch) || scratch_bytes < exact_merge_scratch_bytes(L->m, L->n, L->r))
    return FALQON_ERR_WORKSPACE;
  FALQON_CUDA(launch_exact_merge_prepare(L->wq, L->m, L->n, L->r, scratch, stream));
  return FALQON_OK;
}

int falqon_proxy_update_batched_exact(const falqon_layer* layers, int32_t count, const float* const* dB, float lr, const int64_t* k,
                                      int32_t* const* idx_out, void* const* ws, const size_t* ws_bytes, void* const* scratch,
                                      const size_t* scratch_bytes, int32_t a_prepared, falqon_stream stream) {
  if (count < 0 || !(lr == lr)) return FALQON_ERR_INVALID_ARG;
  if (count == 0) return FALQON_OK;
  if (layers == nullptr || dB == nullptr || k == nullptr || ws == nullptr || ws_bytes == nullptr || scratch == nullptr ||
      scratch_bytes == nullptr)
    return FALQON_ERR_INVALID_ARG;
  for (int32_t i = 0; i < count; ++i) {
    const falqon_layer* L = &layers[i];
    if (!layer_ok(L) || k[i] < 0 || k[i] > L->m || (dB[i] != nullptr && !aligned16(dB[i]))) return FALQON_ERR_INVALID_ARG;
    WorkspaceLayout w;
    if (!make_layout(L->m, L->n, L->r, 1, &w)) return FALQON_ERR_INVALID_ARG;
    if (ws[i] == nullptr || !aligned16(ws[i]) || ws_bytes[i] < w.total) return FALQON_ERR_WORKSPACE;
    if (scratch[i] == nullptr || !aligned16(scratch[i]) || scratch_bytes[i] < exact_merge_scratch_bytes(L->m, L->n, L->r))
      return FALQON_ERR_WORKSPACE;
    for (int32_t j = 0; j < i; ++j)
      if (ws[j] == ws[i] || scratch[j] == scratch[i] || layers[j].wq == L->wq || layers[j].dbuf == L->dbuf) return FALQON_ERR_INVALID_ARG;
  }
  int* status = status_ptr();
  if (status == nullptr) return FALQON_ERR_CUDA;
  for (int32_t first = 0; first < count; first += kProxyBatchMax) {
    const int chunk = count - first < kProxyBatchMax ? count - first : kProxyBatchMax;
    ProxyBatchLayer b[kProxyBatchMax];
    ExactMergeLayer x[kProxyBatchMax];
    bool any_merge = false;
    for (int c = 0; c < chunk; ++c) {
      const int32_t i = first + c;
      const falqon_layer* L = &layers[i];
      WorkspaceLayout w;
      make_layout(L->m, L->n, L->r, 1, &w);
      uint8_t* base = static_cast<uint8_t*>(ws[i]);
      b[c] = ProxyBatchLayer{};
      b[c].wq = L->wq; b[c].dbuf = L->dbuf; b[c].dB = dB[i];
      b[c].row_scales = L->gran == FALQON_PER_ROW ? L->s_w : nullptr;
      b[c].score = reinterpret_cast<float*>(base + w.score);
      b[c].sel_idx = reinterpret_cast<int32_t*>(base + w.sel_idx);
      b[c].idx_out = idx_out != nullptr ? idx_out[i] : nullptr;
      b[c].done_counter = reinterpret_cast<unsigned int*>(base + w.scales + kDoneOffset);
      b[c].group_counters = reinterpret_cast<unsigned int*>(base + w.scales + kGroupCountersOffset);
      b[c].m = L->m; b[c].n = L->n; b[c].r = L->r; b[c].k = k[i];
      x[c] = ExactMergeLayer{L->wq, L->dbuf, b[c].sel_idx, b[c].row_scales, scratch[i], nullptr, nullptr, L->m, L->n, L->r, k[i]};
      any_merge = any_merge || k[i] > 0;
    }
    {
      StageTimer timer(FALQON_STAGE_SGD_SCORE, stream);
      FALQON_CUDA(launch_proxy_update_batched(b, chunk, lr, nullptr, 0, stream));
    }
    if (any_merge) {
      StageTimer timer(FALQON_STAGE_MERGE, stream);
      FALQON_CUDA(launch_merge_exact_batched(x, chunk, a_prepared != 0, status, stream));
    }
  }
  return FALQON_OK;
}

size_t falqon_svd_init_scratch_bytes(int64_t m, int64_t n, int64_t l) {
  if (m < 16 || n < 16 || m % 16 || n % 16 || l < 2 || l % 2 || l > 160) return 0;
  return svd_init_scratch_bytes(m, n, l);
}

int falqon_svd_init(const void* W, falqon_dtype w_dt, int64_t m, int64_t n, const uint8_t* wq, const float* s_w, int64_t r,
                    const float* omega, int64_t l, int32_t power_iters, float* A_hat, float* sigma, void* scratch,
                    size_t scratch_bytes, falqon_stream stream) {
  if (W == nullptr || wq == nullptr || s_w == nullptr || omega == nullptr || A_hat == nullptr || sigma == nullptr ||
      !dtype_ok(w_dt) || m < 16 || n < 16 || m % 16 || n % 16 || r < 1 || l < r || l % 2 || l > 160 || l > m || l > n ||
      power_iters < 0 || power_iters > 16 || !aligned16(W) || !aligned16(wq) || !aligned16(omega) || !aligned16(A_hat))
    return FALQON_ERR_INVALID_ARG;
  if (scratch == nullptr || !aligned16(scratch) || scratch_bytes < svd_init_scratch_bytes(m, n, l)) return FALQON_ERR_WORKSPACE;
  FALQON_CUDA(launch_svd_init(W, w_dt, m, n, wq, s_w, r, omega, l, power_iters, A_hat, sigma, scratch, stream));
  return FALQON_OK;
}

int falqon_tensor_ceiling_ctas(void) { return tensor_ceiling_ctas(); }

int falqon_tensor_ceiling(int64_t kblocks, uint32_t seed, int32_t random_fill, float* sink, double* flops_out,
                          const void* load_src, size_t load_bytes, int32_t bytes_per_kblock, falqon_stream stream) {
  if (bytes_per_kblock == 0) bytes_per_kblock = 32768;
  if (bytes_per_kblock < 16384 || bytes_per_kblock > 32768 || bytes_per_kblock % 16 != 0) return FALQON_ERR_INVALID_ARG;
  if (kblocks < 1 || kblocks > (1 << 20) || random_fill < 0 || random_fill > 2 || (sink != nullptr && !aligned16(sink)))
    return FALQON_ERR_INVALID_ARG;
  if (load_src != nullptr && (!aligned16(load_src) || load_bytes < 32768 || load_bytes % 16384 != 0)) return FALQON_ERR_INVALID_ARG;
  int* status = status_ptr();
  if (status == nullptr) return FALQON_ERR_CUDA;
  if (flops_out != nullptr) *flops_out = tensor_ceiling_flops(static_cast<int>(kblocks));
  FALQON_CUDA(launch_tensor_ceiling(static_cast<int>(kblocks), seed, random_fill, sink, status, load_src, load_bytes, bytes_per_kblock, stream));
  return FALQON_OK;
}

int falqon_selftest_wait_timeout(uint32_t limit_ms, falqon_stream stream) {
  if (limit_ms < 1 || limit_ms > 1000) return FALQON_ERR_INVALID_ARG;
  int* status = status_ptr();
  if (status == nullptr) return FALQON_ERR_CUDA;
  FALQON_CUDA(launch_wait_timeout_selftest(static_cast<uint64_t>(limit_ms) * 1000000ull, status, stream));
  return FALQON_OK;
}

int falqon_last_device_status(falqon_stream stream) {
  if (cudaStreamSynchronize(stream) != cudaSuccess) return FALQON_ERR_CUDA;
  int* p = status_ptr();
  if (p == nullptr) return FALQON_ERR_CUDA;
  int v = 0;
  if (cudaMemcpy(&v, p, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return FALQON_ERR_CUDA;
  if (v != 0) {
    const int zero = 0;
    if (cudaMemcpy(p, &zero, sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) return FALQON_ERR_CUDA;
  }
  return v;
}

int falqon_profile_start(int max_records, unsigned stage_mask) {
  if (g_prof.active || max_records < 1 || max_records > (1 << 20)) return FALQON_ERR_INVALID_ARG;
  g_prof.start = new cudaEvent_t[max_records];
  g_prof.stop = new cudaEvent_t[max_records];
  g_prof.kind = new int[max_records];
  for (int i = 0; i < max_records; ++i) {
    if (cudaEventCreate(&g_prof.start[i]) != cudaSuccess || cudaEventCreate(&g_prof.stop[i]) != cudaSuccess) {
      for (int j = 0; j < i; ++j) { cudaEventDestroy(g_prof.start[j]); cudaEventDestroy(g_prof.stop[j]); }
      delete[] g_prof.start; delete[] g_prof.stop; delete[] g_prof.kind;
      g_prof = ProfileState{};
      return FALQON_ERR_CUDA;
    }
  }
  g_prof.capacity = max_records;
  g_prof.used = 0;
  g_prof.mask = stage_mask;
  g_prof.active = true;
  return FALQON_OK;
}

int falqon_profile_stop(float* ms_out, int* stage_out, int capacity) {
  if (!g_prof.active) return FALQON_ERR_INVALID_ARG;
  g_prof.active = false;
  int count = g_prof.used < capacity ? g_prof.used : capacity;
  if (ms_out == nullptr || stage_out == nullptr) count = 0;
  int rc = count;
  for (int i = 0; i < count; ++i) {
    if (cudaEventSynchronize(g_prof.stop[i]) != cudaSuccess ||
        cudaEventElapsedTime(&ms_out[i], g_prof.start[i], g_prof.stop[i]) != cudaSuccess) {
      rc = FALQON_ERR_CUDA;
      break;
    }
    stage_out[i] = g_prof.kind[i];
  }
  for (int i = 0; i < g_prof.capacity; ++i) { cudaEventDestroy(g_prof.start[i]); cudaEventDestroy(g_prof.stop[i]); }
  delete[] g_prof.start; delete[] g_prof.stop; delete[] g_prof.kind;
  g_prof = ProfileState{};
  return rc;
}

int falqon_launch_count(const char* entry_point, int64_t m, int64_t n, int64_t r, int64_t T, int64_t k) {
  (void)m; (void)n; (void)r; (void)T;
  if (entry_point == nullptr) return 0;
  if (std::strcmp(entry_point, "falqon_quantize") == 0) return 2;           // absmax, cast
  if (std::strcmp(entry_point, "falqon_melded_forward") == 0) return 2;     // fused quantize, GEMM
  // fused quantize (the O_A cast rides on it), dX product (dB rides on it); dB as a kernel of its own where it cannot ride:
  // no dX requested, FALQON_LAYER_DB_OWN_KERNEL
  if (std::strcmp(entry_point, "falqon_melded_backward") == 0) return 2;
  if (std::strcmp(entry_point, "falqon_melded_backward:own_db") == 0) return 3;
  // with FALQON_LAYER_FUSED_CAST: absmax, scale, product / absmax, scale, O_A cast, dX product (casts dY, writes g~), dB
  if (std::strcmp(entry_point, "falqon_melded_forward:fused") == 0) return 3;
  if (std::strcmp(entry_point, "falqon_melded_backward:fused") == 0) return 5;
  if (std::strcmp(entry_point, "falqon_proxy_update") == 0) return k > 0 ? 2 : 1;  // optimizer+score+top-k, merge+clear
  if (std::strcmp(entry_point, "falqon_proxy_update_batched") == 0) return k > 0 ? 2 : 1;   // per 8 layers
  // as the backward: the optimizer step and the scores ride with dB (inside the dX launch, or in the dB kernel)
  if (std::strcmp(entry_point, "falqon_melded_backward_update") == 0) return 2;
  if (std::strcmp(entry_point, "falqon_melded_backward_update:own_db") == 0) return 3;
  if (std::strcmp(entry_point, "falqon_proxy_update_scored") == 0) return k > 0 ? 2 : 0;
  if (std::strcmp(entry_point, "falqon_proxy_update_scored_batched") == 0) return k > 0 ? 2 : 0;
  if (std::strcmp(entry_point, "falqon_proxy_update_static") == 0) return k > 0 ? 4 : 1;   // optimizer+score, top-k, merge, clear (+ one copy of idx)
  return 0;
}

}  // extern "C"
