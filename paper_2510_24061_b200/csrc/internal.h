// Host-side declarations shared by the translation units of libfalqon (not part of the public ABI).
#pragma once

#include <atomic>
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

struct CUtensorMap_st;

namespace falqon {

constexpr int kE4M3 = 0, kE5M2 = 1;
constexpr int kBF16 = 0, kF32 = 1;

inline int64_t round_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }

// Per-device caches (symbol addresses, occupancy figures, configured attributes) are tables of this many entries, indexed
// by the device ordinal; a device beyond it is refused.  The caches are filled on first use and never invalidated: the
// library must not be used across a cudaDeviceReset of a device it has already run on.
constexpr int kMaxDevices = 64;

// The largest dynamic shared-memory size of a kernel is a property of the (kernel, device) pair: set it the first time a
// launch site is used on a device.  `done` is the launch site's own word, one bit per device.
using DeviceMask = std::atomic<unsigned long long>;
template <typename K>
cudaError_t set_max_dynamic_smem(K kernel, int bytes, DeviceMask& done) {
  int dev = 0;
  const bool tracked = cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64;
  const unsigned long long bit = tracked ? 1ull << dev : 0ull;
  if (tracked && (done.load(std::memory_order_acquire) & bit) != 0) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && tracked) done.fetch_or(bit, std::memory_order_release);
  return e;
}

// Launches `kernel` so that it may be scheduled before the previous kernel in the stream has drained
// (programmatic stream serialization).  The kernel itself must call pdl_wait() before it reads or writes
// anything another kernel touches.  cluster_x > 1 adds a thread-block-cluster dimension.
// cluster_x < 0: a COOPERATIVE launch without clusters -- the driver starts the grid only when all of its CTAs can be
// resident at once, which a kernel whose CTAs wait for one another needs.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, int cluster_x,
                       Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  int n = 0;
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster_x < 0) {
    attr[n].id = cudaLaunchAttributeCooperative;
    attr[n].val.cooperative = 1;
    ++n;
  }
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = static_cast<unsigned>(cluster_x);
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = static_cast<unsigned>(n);
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- api.cu: the device status word of the current device (bounded waits that run out report there), or nullptr
int* device_status_ptr();

// ---- quantize.cu
constexpr int kMaxAbsmaxParts = 148 * 8;   // upper bound of the absmax grid = number of partial maxima
// Pass 1 of per-tensor absmax scaling: one partial max (fp32 bit pattern of |x|) per CTA into partial[0..*nparts).
cudaError_t launch_absmax(const void* src, int src_dt, int64_t count, float premul, uint32_t* partial, int* nparts,
                          cudaStream_t stream);
// max |x| of a tensor as an fp32 number in *amax_out (two small launches); partial: kMaxAbsmaxParts words of scratch.
cudaError_t launch_absmax_value(const void* src, int src_dt, int64_t count, uint32_t* partial, float* amax_out,
                                cudaStream_t stream);
// Pass 2: cast with scale = fp8max / max(partial[0..nparts)) when nparts > 0, else with *scale_in.  Writes the
// scale to scale_out / scale_out2 and the absmax to amax_out when non-null; sets *clear_word = 0 when non-null.
cudaError_t launch_cast_per_tensor(const void* src, int src_dt, int64_t count, int fmt, float premul,
                                   const uint32_t* partial, int nparts, const float* scale_in, uint8_t* dst,
                                   float* scale_out, float* scale_out2, float* amax_out, float* clear_word,
                                   cudaStream_t stream);
// The scale of a tensor without its cast (one small CTA): fp8max / amax with amax = max(partial[0..nparts)) when nparts > 0,
// else *amax_in; outputs as launch_cast_per_tensor (all nullable).
cudaError_t launch_scale_prep(const uint32_t* partial, int nparts, const float* amax_in, int fmt, float* scale_out,
                              float* scale_out2, float* amax_out, float* clear_word, cudaStream_t stream);
// A small cast that rides along with a fused quantizer launch (S5a inside S3's kernel): O_A [T][r] fp32 -> E4M3 codes
// written transposed as [r][ldt] with s_OA = 448 / *amax_oa; *amax_copy = *amax_oa.  oa == nullptr: none.
struct OaCastJob {
  const float* oa;
  const float* amax_oa;
  long long T;
  int r;
  long long ldt;
  uint8_t* oaq_t;
  float* s_oa_out;
  float* amax_copy;   // nullable
};
cudaError_t launch_oa_cast(const OaCastJob& job, cudaStream_t stream);   // the same cast as a kernel of its own
// Per-tensor absmax scaling in one kernel (absmax, grid barrier, cast).  `sync` points at 8 bytes of workspace that
// are zero before the call and are left zero by it; `partial` holds up to kMaxAbsmaxParts words.
// col_mul (nullable): column c of the [count / cols][cols] tensor is multiplied by col_mul[c] before everything else.
// oa_cast (nullable): see OaCastJob.
cudaError_t launch_quantize_fused(const void* src, int src_dt, int64_t count, int fmt, uint8_t* dst, uint32_t* partial,
                                  void* sync, float* scale_out, float* scale_out2, float* amax_out, float* clear_word,
                                  int* status, const float* col_mul, int cols, const OaCastJob* oa_cast, cudaStream_t stream);
// Tables for a per-row-scaled backbone (s_w has m + 1 entries): mode 0 -> out[i] = 1/s_w[i]; mode 1 ->
// out[c] = 1/(s_w[min(c,m)] * *s_x) for c < m + r.  Entries up to `padded` are written (zero beyond the table).
cudaError_t launch_scale_table(int mode, const float* s_w, int64_t m, int64_t r, const float* s_x, float* out, int64_t padded,
                               cudaStream_t stream);
cudaError_t launch_quantize_per_row(const void* src, int src_dt, int64_t rows, int64_t cols, int fmt, float premul,
                                    const float* scale_in, uint8_t* dst, float* scale_out, float* amax_out,
                                    cudaStream_t stream);

// ---- gemm_fp8.cu
struct DbFusedProblem;
struct GemmProblem {
  // D[M][N] = A[M][K] * B[N][K]^T with fp32 accumulation on tcgen05
  int64_t M, N, K;
  const uint8_t* a; int64_t lda; int a_fmt;                   // K-major: a[M][lda]
  const uint8_t* b; int64_t ldb; bool b_mn_major; int b_fmt;  // K-major: b[N][ldb]; MN-major: b[K][ldb]
  int block_n;                 // tile width (16..256, multiple of 16)
  // epilogue: columns [0, n_split) -> c0 (bf16 or fp32), columns [n_split, N) -> c1 (fp32) with |max| -> amax1
  void* c0; int64_t ldc0; int c0_dt; int64_t n_split;
  float* c1; int64_t ldc1; uint32_t* amax1_bits;
  const float* scale_a; const float* scale_b;  // device scalars; output *= 1/(sa*sb); scale_b null: 1/sa; both null: none
  const float* col_scale;                      // nullable: per-column factors (N rounded up to 32 entries) instead
  int* status;
  // nullable: the adapter gradient of the same layer, computed by the same launch on the CTA pairs that the last wave of
  // this product's tiles leaves idle (see gemm_db_rider_supported)
  const DbFusedProblem* db_rider;
  // nullable, with db_rider only: the cast of O_A that the rider's B operand needs, done by the same launch too (its
  // epilogue warps, before the first tile is complete); oa_sync: 8 bytes of device memory that are zero between launches
  const OaCastJob* oa_rider;
  void* oa_sync;
};
cudaError_t launch_gemm_fp8(const GemmProblem& p, cudaStream_t stream);
// Whether launch_gemm_fp8 can carry d as p.db_rider: p is an input-gradient product on CTA pairs whose A operand is d's
// g~ (and, with the optimizer step fused into d, r <= 128).
bool gemm_db_rider_supported(const GemmProblem& p, const DbFusedProblem& d);

// ---- gemm_fp8_fused.cu: the same product on CTA pairs with the cast of the A operand fused into the producer.  A arrives
// as bf16 [M][lda16]; converter warps scale it by *a_scale (the scale of Eq. quantize, already on the device) and
// round it to a_fmt straight into the swizzled operand slots, so its codes need never be written to memory.
// p.a / p.lda are ignored; p.scale_a must be a_scale.  emit_dst (nullable): the tiles of output-column block
// emit_n_block (256 columns each) also write the codes they staged to emit_dst[M][emit_ld] (emit_ld >= K).
struct FusedOperand {
  const void* a16; int64_t lda16;
  const float* a_scale;
  uint8_t* emit_dst; int64_t emit_ld; int emit_n_block;
};
// Whether the fused kernel takes this problem (CTA-pair tiling: block_n == 256, N a multiple of 16, K a multiple of 16).
bool gemm_fp8_fused_supported(const GemmProblem& p);
cudaError_t launch_gemm_fp8_fused(const GemmProblem& p, const FusedOperand& f, cudaStream_t stream);
bool make_tensor_map_u16(CUtensorMap_st* map, const void* base, int64_t rows, int64_t cols, int64_t ld, uint32_t box_cols,
                         uint32_t box_rows);
// 2-D uint8 tensor [rows][cols] with row pitch ld bytes; box = box_cols x box_rows, 128-byte swizzle.
bool make_tensor_map(CUtensorMap_st* map, const uint8_t* base, int64_t rows, int64_t cols, int64_t ld, uint32_t box_cols,
                     uint32_t box_rows);
int sm_count();

// ---- gemm_db.cu: S5b in one kernel -- dB = g~^T O~_A / (s_g s_OA) over token slabs, the slab sum taken in slab
// order across a thread-block cluster.
struct DbFusedProblem {
  int64_t m, r, T;
  const uint8_t* gq;           // [T][m] E5M2
  const uint8_t* oaq_t; int64_t ldt;   // [r16][ldt] E4M3 codes of O_A, transposed (rows r.. may hold anything)
  const float* s_oa;           // [1]
  const float* s_g;            // [1]
  const float* row_mul;        // nullable [m]: dB row i is also multiplied by row_mul[i]
  float* dB;                   // [m][r]; nullable when dbuf is given
  int* status;
  // optional, together: the plain-SGD step of Alg. 3 line 4 and the row scores, in the kernel's slab-sum phase
  bool g_is_e4m3;              // the [T][m] operand holds E4M3 codes (the update-A product reads x~ here) instead of E5M2
  float* dbuf;                 // [m][r]: DeltaBuffer <- fma(neg_lr, dB, DeltaBuffer)
  float* score;                // [m]: sum_j |DeltaBuffer_ij|, fp32, j ascending
  float neg_lr;
};
cudaError_t launch_db_fused(const DbFusedProblem& p, cudaStream_t stream);
bool db_fused_update_fits(int64_t m, int64_t r, int64_t T);   // whether the fused step has room in the kernel's shared memory

// ---- update_a.cu: p[j][c] = fma(-lr, g_t[c][j], p[j][c]) for p [rows][cols] and the transposed gradient g_t [cols][rows]
cudaError_t launch_sgd_step_transposed(float* p, const float* g_t, float lr, int64_t rows, int64_t cols, cudaStream_t stream);

// ---- merge_exact.cu: the correctly rounded merge of the selected rows on the tensor cores (guard band + exact fallback).
// scratch: exact_merge_scratch_bytes(m, n, r) bytes, no initialisation needed.  Clears the merged DeltaBuffer rows.
// sums_out (nullable [k][n] fp32): the accumulated sums before rounding; fix_count_out (nullable device [1]): how many
// elements went through the exact fallback.
size_t exact_merge_scratch_bytes(int64_t m, int64_t n, int64_t r);
cudaError_t launch_merge_exact(uint8_t* wq, float* dbuf, const int32_t* sel_idx, int64_t k, int64_t m, int64_t n, int64_t r,
                               const float* row_scales, void* scratch, float* sums_out, unsigned int* fix_count_out, int* status,
                               cudaStream_t stream);

// The same for several layers per launch (three launches for the whole set, plus two per layer when the bf16 copy of A~ has
// not been prepared beforehand).  Layers with k == 0 are skipped.
struct ExactMergeLayer {
  uint8_t* wq;
  float* dbuf;
  const int32_t* sel_idx;
  const float* row_scales;       // nullable
  void* scratch;                 // exact_merge_scratch_bytes(m, n, r)
  float* sums_out;               // nullable
  unsigned int* fix_count_out;   // nullable
  int64_t m, n, r, k;
};
cudaError_t launch_exact_merge_prepare(const uint8_t* wq, int64_t m, int64_t n, int64_t r, void* scratch, cudaStream_t stream);
cudaError_t launch_merge_exact_batched(const ExactMergeLayer* layers, int count, bool a_prepared, int* status, cudaStream_t stream);

// ---- svd_init.cu: A^ = sqrt(S_r) V_r^T of Delta W = W - dec(W~) / s_W by randomized subspace iteration (set-up code).
// omega: [n][l] fp32 Gaussian test matrix drawn by the caller, l even, r <= l <= 160; scratch: svd_init_scratch_bytes.
size_t svd_init_scratch_bytes(int64_t m, int64_t n, int64_t l);
cudaError_t launch_svd_init(const void* w, int w_dt, int64_t m, int64_t n, const uint8_t* wq, const float* s_w, int64_t r,
                            const float* omega, int64_t l, int power_iters, float* a_hat, float* sigma, void* scratch,
                            cudaStream_t stream);

// ---- proxy_update.cu
cudaError_t launch_sgd_score(float* dbuf, const float* dB, float lr, int64_t m, int64_t r, float* score,
                             cudaStream_t stream);
// The k selected rows (ascending) are written to sel_idx and, when idx_copy is non-null, to idx_copy (int32 [k]).
cudaError_t launch_topk(const float* score, int64_t m, int64_t k, int32_t* sel_idx, void* idx_copy, cudaStream_t stream);
cudaError_t launch_merge_rows(uint8_t* wq, float* dbuf, const int32_t* sel_idx, int64_t k, int64_t m, int64_t n,
                              int64_t r, cudaStream_t stream);
// Fused forms used with an initialised workspace: optimizer step + scores + selection in one kernel (done_counter:
// one word, zero between calls), and the merge that also clears the merged DeltaBuffer rows (group_counters:
// merge_group_count(k) words, zero between calls).
int merge_group_count(int64_t k);
cudaError_t launch_zero_rows(float* dbuf, const int32_t* sel_idx, int64_t k, int64_t r, cudaStream_t stream);
cudaError_t launch_sgd_score_topk(float* dbuf, const float* dB, float lr, int64_t m, int64_t r, int64_t k, float* score,
                                  int32_t* sel_idx, int32_t* idx_copy, unsigned int* done_counter, cudaStream_t stream);
// row_scales (nullable, m + 1 entries): per-row mode, DeltaBuffer row i enters the chain times s_w[i] / s_w[m].
// The same kernel with AdamW (decoupled weight decay) as the optimizer; exp_avg / exp_avg_sq are [m][r] fp32 state.
cudaError_t launch_adamw_score_topk(float* dbuf, const float* dB, float* exp_avg, float* exp_avg_sq, float lr, float beta1,
                                    float beta2, float eps, float weight_decay, int64_t step, int64_t m, int64_t r, int64_t k,
                                    float* score, int32_t* sel_idx, int32_t* idx_copy, unsigned int* done_counter,
                                    cudaStream_t stream);
cudaError_t launch_merge_rows_fused(uint8_t* wq, float* dbuf, const int32_t* sel_idx, int64_t k, int64_t m, int64_t n,
                                    int64_t r, unsigned int* group_counters, const float* row_scales, cudaStream_t stream);

// The two fused kernels over up to kProxyBatchMax layers per launch (plain SGD; dB null = no optimizer step for that
// layer).  Every layer brings its own score / selection regions and counters; results are those of the per-layer calls.
constexpr int kProxyBatchMax = 8;
struct ProxyBatchLayer {
  uint8_t* wq;
  float* dbuf;
  const float* dB;
  float* exp_avg;               // AdamW state of this layer (both null for plain SGD)
  float* exp_avg_sq;
  const float* row_scales;      // null for a per-tensor scale
  float* score;
  int32_t* sel_idx;
  int32_t* idx_out;             // nullable
  unsigned int* done_counter;
  unsigned int* group_counters;
  int64_t m, n, r, k;
  bool scored;                  // the optimizer step and the scores are done already (score holds them): selection only
};
// phase 0: optimizer step, scores and selection of every layer; phase 1: the merge of every layer with k > 0.
// adamw == null: plain SGD with `lr`; else AdamW with these hyper-parameters on every layer (lr is then ignored).
struct AdamwHyper {
  float lr, beta1, beta2, eps, weight_decay;
  int64_t step;
};
cudaError_t launch_proxy_update_batched(const ProxyBatchLayer* layers, int count, float lr, const AdamwHyper* adamw, int phase,
                                        cudaStream_t stream);

// Measurement aid: every SM pair issues kblocks x 4 FP8 MMAs (256 x 256 x 32, the product kernels' instruction) on
// operands resident in shared memory.  sink: device [4 * tensor_ceiling_ctas()] floats or null.
int tensor_ceiling_ctas();
double tensor_ceiling_flops(int kblocks);
// load_src / load_bytes: optional buffer (a multiple of 16 KB, at least 32 KB) streamed into the operand slots at the
// rate of a real product's operand traffic.
// bytes_per_kblock: 16384 .. 32768, a multiple of 16 (what one CTA fetches per four MMAs: 32768 for 256 x 256 tiles).
cudaError_t launch_tensor_ceiling(int kblocks, uint32_t seed, int random_fill, float* sink, int* status, const void* load_src,
                                  size_t load_bytes, int bytes_per_kblock, cudaStream_t stream);

// One CTA waits limit_ns on a barrier nobody signals, records the timeout in *status and returns (self-test of the bounded waits).
cudaError_t launch_wait_timeout_selftest(uint64_t limit_ns, int* status, cudaStream_t stream);

}  // namespace falqon
