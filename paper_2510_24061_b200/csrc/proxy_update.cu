// Row-wise proxy update (Alg. 3 lines 4-6, Eq. update of the paper) and the fixed-order reduction of
// the split adapter-gradient partial sums.  Everything that feeds a bit-exact stage is done in fp32
// with an explicit operation order: one fma per DeltaBuffer element, left-to-right row sums, and the
// merge as an fma chain over the rank index.
#include <cmath>

#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

// ---- DeltaBuffer <- fma(-lr, dB, DeltaBuffer); score_i = ((|d_i0| + |d_i1|) + ...) in fp32
constexpr int kScoreRows = 32;
__global__ void __launch_bounds__(256) sgd_score_kernel(float* dbuf, const float* dB,
                                                        float neg_lr, int64_t m, int r, float* score) {
  extern __shared__ float sabs[];  // [kScoreRows][r + 1]
  pdl_trigger();
  pdl_wait();
  const int64_t row0 = (int64_t)blockIdx.x * kScoreRows;
  const int rows = static_cast<int>(min((int64_t)kScoreRows, m - row0));
  const int64_t base = row0 * r;
  for (int e = threadIdx.x; e < rows * r; e += blockDim.x) {
    float d = dbuf[base + e];
    if (dB != nullptr) {
      d = __fmaf_rn(neg_lr, dB[base + e], d);
      dbuf[base + e] = d;
    }
    const int i = e / r, j = e - i * r;
    sabs[i * (r + 1) + j] = fabsf(d);
  }
  __syncthreads();
  if (threadIdx.x < rows) {
    const float* a = sabs + threadIdx.x * (r + 1);
    float s = 0.0f;
#pragma unroll 8
    for (int j = 0; j < r; ++j) s = __fadd_rn(s, a[j]);   // strictly left to right; the loads run ahead
    score[row0 + threadIdx.x] = s;
  }
}

// ---- top-k rows by score (scores are >= +0, so their bit patterns order like the values):
// radix select of the k-th largest value (4 passes of 8 bits), then an index-ordered compaction that
// takes every score above it and the lowest-index rows among the ties.  One CTA.  Thread t owns the
// contiguous rows [t*E, (t+1)*E), so thread order is index order and the compaction needs only two
// CTA-wide scans of per-thread counts.  Output ascending, written to sel_idx and, when given, idx_out.
constexpr int kTopkThreads = 1024;
constexpr int kTopkSmemRows = 48 * 1024;   // scores are staged in shared memory up to this many rows

// Exclusive prefix sums of two ints per thread over the whole CTA (any multiple of 32 threads up to 1024), one pass of
// synchronisation for both.
__device__ __forceinline__ void block_exclusive_scan2(int a, int b, int* sums_a /* [32] */, int* sums_b /* [32] */, int& ex_a,
                                                      int& ex_b) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nwarps = blockDim.x >> 5;
  int ia = a, ib = b;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int ta = __shfl_up_sync(0xFFFFFFFFu, ia, o), tb = __shfl_up_sync(0xFFFFFFFFu, ib, o);
    if (lane >= o) { ia += ta; ib += tb; }
  }
  if (lane == 31) { sums_a[warp] = ia; sums_b[warp] = ib; }
  __syncthreads();
  if (warp == 0) {
    const int wa = lane < nwarps ? sums_a[lane] : 0, wb = lane < nwarps ? sums_b[lane] : 0;
    int xa = wa, xb = wb;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int ta = __shfl_up_sync(0xFFFFFFFFu, xa, o), tb = __shfl_up_sync(0xFFFFFFFFu, xb, o);
      if (lane >= o) { xa += ta; xb += tb; }
    }
    sums_a[lane] = xa - wa;
    sums_b[lane] = xb - wb;
  }
  __syncthreads();
  ex_a = sums_a[warp] + ia - a;
  ex_b = sums_b[warp] + ib - b;
}

// The whole selection, run by one CTA (all of its threads).  s_bits: shared-memory staging for the m scores, or
// null to read them from global memory every time.
__device__ __forceinline__ void topk_block(const float* score, int m, int k, int32_t* sel_idx,
                                           int32_t* idx_out, uint32_t* s_bits) {
  __shared__ int hist[4][256];
  __shared__ int warp_sums_a[32], warp_sums_b[32];
  __shared__ uint32_t s_digit[4], s_remaining[4];
  const uint32_t* gbits = reinterpret_cast<const uint32_t*>(score);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nthreads = blockDim.x;

  for (int i = tid; i < 4 * 256; i += nthreads) (&hist[0][0])[i] = 0;
  // the minimum and maximum are taken while the scores stream in (any assignment of elements to threads will do)
  uint32_t lmin = 0xFFFFFFFFu, lmax = 0u;
  for (int i = tid; i < m; i += nthreads) {
    const uint32_t b = __ldcg(gbits + i);
    if (s_bits != nullptr) s_bits[i] = b;
    lmin = min(lmin, b);
    lmax = max(lmax, b);
  }
  const uint32_t* bits = s_bits != nullptr ? s_bits : gbits;
  const int E = (m + nthreads - 1) / nthreads;
  const int lo = min(tid * E, m), hi = min(lo + E, m);

  // The scores of a layer lie in a narrow range, so their top bits agree: find the highest bit in which any two
  // differ (from the CTA-wide min and max) and run the radix passes only over the bits from there down.  This
  // also keeps the first histogram from collapsing into one or two bins.
  lmin = __reduce_min_sync(0xFFFFFFFFu, lmin);
  lmax = __reduce_max_sync(0xFFFFFFFFu, lmax);
  if (lane == 0) { warp_sums_a[warp] = static_cast<int>(lmin); warp_sums_b[warp] = static_cast<int>(lmax); }
  __syncthreads();
  {
    const int nwarps = nthreads >> 5;
    uint32_t a = lane < nwarps ? static_cast<uint32_t>(warp_sums_a[lane]) : 0xFFFFFFFFu;
    uint32_t b = lane < nwarps ? static_cast<uint32_t>(warp_sums_b[lane]) : 0u;
    lmin = __reduce_min_sync(0xFFFFFFFFu, a);
    lmax = __reduce_max_sync(0xFFFFFFFFu, b);
  }
  __syncthreads();   // warp_sums_* are reused by the scans below
  const uint32_t diff = lmin ^ lmax;
  int top_bits = diff == 0 ? 0 : 32 - __clz(diff);          // number of low bits that can differ
  uint32_t prefix = top_bits >= 32 ? 0u : (lmax >> top_bits) << top_bits;   // the common high bits
  uint32_t mask = top_bits >= 32 ? 0u : ~((1u << top_bits) - 1u);
  uint32_t remaining = static_cast<uint32_t>(k);
  int pass = 0;
  for (int shift = top_bits; shift > 0; ++pass) {
    const int nb = min(8, shift);
    shift -= nb;
    const uint32_t dmask = (1u << nb) - 1u;
    for (int i = lo; i < hi; ++i) {
      const uint32_t b = bits[i];
      if ((b & mask) == prefix) atomicAdd(&hist[pass][(b >> shift) & dmask], 1);
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns bins 255-8l .. 248-8l (descending); find the bin where the running count reaches `remaining`
      int cnt[8], sum = 0;
#pragma unroll
      for (int q = 0; q < 8; ++q) { cnt[q] = hist[pass][255 - (8 * lane + q)]; sum += cnt[q]; }
      int incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
      }
      int above = incl - sum;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        if (static_cast<uint32_t>(above) < remaining && remaining <= static_cast<uint32_t>(above + cnt[q])) {
          s_digit[pass] = static_cast<uint32_t>(255 - (8 * lane + q));
          s_remaining[pass] = remaining - static_cast<uint32_t>(above);
        }
        above += cnt[q];
      }
    }
    __syncthreads();
    prefix |= s_digit[pass] << shift;
    remaining = s_remaining[pass];
    mask |= dmask << shift;
  }
  const uint32_t tau = prefix;                      // bit pattern of the k-th largest score
  const int take_eq = static_cast<int>(remaining);  // how many rows with score == tau are taken

  // index-ordered compaction with ONE scan: rows above tau that precede this thread's range, and rows equal to tau
  // that precede it (of which the first take_eq overall are taken)
  int my_gt = 0, my_eq = 0;
  for (int i = lo; i < hi; ++i) {
    const uint32_t b = bits[i];
    my_gt += b > tau ? 1 : 0;
    my_eq += b == tau ? 1 : 0;
  }
  int gt_before, eq_before;
  block_exclusive_scan2(my_gt, my_eq, warp_sums_a, warp_sums_b, gt_before, eq_before);
  int pos = gt_before + min(eq_before, take_eq);
  int eq_rank = eq_before;
  for (int i = lo; i < hi; ++i) {
    const uint32_t b = bits[i];
    bool selected = b > tau;
    if (b == tau) { selected = eq_rank < take_eq; ++eq_rank; }
    if (selected) {
      sel_idx[pos] = i;
      if (idx_out != nullptr) idx_out[pos] = i;
      ++pos;
    }
  }
}

__global__ void __launch_bounds__(kTopkThreads) topk_kernel(const float* score, int m, int k,
                                                            int32_t* sel_idx, int32_t* idx_out,
                                                            int use_smem) {
  extern __shared__ uint32_t s_bits_dyn[];          // [m] when use_smem
  pdl_wait();      // before the trigger, for the sake of the merge that follows (it reads A~ ahead of its wait)
  pdl_trigger();
  topk_block(score, m, k, sel_idx, idx_out, use_smem ? s_bits_dyn : nullptr);
}

// ---- the optimizer step on one DeltaBuffer element.  kind 0: none (the caller ran its own optimizer), 1: plain
// SGD d = fma(-lr, g, d), 2: AdamW with decoupled weight decay, all fp32 in this order:
//   p = p * decay;  m = fma(beta1, m, (1-beta1) * g);  v = fma(beta2, v, (1-beta2) * (g*g));
//   p = fma(-step_size, m / (sqrt(v) / sqrt_bc2 + eps), p)
struct OptimizerArgs {
  int kind;
  float neg_lr;                                   // SGD
  float beta1, beta2, eps, decay, one_minus_b1, one_minus_b2, neg_step_size, sqrt_bc2;   // AdamW
  float* exp_avg;
  float* exp_avg_sq;
};
__device__ __forceinline__ float optimizer_update(const OptimizerArgs& o, float d, float g, float& ea, float& es) {
  if (o.kind == 1) return __fmaf_rn(o.neg_lr, g, d);
  if (o.kind == 2) {
    const float p1 = __fmul_rn(d, o.decay);
    const float m1 = __fmaf_rn(o.beta1, ea, __fmul_rn(o.one_minus_b1, g));
    const float v1 = __fmaf_rn(o.beta2, es, __fmul_rn(o.one_minus_b2, __fmul_rn(g, g)));
    const float denom = __fadd_rn(__fdiv_rn(__fsqrt_rn(v1), o.sqrt_bc2), o.eps);
    ea = m1;
    es = v1;
    return __fmaf_rn(o.neg_step_size, __fdiv_rn(m1, denom), p1);
  }
  return d;
}

// ---- optimizer step + row scores + selection in ONE kernel: CTAs of 1024 threads take 128 rows each; the CTA
// that finishes last (a counter in the workspace that is zero between calls) runs the selection on all scores.
constexpr int kFusedScoreRows = 128;
// cta / n_ctas: this CTA's position among the CTAs that work on the layer.  fused_smem: [kFusedScoreRows][r + 1]
// floats, later the m staged scores.
__device__ __forceinline__ void score_topk_body(float* dbuf, const float* dB, const OptimizerArgs& opt, int m, int r, int k,
                                                float* score, int32_t* sel_idx, int32_t* idx_out,
                                                unsigned int* done_counter, int use_smem, int cta, int n_ctas,
                                                float* fused_smem) {
  __shared__ int s_last;
  const int row0 = cta * kFusedScoreRows;
  const int rows = min(kFusedScoreRows, m - row0);
  const int64_t base = (int64_t)row0 * r;
  const int total = rows * r;
  constexpr int kBatch = 4;   // loads of four elements per thread are in flight together
  for (int e0 = threadIdx.x; e0 < total; e0 += kBatch * blockDim.x) {
    float d[kBatch], g[kBatch], ea[kBatch], es[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int e = e0 + u * blockDim.x;
      d[u] = 0.0f; g[u] = 0.0f; ea[u] = 0.0f; es[u] = 0.0f;
      if (e < total) {
        d[u] = ld_stream(dbuf + base + e);
        if (opt.kind != 0) g[u] = ld_stream(dB + base + e);
        if (opt.kind == 2) { ea[u] = ld_stream(opt.exp_avg + base + e); es[u] = ld_stream(opt.exp_avg_sq + base + e); }
      }
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int e = e0 + u * blockDim.x;
      if (e < total) {
        float v = d[u];
        if (opt.kind != 0) {
          v = optimizer_update(opt, v, g[u], ea[u], es[u]);
          dbuf[base + e] = v;
          if (opt.kind == 2) { opt.exp_avg[base + e] = ea[u]; opt.exp_avg_sq[base + e] = es[u]; }
        }
        const int i = e / r, j = e - i * r;
        fused_smem[i * (r + 1) + j] = fabsf(v);
      }
    }
  }
  __syncthreads();
  if (threadIdx.x < rows) {
    const float* a = fused_smem + threadIdx.x * (r + 1);
    float s = 0.0f;
#pragma unroll 8
    for (int j = 0; j < r; ++j) s = __fadd_rn(s, a[j]);   // strictly left to right; the loads run ahead
    score[row0 + threadIdx.x] = s;
  }
  if (k <= 0) return;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int prev = atomicAdd(done_counter, 1u);
    s_last = (prev == static_cast<unsigned int>(n_ctas) - 1u) ? 1 : 0;
    if (s_last) *done_counter = 0u;       // back to zero for the next call
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  topk_block(score, m, k, sel_idx, idx_out, use_smem ? reinterpret_cast<uint32_t*>(fused_smem) : nullptr);
}

__global__ void __launch_bounds__(kTopkThreads) sgd_score_topk_kernel(float* dbuf, const float* dB,
                                                                      OptimizerArgs opt, int m, int r, int k,
                                                                      float* score, int32_t* sel_idx,
                                                                      int32_t* idx_out,
                                                                      unsigned int* done_counter, int use_smem) {
  extern __shared__ float fused_smem_dyn[];
  // The wait comes first: the merge that follows reads the A~ rows before its own wait, which is only safe
  // once every earlier kernel on the stream has finished, i.e. once this kernel is past this point.
  pdl_wait();
  pdl_trigger();
  score_topk_body(dbuf, dB, opt, m, r, k, score, sel_idx, idx_out, done_counter, use_smem, blockIdx.x, gridDim.x,
                  fused_smem_dyn);
}

// The same for several layers in one launch: the CTAs of all layers are laid end to end and each finds its layer
// from the table of first-CTA indices.  Plain SGD (or none, where a layer's dB is null).
struct BatchedScoreLayer {
  float* dbuf;
  const float* dB;
  float* exp_avg;
  float* exp_avg_sq;
  float* score;
  int32_t* sel_idx;
  int32_t* idx_out;
  unsigned int* done_counter;
  int m, r, k, cta_begin;
  int scored;      // scores are in place already: the layer's single CTA runs the selection only
};
struct BatchedScoreArgs {
  BatchedScoreLayer layer[kProxyBatchMax];
  int count;
  OptimizerArgs opt;     // the constants shared by all layers; kind and the state pointers are set per layer
};
__global__ void __launch_bounds__(kTopkThreads) score_topk_batched_kernel(const __grid_constant__ BatchedScoreArgs args) {
  extern __shared__ float fused_smem_dyn[];
  pdl_wait();
  pdl_trigger();
  int l = 0;
#pragma unroll 1
  for (int i = 1; i < args.count; ++i) l = static_cast<int>(blockIdx.x) >= args.layer[i].cta_begin ? i : l;
  const BatchedScoreLayer& a = args.layer[l];
  if (a.scored) {
    if (a.k > 0)
      topk_block(a.score, a.m, a.k, a.sel_idx, a.idx_out, a.m <= kTopkSmemRows ? reinterpret_cast<uint32_t*>(fused_smem_dyn) : nullptr);
    return;
  }
  const int n_ctas = (a.m + kFusedScoreRows - 1) / kFusedScoreRows;
  OptimizerArgs opt = args.opt;
  if (a.dB == nullptr) opt.kind = 0;
  opt.exp_avg = a.exp_avg;
  opt.exp_avg_sq = a.exp_avg_sq;
  score_topk_body(a.dbuf, a.dB, opt, a.m, a.r, a.k, a.score, a.sel_idx, a.idx_out, a.done_counter,
                  a.m <= kTopkSmemRows ? 1 : 0, static_cast<int>(blockIdx.x) - a.cta_begin, n_ctas, fused_smem_dyn);
}

// ---- W~[i][:] <- sat_rne_e4m3(W~[i][:] + DeltaBuffer[i][:] * A~) for the selected rows.
// A CTA owns 128 columns and every n_splits-th group of 32 selected rows.  It decodes the r x 128 tile of A~ to fp32 in
// shared memory once (the FP8 decode is the expensive part, so it is shared by all of the CTA's rows), then walks
// its row groups: each thread runs the fp32 fma chains of 4 rows x 8 columns
// (8 x 8 tiles and a hand-pipelined j loop were measured and were no faster).  The chain order (j ascending, seeded
// with the decoded W~) is fixed, so the result is bit-identical to the sequential definition.  The groups are software
// pipelined: while one is in the fma loop, the next one's DeltaBuffer rows arrive by asynchronous copy, its backbone codes
// are in flight to registers, and the row indices of the one after it are being fetched, so that a CTA pays the
// memory latency once, not once per group.  The inner loop needs as many shared-memory wavefronts as it can get: the
// DeltaBuffer rows are read four j at a time, and their pitch of r + 4 floats keeps the two row blocks a warp
// touches in different banks.
constexpr int kMergeRowsPerThread = 4;
constexpr int kMergeTy = 8;
constexpr int kMergeRows = kMergeRowsPerThread * kMergeTy;          // 32 rows per group
constexpr int kMergeRing = 4;                                       // row-index slots: groups t - 1 .. t + 2
constexpr int kMergeTx = 16;
constexpr int kMergeThreads = kMergeTx * kMergeTy;                  // 128
constexpr int kMergeCols = 128;                                     // columns per CTA: thread tx owns 4tx..4tx+3 and 64+4tx..64+4tx+3

__device__ __forceinline__ void decode4(uint32_t w, float (&a)[4]) {
  const float2 p0 = e4m3x2_to_float2(w), p1 = e4m3x2_to_float2(w >> 16);
  a[0] = p0.x; a[1] = p0.y; a[2] = p1.x; a[3] = p1.y;
}

__host__ __device__ constexpr size_t merge_smem_bytes(int64_t r) {
  return sizeof(float) * (static_cast<size_t>(r) * kMergeCols + 2 * static_cast<size_t>(kMergeRows) * (r + 4));
}

// col_tile: which 128 columns; split / n_splits: this CTA takes the row groups split, split + n_splits, ...;
// n_col_tiles: how many CTAs work on one row group.
__device__ __forceinline__ void merge_rows_body(uint8_t* wq, float* dbuf, const int32_t* sel_idx, int k, int64_t m, int64_t n,
                                                int r, unsigned int* group_counters, const float* row_scales, int col_tile,
                                                int split, int n_splits, int n_col_tiles, float* merge_smem) {
  constexpr int kRPT = kMergeRowsPerThread;
  const int pitch = r + 4;
  float* a_tile = merge_smem;                         // [r][kMergeCols] decoded A~
  float* sdb = merge_smem + (size_t)r * kMergeCols;   // [2][kMergeRows][r + 4]
  __shared__ int srow[kMergeRing][kMergeRows];        // row indices of the groups t - 1 (late clearing) .. t + 2
  const int64_t cta_c0 = (int64_t)col_tile * kMergeCols;
  const int cta_cols = static_cast<int>(min((int64_t)kMergeCols, n - cta_c0));   // multiple of 16
  const int groups = (k + kMergeRows - 1) / kMergeRows;
  const int items = split < groups ? (groups - split + n_splits - 1) / n_splits : 0;
  // The A~ rows are decoded BEFORE the wait, while the selection kernel is still running: nothing on the proxy
  // update's path writes them, and the kernel launched before this one (the selection) releases this launch
  // only after its own wait, i.e. after everything earlier on the stream (a set-up cast of A~, say) is done.
  // decode A~ (rows m.. of W~') into shared memory; columns beyond the matrix edge become 0.  The loads of
  // four iterations are issued together so that their latencies overlap.
  const uint8_t* aq = wq + m * n + cta_c0;
  constexpr int kVecPerRow = kMergeCols / 16;
  const int a_vecs = r * kVecPerRow;
  for (int e0 = threadIdx.x; e0 < a_vecs; e0 += 4 * kMergeThreads) {
    uint4 w[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = e0 + u * kMergeThreads;
      const int j = e / kVecPerRow, v = e % kVecPerRow;
      w[u] = make_uint4(0u, 0u, 0u, 0u);
      if (e < a_vecs && v * 16 < cta_cols) w[u] = ld_stream(reinterpret_cast<const uint4*>(aq + (int64_t)j * n + v * 16));
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = e0 + u * kMergeThreads;
      if (e < a_vecs) {
        const int j = e / kVecPerRow, v = e % kVecPerRow;
        float f[4];
        float4* dst = reinterpret_cast<float4*>(a_tile + (size_t)j * kMergeCols + v * 16);
        decode4(w[u].x, f); dst[0] = make_float4(f[0], f[1], f[2], f[3]);
        decode4(w[u].y, f); dst[1] = make_float4(f[0], f[1], f[2], f[3]);
        decode4(w[u].z, f); dst[2] = make_float4(f[0], f[1], f[2], f[3]);
        decode4(w[u].w, f); dst[3] = make_float4(f[0], f[1], f[2], f[3]);
      }
    }
  }
  pdl_wait();
  if (items == 0) return;
  const int tid = threadIdx.x;
  const int tx = tid % kMergeTx, ty = tid / kMergeTx;
  const int lc0 = 4 * tx, lc1 = 64 + 4 * tx;
  const bool ok0 = lc0 < cta_cols, ok1 = lc1 < cta_cols;
  const int q0 = ty * kRPT;
  const int r4 = r >> 2;
  const int d_vecs = kMergeRows * r4;
  // index of selected row q of this CTA's item t (or -1 past the end of the selection / of the items)
  auto fetch_index = [&](int t) -> int {
    const int64_t pos = (int64_t)(split + t * n_splits) * kMergeRows + tid;
    return (t < items && tid < kMergeRows && pos < k) ? ld_stream(sel_idx + pos) : -1;
  };
  // DeltaBuffer rows of the group whose indices are in srow[slot] -> sdb[buf], as asynchronous 16-byte copies
  auto fetch_rows = [&](int slot, int buf) {
    float* dst = sdb + (size_t)buf * kMergeRows * pitch;
    for (int e = tid; e < d_vecs; e += kMergeThreads) {
      const int q = e / r4, j4 = e - q * r4;
      const int row = srow[slot][q];
      if (row >= 0) cp_async16(smem_u32(dst + q * pitch + 4 * j4), dbuf + (int64_t)row * r + 4 * j4);
    }
    cp_async_commit();
  };
  auto fetch_codes = [&](int slot, uint32_t (&w0)[kRPT], uint32_t (&w1)[kRPT]) {
#pragma unroll
    for (int q = 0; q < kRPT; ++q) {
      w0[q] = 0u; w1[q] = 0u;
      const int row = srow[slot][q0 + q];
      if (row >= 0) {
        const uint8_t* p = wq + (int64_t)row * n + cta_c0;
        if (ok0) w0[q] = *reinterpret_cast<const uint32_t*>(p + lc0);
        if (ok1) w1[q] = *reinterpret_cast<const uint32_t*>(p + lc1);
      }
    }
  };
  if (tid < kMergeRows) {
    srow[0][tid] = fetch_index(0);
    srow[1][tid] = fetch_index(1);
  }
  __syncthreads();   // the indices and the A~ tile are visible
  uint32_t w0[kRPT], w1[kRPT];
  fetch_rows(0, 0);
  fetch_codes(0, w0, w1);
  unsigned int pending = 0u;     // warp 0: the counter value its lane 0 drew for the previous group
  bool has_pending = false;
  for (int t = 0; t < items; ++t) {
    const int slot = t % kMergeRing, buf = t & 1;
    const int idx_ahead = fetch_index(t + 2);
    uint32_t nw0[kRPT], nw1[kRPT];
    if (t + 1 < items) {
      fetch_rows((t + 1) % kMergeRing, buf ^ 1);
      fetch_codes((t + 1) % kMergeRing, nw0, nw1);
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    float* db = sdb + (size_t)buf * kMergeRows * pitch;
    if (row_scales != nullptr) {   // per-row mode: c_i = s_w[i] / s_w[m], applied as its own rounded multiply to the
      const float s_a = ld_stream(row_scales + m);                       // chunks this thread copied itself
      for (int e = tid; e < d_vecs; e += kMergeThreads) {
        const int q = e / r4, j4 = e - q * r4;
        const int row = srow[slot][q];
        if (row >= 0) {
          const float c = __fdiv_rn(ld_stream(row_scales + row), s_a);
          float4* p = reinterpret_cast<float4*>(db + q * pitch + 4 * j4);
          float4 d = *p;
          d.x = __fmul_rn(d.x, c); d.y = __fmul_rn(d.y, c); d.z = __fmul_rn(d.z, c); d.w = __fmul_rn(d.w, c);
          *p = d;
        }
      }
    }
    __syncthreads();   // this group's DeltaBuffer rows have landed for every thread
    // accumulators as packed pairs of neighbouring columns: the chains run on the two-wide fp32 fma, every half
    // of which is an ordinary round-to-nearest fma
    uint64_t v[kRPT][4];
#pragma unroll
    for (int q = 0; q < kRPT; ++q) {
      float f[4];
      decode4(w0[q], f); v[q][0] = pack_f32x2(f[0], f[1]); v[q][1] = pack_f32x2(f[2], f[3]);
      decode4(w1[q], f); v[q][2] = pack_f32x2(f[0], f[1]); v[q][3] = pack_f32x2(f[2], f[3]);
    }
    const float* d0 = db + q0 * pitch;
#pragma unroll 1
    for (int j = 0; j < r; j += 4) {
      float4 d4[kRPT];
#pragma unroll
      for (int q = 0; q < kRPT; ++q) d4[q] = *reinterpret_cast<const float4*>(d0 + q * pitch + j);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const ulonglong2 a0 = *reinterpret_cast<const ulonglong2*>(a_tile + (size_t)(j + u) * kMergeCols + lc0);
        const ulonglong2 a1 = *reinterpret_cast<const ulonglong2*>(a_tile + (size_t)(j + u) * kMergeCols + lc1);
#pragma unroll
        for (int q = 0; q < kRPT; ++q) {
          const float d = u == 0 ? d4[q].x : u == 1 ? d4[q].y : u == 2 ? d4[q].z : d4[q].w;
          const uint64_t dd = pack_f32x2(d, d);
          fma_f32x2(v[q][0], dd, a0.x); fma_f32x2(v[q][1], dd, a0.y);
          fma_f32x2(v[q][2], dd, a1.x); fma_f32x2(v[q][3], dd, a1.y);
        }
      }
    }
#pragma unroll
    for (int q = 0; q < kRPT; ++q) {
      const int row = srow[slot][q0 + q];
      if (row >= 0) {
        uint8_t* p = wq + (int64_t)row * n + cta_c0;
        float f[8];
        unpack_f32x2(v[q][0], f[0], f[1]); unpack_f32x2(v[q][1], f[2], f[3]);
        unpack_f32x2(v[q][2], f[4], f[5]); unpack_f32x2(v[q][3], f[6], f[7]);
        if (ok0) *reinterpret_cast<uint32_t*>(p + lc0) = cvt_fp8x4<kE4M3>(f[0], f[1], f[2], f[3]);
        if (ok1) *reinterpret_cast<uint32_t*>(p + lc1) = cvt_fp8x4<kE4M3>(f[4], f[5], f[6], f[7]);
      }
    }
    // With group counters (zero between calls) the CTA that is last to be done with a row group clears the group's
    // DeltaBuffer rows, which saves a separate kernel; every CTA of the group has its copy of them by then.  Warp 0
    // does this alone, and looks at the counter value one group late, so that nobody waits for the atomic.
    if (group_counters != nullptr && tid < 32) {
      auto clear_if_last = [&](int item) {
        unsigned int prev = __shfl_sync(0xFFFFFFFFu, pending, 0);
        if (prev == static_cast<unsigned int>(n_col_tiles) - 1u) {
          const int g = split + item * n_splits;
          if (tid == 0) group_counters[g] = 0u;
          const int s3 = item % kMergeRing;
          for (int e = tid; e < d_vecs; e += 32) {
            const int q = e / r4, j4 = e - q * r4;
            const int row = srow[s3][q];
            if (row >= 0) *reinterpret_cast<float4*>(dbuf + (int64_t)row * r + 4 * j4) = make_float4(0.f, 0.f, 0.f, 0.f);
          }
        }
      };
      if (has_pending) clear_if_last(t - 1);
      if (tid == 0) pending = atomicAdd(&group_counters[split + t * n_splits], 1u);
      has_pending = true;
      if (t + 1 == items) clear_if_last(t);
    }
    // The indices of group t + 2 go into the slot that group t - 2 had; the late clearing of that group ran before
    // the previous iteration's closing barrier.
    if (tid < kMergeRows) srow[(t + 2) % kMergeRing][tid] = idx_ahead;
#pragma unroll
    for (int q = 0; q < kRPT; ++q) { w0[q] = nw0[q]; w1[q] = nw1[q]; }
    __syncthreads();   // everyone is done with sdb[buf]; the new indices are visible
  }
}

__global__ void __launch_bounds__(kMergeThreads) merge_rows_kernel(uint8_t* wq, float* dbuf,
                                                                   const int32_t* sel_idx, int k, int64_t m,
                                                                   int64_t n, int r, unsigned int* group_counters,
                                                                   const float* row_scales) {
  extern __shared__ __align__(16) float merge_smem_dyn[];
  pdl_trigger();
  merge_rows_body(wq, dbuf, sel_idx, k, m, n, r, group_counters, row_scales, blockIdx.x, blockIdx.y, gridDim.y, gridDim.x,
                  merge_smem_dyn);
}

// Several layers in one launch (see score_topk_batched_kernel): a layer's CTAs are numbered column tile fastest.
struct BatchedMergeLayer {
  uint8_t* wq;
  float* dbuf;
  const int32_t* sel_idx;
  unsigned int* group_counters;
  const float* row_scales;
  int64_t m, n;
  int r, k, cta_begin, col_tiles, splits;
};
struct BatchedMergeArgs {
  BatchedMergeLayer layer[kProxyBatchMax];
  int count;
};
__global__ void __launch_bounds__(kMergeThreads) merge_rows_batched_kernel(const __grid_constant__ BatchedMergeArgs args) {
  extern __shared__ __align__(16) float merge_smem_dyn[];
  pdl_trigger();
  int l = 0;
#pragma unroll 1
  for (int i = 1; i < args.count; ++i) l = static_cast<int>(blockIdx.x) >= args.layer[i].cta_begin ? i : l;
  const BatchedMergeLayer& a = args.layer[l];
  const int local = static_cast<int>(blockIdx.x) - a.cta_begin;
  merge_rows_body(a.wq, a.dbuf, a.sel_idx, a.k, a.m, a.n, a.r, a.group_counters, a.row_scales, local % a.col_tiles,
                  local / a.col_tiles, a.splits, a.col_tiles, merge_smem_dyn);
}

__global__ void __launch_bounds__(256) zero_rows_kernel(float* dbuf, const int32_t* sel_idx,
                                                        int k, int r) {
  pdl_trigger();
  pdl_wait();
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < k * r; e += gridDim.x * blockDim.x) {
    const int s = e / r, j = e - s * r;
    dbuf[(int64_t)sel_idx[s] * r + j] = 0.0f;
  }
}

}  // namespace

cudaError_t launch_sgd_score(float* dbuf, const float* dB, float lr, int64_t m, int64_t r, float* score,
                             cudaStream_t stream) {
  const int grid = static_cast<int>((m + kScoreRows - 1) / kScoreRows);
  const size_t smem = sizeof(float) * kScoreRows * (r + 1);
  return launch_pdl(sgd_score_kernel, dim3(grid), dim3(256), smem, stream, 1, dbuf, dB, -lr, m, static_cast<int>(r), score);
}

cudaError_t launch_topk(const float* score, int64_t m, int64_t k, int32_t* sel_idx, void* idx_copy, cudaStream_t stream) {
  const int use_smem = m <= kTopkSmemRows ? 1 : 0;
  const size_t smem = use_smem ? static_cast<size_t>(m) * sizeof(uint32_t) : 0;
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(topk_kernel, static_cast<int>(kTopkSmemRows * sizeof(uint32_t)), configured);
    if (ec != cudaSuccess) return ec;
  }
  return launch_pdl(topk_kernel, dim3(1), dim3(kTopkThreads), smem, stream, 1, score, static_cast<int>(m),
                    static_cast<int>(k), sel_idx, static_cast<int32_t*>(idx_copy), use_smem);
}

namespace {
constexpr int kMergeSmemMax = 200 * 1024;   // r = 256: 128 KB of A~ and two buffers of 33 KB
constexpr int kMergeCtasPerSm = 4;

// How many CTAs may share one column tile (each takes every splits-th row group) so that the whole launch is about one
// wave of resident CTAs: the fewer CTAs, the more groups each one pipelines through.
int merge_splits_budget(int64_t col_tiles_total, int64_t r_max) {
  int64_t per_sm = (227 * 1024) / static_cast<int64_t>(merge_smem_bytes(r_max) + 1024);
  if (per_sm > kMergeCtasPerSm) per_sm = kMergeCtasPerSm;
  if (per_sm < 1) per_sm = 1;
  const int64_t budget = per_sm * sm_count() / (col_tiles_total > 0 ? col_tiles_total : 1);
  return static_cast<int>(budget < 1 ? 1 : budget);
}
// ... but no CTA walks more than kMergeItemsMax groups: with many selected rows and a small rank the groups are short
// and bound by memory latency, which more CTAs (several waves of them) hide better than a longer walk does.
constexpr int kMergeItemsMax = 4;
int merge_splits(int budget, int64_t groups) {
  int64_t splits = (groups + kMergeItemsMax - 1) / kMergeItemsMax;
  if (splits < budget) splits = budget;
  if (splits > groups) splits = groups;
  if (splits > 65535) splits = 65535;
  return static_cast<int>(splits < 1 ? 1 : splits);
}

cudaError_t launch_merge_only(uint8_t* wq, float* dbuf, const int32_t* sel_idx, int64_t k, int64_t m, int64_t n, int64_t r,
                              unsigned int* group_counters, const float* row_scales, cudaStream_t stream) {
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(merge_rows_kernel, kMergeSmemMax, configured);
    if (ec != cudaSuccess) return ec;
  }
  const int64_t col_tiles = (n + kMergeCols - 1) / kMergeCols, groups = (k + kMergeRows - 1) / kMergeRows;
  const int splits = merge_splits(merge_splits_budget(col_tiles, r), groups);
  dim3 grid(static_cast<unsigned>(col_tiles), static_cast<unsigned>(splits));
  return launch_pdl(merge_rows_kernel, grid, dim3(kMergeThreads), merge_smem_bytes(r), stream, 1, wq, dbuf, sel_idx,
                    static_cast<int>(k), m, n, static_cast<int>(r), group_counters, row_scales);
}
}  // namespace

cudaError_t launch_merge_rows(uint8_t* wq, float* dbuf, const int32_t* sel_idx, int64_t k, int64_t m, int64_t n,
                              int64_t r, cudaStream_t stream) {
  cudaError_t e = launch_merge_only(wq, dbuf, sel_idx, k, m, n, r, nullptr, nullptr, stream);
  if (e != cudaSuccess) return e;
  int64_t zb = (k * r + 255) / 256;
  if (zb > 1024) zb = 1024;
  return launch_pdl(zero_rows_kernel, dim3(static_cast<unsigned>(zb)), dim3(256), 0, stream, 1, dbuf, sel_idx,
                    static_cast<int>(k), static_cast<int>(r));
}

cudaError_t launch_zero_rows(float* dbuf, const int32_t* sel_idx, int64_t k, int64_t r, cudaStream_t stream) {
  int64_t zb = (k * r + 255) / 256;
  if (zb > 1024) zb = 1024;
  return launch_pdl(zero_rows_kernel, dim3(static_cast<unsigned>(zb)), dim3(256), 0, stream, 1, dbuf, sel_idx,
                    static_cast<int>(k), static_cast<int>(r));
}

int merge_group_count(int64_t k) { return static_cast<int>((k + kMergeRows - 1) / kMergeRows); }

cudaError_t launch_merge_rows_fused(uint8_t* wq, float* dbuf, const int32_t* sel_idx, int64_t k, int64_t m, int64_t n,
                                    int64_t r, unsigned int* group_counters, const float* row_scales, cudaStream_t stream) {
  return launch_merge_only(wq, dbuf, sel_idx, k, m, n, r, group_counters, row_scales, stream);
}

namespace {
cudaError_t launch_opt_score_topk(float* dbuf, const float* dB, const OptimizerArgs& opt, int64_t m, int64_t r, int64_t k,
                                  float* score, int32_t* sel_idx, int32_t* idx_copy, unsigned int* done_counter,
                                  cudaStream_t stream) {
  const int use_smem = m <= kTopkSmemRows ? 1 : 0;
  size_t smem = sizeof(float) * kFusedScoreRows * (r + 1);
  if (use_smem && static_cast<size_t>(m) * sizeof(uint32_t) > smem) smem = static_cast<size_t>(m) * sizeof(uint32_t);
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(sgd_score_topk_kernel, static_cast<int>(kTopkSmemRows * sizeof(uint32_t)), configured);
    if (ec != cudaSuccess) return ec;
  }
  const int grid = static_cast<int>((m + kFusedScoreRows - 1) / kFusedScoreRows);
  return launch_pdl(sgd_score_topk_kernel, dim3(grid), dim3(kTopkThreads), smem, stream, 1, dbuf, dB, opt,
                    static_cast<int>(m), static_cast<int>(r), static_cast<int>(k), score, sel_idx, idx_copy, done_counter,
                    use_smem);
}
}  // namespace

cudaError_t launch_sgd_score_topk(float* dbuf, const float* dB, float lr, int64_t m, int64_t r, int64_t k, float* score,
                                  int32_t* sel_idx, int32_t* idx_copy, unsigned int* done_counter, cudaStream_t stream) {
  OptimizerArgs opt{};
  opt.kind = dB != nullptr ? 1 : 0;
  opt.neg_lr = -lr;
  return launch_opt_score_topk(dbuf, dB, opt, m, r, k, score, sel_idx, idx_copy, done_counter, stream);
}

namespace {
OptimizerArgs adamw_args(float lr, float beta1, float beta2, float eps, float weight_decay, int64_t step) {
  OptimizerArgs opt{};
  opt.kind = 2;
  opt.beta1 = beta1; opt.beta2 = beta2; opt.eps = eps;
  // derived constants: evaluated in double, rounded once to fp32
  opt.decay = static_cast<float>(1.0 - static_cast<double>(lr) * static_cast<double>(weight_decay));
  opt.one_minus_b1 = static_cast<float>(1.0 - static_cast<double>(beta1));
  opt.one_minus_b2 = static_cast<float>(1.0 - static_cast<double>(beta2));
  opt.neg_step_size = -static_cast<float>(static_cast<double>(lr) / (1.0 - std::pow(static_cast<double>(beta1), static_cast<double>(step))));
  opt.sqrt_bc2 = static_cast<float>(std::sqrt(1.0 - std::pow(static_cast<double>(beta2), static_cast<double>(step))));
  return opt;
}
}  // namespace

cudaError_t launch_adamw_score_topk(float* dbuf, const float* dB, float* exp_avg, float* exp_avg_sq, float lr, float beta1,
                                    float beta2, float eps, float weight_decay, int64_t step, int64_t m, int64_t r, int64_t k,
                                    float* score, int32_t* sel_idx, int32_t* idx_copy, unsigned int* done_counter,
                                    cudaStream_t stream) {
  OptimizerArgs opt = adamw_args(lr, beta1, beta2, eps, weight_decay, step);
  opt.exp_avg = exp_avg;
  opt.exp_avg_sq = exp_avg_sq;
  return launch_opt_score_topk(dbuf, dB, opt, m, r, k, score, sel_idx, idx_copy, done_counter, stream);
}

namespace {
cudaError_t launch_merge_batched(const ProxyBatchLayer* layers, int count, cudaStream_t stream) {
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(merge_rows_batched_kernel, kMergeSmemMax, configured);
    if (ec != cudaSuccess) return ec;
  }
  int64_t col_tiles_total = 0, r_max = 8;
  for (int i = 0; i < count; ++i) {
    if (layers[i].k <= 0) continue;
    col_tiles_total += (layers[i].n + kMergeCols - 1) / kMergeCols;
    if (layers[i].r > r_max) r_max = layers[i].r;
  }
  const int budget = merge_splits_budget(col_tiles_total, r_max);
  BatchedMergeArgs ma{};
  int ctas = 0;
  for (int i = 0; i < count; ++i) {
    const ProxyBatchLayer& L = layers[i];
    if (L.k <= 0) continue;
    BatchedMergeLayer& b = ma.layer[ma.count++];
    b.wq = L.wq; b.dbuf = L.dbuf; b.sel_idx = L.sel_idx; b.group_counters = L.group_counters; b.row_scales = L.row_scales;
    b.m = L.m; b.n = L.n; b.r = static_cast<int>(L.r); b.k = static_cast<int>(L.k);
    b.cta_begin = ctas;
    b.col_tiles = static_cast<int>((L.n + kMergeCols - 1) / kMergeCols);
    const int groups = static_cast<int>((L.k + kMergeRows - 1) / kMergeRows);
    b.splits = merge_splits(budget, groups);
    ctas += b.col_tiles * b.splits;
  }
  if (ma.count == 0) return cudaSuccess;
  return launch_pdl(merge_rows_batched_kernel, dim3(ctas), dim3(kMergeThreads), merge_smem_bytes(r_max), stream, 1, ma);
}
}  // namespace

cudaError_t launch_proxy_update_batched(const ProxyBatchLayer* layers, int count, float lr, const AdamwHyper* adamw, int phase,
                                        cudaStream_t stream) {
  if (count < 1 || count > kProxyBatchMax) return cudaErrorInvalidValue;
  if (phase != 0) return launch_merge_batched(layers, count, stream);
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(score_topk_batched_kernel, static_cast<int>(kTopkSmemRows * sizeof(uint32_t)), configured);
    if (ec != cudaSuccess) return ec;
  }
  BatchedScoreArgs sa{};
  sa.count = count;
  if (adamw != nullptr) {
    sa.opt = adamw_args(adamw->lr, adamw->beta1, adamw->beta2, adamw->eps, adamw->weight_decay, adamw->step);
  } else {
    sa.opt.kind = 1;
    sa.opt.neg_lr = -lr;
  }
  int score_ctas = 0;
  size_t score_smem = 0;
  for (int i = 0; i < count; ++i) {
    const ProxyBatchLayer& L = layers[i];
    BatchedScoreLayer& a = sa.layer[i];
    a.dbuf = L.dbuf; a.dB = L.dB; a.exp_avg = L.exp_avg; a.exp_avg_sq = L.exp_avg_sq; a.score = L.score; a.sel_idx = L.sel_idx; a.idx_out = L.idx_out;
    a.done_counter = L.done_counter;
    a.m = static_cast<int>(L.m); a.r = static_cast<int>(L.r); a.k = static_cast<int>(L.k);
    a.cta_begin = score_ctas;
    a.scored = L.scored ? 1 : 0;
    score_ctas += L.scored ? 1 : static_cast<int>((L.m + kFusedScoreRows - 1) / kFusedScoreRows);
    size_t smem = L.scored ? 0 : sizeof(float) * kFusedScoreRows * (L.r + 1);
    if (L.m <= kTopkSmemRows && static_cast<size_t>(L.m) * sizeof(uint32_t) > smem) smem = static_cast<size_t>(L.m) * sizeof(uint32_t);
    if (smem > score_smem) score_smem = smem;
  }
  return launch_pdl(score_topk_batched_kernel, dim3(score_ctas), dim3(kTopkThreads), score_smem, stream, 1, sa);
}

}  // namespace falqon
