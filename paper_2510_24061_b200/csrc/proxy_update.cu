// Row-wise proxy update (Alg. 3 lines 4-6, Eq. update of the paper) and the fixed-order reduction of
// the split adapter-gradient partial sums.  Everything that feeds a bit-exact stage is done in fp32
// with an explicit operation order: one fma per DeltaBuffer element, left-to-right row sums, and the
// merge as an fma chain over the rank index.
#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

// ---- dB = (sum over splits, in split order) / (s_g * s_OA)
__global__ void __launch_bounds__(256) reduce_db_kernel(const float* __restrict__ partials, int splits, int64_t count,
                                                        const float* __restrict__ s_g, const float* __restrict__ s_oa,
                                                        float* __restrict__ dB) {
  const float inv = 1.0f / (__ldg(s_g) * __ldg(s_oa));
  const int64_t nvec = count / 4;
  for (int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; v < nvec; v += (int64_t)gridDim.x * blockDim.x) {
    float4 acc = reinterpret_cast<const float4*>(partials)[v];
    for (int s = 1; s < splits; ++s) {
      const float4 x = reinterpret_cast<const float4*>(partials + (int64_t)s * count)[v];
      acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
    }
    acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    reinterpret_cast<float4*>(dB)[v] = acc;
  }
}

// ---- DeltaBuffer <- fma(-lr, dB, DeltaBuffer); score_i = ((|d_i0| + |d_i1|) + ...) in fp32
constexpr int kScoreRows = 32;
__global__ void __launch_bounds__(256) sgd_score_kernel(float* __restrict__ dbuf, const float* __restrict__ dB,
                                                        float neg_lr, int64_t m, int r, float* __restrict__ score) {
  extern __shared__ float sabs[];  // [kScoreRows][r + 1]
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
    for (int j = 0; j < r; ++j) s = __fadd_rn(s, a[j]);
    score[row0 + threadIdx.x] = s;
  }
}

// ---- top-k rows by score (scores are >= +0, so their bit patterns order like the values):
// radix select of the k-th largest value, then an index-ordered compaction that takes every score
// above it and the lowest-index rows among the ties.  One CTA; output ascending.
constexpr int kTopkThreads = 1024;
__global__ void __launch_bounds__(kTopkThreads) topk_kernel(const float* __restrict__ score, int m, int k,
                                                            int32_t* __restrict__ sel_idx) {
  __shared__ int hist[256];
  __shared__ uint32_t s_prefix, s_remaining;
  __shared__ int warp_eq[32], warp_sel[32];
  __shared__ int run_eq, run_sel;
  const uint32_t* bits = reinterpret_cast<const uint32_t*>(score);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  uint32_t prefix = 0, mask = 0, remaining = static_cast<uint32_t>(k);
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int i = tid; i < m; i += kTopkThreads) {
      const uint32_t b = bits[i];
      if ((b & mask) == prefix) atomicAdd(&hist[(b >> shift) & 0xFF], 1);
    }
    __syncthreads();
    if (tid == 0) {
      uint32_t rem = remaining;
      int d = 255;
      for (; d > 0; --d) {
        const uint32_t h = static_cast<uint32_t>(hist[d]);
        if (rem <= h) break;
        rem -= h;
      }
      s_prefix = prefix | (static_cast<uint32_t>(d) << shift);
      s_remaining = rem;
    }
    __syncthreads();
    prefix = s_prefix;
    remaining = s_remaining;
    mask |= 0xFFu << shift;
    __syncthreads();
  }
  const uint32_t tau = prefix;      // bit pattern of the k-th largest score
  const int take_eq = static_cast<int>(remaining);  // how many rows with score == tau are taken

  if (tid == 0) { run_eq = 0; run_sel = 0; }
  __syncthreads();
  for (int base = 0; base < m; base += kTopkThreads) {
    const int i = base + tid;
    const uint32_t b = (i < m) ? bits[i] : 0u;
    const bool is_gt = (i < m) && b > tau;
    const bool is_eq = (i < m) && b == tau;
    // rank of this row among the tied rows, in index order
    const uint32_t eq_ballot = __ballot_sync(0xFFFFFFFFu, is_eq);
    if (lane == 0) warp_eq[warp] = __popc(eq_ballot);
    __syncthreads();
    int eq_before = run_eq;
    for (int w = 0; w < warp; ++w) eq_before += warp_eq[w];
    const int eq_rank = eq_before + __popc(eq_ballot & ((1u << lane) - 1u));
    const bool selected = is_gt || (is_eq && eq_rank < take_eq);
    const uint32_t sel_ballot = __ballot_sync(0xFFFFFFFFu, selected);
    if (lane == 0) warp_sel[warp] = __popc(sel_ballot);
    __syncthreads();
    int sel_before = run_sel;
    for (int w = 0; w < warp; ++w) sel_before += warp_sel[w];
    if (selected) sel_idx[sel_before + __popc(sel_ballot & ((1u << lane) - 1u))] = i;
    __syncthreads();
    if (tid == 0) {
      int te = 0, ts = 0;
      for (int w = 0; w < 32; ++w) { te += warp_eq[w]; ts += warp_sel[w]; }
      run_eq += te;
      run_sel += ts;
    }
    __syncthreads();
  }
}

// ---- W~[i][:] <- sat_rne_e4m3(W~[i][:] + DeltaBuffer[i][:] * A~) for the selected rows.
// A CTA owns kMergeRows selected rows x (128 threads x 8 columns); each decoded A~ value is reused for
// all of the CTA's rows.  The chain order (j ascending, seeded with the decoded W~) is fixed.
constexpr int kMergeRows = 4;
constexpr int kMergeThreads = 128;
constexpr int kMergeCols = 8;
__global__ void __launch_bounds__(kMergeThreads) merge_rows_kernel(uint8_t* __restrict__ wq, const float* __restrict__ dbuf,
                                                                   const int32_t* __restrict__ sel_idx, int k, int64_t m,
                                                                   int64_t n, int r) {
  extern __shared__ float sdb[];  // [kMergeRows][r]
  __shared__ int srow[kMergeRows];
  const int g0 = blockIdx.y * kMergeRows;
  const int nrows = min(kMergeRows, k - g0);
  if (threadIdx.x < kMergeRows) srow[threadIdx.x] = (threadIdx.x < nrows) ? sel_idx[g0 + threadIdx.x] : -1;
  __syncthreads();
  for (int e = threadIdx.x; e < kMergeRows * r; e += kMergeThreads) {
    const int q = e / r, j = e - q * r;
    sdb[e] = (q < nrows) ? dbuf[(int64_t)srow[q] * r + j] : 0.0f;
  }
  __syncthreads();
  const int64_t c0 = ((int64_t)blockIdx.x * kMergeThreads + threadIdx.x) * kMergeCols;
  if (c0 >= n) return;
  float v[kMergeRows][kMergeCols];
#pragma unroll
  for (int q = 0; q < kMergeRows; ++q) {
    uint2 w = make_uint2(0u, 0u);
    if (q < nrows) w = *reinterpret_cast<const uint2*>(wq + (int64_t)srow[q] * n + c0);
    const float2 p0 = e4m3x2_to_float2(w.x), p1 = e4m3x2_to_float2(w.x >> 16);
    const float2 p2 = e4m3x2_to_float2(w.y), p3 = e4m3x2_to_float2(w.y >> 16);
    v[q][0] = p0.x; v[q][1] = p0.y; v[q][2] = p1.x; v[q][3] = p1.y;
    v[q][4] = p2.x; v[q][5] = p2.y; v[q][6] = p3.x; v[q][7] = p3.y;
  }
  const uint8_t* aq = wq + m * n + c0;  // rows m.. of W~' are A~
#pragma unroll 4
  for (int j = 0; j < r; ++j) {
    const uint2 w = __ldg(reinterpret_cast<const uint2*>(aq + (int64_t)j * n));
    const float2 p0 = e4m3x2_to_float2(w.x), p1 = e4m3x2_to_float2(w.x >> 16);
    const float2 p2 = e4m3x2_to_float2(w.y), p3 = e4m3x2_to_float2(w.y >> 16);
    const float a[kMergeCols] = {p0.x, p0.y, p1.x, p1.y, p2.x, p2.y, p3.x, p3.y};
#pragma unroll
    for (int q = 0; q < kMergeRows; ++q) {
      const float d = sdb[q * r + j];
#pragma unroll
      for (int c = 0; c < kMergeCols; ++c) v[q][c] = __fmaf_rn(d, a[c], v[q][c]);
    }
  }
#pragma unroll
  for (int q = 0; q < kMergeRows; ++q) {
    if (q < nrows) {
      uint2 o;
      o.x = cvt_fp8x4<kE4M3>(v[q][0], v[q][1], v[q][2], v[q][3]);
      o.y = cvt_fp8x4<kE4M3>(v[q][4], v[q][5], v[q][6], v[q][7]);
      *reinterpret_cast<uint2*>(wq + (int64_t)srow[q] * n + c0) = o;
    }
  }
}

__global__ void __launch_bounds__(256) zero_rows_kernel(float* __restrict__ dbuf, const int32_t* __restrict__ sel_idx,
                                                        int k, int r) {
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < k * r; e += gridDim.x * blockDim.x) {
    const int s = e / r, j = e - s * r;
    dbuf[(int64_t)sel_idx[s] * r + j] = 0.0f;
  }
}

}  // namespace

cudaError_t launch_reduce_db(const float* partials, int splits, int64_t count, const float* s_g, const float* s_oa,
                             float* dB, cudaStream_t stream) {
  int64_t blocks = (count / 4 + 255) / 256;
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (blocks < 1) blocks = 1;
  reduce_db_kernel<<<static_cast<int>(blocks), 256, 0, stream>>>(partials, splits, count, s_g, s_oa, dB);
  return cudaGetLastError();
}

cudaError_t launch_sgd_score(float* dbuf, const float* dB, float lr, int64_t m, int64_t r, float* score,
                             cudaStream_t stream) {
  const int grid = static_cast<int>((m + kScoreRows - 1) / kScoreRows);
  const size_t smem = sizeof(float) * kScoreRows * (r + 1);
  sgd_score_kernel<<<grid, 256, smem, stream>>>(dbuf, dB, -lr, m, static_cast<int>(r), score);
  return cudaGetLastError();
}

size_t topk_scratch_bytes(int64_t m) { (void)m; return 256; }

cudaError_t launch_topk(const float* score, int64_t m, int64_t k, int32_t* sel_idx, void* scratch, cudaStream_t stream) {
  (void)scratch;
  topk_kernel<<<1, kTopkThreads, 0, stream>>>(score, static_cast<int>(m), static_cast<int>(k), sel_idx);
  return cudaGetLastError();
}

cudaError_t launch_merge_rows(uint8_t* wq, float* dbuf, const int32_t* sel_idx, int64_t k, int64_t m, int64_t n,
                              int64_t r, cudaStream_t stream) {
  const int cols_per_block = kMergeThreads * kMergeCols;
  dim3 grid(static_cast<unsigned>((n + cols_per_block - 1) / cols_per_block),
            static_cast<unsigned>((k + kMergeRows - 1) / kMergeRows));
  const size_t smem = sizeof(float) * kMergeRows * r;
  merge_rows_kernel<<<grid, kMergeThreads, smem, stream>>>(wq, dbuf, sel_idx, static_cast<int>(k), m, n,
                                                           static_cast<int>(r));
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  int64_t zb = (k * r + 255) / 256;
  if (zb > 1024) zb = 1024;
  zero_rows_kernel<<<static_cast<int>(zb), 256, 0, stream>>>(dbuf, sel_idx, static_cast<int>(k), static_cast<int>(r));
  return cudaGetLastError();
}

}  // namespace falqon
