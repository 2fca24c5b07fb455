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
// radix select of the k-th largest value (4 passes of 8 bits, histogram in shared memory, the digit
// found with a parallel suffix scan), then an index-ordered compaction that takes every score above
// it and the lowest-index rows among the ties.  One CTA; output ascending, written to sel_idx and,
// when given, to idx_out.
constexpr int kTopkThreads = 1024;

// Exclusive prefix sum of one int per thread over the whole CTA (1024 threads); *total = CTA sum.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums /* [32] */, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int w = warp_sums[lane];
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xFFFFFFFFu, wi, o);
      if (lane >= o) wi += t;
    }
    warp_sums[lane] = wi - w;                 // exclusive offset of each warp
    if (lane == 31) *total = wi;
  }
  __syncthreads();
  const int out = warp_sums[warp] + incl - v;
  __syncthreads();
  return out;
}

__global__ void __launch_bounds__(kTopkThreads) topk_kernel(const float* __restrict__ score, int m, int k,
                                                            int32_t* __restrict__ sel_idx, int32_t* __restrict__ idx_out) {
  __shared__ int hist[256];
  __shared__ int warp_sums[32];
  __shared__ int s_total;
  __shared__ uint32_t s_digit, s_remaining;
  const uint32_t* bits = reinterpret_cast<const uint32_t*>(score);
  const int tid = threadIdx.x;

  uint32_t prefix = 0, mask = 0, remaining = static_cast<uint32_t>(k);
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int i = tid; i < m; i += kTopkThreads) {
      const uint32_t b = bits[i];
      if ((b & mask) == prefix) atomicAdd(&hist[(b >> shift) & 0xFF], 1);
    }
    __syncthreads();
    // thread t < 256 owns bin d = 255 - t, so an exclusive scan over t counts the rows in larger bins
    const int mine = (tid < 256) ? hist[255 - tid] : 0;
    const int above = block_exclusive_scan(mine, warp_sums, &s_total);
    if (tid < 256 && static_cast<uint32_t>(above) < remaining && remaining <= static_cast<uint32_t>(above + mine)) {
      s_digit = static_cast<uint32_t>(255 - tid);
      s_remaining = remaining - static_cast<uint32_t>(above);
    }
    __syncthreads();
    prefix |= s_digit << shift;
    remaining = s_remaining;
    mask |= 0xFFu << shift;
    __syncthreads();
  }
  const uint32_t tau = prefix;                      // bit pattern of the k-th largest score
  const int take_eq = static_cast<int>(remaining);  // how many rows with score == tau are taken

  int run_eq = 0, run_sel = 0;
  for (int base = 0; base < m; base += kTopkThreads) {
    const int i = base + tid;
    const uint32_t b = (i < m) ? bits[i] : 0u;
    const bool is_gt = (i < m) && b > tau;
    const bool is_eq = (i < m) && b == tau;
    const int eq_rank = run_eq + block_exclusive_scan(is_eq ? 1 : 0, warp_sums, &s_total);
    run_eq += s_total;
    const bool selected = is_gt || (is_eq && eq_rank < take_eq);
    __syncthreads();
    const int pos = run_sel + block_exclusive_scan(selected ? 1 : 0, warp_sums, &s_total);
    run_sel += s_total;
    if (selected) {
      sel_idx[pos] = i;
      if (idx_out != nullptr) idx_out[pos] = i;
    }
    __syncthreads();
  }
}

// ---- W~[i][:] <- sat_rne_e4m3(W~[i][:] + DeltaBuffer[i][:] * A~) for the selected rows.
// A CTA owns 8 selected rows x 512 columns.  It first stages the r x 512 tile of A~ in shared memory
// with 16-byte loads that are all in flight together, then each thread runs the fp32 fma chains of
// 4 rows x 8 columns, so every decoded A~ value feeds four chains.  The chain order (j ascending,
// seeded with the decoded W~) is fixed.
constexpr int kMergeRowsPerThread = 4;
constexpr int kMergeRowGroups = 2;
constexpr int kMergeRows = kMergeRowsPerThread * kMergeRowGroups;   // rows per CTA
constexpr int kMergeColsPerThread = 8;
constexpr int kMergeTx = 64;
constexpr int kMergeThreads = kMergeTx * kMergeRowGroups;           // 128
constexpr int kMergeCols = kMergeTx * kMergeColsPerThread;          // 512 columns per CTA

__device__ __forceinline__ void decode8(uint2 w, float (&a)[8]) {
  const float2 p0 = e4m3x2_to_float2(w.x), p1 = e4m3x2_to_float2(w.x >> 16);
  const float2 p2 = e4m3x2_to_float2(w.y), p3 = e4m3x2_to_float2(w.y >> 16);
  a[0] = p0.x; a[1] = p0.y; a[2] = p1.x; a[3] = p1.y; a[4] = p2.x; a[5] = p2.y; a[6] = p3.x; a[7] = p3.y;
}

__global__ void __launch_bounds__(kMergeThreads) merge_rows_kernel(uint8_t* __restrict__ wq, const float* __restrict__ dbuf,
                                                                   const int32_t* __restrict__ sel_idx, int k, int64_t m,
                                                                   int64_t n, int r) {
  extern __shared__ __align__(16) uint8_t merge_smem[];
  uint8_t* a_tile = merge_smem;                                           // [r][kMergeCols] codes of A~
  float* sdb = reinterpret_cast<float*>(merge_smem + (size_t)r * kMergeCols);  // [kMergeRows][r]
  __shared__ int srow[kMergeRows];
  const int g0 = blockIdx.y * kMergeRows;
  const int nrows = min(kMergeRows, k - g0);
  const int64_t cta_c0 = (int64_t)blockIdx.x * kMergeCols;
  const int cta_cols = static_cast<int>(min((int64_t)kMergeCols, n - cta_c0));   // multiple of 16
  if (threadIdx.x < kMergeRows) srow[threadIdx.x] = (threadIdx.x < nrows) ? sel_idx[g0 + threadIdx.x] : -1;
  // stage A~ (rows m.. of W~')
  const uint8_t* aq = wq + m * n + cta_c0;
  const int vec_per_row = cta_cols / 16;
  for (int e = threadIdx.x; e < r * vec_per_row; e += kMergeThreads) {
    const int j = e / vec_per_row, v = e - j * vec_per_row;
    *reinterpret_cast<uint4*>(a_tile + (size_t)j * kMergeCols + v * 16) =
        __ldg(reinterpret_cast<const uint4*>(aq + (int64_t)j * n + v * 16));
  }
  __syncthreads();
  for (int e = threadIdx.x; e < kMergeRows * r; e += kMergeThreads) {
    const int q = e / r, j = e - q * r;
    sdb[e] = (q < nrows) ? dbuf[(int64_t)srow[q] * r + j] : 0.0f;
  }
  __syncthreads();
  const int tx = threadIdx.x % kMergeTx, ty = threadIdx.x / kMergeTx;
  const int lc = tx * kMergeColsPerThread;
  if (lc >= cta_cols) return;
  const int64_t c0 = cta_c0 + lc;
  const int q0 = ty * kMergeRowsPerThread;
  float v[kMergeRowsPerThread][kMergeColsPerThread];
#pragma unroll
  for (int q = 0; q < kMergeRowsPerThread; ++q) {
    uint2 w = make_uint2(0u, 0u);
    if (q0 + q < nrows) w = *reinterpret_cast<const uint2*>(wq + (int64_t)srow[q0 + q] * n + c0);
    decode8(w, v[q]);
  }
  const float* d0 = sdb + q0 * r;
#pragma unroll 4
  for (int j = 0; j < r; ++j) {
    float a[8];
    decode8(*reinterpret_cast<const uint2*>(a_tile + (size_t)j * kMergeCols + lc), a);
#pragma unroll
    for (int q = 0; q < kMergeRowsPerThread; ++q) {
      const float d = d0[q * r + j];
#pragma unroll
      for (int c = 0; c < kMergeColsPerThread; ++c) v[q][c] = __fmaf_rn(d, a[c], v[q][c]);
    }
  }
#pragma unroll
  for (int q = 0; q < kMergeRowsPerThread; ++q) {
    if (q0 + q < nrows) {
      uint2 o;
      o.x = cvt_fp8x4<kE4M3>(v[q][0], v[q][1], v[q][2], v[q][3]);
      o.y = cvt_fp8x4<kE4M3>(v[q][4], v[q][5], v[q][6], v[q][7]);
      *reinterpret_cast<uint2*>(wq + (int64_t)srow[q0 + q] * n + c0) = o;
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
  topk_kernel<<<1, kTopkThreads, 0, stream>>>(score, static_cast<int>(m), static_cast<int>(k), sel_idx,
                                              static_cast<int32_t*>(scratch));
  return cudaGetLastError();
}

cudaError_t launch_merge_rows(uint8_t* wq, float* dbuf, const int32_t* sel_idx, int64_t k, int64_t m, int64_t n,
                              int64_t r, cudaStream_t stream) {
  dim3 grid(static_cast<unsigned>((n + kMergeCols - 1) / kMergeCols),
            static_cast<unsigned>((k + kMergeRows - 1) / kMergeRows));
  const size_t smem = static_cast<size_t>(r) * kMergeCols + sizeof(float) * kMergeRows * r;
  static bool configured = false;
  if (!configured) {
    cudaError_t ea = cudaFuncSetAttribute(merge_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
    if (ea != cudaSuccess) return ea;
    configured = true;
  }
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
