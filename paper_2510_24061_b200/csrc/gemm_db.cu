// Adapter gradient (Eq. lora_backward_modified, Alg. 3):  dB = g~^T O~_A / (s_g s_OA), one kernel.
// The product contracts over the tokens, is skinny (N = r) and therefore bound by how fast g~ streams in, so the
// tokens are split into slabs and a CTA owns one (128-row tile of dB, slab) pair:
//   warp 0      TMA producer: g~ tiles ([tokens][m], read MN-major as the A operand) and O~_A^T tiles (K-major B)
//   warp 1      tcgen05.mma issuer, accumulator 128 x r16 fp32 in TMEM
//   warps 2..5  drain the accumulator and run the slab sum
// The CTAs of one row tile (one per slab) form a thread-block cluster.  Each leaves its 128 x r partial sums in
// its own shared memory; after a cluster barrier, CTA s of the cluster sums rows [s R, (s+1) R) of the tile over
// all slabs, in slab order, reading the other CTAs' partials through distributed shared memory, scales them and
// writes dB.  The sum is deterministic, the reduction is spread over all CTAs, and no partial sum touches global
// memory.  (O~_A is cast, transposed, by a rider of the output-gradient quantizer.)
#include <cuda.h>

#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

constexpr int kDbThreads = 192;
constexpr int kDbEpilogueWarps = 4;
constexpr int kDbBlock = 128;                       // rows of dB per CTA = tokens per k-block = bytes per swizzle row
constexpr uint32_t kDbATileBytes = kDbBlock * kDbBlock;   // 16 KB of g~ per k-block
constexpr int kDbStages = 4;
constexpr int kDbUmmaK = 32;
constexpr int kDbMaxSplits = 4;                     // cluster size: small clusters pack onto the SMs without gaps

struct DbParams {
  int m, r, r16;
  long long T;
  int m_tiles, splits, kblocks_total, kblocks_per_split;   // splits = cluster size (a slab may be empty)
  uint32_t idesc, tmem_cols;
  const float* s_oa;        // [1]
  const float* s_g;         // [1]
  const float* row_mul;     // nullable [m]
  float* dB;                // [m][r], nullable when the update below is fused
  float* dbuf;              // nullable [m][r]: DeltaBuffer <- fma(neg_lr, dB, DeltaBuffer) (Alg. 3 line 4, plain SGD) ...
  float* score;             // ... and [m]: score_i = sum_j |DeltaBuffer_ij|, fp32, j ascending
  float neg_lr;
  int* status;
};

__global__ void __launch_bounds__(kDbThreads, 2)
db_fused_kernel(const __grid_constant__ CUtensorMap tmap_g, const __grid_constant__ CUtensorMap tmap_oa, const DbParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t smem_base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - raw_addr);

  const uint32_t b_tile_bytes = static_cast<uint32_t>(p.r16) * kDbBlock;   // r16 rows of 128 token bytes
  const uint32_t stage_bytes = kDbATileBytes + b_tile_bytes;               // a multiple of 2 KB
  constexpr int S = kDbStages;
  const uint32_t bars = smem_base + S * stage_bytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (S + s); };
  const uint32_t tmem_full_bar = bars + 8u * (2 * S);
  const uint32_t slot_off = S * stage_bytes + 8u * (2 * S + 1);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + slot_off);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    prefetch_tensor_map(&tmap_g);
    prefetch_tensor_map(&tmap_oa);
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);                     // the TMA producer's arrive.expect_tx
      mbar_init(empty_bar(s), 1);                    // one tcgen05.commit
    }
    mbar_init(tmem_full_bar, 1);
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
  pdl_wait();   // everything above is private set-up

  const int m_idx = static_cast<int>(blockIdx.x) / p.splits;     // the cluster = the slabs of one row tile
  const int split = static_cast<int>(cluster_ctarank());
  const int kb_begin = min(split * p.kblocks_per_split, p.kblocks_total);
  const int kb_end = min(kb_begin + p.kblocks_per_split, p.kblocks_total);   // kb_begin == kb_end: an empty slab
  bool aborted = false;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    int stage = 0;
    uint32_t phase = 0;
    for (int kb = kb_begin; kb < kb_end; ++kb) {
      if (!mbar_wait_warp(empty_bar(stage), phase ^ 1u, p.status)) { aborted = true; break; }
      if (elect_one()) {
        mbar_expect_tx(full_bar(stage), stage_bytes);
        tma_load_2d(smem_base + stage * stage_bytes, &tmap_g, full_bar(stage), m_idx * kDbBlock, kb * kDbBlock);
        tma_load_2d(smem_base + stage * stage_bytes + kDbATileBytes, &tmap_oa, full_bar(stage), kb * kDbBlock, 0);
      }
      __syncwarp();
      if (++stage == S) { stage = 0; phase ^= 1u; }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    int stage = 0;
    uint32_t phase = 0;
    const uint64_t a_desc0 = make_smem_desc(smem_base, kDbATileBytes, 1024);          // MN-major: 128 x 128 chunk
    const uint64_t b_desc0 = make_smem_desc(smem_base + kDbATileBytes, 16, 1024);     // K-major
    constexpr uint32_t kAStep = (kDbUmmaK * 128) >> 4;   // per K step, in 16-byte units
    constexpr uint32_t kBStep = kDbUmmaK >> 4;
    for (int kb = kb_begin; kb < kb_end; ++kb) {
      if (!mbar_wait_warp(full_bar(stage), phase, p.status)) { aborted = true; break; }
      tc_fence_after_sync();
      const uint32_t stage_off = (static_cast<uint32_t>(stage) * stage_bytes) >> 4;
      if (elect_one()) {
#pragma unroll
        for (int k = 0; k < kDbBlock / kDbUmmaK; ++k)
          umma_f8(tmem_base, a_desc0 + stage_off + k * kAStep, b_desc0 + stage_off + k * kBStep, p.idesc,
                  (kb > kb_begin || k > 0) ? 1u : 0u);
        umma_commit(empty_bar(stage));
      }
      __syncwarp();
      if (++stage == S) { stage = 0; phase ^= 1u; }
    }
    if (!aborted && kb_end > kb_begin) {
      if (elect_one()) umma_commit(tmem_full_bar);
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    // ---- epilogue: this warp owns TMEM lanes [32 quad, 32 quad + 32) = rows of the tile; the partial sums go to
    // this CTA's shared memory (over the stage buffers, which the finished MMAs no longer read), rows padded by
    // four floats against bank conflicts
    const bool have_acc = kb_end > kb_begin;
    if (!aborted && have_acc && !mbar_wait_warp(tmem_full_bar, 0u, p.status)) aborted = true;
    if (!aborted) {
      tc_fence_after_sync();
      const int quad = warp & 3;
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
      float* my_row = reinterpret_cast<float*>(smem_gen) + (quad * 32 + lane) * (p.r + 4);
      for (int c0 = 0; c0 < p.r; c0 += 32) {
        uint32_t v[32];
        if (have_acc) {
          tmem_ld_32x32b_x32(t_row + static_cast<uint32_t>(c0), v);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = 0u;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (c0 + 4 * i < p.r)
            reinterpret_cast<uint4*>(my_row + c0)[i] = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
      }
      tc_fence_before_sync();
    }
  }

  // ------------------------------------------------------------ slab sum across the cluster (every thread passes
  // both cluster barriers, also after a timeout, so that no CTA of the cluster is left waiting)
  constexpr int kU = 4;   // positions per thread whose loads (all slabs) are issued before the first add
  const int tidc = static_cast<int>(threadIdx.x) - 64;
  const int rows_per_cta = (kDbBlock + p.splits - 1) / p.splits;
  const int r4 = p.r >> 2;
  const int row_begin = split * rows_per_cta;
  const int row_end = min(row_begin + rows_per_cta, kDbBlock);
  // fused optimizer step: the DeltaBuffer values of this thread's first positions are fetched before the cluster barrier,
  // so their latency overlaps the wait for the other slabs
  float4 dpre[kU];
  if (warp >= 2 && p.dbuf != nullptr) {
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int e = tidc + u * kDbEpilogueWarps * 32;
      const int row = m_idx * kDbBlock + row_begin + e / r4;
      dpre[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (e < (row_end - row_begin) * r4 && row < p.m)
        dpre[u] = ld_stream(reinterpret_cast<const float4*>(p.dbuf + static_cast<long long>(row) * p.r + 4 * (e % r4)));
    }
  }
  cluster_arrive();
  cluster_wait();
  if (warp >= 2) {
    const float inv = 1.0f / (ld_stream(p.s_g) * ld_stream(p.s_oa));
    const uint32_t local = smem_base;   // the partial tile starts at the (1 KB aligned) base in every CTA of the cluster
    const int total = (row_end - row_begin) * r4;
    // fused optimizer step: |DeltaBuffer| of this CTA's rows, behind the partial tile, row pitch r + 1 floats
    float* abs_rows = reinterpret_cast<float*>(smem_gen) + kDbBlock * (p.r + 4);
    for (int e0 = tidc; e0 < total; e0 += kU * kDbEpilogueWarps * 32) {
      float4 y[kU][kDbMaxSplits];
#pragma unroll
      for (int u = 0; u < kU; ++u) {
        const int e = e0 + u * kDbEpilogueWarps * 32;
        const int row_l = row_begin + e / r4, c4 = e % r4;
        const uint32_t off = static_cast<uint32_t>(row_l * (p.r + 4) + 4 * c4) * 4u;
#pragma unroll
        for (int sidx = 0; sidx < kDbMaxSplits; ++sidx)
          if (e < total && sidx < p.splits)
            y[u][sidx] = ld_shared_cluster_f32x4(map_to_cta(local + off, static_cast<uint32_t>(sidx)));
      }
#pragma unroll
      for (int u = 0; u < kU; ++u) {
        const int e = e0 + u * kDbEpilogueWarps * 32;
        const int row_l = row_begin + e / r4, c4 = e % r4;
        const int row = m_idx * kDbBlock + row_l;
        if (e >= total || row >= p.m) continue;
        float4 acc = y[u][0];
#pragma unroll
        for (int sidx = 1; sidx < kDbMaxSplits; ++sidx)
          if (sidx < p.splits) { acc.x += y[u][sidx].x; acc.y += y[u][sidx].y; acc.z += y[u][sidx].z; acc.w += y[u][sidx].w; }
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        if (p.row_mul != nullptr) {
          const float f = ld_stream(p.row_mul + row);
          acc.x *= f; acc.y *= f; acc.z *= f; acc.w *= f;
        }
        if (p.dB != nullptr) *reinterpret_cast<float4*>(p.dB + static_cast<long long>(row) * p.r + 4 * c4) = acc;
        if (p.dbuf != nullptr) {   // one fma per element on the value dB holds, exactly as the separate pass would
          float4* dp = reinterpret_cast<float4*>(p.dbuf + static_cast<long long>(row) * p.r + 4 * c4);
          float4 d = e0 == tidc ? dpre[u] : ld_stream(dp);
          d.x = __fmaf_rn(p.neg_lr, acc.x, d.x); d.y = __fmaf_rn(p.neg_lr, acc.y, d.y);
          d.z = __fmaf_rn(p.neg_lr, acc.z, d.z); d.w = __fmaf_rn(p.neg_lr, acc.w, d.w);
          *dp = d;
          float* a = abs_rows + (row_l - row_begin) * (p.r + 1) + 4 * c4;
          a[0] = fabsf(d.x); a[1] = fabsf(d.y); a[2] = fabsf(d.z); a[3] = fabsf(d.w);
        }
      }
    }
    if (p.dbuf != nullptr) {
      asm volatile("bar.sync 1, %0;" ::"n"(kDbEpilogueWarps * 32) : "memory");   // the four epilogue warps only
      const int row_l = row_begin + tidc;
      const int row = m_idx * kDbBlock + row_l;
      if (row_l < row_end && row < p.m) {
        const float* a = abs_rows + tidc * (p.r + 1);
        float sc = 0.0f;
#pragma unroll 8
        for (int j = 0; j < p.r; ++j) sc = __fadd_rn(sc, a[j]);   // strictly left to right
        p.score[row] = sc;
      }
    }
  }
  cluster_arrive();   // nobody leaves (and frees its shared memory) while a neighbour may still read it
  cluster_wait();

  // ------------------------------------------------------------ common exit
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

}  // namespace

namespace {
int db_splits(int64_t m, int64_t T) {
  const int m_tiles = static_cast<int>((m + kDbBlock - 1) / kDbBlock);
  const int kblocks = static_cast<int>((T + kDbBlock - 1) / kDbBlock);
  // slabs per row tile = cluster size: a power of two up to kDbMaxSplits, enough for two CTAs on every SM
  const int want = (2 * sm_count() + m_tiles - 1) / m_tiles;
  int splits = 1;
  while (splits * 2 <= kDbMaxSplits && splits * 2 <= want && splits * 2 <= kblocks) splits *= 2;
  return splits;
}
}  // namespace

// The fused optimizer step parks |DeltaBuffer| of a CTA's rows behind the 128 x (r + 4) partial tile, inside the drained
// operand ring; it needs that much room.
bool db_fused_update_fits(int64_t m, int64_t r, int64_t T) {
  const int splits = db_splits(m, T);
  const int64_t r16 = round_up(r, 16);
  const int64_t ring = static_cast<int64_t>(kDbStages) * (kDbATileBytes + r16 * kDbBlock);
  const int64_t rows_per_cta = (kDbBlock + splits - 1) / splits;
  return 4 * (kDbBlock * (r + 4) + rows_per_cta * (r + 1)) <= ring;
}

cudaError_t launch_db_fused(const DbFusedProblem& q, cudaStream_t stream) {
  if (q.m < 1 || q.T < 1 || q.r < 8 || q.r > 256 || q.r % 8) return cudaErrorInvalidValue;
  DbParams p{};
  p.m = static_cast<int>(q.m); p.r = static_cast<int>(q.r); p.r16 = static_cast<int>(round_up(q.r, 16));
  p.T = q.T;
  p.m_tiles = static_cast<int>((q.m + kDbBlock - 1) / kDbBlock);
  p.kblocks_total = static_cast<int>((q.T + kDbBlock - 1) / kDbBlock);
  const int splits = db_splits(q.m, q.T);
  p.splits = splits;
  p.kblocks_per_split = (p.kblocks_total + splits - 1) / splits;
  // instruction descriptor: fp32 accumulate, A = E5M2 MN-major, B = E4M3 K-major, N = r16, M = 128
  p.idesc = (1u << 4) | (static_cast<uint32_t>(q.g_is_e4m3 ? kE4M3 : kE5M2) << 7) | (static_cast<uint32_t>(kE4M3) << 10) | (1u << 15) |
            (static_cast<uint32_t>(p.r16 >> 3) << 17) | (static_cast<uint32_t>(kDbBlock >> 4) << 24);
  uint32_t cols = 32;
  while (cols < static_cast<uint32_t>(p.r16)) cols <<= 1;
  p.tmem_cols = cols;
  p.s_oa = q.s_oa;
  p.s_g = q.s_g; p.row_mul = q.row_mul; p.dB = q.dB; p.status = q.status;
  p.dbuf = q.dbuf; p.score = q.score; p.neg_lr = q.neg_lr;
  if ((q.dbuf != nullptr) != (q.score != nullptr) || (q.dbuf == nullptr && q.dB == nullptr)) return cudaErrorInvalidValue;
  if (q.dbuf != nullptr && !db_fused_update_fits(q.m, q.r, q.T)) return cudaErrorInvalidValue;
  CUtensorMap tg, toa;
  if (!make_tensor_map(&tg, q.gq, q.T, q.m, q.m, kDbBlock, kDbBlock)) return cudaErrorInvalidValue;
  if (!make_tensor_map(&toa, q.oaq_t, p.r16, q.T, q.ldt, kDbBlock, static_cast<uint32_t>(p.r16))) return cudaErrorInvalidValue;
  const size_t smem = static_cast<size_t>(kDbStages) * (kDbATileBytes + static_cast<size_t>(p.r16) * kDbBlock) + 128 + 1024;
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(db_fused_kernel, 227 * 1024, configured);
    if (ec != cudaSuccess) return ec;
  }
  const unsigned grid = static_cast<unsigned>(p.m_tiles) * static_cast<unsigned>(splits);
  return launch_pdl(db_fused_kernel, dim3(grid), dim3(kDbThreads), smem, stream, splits, tg, toa, p);
}

}  // namespace falqon
