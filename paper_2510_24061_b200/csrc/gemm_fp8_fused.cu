// The FP8 products of the melded layer with the cast of their A operand fused into the producer (Alg. 2 lines 5-6,
// Alg. 3 with Eq. quantize): the activations X (forward) or the output gradient dY (input-gradient product) arrive as
// bf16, and their E4M3 / E5M2 codes exist only in shared memory -- no separate cast pass writes them to memory and reads
// them back.  Same tiling and the same MMA sequence as gemm_fp8_pair_kernel (256 x 256 tiles on CTA pairs,
// tcgen05.mma cta_group::2, double-buffered accumulators in tensor memory), so for the same codes the results are
// the same bit for bit.  Warp roles per CTA:
//   warp 0          TMA producer: per k-block the CTA's 128 x 128 bf16 rows of A (32 KB, no swizzle, onto the
//                   CTA's own "landed" barrier) and its half of the B tile (16 KB of codes, 128-byte swizzle, counted
//                   on the leader's "full" barrier)
//   warp 1          MMA issuer (leader CTA); warps 2, 3 idle
//   warps 4..11     epilogue
//   warps 12..19    converters: wait for the bf16 rows, scale and round them IN PLACE into the swizzled K-major
//                   operand layout (convert_tile.cuh), fence them towards the asynchronous proxy and arrive on the
//                   LEADER's "full" barrier -- the leader's MMAs read the A rows of both CTAs
// A stage is 48 KB (32 KB A, of which the codes take the first half of every 2 KB row group, + 16 KB B); four stages.
// The tiles of one chosen column block can also write the codes they staged to global memory: the adapter-gradient
// product needs g~ as a tensor, and the tests compare the staged codes with the oracle's cast.
// Every wait is bounded; on a timeout the CTA records it, drains and frees its tensor memory.
#include <cuda.h>

#include "convert_tile.cuh"
#include "gemm_common.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

// Warp groups (4 warps each; the register hand-over below works on whole groups): 0 = TMA producer, MMA issuer and two
// idle warps; 1-2 = epilogue; 3-4 = converters.
constexpr int kConvWarps = 8;
constexpr int kEpiFirstWarp = 4;
constexpr int kConvFirstWarp = kEpiFirstWarp + static_cast<int>(kEpilogueWarps);
constexpr int kFusedThreads = 32 * (kConvFirstWarp + kConvWarps);   // 640
// The kernel starts with 96 registers per thread (65536 / 640); the light groups then hand registers to the epilogue.
constexpr int kRegsAtLaunch = 96, kRegsLight = 24, kRegsConv = 80, kRegsEpi = 144;
static_assert(128 * kRegsLight + 32 * kConvWarps * kRegsConv + 32 * static_cast<int>(kEpilogueWarps) * kRegsEpi <=
              kFusedThreads * kRegsAtLaunch, "register pool of the CTA");
constexpr uint32_t kFusedATileBytes = 2 * kATileBytes;                       // bf16 rows; the codes overwrite them
constexpr uint32_t kFusedBTileBytes = 128 * kBlockKBytes;                    // this CTA's half of the B tile
constexpr uint32_t kFusedStageBytes = kFusedATileBytes + kFusedBTileBytes;   // 48 KB
constexpr int kFusedStages = 4;
static_assert(kFusedStages * kFusedStageBytes + kBarrierBytes + kStagingBytes + 1024 <= kSmemBudget, "shared memory");
static_assert(kConvGroupsPerTile % kConvWarps == 0, "row groups per converter warp");

struct FusedParams {
  float const* a_scale;
  uint8_t* emit_dst;
  long long emit_ld;
  int emit_n_block;
};

template <bool kBMn, int kAFmt>
__global__ void __launch_bounds__(kFusedThreads, 1)
gemm_fp8_pair_fused_kernel(const __grid_constant__ CUtensorMap tmap_a16, const __grid_constant__ CUtensorMap tmap_b,
                           const GemmParams p, const FusedParams fp) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t smem_base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - raw_addr);

  constexpr int S = kFusedStages;
  const uint32_t bars = smem_base + static_cast<uint32_t>(S) * kFusedStageBytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };             // leader: B bytes of both CTAs + all converter warps
  auto empty_bar = [&](int s) { return bars + 8u * (S + s); };      // one multicast commit
  auto landed_bar = [&](int s) { return bars + 8u * (2 * S + s); };  // this CTA's bf16 rows have arrived
  auto tmem_full_bar = [&](int a) { return bars + 8u * (3 * S + a); };
  auto tmem_empty_bar = [&](int a) { return bars + 8u * (3 * S + 2 + a); };
  const uint32_t slot_off = static_cast<uint32_t>(S) * kFusedStageBytes + 8u * (3 * S + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + slot_off);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();       // 0 = leader
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    prefetch_tensor_map(&tmap_a16);
    prefetch_tensor_map(&tmap_b);
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1 + 2 * kConvWarps);   // the leader's arrive.expect_tx + one arrival per converter warp of the pair
      mbar_init(empty_bar(s), 1);
      mbar_init(landed_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tmem_full_bar(a), 1);
      mbar_init(tmem_empty_bar(a), 2 * kEpilogueWarps);
    }
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_base + slot_off, kTmemCols);
    tmem_relinquish_pair();
  }
  pdl_trigger();
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive();      // the peer's barriers must be initialised before anything signals them
  cluster_wait();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();   // everything above is private set-up; operands and scales are read only from here on

  const int num_pairs = gridDim.x >> 1;
  const int pair = blockIdx.x >> 1;
  const int total_tiles = p.m_tiles * p.n_tiles;   // m_tiles counts 256-row pair tiles
  bool aborted = false;

  // Register hand-over, first thing in every role: the producer / issuer group and the converters shrink, the
  // epilogue groups grow.
  if (warp < kEpiFirstWarp) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsLight));
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    int stage = 0;
    uint32_t phase = 0;
    for (int tile = pair; tile < total_tiles && !aborted; tile += num_pairs) {
      const int n_idx = tile / p.m_tiles;
      const int m_idx = tile - n_idx * p.m_tiles;
      const int n0 = n_idx * 256;
      const int n_inst = pair_instr_n<kBMn>(p.N - n0);
      const int row0 = m_idx * 256 + static_cast<int>(rank) * kBlockM;
      const int bn0 = n0 + static_cast<int>(rank) * (n_inst >> 1);
      for (int kb = 0; kb < p.kblocks_total; ++kb) {
        if (!mbar_wait_warp(empty_bar(stage), phase ^ 1u, p.status)) { aborted = true; break; }
        if (elect_one()) {
          const uint32_t a_dst = smem_base + static_cast<uint32_t>(stage) * kFusedStageBytes;
          const uint32_t b_dst = a_dst + kFusedATileBytes;
          mbar_expect_tx(landed_bar(stage), kFusedATileBytes);
          tma_load_2d(a_dst, &tmap_a16, landed_bar(stage), kb * kBlockKBytes, row0);   // coordinates in elements
          if (leader) mbar_expect_tx(full_bar(stage), 2 * kFusedBTileBytes);
          const uint32_t fb = map_to_cta(full_bar(stage), 0);
          if (!kBMn) tma_load_2d_pair(b_dst, &tmap_b, fb, kb * kBlockKBytes, bn0);
          else       tma_load_2d_pair(b_dst, &tmap_b, fb, bn0, kb * kBlockKBytes);
        }
        __syncwarp();
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
    }
    for (int i = 0; i < S && !aborted; ++i) {   // tail: every stage released, so no signal can reach a CTA that has left
      if (!mbar_wait_warp(empty_bar(stage), phase ^ 1u, p.status)) aborted = true;
      if (++stage == S) { stage = 0; phase ^= 1u; }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA; one lane issues)
    if (leader) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      const uint64_t a_desc0 = make_smem_desc(smem_base, 16, kConvGroupBytes);   // 8-row groups 2 KB apart
      const uint64_t b_desc0 = kBMn ? make_smem_desc(smem_base + kFusedATileBytes, kMnChunkBytes, 1024)
                                    : make_smem_desc(smem_base + kFusedATileBytes, 16, 1024);
      constexpr uint32_t kAStep = kUmmaK >> 4;
      constexpr uint32_t kBStep = (kBMn ? kUmmaK * 128 : kUmmaK) >> 4;
      for (int tile = pair; tile < total_tiles && !aborted; tile += num_pairs) {
        const int n_idx = tile / p.m_tiles;
        const int n0 = n_idx * 256;
        const int n_inst = pair_instr_n<kBMn>(p.N - n0);
        const uint32_t idesc = p.idesc | (static_cast<uint32_t>(n_inst >> 3) << 17);
        if (!mbar_wait_warp(tmem_empty_bar(acc), acc_phase ^ 1u, p.status)) { aborted = true; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc) * kAccCols;
        for (int kb = 0; kb < p.kblocks_total; ++kb) {
          if (!mbar_wait_warp(full_bar(stage), phase, p.status)) { aborted = true; break; }
          tc_fence_after_sync();
          const uint32_t stage_off = (static_cast<uint32_t>(stage) * kFusedStageBytes) >> 4;
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < kBlockKBytes / kUmmaK; ++k) {
              umma_f8_pair(d_tmem, a_desc0 + stage_off + k * kAStep, b_desc0 + stage_off + k * kBStep, idesc,
                           (kb > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit_pair(empty_bar(stage), 3);
          }
          __syncwarp();
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
        if (aborted) break;
        if (elect_one()) umma_commit_pair(tmem_full_bar(acc), 3);
        __syncwarp();
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  }   // warps 2 and 3 only fill up the first warp group
  } else if (warp < kConvFirstWarp) {
    // ------------------------------------------------------------ epilogue (warps 4..11 of each CTA)
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsEpi));
    const int quad = warp & 3;
    const int col_half = (warp - kEpiFirstWarp) >> 2;
    uint8_t* stage_out = smem_gen + static_cast<uint32_t>(S) * kFusedStageBytes + kBarrierBytes + (warp - kEpiFirstWarp) * kStageOutBytes;
    const bool rescale = p.scale_a != nullptr;
    const float inv = rescale ? 1.0f / (p.scale_b != nullptr ? ld_stream(p.scale_a) * ld_stream(p.scale_b) : ld_stream(p.scale_a)) : 1.0f;
    int acc = 0;
    uint32_t acc_phase = 0;
    uint32_t amax_bits = 0;
    for (int tile = pair; tile < total_tiles && !aborted; tile += num_pairs) {
      const int n_idx = tile / p.m_tiles;
      const int m_idx = tile - n_idx * p.m_tiles;
      if (!mbar_wait(tmem_full_bar(acc), acc_phase, p.status)) { aborted = true; break; }
      tc_fence_after_sync();
      const int row = m_idx * 256 + static_cast<int>(rank) * kBlockM + quad * 32 + lane;
      const bool row_ok = row < p.M;
      const uint32_t t_row = tmem_base + static_cast<uint32_t>(acc) * kAccCols + (static_cast<uint32_t>(quad * 32) << 16);
      const int n0 = n_idx * 256;
      epilogue_tile(p, t_row, row, row_ok, n0, col_half ? 128 : 0, col_half ? 256 : 128, inv, amax_bits, stage_out);
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(tmem_empty_bar(acc), 0));
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    if (p.amax1_bits != nullptr) {
      amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
      if (lane == 0 && amax_bits != 0) atomicMax(p.amax1_bits, amax_bits);
    }
  } else {
    // ------------------------------------------------------------ converters: bf16 rows -> codes, in place
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsConv));
    const int cw = warp - kConvFirstWarp;
    const float s = ld_stream(fp.a_scale);
    const uint32_t full_leader = map_to_cta(full_bar(0), 0);
    int stage = 0;
    uint32_t phase = 0;
    for (int tile = pair; tile < total_tiles && !aborted; tile += num_pairs) {
      const int n_idx = tile / p.m_tiles;
      const int m_idx = tile - n_idx * p.m_tiles;
      const int row0 = m_idx * 256 + static_cast<int>(rank) * kBlockM;
      const bool emit = fp.emit_dst != nullptr && n_idx == fp.emit_n_block;
      for (int kb = 0; kb < p.kblocks_total; ++kb) {
        if (!mbar_wait_warp(landed_bar(stage), phase, p.status)) { aborted = true; break; }
        uint8_t* a_tile = smem_gen + static_cast<uint32_t>(stage) * kFusedStageBytes;
        const int k0 = kb * kBlockKBytes;
#pragma unroll
        for (int g = cw; g < kConvGroupsPerTile; g += 2 * kConvWarps) {   // two row groups in flight per lane
          const int g1 = g + kConvWarps;
          uint4 q0[4], q1[4];
          convert_group_load(a_tile + g * kConvGroupBytes, lane, q0);
          convert_group_load(a_tile + g1 * kConvGroupBytes, lane, q1);
          __syncwarp();      // every lane holds its pieces of both groups: the codes may now overwrite them
          uint8_t* e0 = emit ? fp.emit_dst + static_cast<long long>(row0 + g * 8) * fp.emit_ld + k0 : nullptr;
          uint8_t* e1 = emit ? fp.emit_dst + static_cast<long long>(row0 + g1 * 8) * fp.emit_ld + k0 : nullptr;
          convert_group_store<kAFmt>(a_tile + g * kConvGroupBytes, lane, q0, s, e0, fp.emit_ld, p.M - (row0 + g * 8), p.K - k0);
          convert_group_store<kAFmt>(a_tile + g1 * kConvGroupBytes, lane, q1, s, e1, fp.emit_ld, p.M - (row0 + g1 * 8), p.K - k0);
        }
        fence_proxy_async_smem();    // each lane's codes, towards the tensor core's reads
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(full_leader + 8u * stage);   // CTA-scope release: a cluster-wide one costs ~1000 cycles here
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
    }
  }

  // ------------------------------------------------------------ common exit
  if (aborted) {
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) { }
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive();      // neither CTA frees its TMEM or leaves while the other may still signal it
  cluster_wait();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

template <bool kBMn, int kAFmt>
cudaError_t launch_fused_variant(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& gp, const FusedParams& fp,
                                 int grid, size_t smem, cudaStream_t stream) {
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(gemm_fp8_pair_fused_kernel<kBMn, kAFmt>, static_cast<int>(kSmemBudget), configured);
    if (ec != cudaSuccess) return ec;
  }
  return launch_pdl(gemm_fp8_pair_fused_kernel<kBMn, kAFmt>, dim3(static_cast<unsigned>(grid)), dim3(kFusedThreads), smem, stream, 2,
                    ta, tb, gp, fp);
}

}  // namespace

bool gemm_fp8_fused_supported(const GemmProblem& q) {
  return q.M > 0 && q.N > 0 && q.K > 0 && q.block_n == 256 && q.N % 16 == 0 && q.K % 16 == 0;
}

cudaError_t launch_gemm_fp8_fused(const GemmProblem& q, const FusedOperand& f, cudaStream_t stream) {
  if (!gemm_fp8_fused_supported(q) || f.a16 == nullptr || f.a_scale == nullptr || f.lda16 < q.K || f.lda16 % 8 != 0)
    return cudaErrorInvalidValue;
  if (f.emit_dst != nullptr && (f.emit_ld < q.K || f.emit_ld % 16 != 0)) return cudaErrorInvalidValue;
  GemmParams gp{};
  gp.M = static_cast<int>(q.M); gp.N = static_cast<int>(q.N); gp.K = static_cast<int>(q.K);
  gp.block_n = 256;
  gp.m_tiles = static_cast<int>((q.M + 255) / 256);
  gp.n_tiles = static_cast<int>((q.N + 255) / 256);
  gp.kblocks_total = static_cast<int>((q.K + kBlockKBytes - 1) / kBlockKBytes);
  gp.num_stages = kFusedStages;
  gp.idesc = (1u << 4) | (static_cast<uint32_t>(q.a_fmt) << 7) | (static_cast<uint32_t>(q.b_fmt) << 10) |
             ((q.b_mn_major ? 1u : 0u) << 16) | (static_cast<uint32_t>(256 >> 4) << 24);
  gp.c0 = q.c0; gp.ldc0 = q.ldc0; gp.c0_dt = q.c0_dt; gp.n_split = static_cast<int>(q.n_split);
  gp.c1 = q.c1; gp.ldc1 = q.ldc1; gp.amax1_bits = q.amax1_bits;
  gp.scale_a = q.scale_a; gp.scale_b = q.scale_b; gp.col_scale = q.col_scale;
  gp.status = q.status;
  const FusedParams fp{f.a_scale, f.emit_dst, static_cast<long long>(f.emit_ld), f.emit_dst != nullptr ? f.emit_n_block : -1};
  CUtensorMap ta, tb;
  if (!make_tensor_map_u16(&ta, f.a16, q.M, q.K, f.lda16, kBlockKBytes, kBlockM)) return cudaErrorInvalidValue;
  const bool ok = q.b_mn_major ? make_tensor_map(&tb, q.b, q.K, q.N, q.ldb, 128, kBlockKBytes)
                               : make_tensor_map(&tb, q.b, q.N, q.K, q.ldb, kBlockKBytes, 128);
  if (!ok) return cudaErrorInvalidValue;
  const long long total_tiles = static_cast<long long>(gp.m_tiles) * gp.n_tiles;
  long long pairs = sm_count() / 2;
  if (total_tiles < pairs) pairs = total_tiles;
  const int grid = static_cast<int>(pairs * 2);
  const size_t smem = static_cast<size_t>(kFusedStages) * kFusedStageBytes + kBarrierBytes + kStagingBytes + 1024;
#define FALQON_FUSED_GEMM(MN, FMT) return launch_fused_variant<MN, FMT>(ta, tb, gp, fp, grid, smem, stream)
  if (q.b_mn_major) { if (q.a_fmt == kE4M3) FALQON_FUSED_GEMM(true, kE4M3); FALQON_FUSED_GEMM(true, kE5M2); }
  if (q.a_fmt == kE4M3) FALQON_FUSED_GEMM(false, kE4M3);
  FALQON_FUSED_GEMM(false, kE5M2);
#undef FALQON_FUSED_GEMM
}

}  // namespace falqon
