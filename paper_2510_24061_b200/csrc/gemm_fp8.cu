// FP8 GEMM on the 5th-generation tensor cores (tcgen05.mma kind::f8f6f4, fp32 accumulators in
// tensor memory), operands staged by TMA into 128-byte-swizzled shared-memory tiles.
//
//   D[M][N] = A[M][K] * B[N][K]^T      A, B: E4M3 or E5M2 codes (mixed allowed), D: fp32 in TMEM
//
// One persistent CTA per SM walks a static list of 128 x block_n output tiles.  Warp roles:
//   warp 0      TMA producer (one lane): fills a ring of (A,B) stages, signalled through mbarriers
//   warp 1      allocates TMEM; one lane issues the MMAs and commits them to the barriers
//   warps 2..9  epilogue: tcgen05.ld the accumulator, rescale by 1/(s_a*s_b), store
// The accumulator is double buffered (2 x 256 TMEM columns), so the epilogue of tile i overlaps the
// main loop of tile i+1.  A is K-major (rows along K); B may be K-major or MN-major (rows along N): the
// melded forward reads both K-major, the input gradient reads W~ MN-major (no transposed copy of the
// backbone exists).  The adapter gradient, which reads the output gradient MN-major, rides on the CTA-pair form of the
// input-gradient product (see gemm_fp8_pair_kernel) or runs as a kernel of its own (gemm_db.cu).
// Every mbarrier wait is bounded; on a timeout the CTA records it, drains and frees its TMEM.
#include <cuda.h>

#include <cstdlib>

#include "gemm_common.cuh"
#include "grid_sync.cuh"
#include "internal.h"
#include "oa_cast.cuh"
#include "ptx.cuh"

namespace falqon {
namespace {

template <bool kBMn>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_fp8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t smem_base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - raw_addr);

  const uint32_t b_tile_bytes = static_cast<uint32_t>(p.block_n) * kBlockKBytes;
  const uint32_t stage_bytes = kATileBytes + b_tile_bytes;
  const int S = p.num_stages;
  const uint32_t bars = smem_base + static_cast<uint32_t>(S) * stage_bytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (S + s); };
  auto tmem_full_bar = [&](int a) { return bars + 8u * (2 * S + a); };
  auto tmem_empty_bar = [&](int a) { return bars + 8u * (2 * S + 2 + a); };
  const uint32_t slot_off = static_cast<uint32_t>(S) * stage_bytes + 8u * (2 * S + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + slot_off);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    prefetch_tensor_map(&tmap_a);
    prefetch_tensor_map(&tmap_b);
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tmem_full_bar(a), 1);
      mbar_init(tmem_empty_bar(a), kEpilogueWarps);
    }
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_base + slot_off, kTmemCols);
    tmem_relinquish();
  }
  pdl_trigger();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();   // everything above is private set-up; operands and scales are read only from here on

  const int total_tiles = p.m_tiles * p.n_tiles;
  bool aborted = false;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (whole warp loops, one lane issues)
    int stage = 0;
    uint32_t phase = 0;
    for (int tile = blockIdx.x; tile < total_tiles && !aborted; tile += gridDim.x) {
      const int n_idx = tile / p.m_tiles;
      const int m_idx = tile - n_idx * p.m_tiles;
      for (int kb = 0; kb < p.kblocks_total; ++kb) {
        if (!mbar_wait_warp(empty_bar(stage), phase ^ 1u, p.status)) { aborted = true; break; }
        if (elect_one()) {
          const uint32_t fb = full_bar(stage);
          mbar_expect_tx(fb, stage_bytes);
          const uint32_t a_dst = smem_base + static_cast<uint32_t>(stage) * stage_bytes;
          const uint32_t b_dst = a_dst + kATileBytes;
          tma_load_2d(a_dst, &tmap_a, fb, kb * kBlockKBytes, m_idx * kBlockM);
          if (!kBMn) {
            tma_load_2d(b_dst, &tmap_b, fb, kb * kBlockKBytes, n_idx * p.block_n);
          } else {
            for (int c = 0; c < p.block_n / 128; ++c)
              tma_load_2d(b_dst + c * kMnChunkBytes, &tmap_b, fb, n_idx * p.block_n + c * 128, kb * kBlockKBytes);
          }
        }
        __syncwarp();
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (whole warp loops, one lane issues:
    // warp-uniform control flow keeps the descriptor arithmetic on the uniform datapath)
    int stage = 0;
    uint32_t phase = 0;
    int acc = 0;
    uint32_t acc_phase = 0;
    // descriptors differ between stages and K steps only in the 14-bit start-address field
    const uint64_t a_desc0 = make_smem_desc(smem_base, 16, 1024);
    const uint64_t b_desc0 = kBMn ? make_smem_desc(smem_base + kATileBytes, kMnChunkBytes, 1024)
                                  : make_smem_desc(smem_base + kATileBytes, 16, 1024);
    constexpr uint32_t kAStep = kUmmaK >> 4;   // per K step, in 16-byte units
    constexpr uint32_t kBStep = (kBMn ? kUmmaK * 128 : kUmmaK) >> 4;
    for (int tile = blockIdx.x; tile < total_tiles && !aborted; tile += gridDim.x) {
      if (!mbar_wait_warp(tmem_empty_bar(acc), acc_phase ^ 1u, p.status)) { aborted = true; break; }
      tc_fence_after_sync();
      const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc) * kAccCols;
      for (int kb = 0; kb < p.kblocks_total; ++kb) {
        if (!mbar_wait_warp(full_bar(stage), phase, p.status)) { aborted = true; break; }
        tc_fence_after_sync();
        const uint32_t stage_off = (static_cast<uint32_t>(stage) * stage_bytes) >> 4;
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < kBlockKBytes / kUmmaK; ++k) {
            umma_f8(d_tmem, a_desc0 + stage_off + k * kAStep, b_desc0 + stage_off + k * kBStep, p.idesc,
                    (kb > 0 || k > 0) ? 1u : 0u);
          }
          umma_commit(empty_bar(stage));  // frees the stage once these MMAs have read it
        }
        __syncwarp();
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
      if (aborted) break;
      if (elect_one()) umma_commit(tmem_full_bar(acc));  // accumulator complete
      __syncwarp();
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..9)
    const int quad = warp & 3;  // TMEM lanes [32*quad, 32*quad+32) belong to this warp
    const int col_half = (warp - 2) >> 2;   // warps 2..5 drain the left half of the tile, 6..9 the right half
    uint8_t* stage_out = smem_gen + static_cast<uint32_t>(S) * stage_bytes + kBarrierBytes + (warp - 2) * kStageOutBytes;
    const bool rescale = p.scale_a != nullptr;
    const float inv = rescale ? 1.0f / (p.scale_b != nullptr ? ld_stream(p.scale_a) * ld_stream(p.scale_b) : ld_stream(p.scale_a)) : 1.0f;
    int acc = 0;
    uint32_t acc_phase = 0;
    uint32_t amax_bits = 0;
    for (int tile = blockIdx.x; tile < total_tiles && !aborted; tile += gridDim.x) {
      const int n_idx = tile / p.m_tiles;
      const int m_idx = tile - n_idx * p.m_tiles;
      if (!mbar_wait(tmem_full_bar(acc), acc_phase, p.status)) { aborted = true; break; }
      tc_fence_after_sync();
      const int row = m_idx * kBlockM + quad * 32 + lane;
      const bool row_ok = row < p.M;
      const uint32_t t_row = tmem_base + static_cast<uint32_t>(acc) * kAccCols + (static_cast<uint32_t>(quad * 32) << 16);
      const int n0 = n_idx * p.block_n;
      const int half = (((p.block_n + 1) / 2) + 31) & ~31;   // first-half warps take [0, half), the others [half, block_n)
      epilogue_tile(p, t_row, row, row_ok, n0, col_half ? half : 0, col_half ? p.block_n : half, inv, amax_bits, stage_out);
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(tmem_empty_bar(acc));
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    if (p.amax1_bits != nullptr) {
      amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
      if (lane == 0 && amax_bits != 0) atomicMax(p.amax1_bits, amax_bits);
    }
  }

  // ------------------------------------------------------------ common exit
  if (aborted) {
    // give copies and MMAs in flight time to land before the shared memory and TMEM are released
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) { }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}


// ------------------------------------------------------------------ CTA-pair variant (tensor-bound roles)
// Two CTAs of a cluster compute one 256 x 256 tile with tcgen05.mma cta_group::2: each CTA stages its own
// 128 rows of A and only HALF of the B tile (128 of the 256 N rows), the hardware shares the B halves
// between the two tensor cores, and each CTA keeps its 128 accumulator rows in its own TMEM.  Per MMA a
// CTA now moves (128 + 128) x 32 bytes through shared memory instead of (128 + 256) x 32, which is what
// lets the tensor pipe run ahead of the shared-memory port, and the smaller stage (32 KB) buys a deeper
// ring.  The leader CTA (cluster rank 0) issues all MMAs; TMA loads of both CTAs count their bytes on the
// leader's "full" barrier; MMA completion is multicast to both CTAs' "empty" / "accumulator full"
// barriers; both CTAs' epilogue warps arrive on the leader's "accumulator empty" barrier.
// A is K-major; B is K-major or MN-major.  The last N tile is issued with a narrower instruction N.
constexpr uint32_t kPairStageBytes = kATileBytes + 128 * kBlockKBytes;   // 32 KB per CTA per stage

//
// kRider (the input-gradient product only): the adapter gradient dB = g~^T O~_A / (s_g s_OA) rides on the same launch.
// Its A operand is the product's own A tensor g~ [T][m], read through the same tensor map with the coordinates swapped
// (a box of 128 tokens x 128 bytes of m is an MN-major A tile whose M runs over m and whose K runs over the tokens);
// its B operand is O~_A^T [r16][T], K-major.  One pair tile covers 256 rows of dB and ALL tokens, so no partial
// sums exist and the order of the accumulation is fixed.  The tiles of dB are appended to the tile list from the
// far end of the pairs: the last wave of 256 x 256 tiles leaves the highest-numbered pairs idle, and that is where
// the few microseconds of dB work go -- the launch of a separate kernel (TMEM allocation, two cluster barriers,
// about 12 us for 2 us of traffic) disappears from the step.  pd: the parameter block of that second problem.
// oa_job (oa != nullptr): the cast of O_A that dB's B operand needs has not run yet; the epilogue warps of every CTA do it
// first thing (they have nothing to drain until the first tile is complete), each CTA then counts itself in at oa_sync
// (two words that are zero between launches), and the producers of the pairs that carry dB tiles wait for the whole
// grid's count before their first copy of O~_A^T -- tens of microseconds later, so the (bounded) wait never spins.
template <bool kBMn, bool kRider>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_fp8_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                     const __grid_constant__ CUtensorMap tmap_c, const GemmParams p, const GemmParams pd, const OaCastJob oa_job,
                     GridSync* oa_sync) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t smem_base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - raw_addr);

  const int S = p.num_stages;
  const uint32_t bars = smem_base + static_cast<uint32_t>(S) * kPairStageBytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (S + s); };
  auto tmem_full_bar = [&](int a) { return bars + 8u * (2 * S + a); };
  auto tmem_empty_bar = [&](int a) { return bars + 8u * (2 * S + 2 + a); };
  const uint32_t slot_off = static_cast<uint32_t>(S) * kPairStageBytes + 8u * (2 * S + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + slot_off);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();       // 0 = leader
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    prefetch_tensor_map(&tmap_a);
    prefetch_tensor_map(&tmap_b);
    if (kRider) prefetch_tensor_map(&tmap_c);
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);      // the leader's arrive.expect_tx; bytes from both CTAs
      mbar_init(empty_bar(s), 1);     // one multicast commit
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tmem_full_bar(a), 1);   // one multicast commit
      mbar_init(tmem_empty_bar(a), 2 * kEpilogueWarps);  // the epilogue warps of both CTAs
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
  const int total_tiles = p.m_tiles * p.n_tiles;   // m_tiles counts 256-row pair tiles here
  bool aborted = false;
  // rider: which tiles of dB this pair computes after its own tiles of the product.  The pairs without a tile in the
  // product's last wave (the highest-numbered ones) take up to pd.n_tiles each, round robin from the far end -- that many
  // fit into the time the others spend on their last tile (the host's estimate) -- and what is left goes round robin to
  // all pairs, lowest-numbered first.  The same list in all three roles.
  const int last_wave = total_tiles % num_pairs;
  const int idle_pairs = last_wave == 0 ? num_pairs : num_pairs - last_wave;
  const int idle_rank = num_pairs - 1 - pair;
  const int rider_block1 = kRider ? min(pd.m_tiles, idle_pairs * pd.n_tiles) : 0;
  const int rider_n1 = (kRider && idle_rank < idle_pairs && idle_rank < rider_block1) ? (rider_block1 - idle_rank + idle_pairs - 1) / idle_pairs : 0;
  const int rider_rest = kRider ? pd.m_tiles - rider_block1 : 0;
  const int rider_n2 = pair < rider_rest ? (rider_rest - pair + num_pairs - 1) / num_pairs : 0;
  const int rider_count = rider_n1 + rider_n2;
  auto rider_tile = [&](int i) { return i < rider_n1 ? idle_rank + i * idle_pairs : rider_block1 + pair + (i - rider_n1) * num_pairs; };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (warp 0 of each CTA; one lane issues)
    int stage = 0;
    uint32_t phase = 0;
    for (int tile = pair; tile < total_tiles && !aborted; tile += num_pairs) {
      const int n_idx = tile / p.m_tiles;
      const int m_idx = tile - n_idx * p.m_tiles;
      const int n0 = n_idx * 256;
      const int n_inst = pair_instr_n<kBMn>(p.N - n0);             // instruction N of this tile
      const int row0 = m_idx * 256 + static_cast<int>(rank) * kBlockM;
      const int bn0 = n0 + static_cast<int>(rank) * (n_inst >> 1);  // this CTA's half of the B rows
      for (int kb = 0; kb < p.kblocks_total; ++kb) {
        if (!mbar_wait_warp(empty_bar(stage), phase ^ 1u, p.status)) { aborted = true; break; }
        if (elect_one()) {
          if (leader) mbar_expect_tx(full_bar(stage), 2 * kPairStageBytes);
          const uint32_t fb = map_to_cta(full_bar(stage), 0);
          const uint32_t a_dst = smem_base + static_cast<uint32_t>(stage) * kPairStageBytes;
          const uint32_t b_dst = a_dst + kATileBytes;
          tma_load_2d_pair(a_dst, &tmap_a, fb, kb * kBlockKBytes, row0);
          if (!kBMn) tma_load_2d_pair(b_dst, &tmap_b, fb, kb * kBlockKBytes, bn0);
          else       tma_load_2d_pair(b_dst, &tmap_b, fb, bn0, kb * kBlockKBytes);
        }
        __syncwarp();
        if (++stage == S) { stage = 0; phase ^= 1u; }
      }
    }
    if (kRider && oa_job.oa != nullptr && rider_count > 0 && !aborted) {
      // O~_A^T must be complete, written by every CTA of the grid (all resident: one persistent CTA per SM)
      const uint64_t t0 = global_timer_ns();
      while (ld_acquire_gpu(&oa_sync->arrive) < gridDim.x) {
        __nanosleep(100);
        if (global_timer_ns() - t0 > kWaitLimitNs) { aborted = true; atomicExch(p.status, kStatusTimeout); break; }
      }
      aborted = __any_sync(0xFFFFFFFFu, aborted);
      fence_proxy_async_global();   // the codes were stored by ordinary stores; the bulk tensor copies below read them
    }
    if (kRider) {   // the tiles of dB, from the far end of the pairs
      const int half_rows = pd.block_n >> 1;                                  // this CTA's rows of O~_A^T (block_n = r16)
      const uint32_t rider_bytes = kATileBytes + static_cast<uint32_t>(half_rows) * kBlockKBytes;
      for (int ri = 0; ri < rider_count && !aborted; ++ri) {
        const int j = rider_tile(ri);
        const int mcol0 = j * 256 + static_cast<int>(rank) * kBlockM;        // first of this CTA's 128 rows of dB
        for (int kb = 0; kb < pd.kblocks_total; ++kb) {
          if (!mbar_wait_warp(empty_bar(stage), phase ^ 1u, p.status)) { aborted = true; break; }
          if (elect_one()) {
            if (leader) mbar_expect_tx(full_bar(stage), 2 * rider_bytes);
            const uint32_t fb = map_to_cta(full_bar(stage), 0);
            const uint32_t a_dst = smem_base + static_cast<uint32_t>(stage) * kPairStageBytes;
            tma_load_2d_pair(a_dst, &tmap_a, fb, mcol0, kb * kBlockKBytes);                               // 128 tokens x 128 B of m
            tma_load_2d_pair(a_dst + kATileBytes, &tmap_c, fb, kb * kBlockKBytes, static_cast<int>(rank) * half_rows);
          }
          __syncwarp();
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
      }
    }
    // tail: wait until the MMAs have released every stage, so no completion signal can arrive at a CTA
    // that has already left
    for (int i = 0; i < S && !aborted; ++i) {
      if (!mbar_wait_warp(empty_bar(stage), phase ^ 1u, p.status)) aborted = true;
      if (++stage == S) { stage = 0; phase ^= 1u; }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (warp 1 of the leader CTA; one lane issues)
    if (leader) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      const uint64_t a_desc0 = make_smem_desc(smem_base, 16, 1024);
      const uint64_t b_desc0 = kBMn ? make_smem_desc(smem_base + kATileBytes, kMnChunkBytes, 1024)
                                    : make_smem_desc(smem_base + kATileBytes, 16, 1024);
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
          const uint32_t stage_off = (static_cast<uint32_t>(stage) * kPairStageBytes) >> 4;
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < kBlockKBytes / kUmmaK; ++k) {
              umma_f8_pair(d_tmem, a_desc0 + stage_off + k * kAStep, b_desc0 + stage_off + k * kBStep, idesc,
                           (kb > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit_pair(empty_bar(stage), 3);   // frees the stage in both CTAs
          }
          __syncwarp();
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
        if (aborted) break;
        if (elect_one()) umma_commit_pair(tmem_full_bar(acc), 3);    // accumulators of both CTAs complete
        __syncwarp();
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
      if (kRider) {
        const uint64_t ra_desc0 = make_smem_desc(smem_base, kATileBytes, 1024);          // MN-major: one 128 x 128 chunk
        const uint64_t rb_desc0 = make_smem_desc(smem_base + kATileBytes, 16, 1024);     // K-major
        constexpr uint32_t kRaStep = (kUmmaK * 128) >> 4;   // 32 tokens further down the tile
        constexpr uint32_t kRbStep = kUmmaK >> 4;
        for (int ri = 0; ri < rider_count && !aborted; ++ri) {
        const int j = rider_tile(ri);
          if (!mbar_wait_warp(tmem_empty_bar(acc), acc_phase ^ 1u, p.status)) { aborted = true; break; }
          tc_fence_after_sync();
          const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc) * kAccCols;
          for (int kb = 0; kb < pd.kblocks_total; ++kb) {
            if (!mbar_wait_warp(full_bar(stage), phase, p.status)) { aborted = true; break; }
            tc_fence_after_sync();
            const uint32_t stage_off = (static_cast<uint32_t>(stage) * kPairStageBytes) >> 4;
            if (elect_one()) {
#pragma unroll
              for (int k = 0; k < kBlockKBytes / kUmmaK; ++k)
                umma_f8_pair(d_tmem, ra_desc0 + stage_off + k * kRaStep, rb_desc0 + stage_off + k * kRbStep, pd.idesc,
                             (kb > 0 || k > 0) ? 1u : 0u);
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
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..9 of each CTA)
    const int quad = warp & 3;
    const int col_half = (warp - 2) >> 2;
    if (kRider && oa_job.oa != nullptr) {   // S5a, while the first tile is on its way
      cast_oa_transposed(oa_job, warp - 2, static_cast<int>(kEpilogueWarps));
      __threadfence();
      fence_proxy_async_global();
      asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueWarps * 32) : "memory");   // the eight epilogue warps of this CTA
      if (warp == 2 && lane == 0) {
        __threadfence();
        atomicAdd(&oa_sync->arrive, 1u);
      }
    }
    uint8_t* stage_out = smem_gen + static_cast<uint32_t>(S) * kPairStageBytes + kBarrierBytes + (warp - 2) * kStageOutBytes;
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
    if (kRider) {
      // (with the cast riding in this launch, s_OA is taken from the absmax it was made from, not from the word another CTA wrote)
      const float s_oa = oa_job.oa != nullptr ? scale_from_amax(ld_stream(oa_job.amax_oa), kE4M3) : ld_stream(pd.scale_b);
      const float inv_db = 1.0f / (ld_stream(pd.scale_a) * s_oa);
      uint32_t unused = 0;
      for (int ri = 0; ri < rider_count && !aborted; ++ri) {
        const int j = rider_tile(ri);
        if (!mbar_wait(tmem_full_bar(acc), acc_phase, p.status)) { aborted = true; break; }
        tc_fence_after_sync();
        const int row = j * 256 + static_cast<int>(rank) * kBlockM + quad * 32 + lane;      // row of dB
        const uint32_t t_row = tmem_base + static_cast<uint32_t>(acc) * kAccCols + (static_cast<uint32_t>(quad * 32) << 16);
        // (per-row-scaled backbone: row i of dB is multiplied back by s_w[i], one rounded product of the two factors)
        const float inv_row = pd.row_scale != nullptr && row < pd.M ? __fmul_rn(inv_db, ld_stream(pd.row_scale + row)) : inv_db;
        if (pd.dbuf == nullptr) {
          epilogue_tile(pd, t_row, row, row < pd.M, 0, col_half ? 128 : 0, col_half ? 256 : 128, inv_row, unused, stage_out);
        } else if (col_half == 0) {
          // with the optimizer step (r <= 128: this warp's lanes hold whole rows): dB as above, then one fma per element on
          // the value dB holds, and the row's score accumulated strictly left to right -- what the stand-alone kernels do
          const bool ok = row < pd.M;
          float sc = 0.0f;
          for (int c0 = 0; c0 < pd.N; c0 += 32) {
            uint32_t v[32];
            __syncwarp();
            tmem_ld_32x32b_x32(t_row + static_cast<uint32_t>(c0), v);
            tmem_ld_wait();
            if (ok) {
              const long long off = static_cast<long long>(row) * pd.ldc0 + c0;
              float4* drow = reinterpret_cast<float4*>(pd.dbuf + off);
              float4* grow = pd.c0 != nullptr ? reinterpret_cast<float4*>(static_cast<float*>(pd.c0) + off) : nullptr;
              float4 d[8];
#pragma unroll
              for (int q = 0; q < 8; ++q)
                if (c0 + 4 * q < pd.N) d[q] = ld_stream(drow + q);
#pragma unroll
              for (int q = 0; q < 8; ++q) {
                if (c0 + 4 * q < pd.N) {      // r is a multiple of 8: a group of four is all inside or all outside
                  const float4 g = make_float4(__fmul_rn(__uint_as_float(v[4 * q]), inv_row), __fmul_rn(__uint_as_float(v[4 * q + 1]), inv_row),
                                               __fmul_rn(__uint_as_float(v[4 * q + 2]), inv_row), __fmul_rn(__uint_as_float(v[4 * q + 3]), inv_row));
                  if (grow != nullptr) grow[q] = g;
                  float4 e = d[q];
                  e.x = __fmaf_rn(pd.neg_lr, g.x, e.x); e.y = __fmaf_rn(pd.neg_lr, g.y, e.y);
                  e.z = __fmaf_rn(pd.neg_lr, g.z, e.z); e.w = __fmaf_rn(pd.neg_lr, g.w, e.w);
                  drow[q] = e;
                  sc = __fadd_rn(sc, fabsf(e.x)); sc = __fadd_rn(sc, fabsf(e.y));
                  sc = __fadd_rn(sc, fabsf(e.z)); sc = __fadd_rn(sc, fabsf(e.w));
                }
              }
            }
          }
          if (ok) pd.score[row] = sc;
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(map_to_cta(tmem_empty_bar(acc), 0));
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
    if (p.amax1_bits != nullptr) {
      amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
      if (lane == 0 && amax_bits != 0) atomicMax(p.amax1_bits, amax_bits);
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
  if (kRider && oa_job.oa != nullptr && threadIdx.x == 0) grid_depart(oa_sync);   // the last CTA puts the two words back to zero
}

// ------------------------------------------------------------------ host side

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      ptr = nullptr;
    return reinterpret_cast<EncodeTiledFn>(ptr);
  }();
  return fn;
}

}  // namespace

// 2-D uint8 tensor [rows][cols] with row pitch ld bytes; box = box_cols x box_rows, 128-byte swizzle.
bool make_tensor_map(CUtensorMap* map, const uint8_t* base, int64_t rows, int64_t cols, int64_t ld, uint32_t box_cols,
                     uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld)};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t elem_strides[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides, box, elem_strides,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// 2-D tensor of 16-bit elements [rows][cols] with row pitch ld ELEMENTS; box = box_cols x box_rows elements, no swizzle
// (rows of the box land back to back in shared memory).
bool make_tensor_map_u16(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld, uint32_t box_cols,
                         uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * 2};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t elem_strides[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void*>(base), dims, strides, box, elem_strides,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

int sm_count() {   // of the current device
  static std::atomic<int> counts[64];
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  const bool tracked = dev >= 0 && dev < 64;
  if (tracked && (n = counts[dev].load()) > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
  if (tracked) counts[dev].store(n);
  return n;
}

namespace {

template <bool kBMn>
cudaError_t launch_variant(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& gp, int grid, size_t smem,
                           cudaStream_t stream) {
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(gemm_fp8_kernel<kBMn>, static_cast<int>(kSmemBudget), configured);
    if (ec != cudaSuccess) return ec;
  }
  return launch_pdl(gemm_fp8_kernel<kBMn>, dim3(static_cast<unsigned>(grid)), dim3(kGemmThreads), smem, stream, 1, ta,
                    tb, gp);
}

template <bool kBMn, bool kRider>
cudaError_t launch_pair_variant(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, const GemmParams& gp,
                                const GemmParams& gd, const OaCastJob& oa_job, void* oa_sync, int grid, size_t smem,
                                cudaStream_t stream) {
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(gemm_fp8_pair_kernel<kBMn, kRider>, static_cast<int>(kSmemBudget), configured);
    if (ec != cudaSuccess) return ec;
  }
  return launch_pdl(gemm_fp8_pair_kernel<kBMn, kRider>, dim3(static_cast<unsigned>(grid)), dim3(kGemmThreads), smem, stream, 2,
                    ta, tb, tc, gp, gd, oa_job, static_cast<GridSync*>(oa_sync));
}

bool pair_kernel_disabled() {
  // debugging aid: FALQON_DEBUG_GEMM_1CTA=1 routes every product through the single-CTA kernel
  static const bool off = [] {
    const char* v = std::getenv("FALQON_DEBUG_GEMM_1CTA");
    return v != nullptr && v[0] == '1';
  }();
  return off;
}

cudaError_t launch_gemm_fp8_pair(const GemmProblem& q, cudaStream_t stream) {
  GemmParams gp{};
  gp.M = static_cast<int>(q.M); gp.N = static_cast<int>(q.N); gp.K = static_cast<int>(q.K);
  gp.block_n = 256;
  gp.m_tiles = static_cast<int>((q.M + 255) / 256);
  gp.n_tiles = static_cast<int>((q.N + 255) / 256);
  gp.kblocks_total = static_cast<int>((q.K + kBlockKBytes - 1) / kBlockKBytes);
  int stages = static_cast<int>((kSmemBudget - 1024 - kBarrierBytes - kStagingBytes) / kPairStageBytes);
  if (stages > kMaxStages) stages = kMaxStages;
  gp.num_stages = stages;
  // instruction descriptor without N (set per tile): fp32 accumulate, formats, B major, M = 256
  gp.idesc = (1u << 4) | (static_cast<uint32_t>(q.a_fmt) << 7) | (static_cast<uint32_t>(q.b_fmt) << 10) |
             ((q.b_mn_major ? 1u : 0u) << 16) | (static_cast<uint32_t>(256 >> 4) << 24);
  gp.c0 = q.c0; gp.ldc0 = q.ldc0; gp.c0_dt = q.c0_dt; gp.n_split = static_cast<int>(q.n_split);
  gp.c1 = q.c1; gp.ldc1 = q.ldc1; gp.amax1_bits = q.amax1_bits;
  gp.scale_a = q.scale_a; gp.scale_b = q.scale_b; gp.col_scale = q.col_scale;
  gp.status = q.status;
  CUtensorMap ta, tb;
  if (!make_tensor_map(&ta, q.a, q.M, q.K, q.lda, kBlockKBytes, kBlockM)) return cudaErrorInvalidValue;
  const bool ok = q.b_mn_major ? make_tensor_map(&tb, q.b, q.K, q.N, q.ldb, 128, kBlockKBytes)
                               : make_tensor_map(&tb, q.b, q.N, q.K, q.ldb, kBlockKBytes, 128);
  if (!ok) return cudaErrorInvalidValue;
  const long long total_tiles = static_cast<long long>(gp.m_tiles) * gp.n_tiles;
  long long pairs = sm_count() / 2;
  if (total_tiles < pairs) pairs = total_tiles;
  const int grid = static_cast<int>(pairs * 2);
  const size_t smem = static_cast<size_t>(stages) * kPairStageBytes + kBarrierBytes + kStagingBytes + 1024;
  if (q.db_rider != nullptr) {
    // the adapter gradient as a second problem of the same launch: dB[m][r] = A^T (this product's A, g~ [T][m]) x O~_A^T
    const DbFusedProblem& d = *q.db_rider;
    if (!gemm_db_rider_supported(q, d)) return cudaErrorInvalidValue;
    const int r16 = static_cast<int>(round_up(d.r, 16));
    GemmParams gd{};
    gd.M = static_cast<int>(d.m); gd.N = static_cast<int>(d.r); gd.K = static_cast<int>(d.T);
    gd.block_n = r16;
    gd.m_tiles = static_cast<int>((d.m + 255) / 256);
    gd.kblocks_total = static_cast<int>((d.T + kBlockKBytes - 1) / kBlockKBytes);
    {
      // n_tiles carries the quota of the pairs that idle in the product's last wave: how many tiles of dB (bound by the
      // copies: about 0.17 us per k-block) fit into one tile of the product (bound by the MMAs: about 0.47 us per k-block;
      // both measured), at least one, and no more than an even share of the tiles
      const long long last_wave = total_tiles % pairs;
      const long long idle = last_wave == 0 ? pairs : pairs - last_wave;
      long long cap = static_cast<long long>(2.75 * gp.kblocks_total / gd.kblocks_total);
      const long long share = (gd.m_tiles + idle - 1) / idle;
      if (cap > share) cap = share;
      if (cap < 1) cap = 1;
      gd.n_tiles = static_cast<int>(cap);
    }
    gd.num_stages = stages;
    // fp32 accumulate, A = the product's own A format read MN-major, B = E4M3 K-major, N = r16, M = 256
    gd.idesc = (1u << 4) | (static_cast<uint32_t>(q.a_fmt) << 7) | (static_cast<uint32_t>(kE4M3) << 10) | (1u << 15) |
               (static_cast<uint32_t>(r16 >> 3) << 17) | (static_cast<uint32_t>(256 >> 4) << 24);
    gd.c0 = d.dB; gd.ldc0 = d.r; gd.c0_dt = kF32; gd.n_split = static_cast<int>(d.r);
    gd.scale_a = d.s_g; gd.scale_b = d.s_oa; gd.row_scale = d.row_mul;
    gd.dbuf = d.dbuf; gd.score = d.score; gd.neg_lr = d.neg_lr;
    gd.status = q.status;
    CUtensorMap tc;
    if (!make_tensor_map(&tc, d.oaq_t, r16, d.T, d.ldt, kBlockKBytes, static_cast<uint32_t>(r16 / 2))) return cudaErrorInvalidValue;
    OaCastJob oa_job{};
    if (q.oa_rider != nullptr) {
      if (q.oa_sync == nullptr) return cudaErrorInvalidValue;
      oa_job = *q.oa_rider;
    }
    return launch_pair_variant<true, true>(ta, tb, tc, gp, gd, oa_job, q.oa_sync, grid, smem, stream);
  }
  if (q.b_mn_major) return launch_pair_variant<true, false>(ta, tb, ta, gp, gp, OaCastJob{}, nullptr, grid, smem, stream);
  return launch_pair_variant<false, false>(ta, tb, ta, gp, gp, OaCastJob{}, nullptr, grid, smem, stream);
}

}  // namespace

bool gemm_db_rider_supported(const GemmProblem& q, const DbFusedProblem& d) {
  // the product must run on CTA pairs with an MN-major B (the input-gradient product), its A must be the rider's g~
  // ([T][m], the rider's rows on the product's contraction axis); with the optimizer step fused, a warp must hold whole rows
  // of dB (r <= 128)
  return q.block_n == 256 && q.N % 16 == 0 && !pair_kernel_disabled() && q.b_mn_major && q.a != nullptr && q.a == d.gq &&
         q.M == d.T && q.K == d.m && q.lda == d.m && d.m % 16 == 0 && d.r >= 8 && d.r <= 256 && d.r % 8 == 0 &&
         ((d.dbuf == nullptr && d.score == nullptr && d.dB != nullptr) || (d.dbuf != nullptr && d.score != nullptr && d.r <= 128)) &&
         d.oaq_t != nullptr && d.s_g != nullptr &&
         d.s_oa != nullptr && (q.a_fmt == kE5M2) == !d.g_is_e4m3;
}

cudaError_t launch_gemm_fp8(const GemmProblem& q, cudaStream_t stream) {
  if (q.M <= 0 || q.N <= 0 || q.K <= 0) return cudaErrorInvalidValue;
  if (q.db_rider != nullptr && !gemm_db_rider_supported(q, *q.db_rider)) return cudaErrorInvalidValue;
  if (q.oa_rider != nullptr && q.db_rider == nullptr) return cudaErrorInvalidValue;
  if (q.block_n < 16 || q.block_n > 256 || q.block_n % 16) return cudaErrorInvalidValue;
  if (q.b_mn_major && q.block_n % 128) return cudaErrorInvalidValue;
  // the tensor-bound roles (K-major A, full-width tiles, no token slabs) run on CTA pairs
  if (q.block_n == 256 && q.N % 16 == 0 && !pair_kernel_disabled())
    return launch_gemm_fp8_pair(q, stream);

  GemmParams gp{};
  gp.M = static_cast<int>(q.M); gp.N = static_cast<int>(q.N); gp.K = static_cast<int>(q.K);
  gp.block_n = q.block_n;
  gp.m_tiles = static_cast<int>((q.M + kBlockM - 1) / kBlockM);
  gp.n_tiles = static_cast<int>((q.N + q.block_n - 1) / q.block_n);
  gp.kblocks_total = static_cast<int>((q.K + kBlockKBytes - 1) / kBlockKBytes);
  const uint32_t stage_bytes = kATileBytes + static_cast<uint32_t>(q.block_n) * kBlockKBytes;
  int stages = static_cast<int>((kSmemBudget - 1024 - kBarrierBytes - kStagingBytes) / stage_bytes);
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) return cudaErrorInvalidValue;
  gp.num_stages = stages;
  // instruction descriptor: fp32 accumulate, operand formats and majors, N/8 at bit 17, M/16 at bit 24
  gp.idesc = (1u << 4) | (static_cast<uint32_t>(q.a_fmt) << 7) | (static_cast<uint32_t>(q.b_fmt) << 10) |
             ((q.b_mn_major ? 1u : 0u) << 16) |
             (static_cast<uint32_t>(q.block_n >> 3) << 17) | (static_cast<uint32_t>(kBlockM >> 4) << 24);
  gp.c0 = q.c0; gp.ldc0 = q.ldc0; gp.c0_dt = q.c0_dt; gp.n_split = static_cast<int>(q.n_split);
  gp.c1 = q.c1; gp.ldc1 = q.ldc1; gp.amax1_bits = q.amax1_bits;
  gp.scale_a = q.scale_a; gp.scale_b = q.scale_b; gp.col_scale = q.col_scale;
  gp.status = q.status;

  CUtensorMap ta, tb;
  bool ok;
  ok = make_tensor_map(&ta, q.a, q.M, q.K, q.lda, kBlockKBytes, kBlockM);
  if (!ok) return cudaErrorInvalidValue;
  if (!q.b_mn_major) ok = make_tensor_map(&tb, q.b, q.N, q.K, q.ldb, kBlockKBytes, static_cast<uint32_t>(q.block_n));
  else               ok = make_tensor_map(&tb, q.b, q.K, q.N, q.ldb, 128, kBlockKBytes);
  if (!ok) return cudaErrorInvalidValue;

  const long long total_tiles = static_cast<long long>(gp.m_tiles) * gp.n_tiles;
  int grid = sm_count();
  if (total_tiles < grid) grid = static_cast<int>(total_tiles);
  const size_t smem = static_cast<size_t>(stages) * stage_bytes + kBarrierBytes + kStagingBytes + 1024;
  if (q.b_mn_major) return launch_variant<true>(ta, tb, gp, grid, smem, stream);
  return launch_variant<false>(ta, tb, gp, grid, smem, stream);
}

}  // namespace falqon
