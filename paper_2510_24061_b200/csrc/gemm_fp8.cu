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
// backbone exists).  (The adapter gradient, which reads the output gradient MN-major, has its own kernel.)
// Every mbarrier wait is bounded; on a timeout the CTA records it, drains and frees its TMEM.
#include <cuda.h>

#include <cstdlib>

#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

constexpr int kGemmThreads = 320;          // warp 0 TMA, warp 1 MMA, warps 2..9 epilogue
constexpr uint32_t kEpilogueWarps = 8;
constexpr int kBlockM = 128;
constexpr int kBlockKBytes = 128;          // one 128-byte swizzle row of FP8 = 128 elements of K
constexpr int kUmmaK = 32;                 // K per tcgen05.mma for 8-bit operands
constexpr uint32_t kATileBytes = kBlockM * kBlockKBytes;   // 16 KB
constexpr uint32_t kMnChunkBytes = 128 * kBlockKBytes;     // a 128(K) x 128(M/N) chunk of an MN-major tile
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kAccCols = 256;
constexpr int kMaxStages = 8;
constexpr uint32_t kSmemBudget = 227 * 1024;
constexpr uint32_t kBarrierBytes = 256;
constexpr uint32_t kStageOutBytes = 32 * 128;                       // per epilogue warp: 32 rows x 128 B
constexpr uint32_t kStagingBytes = kEpilogueWarps * kStageOutBytes;  // 32 KB behind the barriers

struct GemmParams {
  int M, N, K;
  int m_tiles, n_tiles;
  int kblocks_total;
  int block_n;
  int num_stages;
  uint32_t idesc;
  // epilogue
  void* c0; long long ldc0; int c0_dt; int n_split;
  float* c1; long long ldc1; uint32_t* amax1_bits;
  const float* scale_a; const float* scale_b;
  const float* col_scale;
  int* status;
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// Stores 32 consecutive output columns [col0, col0+32) of one row: columns below n_split go to c0 (bf16 or
// fp32, 16-byte stores when aligned), the rest up to N go to c1 (fp32) and feed the running |max|.
__device__ __forceinline__ void epilogue_store32(const GemmParams& p, int row, int col0, const float (&f)[32],
                                                 uint32_t& amax_bits) {
  if (col0 + 32 <= p.n_split) {
    if (p.c0_dt == kBF16) {
      uint16_t* dst = static_cast<uint16_t*>(p.c0) + (long long)row * p.ldc0 + col0;
      if ((reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint4 o;
          o.x = pack_bf16x2(f[8 * i + 0], f[8 * i + 1]);
          o.y = pack_bf16x2(f[8 * i + 2], f[8 * i + 3]);
          o.z = pack_bf16x2(f[8 * i + 4], f[8 * i + 5]);
          o.w = pack_bf16x2(f[8 * i + 6], f[8 * i + 7]);
          reinterpret_cast<uint4*>(dst)[i] = o;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) dst[i] = static_cast<uint16_t>(pack_bf16x2(f[i], 0.0f) & 0xFFFF);
      }
    } else {
      float* dst = static_cast<float*>(p.c0) + (long long)row * p.ldc0 + col0;
      if ((reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i)
          reinterpret_cast<float4*>(dst)[i] = make_float4(f[4 * i], f[4 * i + 1], f[4 * i + 2], f[4 * i + 3]);
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) dst[i] = f[i];
      }
    }
  } else {
    // chunk touches the O | O_A boundary or the ragged right edge: element by element
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const int col = col0 + i;
      if (col < p.n_split) {
        const long long off = (long long)row * p.ldc0 + col;
        if (p.c0_dt == kBF16) static_cast<uint16_t*>(p.c0)[off] = static_cast<uint16_t>(pack_bf16x2(f[i], 0.0f) & 0xFFFF);
        else static_cast<float*>(p.c0)[off] = f[i];
      } else if (col < p.N) {
        p.c1[(long long)row * p.ldc1 + (col - p.n_split)] = f[i];
        amax_bits = max(amax_bits, __float_as_uint(f[i]) & 0x7FFFFFFFu);
      }
    }
  }
}

// Drains columns [col_begin, col_end) of one accumulator tile for this warp's 32 rows.  tcgen05.ld of the next
// 32-column chunk is in flight while the current one is rescaled.  Chunks that lie wholly inside the main
// output (c0) are transposed through a 32 x 128-byte per-warp staging buffer in shared memory (16-byte pieces
// XOR-swizzled by row, so neither side has bank conflicts) and leave as full 128-byte lines: a store
// instruction then covers 4 rows x 128 B instead of 32 rows x 16 B.  Chunks that touch the O | O_A boundary
// or the ragged right edge take the element-wise path.
__device__ __forceinline__ void epilogue_tile(const GemmParams& p, uint32_t t_row, int row, bool row_ok, int n0,
                                              int col_begin, int col_end, float inv, uint32_t& amax_bits,
                                              uint8_t* stage_out) {
  const int last = min(col_end, p.N - n0);    // warp-uniform: columns at or beyond N hold nothing
  if (col_begin >= last) return;
  const int lane = threadIdx.x & 31;
  const bool bf16 = p.c0_dt == kBF16;
  const int esize = bf16 ? 2 : 4;
  const int chunks_per_flush = bf16 ? 2 : 1;  // 64 bf16 or 32 fp32 columns fill the 128-byte rows
  int pending = 0;                            // chunks staged and not yet flushed
  int flush_col = 0;                          // first output column of the staged data

  auto flush = [&]() {
    if (pending == 0) return;
    __syncwarp();
    const int row_base = row - lane;
    const int bytes_per_row = pending * 32 * esize;       // 64 or 128
    const int lanes_per_row = bytes_per_row >> 4;          // 4 or 8
    const int rows_per_inst = 32 / lanes_per_row;          // 8 or 4
    const int piece = lane % lanes_per_row;
    uint8_t* c0 = static_cast<uint8_t*>(p.c0) +
                  (long long)flush_col * esize + (long long)piece * 16;
    for (int r0 = 0; r0 < 32; r0 += rows_per_inst) {
      const int r = r0 + lane / lanes_per_row;
      const uint4 val = *reinterpret_cast<const uint4*>(stage_out + r * 128 + ((piece ^ (r & 7)) << 4));
      if (row_base + r < p.M) *reinterpret_cast<uint4*>(c0 + (long long)(row_base + r) * p.ldc0 * esize) = val;
    }
    __syncwarp();
    pending = 0;
  };

  auto drain = [&](const uint32_t (&v)[32], int c) {
    const int col0 = n0 + c;
    float f[32];
    if (p.col_scale != nullptr) {   // per-column factors (table padded to a multiple of 32 beyond N)
      const float4* cs = reinterpret_cast<const float4*>(p.col_scale + col0);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float4 s4 = ld_stream(cs + i);
        f[4 * i] = __uint_as_float(v[4 * i]) * s4.x; f[4 * i + 1] = __uint_as_float(v[4 * i + 1]) * s4.y;
        f[4 * i + 2] = __uint_as_float(v[4 * i + 2]) * s4.z; f[4 * i + 3] = __uint_as_float(v[4 * i + 3]) * s4.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) f[i] = __uint_as_float(v[i]) * inv;
    }
    const bool fast = col0 + 32 <= p.n_split && ((p.ldc0 * esize) & 15) == 0 &&
                      (reinterpret_cast<uintptr_t>(p.c0) & 15) == 0;
    if (fast) {   // warp-uniform
      if (pending == 0) flush_col = col0;
      uint8_t* my = stage_out + lane * 128;
      const int sw = lane & 7;
      if (bf16) {
        const int base_piece = pending * 4;               // this chunk's 64 bytes
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint4 o;
          o.x = pack_bf16x2(f[8 * j + 0], f[8 * j + 1]);
          o.y = pack_bf16x2(f[8 * j + 2], f[8 * j + 3]);
          o.z = pack_bf16x2(f[8 * j + 4], f[8 * j + 5]);
          o.w = pack_bf16x2(f[8 * j + 6], f[8 * j + 7]);
          *reinterpret_cast<uint4*>(my + (((base_piece + j) ^ sw) << 4)) = o;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j)
          *reinterpret_cast<float4*>(my + ((j ^ sw) << 4)) = make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]);
      }
      ++pending;
      if (pending == chunks_per_flush) flush();
    } else {
      flush();
      if (row_ok) epilogue_store32(p, row, col0, f, amax_bits);
    }
  };

  uint32_t va[32], vb[32];
  __syncwarp();
  tmem_ld_32x32b_x32(t_row + col_begin, va);
  tmem_ld_wait();
  for (int c = col_begin; c < last; c += 64) {
    const bool more1 = c + 32 < last;      // warp-uniform
    __syncwarp();
    if (more1) tmem_ld_32x32b_x32(t_row + c + 32, vb);
    drain(va, c);
    if (!more1) break;
    tmem_ld_wait();
    const bool more2 = c + 64 < last;
    __syncwarp();
    if (more2) tmem_ld_32x32b_x32(t_row + c + 64, va);
    drain(vb, c + 32);
    if (more2) tmem_ld_wait();
  }
  flush();
}

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

// Instruction N of a pair tile with `remaining` valid columns: a multiple of 16 (each CTA supplies N/2 rows of
// B, a whole number of 8-row swizzle groups); with an MN-major B each half must also start on a 16-byte
// boundary of the N axis for the TMA copy, so N is a multiple of 32 there.
template <bool kBMn>
__device__ __forceinline__ int pair_instr_n(int remaining) {
  const int gran = kBMn ? 32 : 16;
  return min(256, (remaining + gran - 1) / gran * gran);
}

template <bool kBMn>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_fp8_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                     const GemmParams p) {
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
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..9 of each CTA)
    const int quad = warp & 3;
    const int col_half = (warp - 2) >> 2;
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

template <bool kBMn>
cudaError_t launch_pair_variant(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& gp, int grid, size_t smem,
                                cudaStream_t stream) {
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(gemm_fp8_pair_kernel<kBMn>, static_cast<int>(kSmemBudget), configured);
    if (ec != cudaSuccess) return ec;
  }
  return launch_pdl(gemm_fp8_pair_kernel<kBMn>, dim3(static_cast<unsigned>(grid)), dim3(kGemmThreads), smem, stream, 2, ta, tb,
                    gp);
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
  if (q.b_mn_major) return launch_pair_variant<true>(ta, tb, gp, grid, smem, stream);
  return launch_pair_variant<false>(ta, tb, gp, grid, smem, stream);
}

}  // namespace

cudaError_t launch_gemm_fp8(const GemmProblem& q, cudaStream_t stream) {
  if (q.M <= 0 || q.N <= 0 || q.K <= 0) return cudaErrorInvalidValue;
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
