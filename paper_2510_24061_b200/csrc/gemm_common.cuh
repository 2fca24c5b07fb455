// Pieces shared by the FP8 product kernels (gemm_fp8.cu, gemm_fp8_fused.cu): tile constants, the kernel
// parameter block and the epilogue that drains an accumulator tile from tensor memory.  Device code only.
#pragma once

#include <cstdint>

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
  const float* row_scale;   // nullable, used by the adapter-gradient rider only: output row i is also multiplied by row_scale[i]
  // nullable (together), the rider only: DeltaBuffer <- fma(neg_lr, dB, DeltaBuffer) on the rows it has just computed (Alg. 3
  // line 4, plain SGD), and score[i] = sum_j |DeltaBuffer[i][j]| in fp32, j ascending
  float* dbuf; float* score; float neg_lr;
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


// Instruction N of a pair tile with `remaining` valid columns: a multiple of 16 (each CTA supplies N/2 rows of
// B, a whole number of 8-row swizzle groups); with an MN-major B each half must also start on a 16-byte
// boundary of the N axis for the TMA copy, so N is a multiple of 32 there.
template <bool kBMn>
__device__ __forceinline__ int pair_instr_n(int remaining) {
  const int gran = kBMn ? 32 : 16;
  return min(256, (remaining + gran - 1) / gran * gran);
}

}  // namespace
}  // namespace falqon
