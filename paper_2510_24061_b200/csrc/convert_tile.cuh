// The cast of Eq. quantize applied to an operand tile that is already in shared memory: bf16 values times the
// tensor's scale (one rounded fp32 multiply), rounded to nearest even and saturated to E4M3 / E5M2, written in the
// 128-byte-swizzled K-major layout that tcgen05.mma reads.  Used by the converting producer of the fused products.
//
// Source tile: rows of 128 bf16 (256 bytes), back to back, as a bulk tensor copy without swizzle leaves them; eight
// rows form a 2048-byte group.  The codes of a group go IN PLACE into the first 1024 bytes of that group -- eight
// rows of 128 bytes, the 16-byte pieces of row i XOR-swizzled by i, which is the tensor core's 128-byte swizzle for
// a tile whose 8-row groups lie 2048 bytes apart (stride-dimension byte offset 2048 in the matrix descriptor).
// One warp converts a group: every lane first loads its four 16-byte pieces (lane l takes pieces l, l+32, l+64,
// l+96 of the 128 in the group: conflict-free 512-byte wavefronts), the warp synchronises, and only then are the
// codes stored (8 bytes per piece; a half-warp covers one 128-byte row, so the stores are conflict-free too).
#pragma once

#include <cstdint>

#include "ptx.cuh"

namespace falqon {

constexpr uint32_t kConvGroupBytes = 2048;   // 8 rows x 128 bf16
constexpr int kConvGroupsPerTile = 16;       // 128 rows

__device__ __forceinline__ void convert_group_load(const uint8_t* group, int lane, uint4 (&q)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) q[i] = *reinterpret_cast<const uint4*>(group + (lane + 32 * i) * 16);
}

// Eight bf16 values (one 16-byte piece) -> eight codes.
template <int kFmt>
__device__ __forceinline__ uint2 convert_piece(const uint4& q, float s) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
  const uint64_t s2 = pack_f32x2(s, s);
  float x[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {   // two rounded multiplies per instruction (each half an ordinary RN product)
    uint64_t v = pack_f32x2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
    asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(v) : "l"(s2));
    unpack_f32x2(v, x[2 * i], x[2 * i + 1]);
  }
  uint2 o;
  o.x = cvt_fp8x4<kFmt>(x[0], x[1], x[2], x[3]);
  o.y = cvt_fp8x4<kFmt>(x[4], x[5], x[6], x[7]);
  return o;
}

// Converts and stores the four pieces a lane loaded.  emit (nullable): the codes also go to global memory,
// emit points at the code of (first row of the group, first K element of the tile); rows at or beyond rows_left and K
// elements at or beyond k_left are skipped (K extents are multiples of 8, so a piece is all inside or all outside).
template <int kFmt>
__device__ __forceinline__ void convert_group_store(uint8_t* group, int lane, const uint4 (&q)[4], float s, uint8_t* emit,
                                                    long long emit_ld, int rows_left, int k_left) {
  const int c16 = lane & 15;               // which 16-byte piece of the bf16 row = which 8 K elements
  const int chunk = c16 >> 1, half = c16 & 1;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = 2 * i + (lane >> 4);
    const uint2 o = convert_piece<kFmt>(q[i], s);
    *reinterpret_cast<uint2*>(group + row * 128 + ((chunk ^ row) << 4) + half * 8) = o;
    if (emit != nullptr && row < rows_left && c16 * 8 < k_left)
      *reinterpret_cast<uint2*>(emit + row * emit_ld + c16 * 8) = o;
  }
}

}  // namespace falqon
