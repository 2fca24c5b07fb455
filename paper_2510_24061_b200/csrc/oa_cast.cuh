// The cast of O_A (S5a of the backward: O~_A = Q_e4m3(O_A) with s_OA = 448 / amax(O_A), Eq. quantize) as a device
// function that other kernels carry along: the output-gradient quantizer (warps that idle at its grid barrier), the
// input-gradient product (its epilogue warps, idle while the first tile is computed), and a small kernel of its own.
#pragma once

#include <cstdint>

#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

// O_A [T][r] fp32 -> E4M3 codes with s_OA = 448 / amax(O_A), stored
// TRANSPOSED as [r][ldt] so that the adapter-gradient product reads them K-major.  One warp converts a tile of
// 32 tokens (warp w of the rider_warps warps of a CTA that take part): lane (tg, jq) takes tokens 4 tg .. 4 tg + 3 and columns 16 jq .. 16 jq + 15 of every block of 64
// columns, so the codes of four consecutive tokens of one column form one 32-bit store.  Tokens at or beyond T
// give zero codes (they land in the padding of the row pitch, a multiple of 16).
__device__ __forceinline__ void cast_oa_transposed(const OaCastJob& job, int w, int rider_warps) {
  const int lane = threadIdx.x & 31;
  const int tg = lane >> 2, jq = lane & 3;
  const float amax = ld_stream(job.amax_oa);
  const float s_oa = scale_from_amax(amax, kE4M3);
  if (blockIdx.x == 0 && w == 0 && lane == 0) {
    *job.s_oa_out = s_oa;
    if (job.amax_copy != nullptr) *job.amax_copy = amax;
  }
  const long long n_tiles = (job.T + 31) / 32;
  const int r16 = (job.r + 15) & ~15;
  // consecutive tiles go to different CTAs, so a small O_A costs every CTA at most one tile on one warp
  for (long long tile = static_cast<long long>(w) * gridDim.x + blockIdx.x; tile < n_tiles;
       tile += static_cast<long long>(rider_warps) * gridDim.x) {
    const long long t0 = tile * 32 + 4 * tg;
    for (int jb = 0; jb < r16; jb += 64) {
      const int j0 = jb + 16 * jq;
      if (j0 >= job.r) continue;
      float4 x[4][4];
#pragma unroll
      for (int a = 0; a < 4; ++a) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          x[a][q] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (t0 + a < job.T && j0 + 4 * q < job.r)    // r is a multiple of 8: a float4 is all inside or all outside
            x[a][q] = ld_stream(reinterpret_cast<const float4*>(job.oa + (t0 + a) * job.r + j0) + q);
        }
      }
      if (t0 >= job.ldt) continue;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float c[4][4] = {{x[0][q].x, x[1][q].x, x[2][q].x, x[3][q].x}, {x[0][q].y, x[1][q].y, x[2][q].y, x[3][q].y},
                               {x[0][q].z, x[1][q].z, x[2][q].z, x[3][q].z}, {x[0][q].w, x[1][q].w, x[2][q].w, x[3][q].w}};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int j = j0 + 4 * q + e;
          if (j < job.r)
            *reinterpret_cast<uint32_t*>(job.oaq_t + static_cast<long long>(j) * job.ldt + t0) =
                cvt_fp8x4<kE4M3>(__fmul_rn(c[e][0], s_oa), __fmul_rn(c[e][1], s_oa), __fmul_rn(c[e][2], s_oa), __fmul_rn(c[e][3], s_oa));
        }
      }
    }
  }
}

}  // namespace
}  // namespace falqon
