// A measurement, not a step of the method: how fast the FP8 tensor pipe of this GPU runs when nothing but the
// pipe limits it.  Every SM pair issues the same 256 x 256 x 32 tcgen05.mma (kind::f8f6f4, E4M3 x E4M3, fp32
// accumulators in TMEM, cta_group::2) that the melded forward and input-gradient products issue, on operand tiles that
// stay in shared memory: no global loads, no epilogue.  The operands are filled once: with zeros, with uniformly random
// E4M3 codes, or with the codes of a bell-shaped variable under absmax scaling (the switching activity of the data
// decides the power, and the power cap decides the clock).  The
// throughput of a sequence of such launches is the ceiling the products' roofline fraction is quoted against.
#include "internal.h"
#include "ptx.cuh"

namespace falqon {
namespace {

constexpr int kCeilThreads = 128;
constexpr int kCeilStages = 6;                       // operand slots the issuer cycles through, as the products' pipeline does
constexpr uint32_t kCeilTileBytes = 128 * 128;       // 128 rows x 128 bytes of K (one swizzle row), per CTA
constexpr uint32_t kCeilStageBytes = 2 * kCeilTileBytes;   // this CTA's half of A and of B
constexpr uint32_t kCeilTmemCols = 512;              // two 256-column accumulators
constexpr int kCeilKBlocksPerTile = 32;              // a fresh accumulation every 32 k-blocks (K = 4096)
constexpr size_t kCeilSmem = kCeilStages * kCeilStageBytes + 128 + 1024;

__device__ __forceinline__ uint32_t mix32(uint32_t x) {
  x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
  return x;
}

// load_src / load_chunks: optional.  When given, warp 0 of every CTA also streams 16 KB + second_copy_bytes (2 x 16 KB
// for the traffic of a 256 x 256 tile, less for that of wider tiles) per k-block from that buffer
// (load_chunks chunks of 16 KB) into the operand slots, paced by the MMAs like the producer of a real product is: the
// traffic from L2 into shared memory of a 256 x 256 tile pipeline, without its dependencies (the MMAs read whatever the
// slots hold, so the sums are then not reproducible).
__global__ void __launch_bounds__(kCeilThreads, 1) tensor_ceiling_kernel(int kblocks, uint32_t seed, int random_fill,
                                                                         float* sink, int* status, const uint8_t* load_src,
                                                                         uint32_t load_chunks, uint32_t second_copy_bytes) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t smem_base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - raw_addr);
  const uint32_t bars = smem_base + kCeilStages * kCeilStageBytes;
  auto done_bar = [&](int s) { return bars + 8u * s; };
  auto load_bar = [&](int s) { return bars + 8u * (kCeilStages + s); };
  const uint32_t slot_off = kCeilStages * kCeilStageBytes + 16u * kCeilStages;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + slot_off);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool leader = cluster_ctarank() == 0;

  // operands: zeros, or codes whose exponent field is drawn from the middle of the range (no NaN codes, no overflow of
  // the fp32 accumulators within one accumulation)
  uint32_t* words = reinterpret_cast<uint32_t*>(smem_gen);
  for (uint32_t i = threadIdx.x; i < kCeilStages * kCeilStageBytes / 4; i += kCeilThreads) {
    uint32_t w = 0u;
    if (random_fill == 1) {          // uniform codes
      w = mix32(seed ^ (blockIdx.x * 0x9E3779B9u) ^ (i * 0x85EBCA6Bu));
      w = (w & 0xBFBFBFBFu) | ((w >> 1) & 0x20202020u);   // exponent's top bit cleared: magnitudes below 2
    } else if (random_fill == 2) {   // codes of a bell-shaped variable quantized with absmax scaling, as activations are:
      float f[4];                    // sum of four uniforms, standard deviation 448 / 5.5, clipped by the cast at +-448
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const uint32_t h = mix32(seed ^ (blockIdx.x * 0x9E3779B9u) ^ ((4u * i + b) * 0x85EBCA6Bu));
        const float u = static_cast<float>((h & 0xFFu) + ((h >> 8) & 0xFFu) + ((h >> 16) & 0xFFu) + (h >> 24)) - 510.0f;
        f[b] = u * (448.0f / 5.5f / 147.8f);               // the sum has standard deviation 147.8
      }
      w = cvt_fp8x4<0>(f[0], f[1], f[2], f[3]);
    }
    words[i] = w;
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> visible to the tensor pipe
  if (threadIdx.x == 0) {
    for (int s = 0; s < kCeilStages; ++s) { mbar_init(done_bar(s), 1); mbar_init(load_bar(s), 1); }
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_base + slot_off, kCeilTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  bool aborted = false;
  if (warp == 0 && load_src != nullptr) {
    // the stand-in for a TMA producer: slot s is refilled once the MMAs that used it are done (the same condition a
    // real producer waits for) and its own previous copies have landed
    int stage = 0;
    uint32_t phase = 0, lphase = 0;
    uint32_t chunk = (blockIdx.x * 2654435761u) % load_chunks;
    for (int kb = 0; kb < kblocks && !aborted; ++kb) {
      if (!mbar_wait_warp(done_bar(stage), phase ^ 1u, status)) { aborted = true; break; }
      if (!mbar_wait_warp(load_bar(stage), lphase ^ 1u, status)) { aborted = true; break; }
      if (elect_one()) {
        const uint32_t dst = smem_base + static_cast<uint32_t>(stage) * kCeilStageBytes;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_expect_tx(load_bar(stage), kCeilTileBytes + second_copy_bytes);
        bulk_load_1d(dst, load_src + static_cast<size_t>(chunk) * kCeilTileBytes, kCeilTileBytes, load_bar(stage));
        const uint32_t chunk2 = chunk + 1 < load_chunks ? chunk + 1 : 0;
        if (second_copy_bytes > 0)
          bulk_load_1d(dst + kCeilTileBytes, load_src + static_cast<size_t>(chunk2) * kCeilTileBytes, second_copy_bytes, load_bar(stage));
      }
      __syncwarp();
      chunk += 2;
      if (chunk >= load_chunks) chunk -= load_chunks;
      if (++stage == kCeilStages) { stage = 0; phase ^= 1u; lphase ^= 1u; }
    }
    // every copy has landed before the CTA leaves
    for (int i = 0; i < kCeilStages && !aborted; ++i) {
      if (!mbar_wait_warp(load_bar(stage), lphase ^ 1u, status)) aborted = true;
      if (++stage == kCeilStages) { stage = 0; lphase ^= 1u; }
    }
  }
  if (warp == 1) {
    int stage = 0;
    uint32_t phase = 0;
    if (leader) {
      const uint64_t a_desc0 = make_smem_desc(smem_base, 16, 1024);
      const uint64_t b_desc0 = make_smem_desc(smem_base + kCeilTileBytes, 16, 1024);
      // E4M3 x E4M3 -> fp32, both operands K-major, N = 256, M = 256 over the pair
      const uint32_t idesc = (1u << 4) | (static_cast<uint32_t>(256 >> 3) << 17) | (static_cast<uint32_t>(256 >> 4) << 24);
      for (int kb = 0; kb < kblocks; ++kb) {
        // without the load stream: at most kCeilStages commits in flight; with it: the slot's copies have landed
        const bool ok = load_src != nullptr ? mbar_wait_warp(load_bar(stage), phase, status)
                                            : mbar_wait_warp(done_bar(stage), phase ^ 1u, status);
        if (!ok) { aborted = true; break; }
        tc_fence_after_sync();
        const int in_tile = kb % kCeilKBlocksPerTile;
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>((kb / kCeilKBlocksPerTile) & 1) * 256u;
        const uint32_t stage_off = (static_cast<uint32_t>(stage) * kCeilStageBytes) >> 4;
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_f8_pair(d_tmem, a_desc0 + stage_off + 2u * k, b_desc0 + stage_off + 2u * k, idesc, (in_tile > 0 || k > 0) ? 1u : 0u);
          umma_commit_pair(done_bar(stage), 3);
        }
        __syncwarp();
        if (++stage == kCeilStages) { stage = 0; phase ^= 1u; }
      }
    } else {
      stage = kblocks % kCeilStages;
      phase = static_cast<uint32_t>(kblocks / kCeilStages) & 1u;
    }
    // both CTAs: every slot's last commit has arrived here before anyone leaves
    for (int i = 0; i < kCeilStages && !aborted; ++i) {
      if (!mbar_wait_warp(done_bar(stage), phase ^ 1u, status)) aborted = true;
      if (++stage == kCeilStages) { stage = 0; phase ^= 1u; }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  tc_fence_after_sync();
  // one look at the accumulators, so that the products are observable
  {
    uint32_t v[32];
    tmem_ld_32x32b_x32(tmem_base + (static_cast<uint32_t>(warp * 32) << 16), v);
    tmem_ld_wait();
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < 32; ++i) s += __uint_as_float(v[i]);
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    if (lane == 0 && sink != nullptr) sink[blockIdx.x * 4 + warp] = s;
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, kCeilTmemCols);
  }
}

// A self-test of the bounded waits, not a measurement: one CTA waits on a barrier that nobody ever arrives on.  The wait
// gives up after limit_ns, records the timeout in the status word and the kernel returns; the context stays usable.
__global__ void __launch_bounds__(32) wait_timeout_selftest_kernel(uint64_t limit_ns, int* status) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    mbar_fence_init();
  }
  __syncwarp();
  mbar_wait_for(smem_u32(&bar), 0u, status, limit_ns);
}

}  // namespace

cudaError_t launch_wait_timeout_selftest(uint64_t limit_ns, int* status, cudaStream_t stream) {
  wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(limit_ns, status);
  return cudaGetLastError();
}

int tensor_ceiling_ctas() { return (sm_count() / 2) * 2; }

double tensor_ceiling_flops(int kblocks) {   // of one launch: every pair issues kblocks x 4 MMAs of 256 x 256 x 32
  return static_cast<double>(tensor_ceiling_ctas() / 2) * kblocks * 4.0 * 2.0 * 256.0 * 256.0 * 32.0;
}

cudaError_t launch_tensor_ceiling(int kblocks, uint32_t seed, int random_fill, float* sink, int* status, const void* load_src,
                                  size_t load_bytes, int bytes_per_kblock, cudaStream_t stream) {
  static DeviceMask configured{0};
  {
    const cudaError_t ec = set_max_dynamic_smem(tensor_ceiling_kernel, static_cast<int>(kCeilSmem), configured);
    if (ec != cudaSuccess) return ec;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(tensor_ceiling_ctas()));
  cfg.blockDim = dim3(kCeilThreads);
  cfg.dynamicSmemBytes = kCeilSmem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const uint32_t load_chunks = load_src != nullptr ? static_cast<uint32_t>(load_bytes / kCeilTileBytes) : 0u;
  return cudaLaunchKernelEx(&cfg, tensor_ceiling_kernel, kblocks, seed, random_fill, sink, status,
                            load_chunks >= 2 ? static_cast<const uint8_t*>(load_src) : nullptr, load_chunks,
                            static_cast<uint32_t>(bytes_per_kblock) - kCeilTileBytes);
}

}  // namespace falqon
