// falqon_proxy_update_static: the row-wise proxy update for callers that cannot hand the library a
// workspace because they cannot allocate device memory themselves.
//
// Who that is: code that runs as a guest inside another runtime -- a training framework's custom-op
// hook, an inference server's plug-in slot -- where the host's caching allocator has already claimed
// the device's memory and the guest has no handle to it.  A cudaMalloc from such a guest either fails
// (nothing is left outside the host's pool) or stalls every stream of the device while the driver
// maps the memory, in the middle of a training step.  For them the scratch that
// falqon_proxy_update takes from its workspace argument (the m row scores and the list of selected
// rows) lives in a fixed array inside the library image instead.
//
// The array is a file-scope __device__ object: every GPU that loads the library carries its 128 KB
// from load until the process ends.  Its name is only a host-side handle, not a device address, so the
// address is looked up once per device with cudaGetSymbolAddress -- with that device current -- and the
// kernels are given the looked-up pointer.  That look-up happens in the FIRST call made on a device;
// make that first call outside any stream capture.
//
// All calls on a device share the one array and it keeps whatever the previous call left in it.  The
// update writes every score before reading any and writes the selected-row list before using it, so
// nothing has to start at zero; but two calls whose kernels overlap on the GPU (different streams, no
// ordering between them) race on the array and corrupt each other's selection.  Order them.
//
// No cudaMalloc, cudaFree or allocating library routine is called on this path.
#include <mutex>

#include "../../include/falqon.h"
#include "internal.h"

namespace {

constexpr int64_t kMaxRows = FALQON_STATIC_MAX_ROWS;
constexpr size_t kScoreBytes = static_cast<size_t>(kMaxRows) * sizeof(float);
constexpr size_t kScratchBytes = 2 * kScoreBytes;   // scores, then selected row indices

static __device__ __align__(256) unsigned char g_proxy_scratch[kScratchBytes];

using falqon::kMaxDevices;
std::mutex g_lookup_mutex;
unsigned char* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the CURRENT device (looked up once per device), or nullptr.
unsigned char* scratch_on_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_lookup_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    unsigned char* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_proxy_scratch) != cudaSuccess) return nullptr;
    g_scratch_addr[dev] = ptr;
  }
  return g_scratch_addr[dev];
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace

extern "C" int falqon_proxy_update_static(const falqon_layer* L, const float* dB, float lr, int64_t k, int32_t* idx_out,
                                          falqon_stream stream) {
  using namespace falqon;
  if (L == nullptr || L->wq == nullptr || L->s_w == nullptr || L->dbuf == nullptr || !aligned16(L->wq) ||
      !aligned16(L->dbuf) || L->m < 16 || L->n < 16 || L->m % 16 != 0 || L->n % 16 != 0 || L->r < 8 || L->r > 256 ||
      L->r % 8 != 0 || L->n >= (1ll << 30) || k < 0 || k > L->m || !(lr == lr) || (dB != nullptr && !aligned16(dB)))
    return FALQON_ERR_INVALID_ARG;
  if (L->m > kMaxRows) return FALQON_ERR_UNSUPPORTED;   // the built-in scratch holds FALQON_STATIC_MAX_ROWS rows
  if (L->gran != FALQON_PER_TENSOR) return FALQON_ERR_UNSUPPORTED;   // per-tensor scaled layers only
  unsigned char* scratch = scratch_on_current_device();
  if (scratch == nullptr) return FALQON_ERR_CUDA;
  float* score = reinterpret_cast<float*>(scratch);
  int32_t* sel = reinterpret_cast<int32_t*>(scratch + kScoreBytes);
  const int64_t m = L->m, n = L->n, r = L->r;
  if (launch_sgd_score(L->dbuf, dB, lr, m, r, score, stream) != cudaSuccess) return FALQON_ERR_CUDA;
  if (k > 0) {
    if (launch_topk(score, m, k, sel, nullptr, stream) != cudaSuccess) return FALQON_ERR_CUDA;
    if (launch_merge_rows(L->wq, L->dbuf, sel, k, m, n, r, stream) != cudaSuccess) return FALQON_ERR_CUDA;
    if (idx_out != nullptr &&
        cudaMemcpyAsync(idx_out, sel, static_cast<size_t>(k) * sizeof(int32_t), cudaMemcpyDeviceToDevice, stream) !=
            cudaSuccess)
      return FALQON_ERR_CUDA;
  }
  return FALQON_OK;
}
