// loki_alloc_solve_static: the allocation search for callers that must not
// allocate device memory.  All working memory of the call -- stage demands, level
// status, the per-block partial keys of the scoring kernel and the reduced keys --
// lives in one fixed array that is part of the library image.
#include <mutex>

#include "loki_internal.h"

using namespace loki;

namespace {

constexpr int kStaticMaxLevels = 64;    // demand levels per call
constexpr int kStaticMaxBlocks = 256;   // thread blocks of the scoring kernel

// Layout of the fixed working memory.
struct StaticScratch {
  int64_t dem64[kStaticMaxLevels * kMaxTasks];          //   4 KiB
  int32_t status[kStaticMaxLevels];                     // 256 B
  Key final_key[kStaticMaxLevels];                      //   1 KiB
  Key partial[kStaticMaxBlocks * kStaticMaxLevels];     // 256 KiB
};

// 267,520 bytes, held by every GPU that loads the library until the process exits.
// In host code this name is only a stand-in for the symbol: the device address
// comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

constexpr int kMaxDev = 64;
std::mutex g_setup_mutex;
StaticScratch* g_scratch_addr[kMaxDev];   // device address of the array, per device

}  // namespace

namespace loki {

// Once per device, with that device current: resolve the array's device address.  Looking the
// symbol up is what makes the driver load this part of the library onto the device and back
// the array with memory, so it is done by loki_alloc_create, while the caller may still
// allocate, and never by loki_alloc_solve_static itself.
int static_scratch_prepare(int device) {
  if (device < 0 || device >= kMaxDev) return LOKI_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_addr[device] != nullptr) return LOKI_OK;
  void* ptr = nullptr;
  const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
  if (e != cudaSuccess || ptr == nullptr) {
    cudaGetLastError();
    return LOKI_ERR_CUDA;
  }
  g_scratch_addr[device] = static_cast<StaticScratch*>(ptr);
  return LOKI_OK;
}

}  // namespace loki

extern "C" int loki_alloc_solve_static(const loki_alloc_t* h, const int64_t* d_demand_mqps,
                                       int32_t n_levels, void* cuda_stream,
                                       loki_config_t* d_out) {
  if (!h || !d_demand_mqps || !d_out) return LOKI_ERR_INVALID_ARG;
  if (n_levels < 1) return LOKI_ERR_INVALID_ARG;
  if (n_levels > kStaticMaxLevels) return LOKI_ERR_RANGE;   // beyond the fixed array
  HandleView v;
  if (!handle_view(h, &v)) return LOKI_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return LOKI_ERR_CUDA; }
  if (dev != v.device) return LOKI_ERR_INVALID_ARG;
  StaticScratch* s = nullptr;
  {
    // resolved when the handle was created on this device; nothing is looked up or loaded here
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    s = g_scratch_addr[dev];
  }
  if (s == nullptr) return LOKI_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  v.dev.partial_keys = (int64_t)kStaticMaxBlocks * kStaticMaxLevels;   // the checked build's bound: the fixed array's
  int n_blocks = v.n_sms * 2;
  if (n_blocks > kStaticMaxBlocks) n_blocks = kStaticMaxBlocks;
  if (n_blocks < 1) n_blocks = 1;
  // Every word of the array that a kernel below reads is written earlier in this
  // same call (each scoring block stores a key for each level, empty or not), so
  // nothing left behind by the previous call is consumed and no clearing is needed.
  if (launch_prepare_levels(v.dev, d_demand_mqps, n_levels, s->dem64, s->status, nullptr, nullptr,
                            1, st) != cudaSuccess ||
      launch_generic_score(v.dev, s->dem64, s->status, n_levels, n_blocks, s->partial, st) != cudaSuccess ||
      launch_finish(v.dev, s->partial, n_blocks, 0, 0, n_levels, d_demand_mqps, nullptr, s->final_key, d_out,
                    st) != cudaSuccess) {
    cudaGetLastError();
    return LOKI_ERR_CUDA;
  }
  return LOKI_OK;
}
