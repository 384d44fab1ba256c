// avggt_build_kv_noalloc: the K/V compaction + mean reduction for callers that cannot
// hand the library a workspace.
//
// Some callers have no device memory to lend and may not create any: a host program whose
// memory manager has handed out all of the GPU's memory before this library is loaded, a
// plugin that runs inside somebody else's process under a fixed memory budget, or a
// latency-critical loop in which cudaMalloc (which synchronises the device) is off limits.
// For them the per-block partial sums of the mean reduction live in a fixed array that is
// part of the library image itself.  Every GPU that loads the library holds that array
// (kStaticScratchBytes, about 2.3 MiB) from load until the process exits, whether or not
// this entry point is ever called.
#include <mutex>

#include <cuda_runtime.h>

#include "internal.h"

namespace avggt {
namespace {

// Capacity: partial rows of 2 * H * d floats, one per thread block of the compaction kernel.
constexpr int kStaticMaxCols2 = 2 * 16 * 64;   // H * d <= 1024
constexpr int kStaticMaxBlocks = 296;          // four blocks per SM on up to 74 SMs' worth of grid (see the entry point)
constexpr size_t kStaticScratchBytes = static_cast<size_t>(kStaticMaxBlocks) * kStaticMaxCols2 * sizeof(float);

// In host code this name is only a handle for the runtime's symbol lookup, not a device
// address: it must never be passed to a kernel.  The device address is looked up below.
static __device__ __align__(256) float g_static_scratch[static_cast<size_t>(kStaticMaxBlocks) * kStaticMaxCols2];

struct PerDevice {
  bool ready = false;
  void* scratch = nullptr;   // device address of g_static_scratch on this device
};

std::mutex g_mu;
PerDevice g_dev[64];

// First call on a device: look up the array's address on that device, which must be the
// current one and an sm_100 part (the caller has checked).  Nothing here allocates.  The address
// is kept for the life of the process; a cudaDeviceReset invalidates it.
int setup_current_device(PerDevice** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return record_cuda(e);
  if (dev < 0 || dev >= 64) return AVGGT_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  PerDevice& pd = g_dev[dev];
  if (!pd.ready) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return record_cuda(e);
    if (ptr == nullptr) return record_message("cudaGetSymbolAddress returned a null address");
    pd.scratch = ptr;
    pd.ready = true;
  }
  *out = &pd;
  return AVGGT_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace
}  // namespace avggt

using namespace avggt;

extern "C" int avggt_build_kv_noalloc(const avggt_params* p, const void* K, const void* V, void* Kc, void* Vc,
                                      int32_t* idx, float* kmean, float* vmean, void* cuda_stream) {
  Plan pl;
  int rc = make_plan(p, &pl);
  if (rc != AVGGT_OK) return rc;
  if (!K || !V || !Kc || !Vc) return AVGGT_ERR_INVALID_ARG;
  if (pl.mean_fill != 0 && (!kmean || !vmean)) return AVGGT_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(Kc) || !aligned16(Vc) ||
      (reinterpret_cast<uintptr_t>(idx) & 3u) || !aligned16(kmean) || !aligned16(vmean))
    return AVGGT_ERR_ALIGNMENT;
  // the fixed array holds rows of at most kStaticMaxCols2 floats
  if (2 * pl.H * pl.d > kStaticMaxCols2) return AVGGT_ERR_STATIC_SCRATCH;
  // the device is checked before the symbol lookup: on another architecture the library holds no
  // image of the array and the lookup itself would fail with an unrelated CUDA error
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != AVGGT_OK) return rc;
  PerDevice* pd = nullptr;
  rc = setup_current_device(&pd);
  if (rc != AVGGT_OK) return rc;
  // The compaction kernel runs four blocks per SM it is told about; telling it about fewer SMs
  // keeps its partial rows within the fixed array.
  int sm_eff = di.sm_count;
  if (sm_eff > kStaticMaxBlocks / 4) sm_eff = kStaticMaxBlocks / 4;
  if (build_kv_ws_bytes(pl, sm_eff) > kStaticScratchBytes) return AVGGT_ERR_STATIC_SCRATCH;
  return record_cuda(launch_build_kv(pl, sm_eff, K, V, Kc, Vc, idx, kmean, vmean, pd->scratch,
                                     static_cast<cudaStream_t>(cuda_stream)));
}
