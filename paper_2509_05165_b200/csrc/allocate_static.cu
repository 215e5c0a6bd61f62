// kvc_allocate_static: the budget allocation of Eqs. 20-22 for callers that cannot hand over a
// workspace because they cannot allocate device memory.  Its scratch (the digit histograms of
// the radix select) lives in a fixed array inside the library image.
#include <mutex>

#include "kvc_internal.cuh"

namespace kvc {
namespace {

// Scratch of the select: KVC_STATIC_MAX_BATCH sequences x 4 passes x 256 bins x 4 bytes = 256 KiB.
// Every device that loads the library holds one copy until the process exits.
constexpr size_t kStaticScratchWords = (size_t)KVC_STATIC_MAX_BATCH * 4 * 256;
static __device__ __align__(256) unsigned int g_static_scratch[kStaticScratchWords];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices];     // device address of g_static_scratch on each device, once known

// The array's name is only a host-side handle here; the device address has to be asked for,
// once per device and with that device current.
kvc_status static_scratch(void** out) {
  int dev = 0;
  KVC_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) {
    set_error("kvc_allocate_static: device ordinal %d beyond the %d this entry point tracks", dev, kMaxDevices);
    return KVC_ERR_UNSUPPORTED;
  }
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    KVC_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
    if (p == nullptr) {
      set_error("kvc_allocate_static: no device address for the static scratch on device %d", dev);
      return KVC_ERR_CUDA;
    }
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return KVC_OK;
}

}  // namespace
}  // namespace kvc

using namespace kvc;

extern "C" kvc_status kvc_allocate_static(const kvc_desc* d, const float* composite, int64_t budget,
                                          int32_t* n_keep, int64_t* offsets, void* stream) {
  Problem P;
  kvc_status s;
  if ((s = resolve_desc(d, &P)) != KVC_OK) return s;
  if (!composite || !n_keep || !offsets) {
    set_error("composite, n_keep or offsets is NULL");
    return KVC_ERR_INVALID_ARG;
  }
  if ((s = require_budget(P, budget)) != KVC_OK) return s;
  if (P.Bt > KVC_STATIC_MAX_BATCH) {
    set_error("kvc_allocate_static: batch %d exceeds KVC_STATIC_MAX_BATCH = %d (its scratch has a fixed size; "
              "use kvc_allocate with a workspace)", P.Bt, KVC_STATIC_MAX_BATCH);
    return KVC_ERR_UNSUPPORTED;
  }
  const size_t need = allocate_workspace_bytes(P);
  if (need > kStaticScratchWords * sizeof(unsigned int)) {
    set_error("kvc_allocate_static: %zu bytes of scratch needed, %zu built in", need,
              kStaticScratchWords * sizeof(unsigned int));
    return KVC_ERR_UNSUPPORTED;
  }
  if ((s = require_device()) != KVC_OK) return s;
  void* scratch = nullptr;
  if ((s = static_scratch(&scratch)) != KVC_OK) return s;
  // launch_allocate zeroes the histograms it uses (stream-ordered) before the first kernel
  return launch_allocate(P, composite, budget, 1, P.min_keep, n_keep, reinterpret_cast<long long*>(offsets), scratch,
                         kStaticScratchWords * sizeof(unsigned int), (cudaStream_t)stream, SelectPath::kHistograms);
}
