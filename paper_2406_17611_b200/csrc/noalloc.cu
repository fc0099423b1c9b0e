// Halo exchange round trip for callers that cannot allocate device memory.
//
// varco_compress followed by varco_decompress needs a packed buffer of H_total * k elements
// between the two kernels, which the caller normally allocates.  Some callers cannot: code that
// runs inside a region where cudaMalloc is forbidden or would synchronise the device (a
// latency-critical serving loop, a library hook invoked while another framework owns the memory
// pool, a process whose allocator has already handed all device memory to a caching pool).  For
// them this file keeps the packed buffer in a fixed array that is part of the library image.
#include <mutex>

#include "device_common.cuh"
#include "kernels.h"

namespace {

constexpr size_t kScratchBytes = VARCO_NOALLOC_SCRATCH_BYTES;

// Lives in the global memory of every GPU that loads the library, until the process exits.
static __device__ __align__(256) unsigned char g_exchange_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void *g_scratch_addr[kMaxDevices] = {};

// The array's name is a host-side handle here, not a device address: resolve it once per device,
// with that device current, and hand the resolved pointer to the kernels.
int scratch_for_current_device(void **out) {
  int dev = 0;
  VARCO_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return VARCO_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void *ptr = nullptr;
    VARCO_CUDA_CHECK(cudaGetSymbolAddress(&ptr, g_exchange_scratch));
    if (!ptr) return VARCO_CUDA;
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return VARCO_OK;
}

}  // namespace

extern "C" int varco_exchange_noalloc(const varco_plan_t *plan, const void *X, int64_t ld, int32_t F,
                                      varco_dtype_t dtype, varco_ratio_t c, varco_key_t key, void *Xhalo,
                                      int64_t ld_halo, uint64_t *bytes, void *stream) {
  if (!plan || (dtype != VARCO_F32 && dtype != VARCO_BF16)) return VARCO_INVALID_ARG;
  const int es = dtype == VARCO_F32 ? 4 : 2, V = 16 / es;
  const int k = varco_kept_internal(F, c);
  if (k < 0) return VARCO_INVALID_ARG;
  if (F > 2048) return VARCO_UNSUPPORTED;
  auto bad = [&](const void *p, int64_t l) {
    return !p || (reinterpret_cast<uintptr_t>(p) & 15u) != 0 || l < F || (l % V) != 0;
  };
  if (bad(X, ld) || (plan->H > 0 && bad(Xhalo, ld_halo))) return VARCO_INVALID_ARG;
  if (!plan->uploaded) return VARCO_NOT_UPLOADED;
  const int64_t kstride = round_up64(k, V);
  const uint64_t need = (uint64_t)plan->H * (uint64_t)kstride * (uint64_t)es;
  if (need > kScratchBytes) return VARCO_WORKSPACE_TOO_SMALL;   // beyond the built-in scratch
  if (bytes) *bytes = (uint64_t)plan->H * (uint64_t)k * (uint64_t)es;
  void *packed = nullptr;
  int rc = scratch_for_current_device(&packed);
  if (rc != VARCO_OK) return rc;
  // every packed element that decompress reads is written by compress first: nothing to clear
  rc = varco_launch_compress_rows(plan, X, ld, F, k, dtype, key, packed, kstride, 0, nullptr, 0, (cudaStream_t)stream);
  if (rc != VARCO_OK) return rc;
  return varco_launch_decompress_slots(plan, packed, kstride, 0, F, k, dtype, key, Xhalo, ld_halo, nullptr, 0,
                                       (cudaStream_t)stream);
}
