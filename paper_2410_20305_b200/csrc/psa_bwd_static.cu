// psa_bwd_static_scratch: the backward pass for callers that cannot hand over a
// workspace.  Same computation and same kernels as psa_bwd; the fp32 dq accumulator
// and the delta vector live in a fixed array inside the library's device image
// instead of a caller-provided buffer.  No counterpart in the paper.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <mutex>

#include "psa_internal.h"

namespace {

// Built-in scratch: 32 MiB per GPU that loads this library, held until the process exits.
constexpr size_t kStaticScratchBytes = size_t(PSA_STATIC_SCRATCH_BYTES);
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device
std::mutex g_scratch_mutex;

// In host code `g_static_scratch` is only a handle for the runtime, not a device address.
// The address is looked up once per device, with that device current.
psa_status_t static_scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PSA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) {
      if (std::getenv("PSA_DEBUG"))
        std::fprintf(stderr, "libpsa: cudaGetSymbolAddress(static scratch): %s\n", cudaGetErrorString(e));
      return PSA_ERR_CUDA;
    }
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return PSA_OK;
}

inline bool misaligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }

}  // namespace

extern "C" psa_status_t psa_bwd_static_scratch(const psa_plan_t* plan, const void* d_o, const void* q,
                                               const void* k, const void* v, const void* o, const float* lse,
                                               void* dq, void* dk, void* dv, int32_t* device_status,
                                               void* stream) {
  if (!plan) return PSA_ERR_INVALID_ARG;
  if (plan->T == 0) return PSA_OK;
  if (!plan->d_blob) return PSA_ERR_INVALID_ARG;
  if (!d_o || !q || !k || !v || !o || !lse || !dq || !dk || !dv) return PSA_ERR_INVALID_ARG;
  if (misaligned(d_o, 16) || misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(o, 16) ||
      misaligned(dq, 16) || misaligned(dk, 16) || misaligned(dv, 16) || misaligned(lse, 4))
    return PSA_ERR_ALIGNMENT;
  if (plan->bwd_workspace_bytes > kStaticScratchBytes) {
    if (std::getenv("PSA_DEBUG"))
      std::fprintf(stderr, "libpsa: psa_bwd_static_scratch: this plan needs %zu bytes of scratch, the built-in "
                           "buffer holds %zu; use psa_bwd with a caller-provided workspace\n",
                   plan->bwd_workspace_bytes, kStaticScratchBytes);
    return PSA_ERR_UNSUPPORTED;
  }
  // The plan's tile map and the scratch array must be on the same device as the launch.
  if (!psa::plan_on_current_device(plan)) return PSA_ERR_INVALID_ARG;
  void* scratch = nullptr;
  const psa_status_t st = static_scratch_address(&scratch);
  if (st != PSA_OK) return st;
  // launch_bwd clears the dq accumulator itself (it must start at zero) and overwrites delta,
  // so whatever the previous call left in the array does not matter.
  psa::note_plan_use(plan, stream);
  return psa::launch_bwd(plan, d_o, q, k, v, o, lse, dq, dk, dv, scratch, false, device_status, stream);
}
