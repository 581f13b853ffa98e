// extern "C" entry points psa_fwd / psa_bwd: argument validation, then the launchers.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>

#include "psa_internal.h"

namespace {
inline bool misaligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }
}  // namespace

extern "C" psa_status_t psa_fwd(const psa_plan_t* plan, const void* q, const void* k, const void* v, void* o,
                                float* lse, int32_t* device_status, void* stream) {
  if (!plan) return PSA_ERR_INVALID_ARG;
  if (plan->T == 0) return PSA_OK;
  if (!plan->d_blob) return PSA_ERR_INVALID_ARG;  // host-only plan: upload it first
  if (!q || !k || !v || !o || !lse) return PSA_ERR_INVALID_ARG;
  if (misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(o, 16) || misaligned(lse, 4))
    return PSA_ERR_ALIGNMENT;
  return psa::launch_fwd(plan, q, k, v, o, lse, device_status, stream);
}

extern "C" psa_status_t psa_bwd(const psa_plan_t* plan, const void* d_o, const void* q, const void* k,
                                const void* v, const void* o, const float* lse, void* dq, void* dk, void* dv,
                                void* workspace, int32_t* device_status, void* stream) {
  if (!plan) return PSA_ERR_INVALID_ARG;
  if (plan->T == 0) return PSA_OK;
  if (!plan->d_blob) return PSA_ERR_INVALID_ARG;
  if (!d_o || !q || !k || !v || !o || !lse || !dq || !dk || !dv || !workspace) return PSA_ERR_INVALID_ARG;
  if (misaligned(d_o, 16) || misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(o, 16) ||
      misaligned(dq, 16) || misaligned(dk, 16) || misaligned(dv, 16) || misaligned(lse, 4) ||
      misaligned(workspace, 256))
    return PSA_ERR_ALIGNMENT;
  return psa::launch_bwd(plan, d_o, q, k, v, o, lse, dq, dk, dv, workspace, device_status, stream);
}

namespace psa {
psa_status_t check_last_cuda_error(const char* where) {
  const cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) return PSA_OK;
  if (std::getenv("PSA_DEBUG")) std::fprintf(stderr, "libpsa: %s: %s\n", where, cudaGetErrorString(e));
  return PSA_ERR_CUDA;
}

ProfileEvents g_profile[3] = {{nullptr, nullptr}, {nullptr, nullptr}, {nullptr, nullptr}};
ProfileScope::ProfileScope(int which, void* s) : ev(g_profile[which]), stream(s) {
  if (ev.start) cudaEventRecord(cudaEvent_t(ev.start), cudaStream_t(stream));
}
ProfileScope::~ProfileScope() {
  if (ev.stop) cudaEventRecord(cudaEvent_t(ev.stop), cudaStream_t(stream));
}
}  // namespace psa

extern "C" psa_status_t psa_profile_events(int32_t which, void* start, void* stop) {
  if (which < 0 || which > 2 || ((start == nullptr) != (stop == nullptr))) return PSA_ERR_INVALID_ARG;
  psa::g_profile[which] = psa::ProfileEvents{start, stop};
  return PSA_OK;
}
