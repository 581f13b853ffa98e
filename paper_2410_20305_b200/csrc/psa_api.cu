// extern "C" entry points psa_fwd / psa_bwd / psa_step_host: argument validation, then the launchers.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>

#include "psa_internal.h"

namespace {
inline bool misaligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }
}  // namespace

namespace psa {
// The plan's device blob lives on the device that was current when it was uploaded; a launch
// from another device would hand the kernels pointers that mean nothing there.
bool plan_on_current_device(const psa_plan_t* plan) {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess && dev == plan->device;
}
}  // namespace psa

extern "C" psa_status_t psa_fwd(const psa_plan_t* plan, const void* q, const void* k, const void* v, void* o,
                                float* lse, int32_t* device_status, void* stream) {
  if (!plan) return PSA_ERR_INVALID_ARG;
  if (plan->T == 0) return PSA_OK;
  if (!plan->d_blob) return PSA_ERR_INVALID_ARG;  // host-only plan: upload it first
  if (!q || !k || !v || !o || !lse) return PSA_ERR_INVALID_ARG;
  if (misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(o, 16) || misaligned(lse, 4))
    return PSA_ERR_ALIGNMENT;
  if (!psa::plan_on_current_device(plan)) return PSA_ERR_INVALID_ARG;
  psa::note_plan_use(plan, stream);
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
  if (!psa::plan_on_current_device(plan)) return PSA_ERR_INVALID_ARG;
  psa::note_plan_use(plan, stream);
  return psa::launch_bwd(plan, d_o, q, k, v, o, lse, dq, dk, dv, workspace, false, device_status, stream);
}

extern "C" psa_status_t psa_bwd_f32(const psa_plan_t* plan, const void* d_o, const void* q, const void* k,
                                    const void* v, const void* o, const float* lse, float* dq, float* dk,
                                    float* dv, void* workspace, int32_t* device_status, void* stream) {
  if (!plan) return PSA_ERR_INVALID_ARG;
  if (plan->T == 0) return PSA_OK;
  if (!plan->d_blob) return PSA_ERR_INVALID_ARG;
  if (!d_o || !q || !k || !v || !o || !lse || !dq || !dk || !dv || !workspace) return PSA_ERR_INVALID_ARG;
  if (misaligned(d_o, 16) || misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(o, 16) ||
      misaligned(dq, 16) || misaligned(dk, 16) || misaligned(dv, 16) || misaligned(lse, 4) ||
      misaligned(workspace, 256))
    return PSA_ERR_ALIGNMENT;
  if (!psa::plan_on_current_device(plan)) return PSA_ERR_INVALID_ARG;
  psa::note_plan_use(plan, stream);
  return psa::launch_bwd(plan, d_o, q, k, v, o, lse, dq, dk, dv, workspace, true, device_status, stream);
}

namespace {
// Arena of psa_step_host: the nine tensors and the backward scratch, each 256-byte aligned.
struct StepArena {
  size_t q, k, v, d_o, o, lse, dq, dk, dv, ws, bytes;
};
StepArena step_arena_layout(const psa_plan_t* plan) {
  auto up = [](size_t x) { return (x + 255) & ~size_t(255); };
  const size_t nq = size_t(plan->T) * plan->Hq * plan->d * 2, nk = size_t(plan->T) * plan->Hkv * plan->d * 2;
  StepArena a;
  size_t off = 0;
  auto take = [&](size_t n) { const size_t at = off; off += up(n); return at; };
  a.q = take(nq); a.k = take(nk); a.v = take(nk); a.d_o = take(nq); a.o = take(nq);
  a.lse = take(size_t(plan->Hq) * plan->T * 4);
  a.dq = take(nq); a.dk = take(nk); a.dv = take(nk);
  a.ws = take(plan->bwd_workspace_bytes);
  a.bytes = off;
  return a;
}
}  // namespace

extern "C" size_t psa_step_host_arena_bytes(const psa_plan_t* plan) {
  return plan ? step_arena_layout(plan).bytes : 0;
}

extern "C" psa_status_t psa_step_host(const psa_plan_t* plan, const void* h_q, const void* h_k, const void* h_v,
                                      const void* h_do, void* h_o, float* h_lse, void* h_dq, void* h_dk,
                                      void* h_dv, void* arena, size_t arena_bytes, int32_t* device_status,
                                      void* stream) {
  if (!plan) return PSA_ERR_INVALID_ARG;
  if (plan->T == 0) return PSA_OK;
  if (!plan->d_blob) return PSA_ERR_INVALID_ARG;
  if (!h_q || !h_k || !h_v || !h_do || !h_o || !h_lse || !h_dq || !h_dk || !h_dv || !arena) return PSA_ERR_INVALID_ARG;
  const StepArena a = step_arena_layout(plan);
  if (arena_bytes < a.bytes) return PSA_ERR_INVALID_ARG;
  if (misaligned(arena, 256)) return PSA_ERR_ALIGNMENT;
  if (!psa::plan_on_current_device(plan)) return PSA_ERR_INVALID_ARG;
  psa::note_plan_use(plan, stream);
  char* base = static_cast<char*>(arena);
  const cudaStream_t st = cudaStream_t(stream);
  const size_t nq = size_t(plan->T) * plan->Hq * plan->d * 2, nk = size_t(plan->T) * plan->Hkv * plan->d * 2;
  const size_t nl = size_t(plan->Hq) * plan->T * 4;
  auto copy = [&](void* dst, const void* src, size_t n, cudaMemcpyKind kind) {
    return cudaMemcpyAsync(dst, src, n, kind, st) == cudaSuccess;
  };
  if (!copy(base + a.q, h_q, nq, cudaMemcpyHostToDevice) || !copy(base + a.k, h_k, nk, cudaMemcpyHostToDevice) ||
      !copy(base + a.v, h_v, nk, cudaMemcpyHostToDevice) || !copy(base + a.d_o, h_do, nq, cudaMemcpyHostToDevice))
    return psa::check_last_cuda_error("psa_step_host copy in");
  psa_status_t rc = psa::launch_fwd(plan, base + a.q, base + a.k, base + a.v, base + a.o,
                                    reinterpret_cast<float*>(base + a.lse), device_status, stream);
  if (rc != PSA_OK) return rc;
  // o and lse are final after the forward: their copies out can leave before the backward runs.
  if (!copy(h_o, base + a.o, nq, cudaMemcpyDeviceToHost) || !copy(h_lse, base + a.lse, nl, cudaMemcpyDeviceToHost))
    return psa::check_last_cuda_error("psa_step_host copy out");
  rc = psa::launch_bwd(plan, base + a.d_o, base + a.q, base + a.k, base + a.v, base + a.o,
                       reinterpret_cast<const float*>(base + a.lse), base + a.dq, base + a.dk, base + a.dv,
                       base + a.ws, false, device_status, stream);
  if (rc != PSA_OK) return rc;
  if (!copy(h_dq, base + a.dq, nq, cudaMemcpyDeviceToHost) || !copy(h_dk, base + a.dk, nk, cudaMemcpyDeviceToHost) ||
      !copy(h_dv, base + a.dv, nk, cudaMemcpyDeviceToHost))
    return psa::check_last_cuda_error("psa_step_host copy out");
  return PSA_OK;
}

namespace psa {
psa_status_t check_last_cuda_error(const char* where) {
  const cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) return PSA_OK;
  if (std::getenv("PSA_DEBUG")) std::fprintf(stderr, "libpsa: %s: %s\n", where, cudaGetErrorString(e));
  return PSA_ERR_CUDA;
}

ProfileEvents g_profile[5] = {{nullptr, nullptr}, {nullptr, nullptr}, {nullptr, nullptr}, {nullptr, nullptr},
                              {nullptr, nullptr}};
ProfileScope::ProfileScope(int which, void* s) : ev(g_profile[which]), stream(s) {
  if (ev.start) cudaEventRecord(cudaEvent_t(ev.start), cudaStream_t(stream));
}
ProfileScope::~ProfileScope() {
  if (ev.stop) cudaEventRecord(cudaEvent_t(ev.stop), cudaStream_t(stream));
}
}  // namespace psa

extern "C" psa_status_t psa_profile_events(int32_t which, void* start, void* stop) {
  if (which < 0 || which > 4 || ((start == nullptr) != (stop == nullptr))) return PSA_ERR_INVALID_ARG;
  psa::g_profile[which] = psa::ProfileEvents{start, stop};
  return PSA_OK;
}
