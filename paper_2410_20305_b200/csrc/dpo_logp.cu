// dpo_logp: per-response summed log-probabilities (Section 2.1; responses are
// recovered from their boundaries, Section 3.2).  HBM-bound: one small CTA streams one
// live logits row exactly once with 16-byte coalesced loads, keeps a running
// (max, sum of exp) per thread in fp32, merges across the warp with shuffles and
// across warps through shared memory, and adds  logit[target] - lse  into
// out[segment] with one atomic per scored label.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cmath>

#include "psa.h"
#include "psa_internal.h"

namespace psa {
namespace {

// 128 threads x 4 loads in flight measured best on B200 (6.86 TB/s on 8192 x 128256 bf16; 256 x 4: 6.71,
// 512 x 4: 5.5, 1024 x 4: 4.6): small CTAs keep many rows in flight per SM and retire unevenly.
constexpr int kLogpThreads = 128;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Streaming 16-byte load that does not linger in L1.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

template <typename T>
struct Vec;  // 16 bytes of logits -> floats
template <>
struct Vec<float> {
  static constexpr int kElems = 4;
  __device__ static void unpack(const uint4& v, float* x) {
    x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y);
    x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
  }
  __device__ static float load1(const float* p) { return *p; }
};
template <>
struct Vec<__nv_bfloat16> {
  static constexpr int kElems = 8;
  __device__ static void unpack(const uint4& v, float* x) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(w[i] << 16);
      x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static float load1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
};

// Running log2-domain (max, sum): sum = sum_i 2^(y_i - m), y = x * log2(e).
struct MaxSum {
  float m, s;
  __device__ void merge(float m2, float s2) {
    const float mn = fmaxf(m, m2);
    if (mn == -INFINITY) return;
    s = s * ex2_approx(m - mn) + s2 * ex2_approx(m2 - mn);
    m = mn;
  }
};

template <typename T, int kUnroll>
__global__ void __launch_bounds__(kLogpThreads)
dpo_logp_kernel(const T* __restrict__ logits, int64_t vocab, int64_t row_stride, const int32_t* __restrict__ targets,
                const int32_t* __restrict__ segment_ids, const int32_t* __restrict__ fork_rows,
                const int32_t* __restrict__ fork_targets, const int32_t* __restrict__ fork_segments, int32_t n_forks,
                int32_t n_segments, float* __restrict__ out, int32_t* __restrict__ status) {
  constexpr int E = Vec<T>::kElems;
  const int64_t row = blockIdx.x;
  const int32_t seg = segment_ids[row];
  // Which labels does this row score?  (At most a handful of forks exist per pack.)
  int32_t fork = -1;
  for (int f = 0; f < n_forks; ++f)
    if (fork_rows[f] == row) fork = f;  // block-uniform
  if (seg < 0 && fork < 0) return;     // dead row: its logits are never read

  const T* x = logits + row * row_stride;
  const uint4* xv = reinterpret_cast<const uint4*>(x);
  const int64_t n_vec = vocab / E;
  MaxSum acc{-INFINITY, 0.f};

  // Main loop: kUnroll independent 16-byte loads in flight per thread.
  int64_t i = threadIdx.x;
  for (; i + int64_t(kUnroll - 1) * kLogpThreads < n_vec; i += int64_t(kUnroll) * kLogpThreads) {
    uint4 v[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) v[u] = ld_stream(xv + i + int64_t(u) * kLogpThreads);
    float y[kUnroll * E];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) Vec<T>::unpack(v[u], y + u * E);
    float mx = y[0];
#pragma unroll
    for (int j = 1; j < kUnroll * E; ++j) mx = fmaxf(mx, y[j]);
    mx *= kLog2e;
    // One rescale of the running sum per chunk, one exponential per element.
    const float mn = fmaxf(acc.m, mx);
    // A chunk of -inf logits (banned or padded vocabulary entries) before anything finite:
    // the shift is taken against 0 instead, so that (-inf) - (-inf) never forms; every term is 0.
    const float sh = (mn == -INFINITY) ? 0.f : mn;
    float s = acc.s * ex2_approx(acc.m - sh);
#pragma unroll
    for (int j = 0; j < kUnroll * E; ++j) s += ex2_approx(fmaf(y[j], kLog2e, -sh));
    acc.m = mn;
    acc.s = s;
  }
  for (; i < n_vec; i += kLogpThreads) {
    float y[E];
    Vec<T>::unpack(ld_stream(xv + i), y);
#pragma unroll
    for (int j = 0; j < E; ++j) acc.merge(y[j] * kLog2e, 1.f);
  }
  for (int64_t j = n_vec * E + threadIdx.x; j < vocab; j += kLogpThreads)  // ragged tail of the row
    acc.merge(Vec<T>::load1(x + j) * kLog2e, 1.f);

  // Warp merge by shuffles, then across warps through shared memory.
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, acc.m, o);
    const float s2 = __shfl_xor_sync(0xffffffffu, acc.s, o);
    acc.merge(m2, s2);
  }
  __shared__ float sm_m[kLogpThreads / 32], sm_s[kLogpThreads / 32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { sm_m[warp] = acc.m; sm_s[warp] = acc.s; }
  __syncthreads();
  if (warp == 0) {
    MaxSum t{-INFINITY, 0.f};
    if (lane < kLogpThreads / 32) { t.m = sm_m[lane]; t.s = sm_s[lane]; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, t.m, o);
      const float s2 = __shfl_xor_sync(0xffffffffu, t.s, o);
      t.merge(m2, s2);
    }
    if (lane == 0) {
      const float lse = (t.m + log2f(t.s)) * kLn2;  // natural log of sum exp(x)
      auto score = [&](int32_t y, int32_t g) {
        if (g < 0) return;
        if (g >= n_segments) { if (status) atomicOr(status, PSA_DEVSTAT_BAD_SEGMENT); return; }
        if (y < 0 || y >= vocab) { if (status) atomicOr(status, PSA_DEVSTAT_BAD_TARGET); return; }
        atomicAdd(out + g, Vec<T>::load1(x + y) - lse);
      };
      score(targets[row], seg);
      if (fork >= 0) {
        // Several forks may name the same row only if the caller built them so; score each.
        for (int f = 0; f < n_forks; ++f)
          if (fork_rows[f] == row) score(fork_targets[f], fork_segments[f]);
      }
    }
  }
}

}  // namespace
}  // namespace psa

extern "C" psa_status_t dpo_logp(const void* logits, int32_t logits_dtype, int64_t n_rows, int64_t vocab,
                                 int64_t row_stride, const int32_t* targets, const int32_t* segment_ids,
                                 const int32_t* fork_rows, const int32_t* fork_targets,
                                 const int32_t* fork_segments, int32_t n_forks, int32_t n_segments, float* out,
                                 int32_t* device_status, void* stream) {
  if (n_rows < 0 || vocab <= 0 || row_stride < vocab || n_forks < 0 || n_segments < 0) return PSA_ERR_INVALID_ARG;
  if (n_segments > 0 && !out) return PSA_ERR_INVALID_ARG;
  if (n_rows > 0 && (!logits || !targets || !segment_ids)) return PSA_ERR_INVALID_ARG;
  if (n_forks > 0 && (!fork_rows || !fork_targets || !fork_segments)) return PSA_ERR_INVALID_ARG;
  if (logits_dtype != PSA_DTYPE_F32 && logits_dtype != PSA_DTYPE_BF16) return PSA_ERR_INVALID_ARG;
  if (n_rows > 0x7fffffffLL) return PSA_ERR_UNSUPPORTED;
  const int64_t esz = logits_dtype == PSA_DTYPE_F32 ? 4 : 2;
  // the stride is not used when there is a single row
  if ((reinterpret_cast<uintptr_t>(logits) & 15) || (n_rows > 1 && ((row_stride * esz) & 15))) return PSA_ERR_ALIGNMENT;
  cudaStream_t st = cudaStream_t(stream);
  if (n_segments > 0 && cudaMemsetAsync(out, 0, sizeof(float) * size_t(n_segments), st) != cudaSuccess)
    return PSA_ERR_CUDA;
  if (n_rows == 0) return PSA_OK;
  const unsigned grid = unsigned(n_rows);
  psa::ProfileScope prof(2, stream);
  if (logits_dtype == PSA_DTYPE_F32)
    psa::dpo_logp_kernel<float, 4><<<grid, psa::kLogpThreads, 0, st>>>(
        static_cast<const float*>(logits), vocab, row_stride, targets, segment_ids, fork_rows, fork_targets,
        fork_segments, n_forks, n_segments, out, device_status);
  else
    psa::dpo_logp_kernel<__nv_bfloat16, 4><<<grid, psa::kLogpThreads, 0, st>>>(
        static_cast<const __nv_bfloat16*>(logits), vocab, row_stride, targets, segment_ids, fork_rows, fork_targets,
        fork_segments, n_forks, n_segments, out, device_status);
  return psa::check_last_cuda_error("dpo_logp launch");
}
