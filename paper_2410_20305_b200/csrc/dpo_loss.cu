// dpo_loss / simpo_loss / orpo_loss / dpo_logp_bwd: the DPO loss of Eq. 1 (Section 2.1; the printed ratio of logs is
// read as  -log sigmoid(beta * [(lp_theta(c) - lp_ref(c)) - (lp_theta(r) - lp_ref(r))]),
// averaged over the samples) and its gradient back into the logits,
//     dlogits[t][v] = sum over labels (t, y, g) scored by row t of  coef[g] * (1[v == y] - softmax(logits[t])[v]).
// dpo_logp_bwd is HBM-bound: every live row is read once from DRAM (the second sweep is meant to
// hit L2: one 1024-thread CTA per SM keeps 148 rows in flight, the first sweep loads with an
// evict-last policy, the second with evict-first, and the gradient is written with streaming
// stores) and written once; rows that score nothing are only written (zeros).
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cmath>

#include "psa.h"
#include "psa_internal.h"

namespace psa {
namespace {

constexpr int kBwdLogpThreads = 1024;   // one CTA per SM: 148 rows (38 MB) in flight, well inside L2
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint4 ld_16_keep(const uint4* p) {   // first sweep: ask L2 to keep the line for the second
  uint4 v;
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  asm volatile("ld.global.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(pol));
  return v;
}
__device__ __forceinline__ uint4 ld_16_last(const uint4* p) {   // second sweep: the line is not needed again
  uint4 v;
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(pol));
  return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

template <typename T>
struct Elem;
template <>
struct Elem<float> {
  static constexpr int kVec = 4;
  __device__ static void unpack(const uint4& v, float* x) {
    x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
  }
  __device__ static uint4 pack(const float* x) {
    return make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]), __float_as_uint(x[3]));
  }
  __device__ static float load1(const float* p) { return *p; }
  __device__ static void store1(float* p, float x) { *p = x; }
};
template <>
struct Elem<__nv_bfloat16> {
  static constexpr int kVec = 8;
  __device__ static void unpack(const uint4& v, float* x) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(w[i] << 16);
      x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static uint4 pack(const float* x) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 b = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&b);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
  __device__ static float load1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
  __device__ static void store1(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }
};

struct MaxSum {
  float m, s;
  __device__ void merge(float m2, float s2) {
    const float mn = fmaxf(m, m2);
    if (mn == -INFINITY) return;
    s = s * ex2_approx(m - mn) + s2 * ex2_approx(m2 - mn);
    m = mn;
  }
};

// One block; n_samples is small.
__global__ void dpo_loss_kernel(const float* __restrict__ pol, const float* __restrict__ ref, int n, float beta,
                                float* __restrict__ loss, float* __restrict__ coef) {
  __shared__ float part[32];
  float acc = 0.f;
  for (int s = threadIdx.x; s < n; s += blockDim.x) {
    const float z = beta * ((pol[2 * s] - ref[2 * s]) - (pol[2 * s + 1] - ref[2 * s + 1]));
    const float e = expf(-fabsf(z));
    acc += fmaxf(-z, 0.f) + log1pf(e);                   // -log sigmoid(z)
    const float sig_neg = expf(-fmaxf(z, 0.f)) / (1.f + e);   // sigmoid(-z)
    coef[2 * s] = -beta * sig_neg / float(n);
    coef[2 * s + 1] = beta * sig_neg / float(n);
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x < 32) {
    float t = threadIdx.x < (blockDim.x >> 5) ? part[threadIdx.x] : 0.f;
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (threadIdx.x == 0) *loss = n > 0 ? t / float(n) : 0.f;
  }
}

// Length-normalised, reference-free variant (SimPO); one block.
__global__ void simpo_loss_kernel(const float* __restrict__ pol, const int32_t* __restrict__ len, int n, float beta,
                                  float gamma, float* __restrict__ loss, float* __restrict__ coef,
                                  int32_t* __restrict__ status) {
  __shared__ float part[32];
  float acc = 0.f;
  for (int s = threadIdx.x; s < n; s += blockDim.x) {
    const int lc = len[2 * s], lr = len[2 * s + 1];
    if (lc < 1 || lr < 1) {
      if (status) atomicOr(status, PSA_DEVSTAT_BAD_SEGMENT);
      coef[2 * s] = 0.f;
      coef[2 * s + 1] = 0.f;
      continue;
    }
    const float z = beta * (pol[2 * s] / float(lc) - pol[2 * s + 1] / float(lr)) - gamma;
    const float e = expf(-fabsf(z));
    acc += fmaxf(-z, 0.f) + log1pf(e);                   // -log sigmoid(z)
    const float sig_neg = expf(-fmaxf(z, 0.f)) / (1.f + e);   // sigmoid(-z)
    coef[2 * s] = -beta * sig_neg / (float(n) * float(lc));
    coef[2 * s + 1] = beta * sig_neg / (float(n) * float(lr));
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x < 32) {
    float t = threadIdx.x < (blockDim.x >> 5) ? part[threadIdx.x] : 0.f;
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (threadIdx.x == 0) *loss = n > 0 ? t / float(n) : 0.f;
  }
}

// Odds-ratio variant (ORPO); one block.
__global__ void orpo_loss_kernel(const float* __restrict__ pol, const int32_t* __restrict__ len, int n, float lam,
                                 float* __restrict__ loss, float* __restrict__ coef, int32_t* __restrict__ status) {
  __shared__ float part[32];
  float acc = 0.f;
  for (int s = threadIdx.x; s < n; s += blockDim.x) {
    const int lc = len[2 * s], lr = len[2 * s + 1];
    if (lc < 1 || lr < 1) {
      if (status) atomicOr(status, PSA_DEVSTAT_BAD_SEGMENT);
      coef[2 * s] = 0.f;
      coef[2 * s + 1] = 0.f;
      continue;
    }
    const float ac = pol[2 * s] / float(lc), ar = pol[2 * s + 1] / float(lr);
    const float qc = -expm1f(ac), qr = -expm1f(ar);          // 1 - P
    const float z = (ac - logf(qc)) - (ar - logf(qr));       // log odds ratio
    const float e = expf(-fabsf(z));
    acc += -ac + lam * (fmaxf(-z, 0.f) + log1pf(e));
    const float sig_neg = expf(-fmaxf(z, 0.f)) / (1.f + e);   // sigmoid(-z)
    coef[2 * s] = (-1.f - lam * sig_neg / qc) / (float(n) * float(lc));
    coef[2 * s + 1] = (lam * sig_neg / qr) / (float(n) * float(lr));
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x < 32) {
    float t = threadIdx.x < (blockDim.x >> 5) ? part[threadIdx.x] : 0.f;
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (threadIdx.x == 0) *loss = n > 0 ? t / float(n) : 0.f;
  }
}

template <typename T>
__global__ void __launch_bounds__(kBwdLogpThreads, 1)
dpo_logp_bwd_kernel(const T* __restrict__ logits, int64_t vocab, int64_t row_stride, const int32_t* __restrict__ targets,
                    const int32_t* __restrict__ segment_ids, const int32_t* __restrict__ fork_rows,
                    const int32_t* __restrict__ fork_targets, const int32_t* __restrict__ fork_segments,
                    int32_t n_forks, int32_t n_segments, const float* __restrict__ coef, T* __restrict__ dlogits,
                    int32_t* __restrict__ status) {
  constexpr int E = Elem<T>::kVec;
  constexpr int kMaxLabels = 4;   // labels scored by one row: its own plus forks
  const int64_t row = blockIdx.x;
  const T* x = logits + row * row_stride;
  T* dx = dlogits + row * row_stride;
  const int64_t n_vec = vocab / E;

  // Labels of this row (block-uniform): (target, coefficient); invalid ones are reported and skipped.
  int32_t lab_y[kMaxLabels];
  float lab_c[kMaxLabels];
  int n_lab = 0;
  float csum = 0.f;
  auto add_label = [&](int32_t y, int32_t g) {
    if (g < 0) return;
    if (g >= n_segments) { if (status && threadIdx.x == 0) atomicOr(status, PSA_DEVSTAT_BAD_SEGMENT); return; }
    if (y < 0 || y >= vocab) { if (status && threadIdx.x == 0) atomicOr(status, PSA_DEVSTAT_BAD_TARGET); return; }
    if (n_lab < kMaxLabels) {
      lab_y[n_lab] = y;
      lab_c[n_lab] = coef[g];
      csum += coef[g];
      ++n_lab;
    }
  };
  add_label(targets[row], segment_ids[row]);
  for (int f = 0; f < n_forks; ++f)
    if (fork_rows[f] == row) add_label(fork_targets[f], fork_segments[f]);

  if (n_lab == 0) {   // nothing scored here: the gradient row is zero, the logits are not read
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    for (int64_t i = threadIdx.x; i < n_vec; i += kBwdLogpThreads) st_stream(reinterpret_cast<uint4*>(dx) + i, z);
    for (int64_t j = n_vec * E + threadIdx.x; j < vocab; j += kBwdLogpThreads) Elem<T>::store1(dx + j, 0.f);
    return;
  }

  // ---- sweep 1: log-sum-exp of the row (log2 domain)
  const uint4* xv = reinterpret_cast<const uint4*>(x);
  MaxSum acc{-INFINITY, 0.f};
  for (int64_t i = threadIdx.x; i < n_vec; i += kBwdLogpThreads) {
    float y[E];
    Elem<T>::unpack(ld_16_keep(xv + i), y);
    float mx = y[0];
#pragma unroll
    for (int j = 1; j < E; ++j) mx = fmaxf(mx, y[j]);
    mx *= kLog2e;
    const float mn = fmaxf(acc.m, mx);
    // A chunk of -inf logits (banned or padded vocabulary entries) before anything finite:
    // the shift is taken against 0 instead, so that (-inf) - (-inf) never forms; every term is 0.
    const float sh = (mn == -INFINITY) ? 0.f : mn;
    float s = acc.s * ex2_approx(acc.m - sh);
#pragma unroll
    for (int j = 0; j < E; ++j) s += ex2_approx(fmaf(y[j], kLog2e, -sh));
    acc.m = mn;
    acc.s = s;
  }
  for (int64_t j = n_vec * E + threadIdx.x; j < vocab; j += kBwdLogpThreads)
    acc.merge(Elem<T>::load1(x + j) * kLog2e, 1.f);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, acc.m, o);
    const float s2 = __shfl_xor_sync(0xffffffffu, acc.s, o);
    acc.merge(m2, s2);
  }
  __shared__ float sm_m[kBwdLogpThreads / 32], sm_s[kBwdLogpThreads / 32];
  __shared__ float sm_lse2;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { sm_m[warp] = acc.m; sm_s[warp] = acc.s; }
  __syncthreads();
  if (warp == 0) {
    MaxSum t{-INFINITY, 0.f};
    if (lane < kBwdLogpThreads / 32) { t.m = sm_m[lane]; t.s = sm_s[lane]; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, t.m, o);
      const float s2 = __shfl_xor_sync(0xffffffffu, t.s, o);
      t.merge(m2, s2);
    }
    if (lane == 0) sm_lse2 = t.m + log2f(t.s);   // log2 sum_v 2^(x_v log2 e)
  }
  __syncthreads();
  const float lse2 = sm_lse2;

  // ---- sweep 2: -csum * softmax, streamed out (the row comes from L2 this time)
  for (int64_t i = threadIdx.x; i < n_vec; i += kBwdLogpThreads) {
    float y[E];
    Elem<T>::unpack(ld_16_last(xv + i), y);
#pragma unroll
    for (int j = 0; j < E; ++j) y[j] = -csum * ex2_approx(fmaf(y[j], kLog2e, -lse2));
    st_stream(reinterpret_cast<uint4*>(dx) + i, Elem<T>::pack(y));
  }
  for (int64_t j = n_vec * E + threadIdx.x; j < vocab; j += kBwdLogpThreads)
    Elem<T>::store1(dx + j, -csum * ex2_approx(fmaf(Elem<T>::load1(x + j), kLog2e, -lse2)));
  __syncthreads();   // the label positions are rewritten below by one thread
  if (threadIdx.x == 0) {
    for (int a = 0; a < n_lab; ++a) {
      float add = 0.f;   // labels of this row that name the same token share one element
      for (int b = 0; b < n_lab; ++b)
        if (lab_y[b] == lab_y[a]) add += lab_c[b];
      const float p = ex2_approx(fmaf(Elem<T>::load1(x + lab_y[a]), kLog2e, -lse2));
      Elem<T>::store1(dx + lab_y[a], add - csum * p);
    }
  }
}

}  // namespace
}  // namespace psa

extern "C" psa_status_t dpo_loss(const float* policy_logps, const float* ref_logps, int32_t n_samples, float beta,
                                 float* loss, float* coef, void* stream) {
  if (n_samples < 0 || !loss || (n_samples > 0 && (!policy_logps || !ref_logps || !coef))) return PSA_ERR_INVALID_ARG;
  psa::dpo_loss_kernel<<<1, 256, 0, cudaStream_t(stream)>>>(policy_logps, ref_logps, n_samples, beta, loss, coef);
  return psa::check_last_cuda_error("dpo_loss launch");
}

extern "C" psa_status_t simpo_loss(const float* policy_logps, const int32_t* lengths, int32_t n_samples, float beta,
                                   float gamma, float* loss, float* coef, int32_t* device_status, void* stream) {
  if (n_samples < 0 || !loss || (n_samples > 0 && (!policy_logps || !lengths || !coef))) return PSA_ERR_INVALID_ARG;
  psa::simpo_loss_kernel<<<1, 256, 0, cudaStream_t(stream)>>>(policy_logps, lengths, n_samples, beta, gamma, loss, coef,
                                                             device_status);
  return psa::check_last_cuda_error("simpo_loss launch");
}

extern "C" psa_status_t orpo_loss(const float* policy_logps, const int32_t* lengths, int32_t n_samples, float lambda,
                                  float* loss, float* coef, int32_t* device_status, void* stream) {
  if (n_samples < 0 || !loss || (n_samples > 0 && (!policy_logps || !lengths || !coef))) return PSA_ERR_INVALID_ARG;
  psa::orpo_loss_kernel<<<1, 256, 0, cudaStream_t(stream)>>>(policy_logps, lengths, n_samples, lambda, loss, coef,
                                                            device_status);
  return psa::check_last_cuda_error("orpo_loss launch");
}

extern "C" psa_status_t dpo_logp_bwd(const void* logits, int32_t logits_dtype, int64_t n_rows, int64_t vocab,
                                     int64_t row_stride, const int32_t* targets, const int32_t* segment_ids,
                                     const int32_t* fork_rows, const int32_t* fork_targets,
                                     const int32_t* fork_segments, int32_t n_forks, int32_t n_segments,
                                     const float* coef, void* dlogits, int32_t* device_status, void* stream) {
  if (n_rows < 0 || vocab <= 0 || row_stride < vocab || n_forks < 0 || n_segments < 0) return PSA_ERR_INVALID_ARG;
  if (n_rows > 0 && (!logits || !targets || !segment_ids || !dlogits)) return PSA_ERR_INVALID_ARG;
  if (n_segments > 0 && !coef) return PSA_ERR_INVALID_ARG;
  if (n_forks > 0 && (!fork_rows || !fork_targets || !fork_segments)) return PSA_ERR_INVALID_ARG;
  if (logits_dtype != PSA_DTYPE_F32 && logits_dtype != PSA_DTYPE_BF16) return PSA_ERR_INVALID_ARG;
  if (n_rows > 0x7fffffffLL) return PSA_ERR_UNSUPPORTED;
  const int64_t esz = logits_dtype == PSA_DTYPE_F32 ? 4 : 2;
  if ((reinterpret_cast<uintptr_t>(logits) & 15) || (reinterpret_cast<uintptr_t>(dlogits) & 15) ||
      (n_rows > 1 && ((row_stride * esz) & 15)))   // the stride is not used when there is a single row
    return PSA_ERR_ALIGNMENT;
  if (n_rows == 0) return PSA_OK;
  cudaStream_t st = cudaStream_t(stream);
  const unsigned grid = unsigned(n_rows);
  if (logits_dtype == PSA_DTYPE_F32)
    psa::dpo_logp_bwd_kernel<float><<<grid, psa::kBwdLogpThreads, 0, st>>>(
        static_cast<const float*>(logits), vocab, row_stride, targets, segment_ids, fork_rows, fork_targets,
        fork_segments, n_forks, n_segments, coef, static_cast<float*>(dlogits), device_status);
  else
    psa::dpo_logp_bwd_kernel<__nv_bfloat16><<<grid, psa::kBwdLogpThreads, 0, st>>>(
        static_cast<const __nv_bfloat16*>(logits), vocab, row_stride, targets, segment_ids, fork_rows, fork_targets,
        fork_segments, n_forks, n_segments, coef, static_cast<__nv_bfloat16*>(dlogits), device_status);
  return psa::check_last_cuda_error("dpo_logp_bwd launch");
}
