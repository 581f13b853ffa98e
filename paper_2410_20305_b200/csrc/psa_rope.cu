// psa_position_ids / psa_rope: position ids of the shared layout (Section 3.1: the positions
// are set so that each response sees what it would see in the paired format, i.e. the
// rejected tokens restart right after the prompt) and the rotary embedding applied with them,
// "rotate-half" convention: with x = [x1 | x2] split at d/2 and angle_i = pos * theta^(-2i/d),
//     y1 = x1 cos - x2 sin,   y2 = x2 cos + x1 sin.
// HBM-bound, one CTA per token: the d/2 (cos, sin) pairs are computed once in shared memory
// and applied to all heads with 16-byte loads and stores.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cmath>

#include "psa.h"
#include "psa_internal.h"

namespace psa {
namespace {

constexpr int kRopeThreads = 256;
constexpr int kRopeMaxTokens = 8;   // tokens per CTA when a token alone does not fill it

// One CTA rotates `tpc` consecutive tokens (all heads): the angles of a token are computed once,
// into shared memory, and shared by its heads; with few heads several tokens share a CTA so that
// every thread has a 16-byte pair to work on.
__global__ void __launch_bounds__(kRopeThreads)
psa_rope_kernel(const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ y,
                const int32_t* __restrict__ position_ids, int64_t n_tokens, int32_t tpc, int32_t H, int32_t d,
                float log2_theta) {
  __shared__ float s_cos[kRopeMaxTokens * 128], s_sin[kRopeMaxTokens * 128];   // d/2 <= 128 per token
  const int64_t t0 = int64_t(blockIdx.x) * tpc;
  const int n_tok = int(min(int64_t(tpc), n_tokens - t0));
  const int half = d / 2;
  for (int i = threadIdx.x; i < n_tok * half; i += kRopeThreads) {
    const int tk = i / half, j = i % half;
    const float pos = float(position_ids[t0 + tk]);
    const float inv_freq = exp2f(-log2_theta * (2.0f * float(j) / float(d)));
    sincosf(pos * inv_freq, &s_sin[tk * 128 + j], &s_cos[tk * 128 + j]);
  }
  __syncthreads();
  const int vec_per_half = half / 8;            // 16-byte vectors in x1 (and in x2) of one head
  const int pairs_per_token = H * vec_per_half;
  const int n_pairs = n_tok * pairs_per_token;
  for (int p = threadIdx.x; p < n_pairs; p += kRopeThreads) {
    const int tk = p / pairs_per_token, q = p % pairs_per_token;
    const int h = q / vec_per_half, c = (q % vec_per_half) * 8;
    const __nv_bfloat16* xt = x + (t0 + tk) * int64_t(H) * d;
    __nv_bfloat16* yt = y + (t0 + tk) * int64_t(H) * d;
    const float* cs = s_cos + tk * 128;
    const float* sn = s_sin + tk * 128;
    const uint4 a = *reinterpret_cast<const uint4*>(xt + h * d + c);
    const uint4 b = *reinterpret_cast<const uint4*>(xt + h * d + half + c);
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
    uint32_t ow1[4], ow2[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float x1l = __uint_as_float(aw[i] << 16), x1h = __uint_as_float(aw[i] & 0xffff0000u);
      const float x2l = __uint_as_float(bw[i] << 16), x2h = __uint_as_float(bw[i] & 0xffff0000u);
      const float cl = cs[c + 2 * i], sl = sn[c + 2 * i], ch = cs[c + 2 * i + 1], sh = sn[c + 2 * i + 1];
      __nv_bfloat162 o1 = __floats2bfloat162_rn(x1l * cl - x2l * sl, x1h * ch - x2h * sh);
      __nv_bfloat162 o2 = __floats2bfloat162_rn(x2l * cl + x1l * sl, x2h * ch + x1h * sh);
      ow1[i] = *reinterpret_cast<uint32_t*>(&o1);
      ow2[i] = *reinterpret_cast<uint32_t*>(&o2);
    }
    *reinterpret_cast<uint4*>(yt + h * d + c) = make_uint4(ow1[0], ow1[1], ow1[2], ow1[3]);
    *reinterpret_cast<uint4*>(yt + h * d + half + c) = make_uint4(ow2[0], ow2[1], ow2[2], ow2[3]);
  }
}

}  // namespace
}  // namespace psa

extern "C" psa_status_t psa_position_ids(const int32_t* cu_seqlens, const int32_t* prefix_len,
                                         const int32_t* chosen_len, const int32_t* rejected_len,
                                         int32_t n_samples, int32_t* position_ids) {
  if (n_samples < 0 || !cu_seqlens) return PSA_ERR_INVALID_ARG;
  if (n_samples > 0 && (!prefix_len || !chosen_len || !rejected_len || !position_ids)) return PSA_ERR_INVALID_ARG;
  if (cu_seqlens[0] != 0) return PSA_ERR_INCONSISTENT_LENGTHS;
  for (int s = 0; s < n_samples; ++s) {
    const int32_t P = prefix_len[s], C = chosen_len[s], R = rejected_len[s];
    if (P < 0 || C < 0 || R < 0) return PSA_ERR_INVALID_ARG;
    if (int64_t(cu_seqlens[s + 1]) - cu_seqlens[s] != int64_t(P) + C + R) return PSA_ERR_INCONSISTENT_LENGTHS;
  }
  for (int s = 0; s < n_samples; ++s) {
    const int32_t P = prefix_len[s], C = chosen_len[s], R = rejected_len[s];
    int32_t* p = position_ids + cu_seqlens[s];
    for (int32_t i = 0; i < P + C; ++i) p[i] = i;
    for (int32_t j = 0; j < R; ++j) p[P + C + j] = P + j;   // rejected restarts right after the prompt
  }
  return PSA_OK;
}

extern "C" psa_status_t psa_rope(const void* x, void* y, const int32_t* position_ids, int64_t n_tokens,
                                 int32_t n_heads, int32_t head_dim, float rope_theta, void* stream) {
  if (n_tokens < 0 || n_heads <= 0 || rope_theta <= 0.f) return PSA_ERR_INVALID_ARG;
  if (head_dim <= 0 || head_dim % 16 != 0 || head_dim > 256) return PSA_ERR_UNSUPPORTED;
  if (n_tokens == 0) return PSA_OK;
  if (!x || !y || !position_ids) return PSA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(x) & 15) || (reinterpret_cast<uintptr_t>(y) & 15)) return PSA_ERR_ALIGNMENT;
  if (n_tokens > 0x7fffffffLL) return PSA_ERR_UNSUPPORTED;
  const int pairs_per_token = n_heads * (head_dim / 16);
  int tpc = psa::kRopeThreads / pairs_per_token;
  tpc = tpc < 1 ? 1 : (tpc > psa::kRopeMaxTokens ? psa::kRopeMaxTokens : tpc);
  const int64_t grid = (n_tokens + tpc - 1) / tpc;
  psa::psa_rope_kernel<<<unsigned(grid), psa::kRopeThreads, 0, cudaStream_t(stream)>>>(
      static_cast<const __nv_bfloat16*>(x), static_cast<__nv_bfloat16*>(y), position_ids, n_tokens, tpc, n_heads,
      head_dim, log2f(rope_theta));
  return psa::check_last_cuda_error("psa_rope launch");
}
