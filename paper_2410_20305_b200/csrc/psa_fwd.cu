// psa_fwd: attention forward under the prefix-sharing mask with packing
// (Algorithm 3; Section 3.1), one CTA per (query tile, query head).
//
// Warp roles (192 threads):
//   warp 0      TMA producer: Q once, then K_j and V_j of every live key tile
//   warp 1      UMMA issuer:  S = Q K_j^T  and  O += P V_j  (tcgen05, accumulators in TMEM)
//   warps 2..5  softmax: one thread per query row; S is read from TMEM, masked in
//               registers when the tile is PARTIAL, turned into P = exp2(S*c - m*c)
//               in fp32 and written back to TMEM as bf16 (over S) for the second UMMA.
// Two CTAs share an SM (96 KB of shared memory and 256 TMEM columns each for
// head_dim 128), so one CTA's softmax overlaps the other's UMMAs.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <type_traits>

#include "psa_device.cuh"
#include "psa_internal.h"
#include "psa_tensormap.h"

namespace psa {
namespace {

using namespace dev;

constexpr int kFwdThreads = 192;
constexpr uint32_t kTmemCols = 256;   // S: columns [0,128), O: columns [128, 128+D)
constexpr uint32_t kColS = 0, kColO = 128;

struct FwdParams {
  const TileRec* tiles;
  const int32_t* entries;
  __nv_bfloat16* o;
  float* lse;
  int32_t* status;
  int32_t T, Hq, Hkv;
  float scale_log2;  // softmax_scale * log2(e)
};

template <int D>
struct FwdSmem {
  static constexpr int kSub = D / 64;                 // 64-column (128-byte) sub-tiles per row
  static constexpr int kTileBytes = kTile * D * 2;    // one Q / K / V tile
  static constexpr int kSubBytes = kTile * 128;       // one sub-tile: 128 rows x 128 bytes
  static constexpr int kQ = 0, kK = kTileBytes, kV = 2 * kTileBytes;
  static constexpr int kBars = 3 * kTileBytes;        // 8 mbarriers
  static constexpr int kTmemSlot = kBars + 64;
  static constexpr int kAbort = kTmemSlot + 4;
  static constexpr int kBytes = kBars + 128;
  // Request enough that at most two CTAs fit on an SM: their TMEM allocations
  // (256 columns each) then always succeed without waiting.
  static constexpr int kRequest = (kBytes + 1024 > 100 * 1024) ? kBytes + 1024 : 100 * 1024;
};

enum { BAR_Q_FULL = 0, BAR_K_FULL, BAR_V_FULL, BAR_K_EMPTY, BAR_V_EMPTY, BAR_S_FULL, BAR_P_FULL, BAR_O_FULL };

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 2)
psa_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const FwdParams prm) {
  using L = FwdSmem<D>;
  extern __shared__ uint8_t smem_raw[];
  // 128-byte-swizzled tiles need 1024-byte alignment.
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base + L::kQ, sK = base + L::kK, sV = base + L::kV;
  const uint32_t bars = base + L::kBars;
  auto bar = [&](int i) { return bars + 8u * i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_base + L::kTmemSlot);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_base + L::kAbort);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile_idx = blockIdx.x / prm.Hq;
  const int h = blockIdx.x % prm.Hq;
  const int hk = h / (prm.Hq / prm.Hkv);
  const TileRec rec = prm.tiles[tile_idx];
  const int32_t* ent = prm.entries + rec.list_off;
  const int n_it = rec.list_cnt;
  const WaitCtx wctx{abort_flag, prm.status};

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(bar(BAR_Q_FULL), 1);
    mbar_init(bar(BAR_K_FULL), 1);
    mbar_init(bar(BAR_V_FULL), 1);
    mbar_init(bar(BAR_K_EMPTY), 1);
    mbar_init(bar(BAR_V_EMPTY), 1);
    mbar_init(bar(BAR_S_FULL), 1);
    mbar_init(bar(BAR_P_FULL), 128);
    mbar_init(bar(BAR_O_FULL), 1);
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_q);
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_v);
      mbar_expect_tx(bar(BAR_Q_FULL), L::kTileBytes);
      for (int s = 0; s < L::kSub; ++s) tma_load_3d(sQ + s * L::kSubBytes, &tm_q, s * 64, h, rec.row0, bar(BAR_Q_FULL));
      for (int it = 0; it < n_it; ++it) {
        const int krow = rec.ds + (ent[it] >> 2) * kTile;
        if (it > 0) mbar_wait(bar(BAR_K_EMPTY), (it - 1) & 1, wctx);
        mbar_expect_tx(bar(BAR_K_FULL), L::kTileBytes);
        for (int s = 0; s < L::kSub; ++s) tma_load_3d(sK + s * L::kSubBytes, &tm_k, s * 64, hk, krow, bar(BAR_K_FULL));
        if (it > 0) mbar_wait(bar(BAR_V_EMPTY), (it - 1) & 1, wctx);
        mbar_expect_tx(bar(BAR_V_FULL), L::kTileBytes);
        for (int s = 0; s < L::kSub; ++s) tma_load_3d(sV + s * L::kSubBytes, &tm_v, s * 64, hk, krow, bar(BAR_V_FULL));
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = umma_idesc_bf16(kTile, kTile, false, false);  // Q, K both K-major
      constexpr uint32_t idesc_o = umma_idesc_bf16(kTile, D, false, true);       // P (TMEM), V MN-major
      mbar_wait(bar(BAR_Q_FULL), 0, wctx);
      for (int it = 0; it < n_it; ++it) {
        mbar_wait(bar(BAR_K_FULL), it & 1, wctx);
        // The S columns are also where P_{it-1} lives.  UMMAs issued by one thread execute in
        // issue order, so this S = Q K^T cannot overwrite P before the previous P V has read it.
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * L::kSubBytes + (kk & 3) * 32;
          umma_ss(tmem + kColS, smem_desc_sw128(sQ + off, 16, 1024), smem_desc_sw128(sK + off, 16, 1024), idesc_s,
                  kk > 0);
        }
        umma_commit(bar(BAR_K_EMPTY));
        umma_commit(bar(BAR_S_FULL));
        mbar_wait(bar(BAR_V_FULL), it & 1, wctx);
        mbar_wait(bar(BAR_P_FULL), it & 1, wctx);
        tc_fence_after();
        // PRECISE tiles carry P as two bf16 terms: columns [0,64) and [64,128) of the S region.
        const int n_terms = (ent[it] & 2) ? 2 : 1;
        for (int term = 0; term < n_terms; ++term) {
#pragma unroll
          for (int kk = 0; kk < kTile / 16; ++kk) {
            // A: 16 keys of P = 8 TMEM columns (two bf16 per column).  B: 16 key rows of V.
            umma_ts(tmem + kColO, tmem + kColS + term * 64 + kk * 8,
                    smem_desc_sw128(sV + kk * 2048, L::kSubBytes, 1024), idesc_o, (it > 0) || (kk > 0) || (term > 0));
          }
        }
        umma_commit(bar(BAR_V_EMPTY));
        umma_commit(bar(BAR_O_FULL));
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ softmax, one row per thread
    const int quarter = warp & 3;                 // TMEM lanes this warp may touch
    const int r = quarter * 32 + lane;            // row within the tile
    const uint32_t lane_base = uint32_t(quarter * 32) << 16;
    const int q_local = rec.local0 + r;
    const bool row_valid = q_local < rec.len;
    const float c = prm.scale_log2;
    float m_run = -INFINITY, l_run = 0.f;

    for (int it = 0; it < n_it; ++it) {
      const int e = ent[it];
      const int k0 = (e >> 2) * kTile;
      const bool precise = (e & 2) != 0;
      mbar_wait(bar(BAR_S_FULL), it & 1, wctx);
      tc_fence_after();
      float s[kTile];
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t v[32];
        tmem_ld32_wait(tmem + lane_base + kColS + ch * 32, v);
#pragma unroll
        for (int i = 0; i < 32; ++i) s[ch * 32 + i] = __uint_as_float(v[i]);
      }
      if (e & 1) {
        // Allowed keys of this row, relative to the tile: [0, a) and [b, cc).
        int a, b, cc;
        if (q_local < rec.rs) { a = q_local + 1 - k0; b = 0; cc = 0; }
        else { a = rec.cs - k0; b = rec.rs - k0; cc = q_local + 1 - k0; }
        const uint32_t span = uint32_t(cc - b);
#pragma unroll
        for (int i = 0; i < kTile; ++i) {
          const bool ok = (i < a) || (uint32_t(i - b) < span);
          s[i] = ok ? s[i] : -INFINITY;
        }
      }
      float mx = s[0];
#pragma unroll
      for (int i = 1; i < kTile; ++i) mx = fmaxf(mx, s[i]);
      const float m_new = fmaxf(m_run, mx);
      // Keep a stale maximum while it is within 2^8 of the true one: P stays <= 256
      // and the accumulator needs no rescaling.  (-inf) - (-inf) is NaN -> false.
      const bool grow = (m_new - m_run) * c > 8.0f;
      float alpha = 1.f;
      if (grow) {
        alpha = ex2_approx((m_run - m_new) * c);   // m_run = -inf -> 0
        m_run = m_new;
        l_run *= alpha;
      }
      if (it > 0 && __any_sync(0xffffffffu, grow)) {
        mbar_wait(bar(BAR_O_FULL), (it - 1) & 1, wctx);
        tc_fence_after();
#pragma unroll
        for (int ch = 0; ch < D / 32; ++ch) {
          uint32_t v[32];
          tmem_ld32_wait(tmem + lane_base + kColO + ch * 32, v);
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
          tmem_st32(tmem + lane_base + kColO + ch * 32, v);
        }
      }
      const float mc = (m_run == -INFINITY) ? 0.f : m_run * c;
      float sum = 0.f;
      // P -> bf16 over the S columns ([0,64)); PRECISE tiles also store the rounding residual as a
      // second bf16 term in columns [64,128).  Two instantiations keep the common path lean.
      auto write_p = [&](auto precise_tag) {
        constexpr bool kPrecise = decltype(precise_tag)::value;
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t v[32], vr[kPrecise ? 32 : 1];
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float p0 = ex2_approx(fmaf(s[ch * 64 + 2 * i], c, -mc));
            const float p1 = ex2_approx(fmaf(s[ch * 64 + 2 * i + 1], c, -mc));
            sum += p0 + p1;
            v[i] = pack_bf16x2(p0, p1);
            if constexpr (kPrecise) vr[i] = pack_bf16x2_residual(p0, p1, v[i]);
          }
          tmem_st32(tmem + lane_base + kColS + ch * 32, v);
          if constexpr (kPrecise) tmem_st32(tmem + lane_base + kColS + 64 + ch * 32, vr);
        }
      };
      if (precise) write_p(std::true_type{}); else write_p(std::false_type{});
      l_run += sum;
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar(BAR_P_FULL));
    }

    // ---- epilogue: O / l -> bf16, lse
    if (n_it > 0) {
      mbar_wait(bar(BAR_O_FULL), (n_it - 1) & 1, wctx);
      tc_fence_after();
    }
    const float inv_l = 1.f / l_run;
    const int64_t row = int64_t(rec.row0) + r;
    __nv_bfloat16* orow = prm.o + (row * prm.Hq + h) * D;
#pragma unroll
    for (int ch = 0; ch < D / 32; ++ch) {
      uint32_t v[32];
      tmem_ld32_wait(tmem + lane_base + kColO + ch * 32, v);
      if (row_valid) {
        uint4* dst = reinterpret_cast<uint4*>(orow + ch * 32);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint4 w;
          w.x = pack_bf16x2(__uint_as_float(v[8 * i + 0]) * inv_l, __uint_as_float(v[8 * i + 1]) * inv_l);
          w.y = pack_bf16x2(__uint_as_float(v[8 * i + 2]) * inv_l, __uint_as_float(v[8 * i + 3]) * inv_l);
          w.z = pack_bf16x2(__uint_as_float(v[8 * i + 4]) * inv_l, __uint_as_float(v[8 * i + 5]) * inv_l);
          w.w = pack_bf16x2(__uint_as_float(v[8 * i + 6]) * inv_l, __uint_as_float(v[8 * i + 7]) * inv_l);
          dst[i] = w;
        }
      }
    }
    if (row_valid) {
      const float mc = (m_run == -INFINITY) ? 0.f : m_run * c;
      prm.lse[int64_t(h) * prm.T + row] = (mc + log2f(l_run)) * 0.6931471805599453f;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

template <int D>
psa_status_t launch_fwd_t(const psa_plan_t* plan, const void* q, const void* k, const void* v, void* o, float* lse,
                          int32_t* device_status, cudaStream_t stream) {
  using L = FwdSmem<D>;
  CUtensorMap tm_q, tm_k, tm_v;
  if (!make_tile_map_bf16(&tm_q, q, plan->T, plan->Hq, D) || !make_tile_map_bf16(&tm_k, k, plan->T, plan->Hkv, D) ||
      !make_tile_map_bf16(&tm_v, v, plan->T, plan->Hkv, D))
    return PSA_ERR_CUDA;
  if (cudaFuncSetAttribute(psa_fwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kRequest) != cudaSuccess)
    return PSA_ERR_CUDA;
  FwdParams prm;
  prm.tiles = plan->d_q_tiles;
  prm.entries = plan->d_fwd_entries;
  prm.o = static_cast<__nv_bfloat16*>(o);
  prm.lse = lse;
  prm.status = device_status;
  prm.T = plan->T;
  prm.Hq = plan->Hq;
  prm.Hkv = plan->Hkv;
  prm.scale_log2 = plan->scale * 1.4426950408889634f;
  const unsigned grid = unsigned(plan->q_tiles.size()) * unsigned(plan->Hq);
  {
    ProfileScope prof(0, stream);
    psa_fwd_kernel<D><<<grid, kFwdThreads, L::kRequest, stream>>>(tm_q, tm_k, tm_v, prm);
  }
  return check_last_cuda_error("psa_fwd launch");
}

}  // namespace

psa_status_t launch_fwd(const psa_plan_t* plan, const void* q, const void* k, const void* v, void* o, float* lse,
                        int32_t* device_status, void* stream) {
  if (plan->d == 128) return launch_fwd_t<128>(plan, q, k, v, o, lse, device_status, cudaStream_t(stream));
  return launch_fwd_t<64>(plan, q, k, v, o, lse, device_status, cudaStream_t(stream));
}

}  // namespace psa
