// psa_bwd: exact gradient of psa_fwd under the prefix-sharing mask with packing
// (Algorithm 3; Section 3.1).  Probabilities are recomputed from lse.
//
//   1. preprocess:  delta[h][t] = dO[t,h,:] . O[t,h,:]   (fp32), dq_accum = 0
//   2. main kernel: one CTA per (key tile j, kv head); it walks the query heads of the
//      group and, for each, the live query tiles i of the transposed tile map.  All
//      products are formed transposed (rows = keys) so that dK and dV accumulate in
//      TMEM for the whole CTA lifetime and need no atomics:
//          S^T  = K Q^T          dP^T = V dO^T
//          P^T  = exp2(S^T c - lse log2e)   (masked per element in PARTIAL tiles)
//          dS^T = P^T * (dP^T - delta)
//          dV  += P^T dO         dK  += dS^T Q          dQ_i = dS K  (added into dq_accum)
//   3. convert:     dq = bf16(dq_accum)
//
// Warp roles of the main kernel (320 threads, one CTA per SM):
//   warp 0      TMA producer: K, V once; Q and dO double-buffered per iteration
//   warp 1      UMMA issuer (tcgen05, all five products)
//   warps 2..5  compute: one thread per key row; P^T -> TMEM (bf16, over S^T),
//               dS^T -> shared memory (bf16, 128-byte swizzle) for the dK and dQ products
//   warps 6..9  dQ drain: TMEM -> registers -> vector red.add into the fp32 dq_accum
// TMEM columns: [0,128) S^T / P^T, [128,256) dP^T / dQ, [256,256+D) dV, [384,384+D) dK.
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

constexpr int kBwdThreads = 320;
constexpr uint32_t kBwdTmemCols = 512;
constexpr uint32_t kColS = 0, kColDP = 128, kColDV = 256, kColDK = 384;
constexpr float kLog2e = 1.4426950408889634f;

struct BwdParams {
  const TileRec* tiles;     // key tiles
  const int32_t* entries;   // (query tile << 2) | (precise << 1) | needs_mask
  const float* lse;         // [Hq, T]
  const float* delta;       // [Hq, T]
  float* dq_accum;          // [T, Hq, D] fp32
  __nv_bfloat16* dk;
  __nv_bfloat16* dv;
  int32_t* status;
  int32_t T, Hq, Hkv;
  float scale, scale_log2;
};

template <int D>
struct BwdSmem {
  static constexpr int kSub = D / 64;
  static constexpr int kTileBytes = kTile * D * 2;      // K, V, Q, dO tiles
  static constexpr int kSubBytes = kTile * 128;
  static constexpr int kDsBytes = kTile * kTile * 2;    // dS^T tile, 128 x 128 bf16
  static constexpr int kK = 0, kV = kTileBytes, kQ = 2 * kTileBytes, kDO = 4 * kTileBytes, kDS = 6 * kTileBytes;
  static constexpr int kBars = kDS + kDsBytes;          // 16 mbarriers
  static constexpr int kTmemSlot = kBars + 128;
  static constexpr int kAbort = kTmemSlot + 4;
  static constexpr int kLse = kBars + 256;              // [2][128] floats
  static constexpr int kDelta = kLse + 1024;            // [2][128] floats
  static constexpr int kBytes = kDelta + 1024;
  // More than half an SM's shared memory: exactly one CTA per SM, so the
  // 512-column TMEM allocation never has to wait for a neighbour.
  static constexpr int kRequest = kBytes > 120 * 1024 ? kBytes : 120 * 1024;
};

enum {
  B_KV_FULL = 0, B_Q_FULL0, B_Q_FULL1, B_DO_FULL0, B_DO_FULL1, B_QDO_EMPTY0, B_QDO_EMPTY1,
  B_S_FULL, B_DP_FULL, B_P_FULL, B_DS_FULL, B_DS_EMPTY, B_DQ_FULL, B_DQ_EMPTY, B_COUNT
};

__device__ __forceinline__ void red_add_v4(float* p, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int n) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory");
}

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
psa_bwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
               const BwdParams prm) {
  using L = BwdSmem<D>;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  const uint32_t sK = base + L::kK, sV = base + L::kV, sDS = base + L::kDS;
  auto sQ = [&](int st) { return base + L::kQ + st * L::kTileBytes; };
  auto sDO = [&](int st) { return base + L::kDO + st * L::kTileBytes; };
  auto bar = [&](int i) { return base + L::kBars + 8u * i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_raw + L::kTmemSlot);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_raw + L::kAbort);
  float* s_lse = reinterpret_cast<float*>(smem_raw + L::kLse);
  float* s_delta = reinterpret_cast<float*>(smem_raw + L::kDelta);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile_idx = blockIdx.x / prm.Hkv;
  const int hk = blockIdx.x % prm.Hkv;
  const int g = prm.Hq / prm.Hkv;
  const TileRec rec = prm.tiles[tile_idx];
  const int32_t* ent = prm.entries + rec.list_off;
  const int n_list = rec.list_cnt;
  const int n_it = n_list * g;
  const WaitCtx wctx{abort_flag, prm.status};

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    // The swizzled tiles need a 1024-byte aligned base; report instead of computing garbage.
    if (base & 1023u) {
      *abort_flag = 1;
      if (prm.status) atomicOr(prm.status, PSA_DEVSTAT_WAIT_EXPIRED);
    }
    for (int i = 0; i < B_COUNT; ++i) {
      const bool many = (i == B_P_FULL || i == B_DS_FULL || i == B_DQ_EMPTY);
      mbar_init(bar(i), many ? 128 : 1);
    }
    fence_mbar_init();
  }
  if (warp == 0) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kBwdTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // Iteration it -> (query head of the group, entry of the list).
  auto head_of = [&](int it) { return hk * g + it / n_list; };
  auto entry_of = [&](int it) { return ent[it % n_list]; };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_q);
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_v);
      tma_prefetch_desc(&tm_do);
      mbar_expect_tx(bar(B_KV_FULL), 2 * L::kTileBytes);
      for (int s = 0; s < L::kSub; ++s) tma_load_3d(sK + s * L::kSubBytes, &tm_k, s * 64, hk, rec.row0, bar(B_KV_FULL));
      for (int s = 0; s < L::kSub; ++s) tma_load_3d(sV + s * L::kSubBytes, &tm_v, s * 64, hk, rec.row0, bar(B_KV_FULL));
      for (int it = 0; it < n_it; ++it) {
        const int st = it & 1;
        const int h = head_of(it);
        const int qrow = rec.ds + (entry_of(it) >> 2) * kTile;
        if (it >= 2) mbar_wait(bar(B_QDO_EMPTY0 + st), ((it >> 1) - 1) & 1, wctx);
        mbar_expect_tx(bar(B_Q_FULL0 + st), L::kTileBytes);
        for (int s = 0; s < L::kSub; ++s) tma_load_3d(sQ(st) + s * L::kSubBytes, &tm_q, s * 64, h, qrow, bar(B_Q_FULL0 + st));
        mbar_expect_tx(bar(B_DO_FULL0 + st), L::kTileBytes);
        for (int s = 0; s < L::kSub; ++s) tma_load_3d(sDO(st) + s * L::kSubBytes, &tm_do, s * 64, h, qrow, bar(B_DO_FULL0 + st));
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_st = umma_idesc_bf16(kTile, kTile, false, false);  // K/V and Q/dO, all K-major
      constexpr uint32_t idesc_dv = umma_idesc_bf16(kTile, D, false, true);       // P^T (TMEM) x dO (MN-major)
      constexpr uint32_t idesc_dk = umma_idesc_bf16(kTile, D, false, true);       // dS^T (K-major) x Q (MN-major)
      constexpr uint32_t idesc_dq = umma_idesc_bf16(kTile, D, true, true);        // dS (MN-major) x K (MN-major)
      mbar_wait(bar(B_KV_FULL), 0, wctx);
      uint32_t ds_ph = 0;  // running parity of B_DS_FULL (it completes twice in a PRECISE iteration)
      for (int it = 0; it < n_it; ++it) {
        const int st = it & 1, ph = (it >> 1) & 1;
        // PRECISE tiles carry P^T and dS^T as two bf16 terms each.
        const int n_terms = (entry_of(it) & 2) ? 2 : 1;
        // S^T = K Q^T.  (Its columns held P^T of the previous iteration; the dV product that
        // read it was issued earlier by this thread and UMMAs execute in issue order.)
        mbar_wait(bar(B_Q_FULL0 + st), ph, wctx);
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * L::kSubBytes + (kk & 3) * 32;
          umma_ss(tmem + kColS, smem_desc_sw128(sK + off, 16, 1024), smem_desc_sw128(sQ(st) + off, 16, 1024), idesc_st,
                  kk > 0);
        }
        umma_commit(bar(B_S_FULL));
        // dP^T = V dO^T into the columns the previous dQ occupied: wait until it was drained.
        mbar_wait(bar(B_DO_FULL0 + st), ph, wctx);
        if (it > 0) mbar_wait(bar(B_DQ_EMPTY), (it - 1) & 1, wctx);
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * L::kSubBytes + (kk & 3) * 32;
          umma_ss(tmem + kColDP, smem_desc_sw128(sV + off, 16, 1024), smem_desc_sw128(sDO(st) + off, 16, 1024),
                  idesc_st, kk > 0);
        }
        umma_commit(bar(B_DP_FULL));
        // dV += P^T dO   (reduction over the 128 query rows, 16 per instruction)
        mbar_wait(bar(B_P_FULL), it & 1, wctx);
        tc_fence_after();
        for (int term = 0; term < n_terms; ++term) {   // second term: columns [64,128) of the S region
#pragma unroll
          for (int kk = 0; kk < kTile / 16; ++kk)
            umma_ts(tmem + kColDV, tmem + kColS + term * 64 + kk * 8,
                    smem_desc_sw128(sDO(st) + kk * 2048, L::kSubBytes, 1024), idesc_dv,
                    (it > 0) || (kk > 0) || (term > 0));
        }
        // dK += dS^T Q ; dQ = dS K.  The two terms of a PRECISE tile pass through the one
        // shared-memory buffer one after the other.
        for (int term = 0; term < n_terms; ++term) {
          mbar_wait(bar(B_DS_FULL), ds_ph, wctx);
          ds_ph ^= 1;
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < kTile / 16; ++kk)
            umma_ss(tmem + kColDK, smem_desc_sw128(sDS + (kk >> 2) * 16384 + (kk & 3) * 32, 16, 1024),
                    smem_desc_sw128(sQ(st) + kk * 2048, L::kSubBytes, 1024), idesc_dk,
                    (it > 0) || (kk > 0) || (term > 0));
#pragma unroll
          for (int kk = 0; kk < kTile / 16; ++kk)
            umma_ss(tmem + kColDP, smem_desc_sw128(sDS + kk * 2048, 16384, 1024),
                    smem_desc_sw128(sK + kk * 2048, L::kSubBytes, 1024), idesc_dq, (kk > 0) || (term > 0));
          if (term + 1 < n_terms) umma_commit(bar(B_DS_EMPTY));
        }
        umma_commit(bar(B_DQ_FULL));
        umma_commit(bar(B_QDO_EMPTY0 + st));
      }
    }
    __syncwarp();
  } else if (warp < 6) {
    // ------------------------------------------------------------ compute, one key row per thread
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;
    const uint32_t lane_base = uint32_t(quarter * 32) << 16;
    const int ct = threadIdx.x - 64;                    // 0..127 among the compute threads
    const int kv_local = rec.local0 + r;
    const bool kv_valid = kv_local < rec.len;
    // Queries allowed to see this key: [kv_local, qend).
    const int qend = (kv_local >= rec.cs && kv_local < rec.rs) ? rec.rs : rec.len;
    const float cl = prm.scale_log2;

    auto load_stats = [&](int it, float& l2, float& dl) {
      const int64_t qrow = int64_t(rec.ds) + (entry_of(it) >> 2) * kTile + ct;
      l2 = 0.f;
      dl = 0.f;
      if (qrow < prm.T) {
        const int64_t idx = int64_t(head_of(it)) * prm.T + qrow;
        l2 = prm.lse[idx] * kLog2e;
        dl = prm.delta[idx];
      }
    };
    {
      float l2, dl;
      load_stats(0, l2, dl);
      s_lse[ct] = l2;
      s_delta[ct] = dl;
    }
    named_bar_sync(1, 128);

    uint32_t dse_ph = 0;  // running parity of B_DS_EMPTY

    // One iteration = one (query head, query tile).  Two instantiations: PRECISE tiles carry
    // P^T and dS^T as two bf16 terms (and recompute delta exactly for a sample's first query
    // tile); keeping that out of the common instantiation keeps its register use down.
    auto iteration = [&](int it, auto precise_tag) {
      constexpr bool kPrecise = decltype(precise_tag)::value;
      const int st = it & 1;
      const int e = entry_of(it);
      const int q0 = (e >> 2) * kTile;
      float nl2 = 0.f, ndl = 0.f;
      if (it + 1 < n_it) load_stats(it + 1, nl2, ndl);

      mbar_wait(bar(B_S_FULL), it & 1, wctx);
      tc_fence_after();
      float p[kTile];
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t v[32];
        tmem_ld32(tmem + lane_base + kColS + ch * 32, v);
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) p[ch * 32 + i] = __uint_as_float(v[i]);
      }
      {
        const float4* l4 = reinterpret_cast<const float4*>(s_lse + st * kTile);
#pragma unroll
        for (int i = 0; i < kTile / 4; ++i) {
          const float4 l = l4[i];
          p[4 * i + 0] = ex2_approx(fmaf(p[4 * i + 0], cl, -l.x));
          p[4 * i + 1] = ex2_approx(fmaf(p[4 * i + 1], cl, -l.y));
          p[4 * i + 2] = ex2_approx(fmaf(p[4 * i + 2], cl, -l.z));
          p[4 * i + 3] = ex2_approx(fmaf(p[4 * i + 3], cl, -l.w));
        }
      }
      if (e & 1) {
        const int lo = kv_local - q0;                        // first allowed column (causal)
        const int hi = qend - q0;                            // one past the last allowed column
        const uint32_t span = hi > lo ? uint32_t(hi - lo) : 0u;
#pragma unroll
        for (int i = 0; i < kTile; ++i) p[i] = (uint32_t(i - lo) < span) ? p[i] : 0.f;
      }
#pragma unroll
      for (int ch = 0; ch < 2; ++ch) {
        uint32_t v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = pack_bf16x2(p[ch * 64 + 2 * i], p[ch * 64 + 2 * i + 1]);
        tmem_st32(tmem + lane_base + kColS + ch * 32, v);
        if constexpr (kPrecise) {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = pack_bf16x2_residual(p[ch * 64 + 2 * i], p[ch * 64 + 2 * i + 1], v[i]);
          tmem_st32(tmem + lane_base + kColS + 64 + ch * 32, v);
        }
      }
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar(B_P_FULL));

      // dS^T = P^T * (dP^T - delta) -> shared memory.  The buffer is free: S^T of this
      // iteration completed after the previous iteration's dK / dQ products.
      mbar_wait(bar(B_DP_FULL), it & 1, wctx);
      tc_fence_after();
      if constexpr (kPrecise) {
        if ((e >> 2) == 0) {
          // Rows of a sample's first query tile see only this key tile, and they are the rows
          // with few keys, where delta = dO . O computed from the bf16-rounded O is the largest
          // error left.  Recompute it exactly here:  delta_i = sum_j P_ij dP_ij  (fp32).
          // Column sums over the 128 key rows: transpose-reduce inside each warp, then add the
          // four warps through the (still unused) dS buffer.
          float* scratch = reinterpret_cast<float*>(smem_raw + L::kDS);
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            uint32_t v[32];
            tmem_ld32(tmem + lane_base + kColDP + ch * 32, v);
            tc_wait_ld();
            float t[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) t[i] = p[ch * 32 + i] * __uint_as_float(v[i]);
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) {
              const bool up = (lane & off) != 0;
#pragma unroll
              for (int kq = 0; kq < off; ++kq) {
                const float send = up ? t[kq] : t[kq + off];
                const float keep = up ? t[kq + off] : t[kq];
                t[kq] = keep + __shfl_xor_sync(0xffffffffu, send, off);
              }
            }
            scratch[quarter * kTile + ch * 32 + lane] = t[0];   // lane l now holds column ch*32 + l
          }
          named_bar_sync(1, 128);
          const float dsum = scratch[ct] + scratch[kTile + ct] + scratch[2 * kTile + ct] + scratch[3 * kTile + ct];
          s_delta[st * kTile + ct] = dsum;
          named_bar_sync(1, 128);
        }
      }
      const float4* d4 = reinterpret_cast<const float4*>(s_delta + st * kTile);
      uint32_t ds_lo[kPrecise ? 64 : 1];  // second bf16 term of dS^T
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t v[32];
        tmem_ld32(tmem + lane_base + kColDP + ch * 32, v);
        tc_wait_ld();
        uint32_t w[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float4 dl = d4[ch * 8 + i];
          const float a0 = p[ch * 32 + 4 * i + 0] * (__uint_as_float(v[4 * i + 0]) - dl.x);
          const float a1 = p[ch * 32 + 4 * i + 1] * (__uint_as_float(v[4 * i + 1]) - dl.y);
          const float a2 = p[ch * 32 + 4 * i + 2] * (__uint_as_float(v[4 * i + 2]) - dl.z);
          const float a3 = p[ch * 32 + 4 * i + 3] * (__uint_as_float(v[4 * i + 3]) - dl.w);
          w[2 * i] = pack_bf16x2(a0, a1);
          w[2 * i + 1] = pack_bf16x2(a2, a3);
          if constexpr (kPrecise) {
            ds_lo[ch * 16 + 2 * i] = pack_bf16x2_residual(a0, a1, w[2 * i]);
            ds_lo[ch * 16 + 2 * i + 1] = pack_bf16x2_residual(a2, a3, w[2 * i + 1]);
          }
        }
        // Row r of the 128 x 128 bf16 tile: 64-column half (ch >> 1), 16-byte chunks
        // (ch & 1) * 4 .. + 3, each stored at chunk index XOR (r & 7)  (128-byte swizzle).
        const uint32_t row_addr = sDS + (ch >> 1) * 16384 + r * 128;
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
          const uint32_t chunk = uint32_t((ch & 1) * 4 + c4) ^ uint32_t(r & 7);
          st_shared_v4(row_addr + chunk * 16, w[4 * c4], w[4 * c4 + 1], w[4 * c4 + 2], w[4 * c4 + 3]);
        }
      }
      fence_proxy_async_smem();
      tc_fence_before();
      mbar_arrive(bar(B_DS_FULL));
      if constexpr (kPrecise) {
        // second term: same buffer, once the products of the first term have read it
        mbar_wait(bar(B_DS_EMPTY), dse_ph, wctx);
        dse_ph ^= 1;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          const uint32_t row_addr = sDS + (ch >> 1) * 16384 + r * 128;
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            const uint32_t chunk = uint32_t((ch & 1) * 4 + c4) ^ uint32_t(r & 7);
            st_shared_v4(row_addr + chunk * 16, ds_lo[ch * 16 + 4 * c4], ds_lo[ch * 16 + 4 * c4 + 1],
                         ds_lo[ch * 16 + 4 * c4 + 2], ds_lo[ch * 16 + 4 * c4 + 3]);
          }
        }
        fence_proxy_async_smem();
        mbar_arrive(bar(B_DS_FULL));
      }

      s_lse[(st ^ 1) * kTile + ct] = nl2;
      s_delta[(st ^ 1) * kTile + ct] = ndl;
      named_bar_sync(1, 128);
    };
    for (int it = 0; it < n_it; ++it) {
      if (entry_of(it) & 2) iteration(it, std::true_type{});
      else iteration(it, std::false_type{});
    }

    // ---- epilogue: dV, dK (scaled) -> bf16
    mbar_wait(bar(B_DQ_FULL), (n_it - 1) & 1, wctx);
    tc_fence_after();
    const int64_t row = int64_t(rec.row0) + r;
    __nv_bfloat16* dv_row = prm.dv + (row * prm.Hkv + hk) * D;
    __nv_bfloat16* dk_row = prm.dk + (row * prm.Hkv + hk) * D;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      const float mul = which ? prm.scale : 1.f;
      __nv_bfloat16* dst_row = which ? dk_row : dv_row;
#pragma unroll
      for (int ch = 0; ch < D / 32; ++ch) {
        uint32_t v[32];
        tmem_ld32(tmem + lane_base + (which ? kColDK : kColDV) + ch * 32, v);
        tc_wait_ld();
        if (kv_valid) {
          uint4* dst = reinterpret_cast<uint4*>(dst_row + ch * 32);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 w;
            w.x = pack_bf16x2(__uint_as_float(v[8 * i + 0]) * mul, __uint_as_float(v[8 * i + 1]) * mul);
            w.y = pack_bf16x2(__uint_as_float(v[8 * i + 2]) * mul, __uint_as_float(v[8 * i + 3]) * mul);
            w.z = pack_bf16x2(__uint_as_float(v[8 * i + 4]) * mul, __uint_as_float(v[8 * i + 5]) * mul);
            w.w = pack_bf16x2(__uint_as_float(v[8 * i + 6]) * mul, __uint_as_float(v[8 * i + 7]) * mul);
            dst[i] = w;
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------ dQ drain, one query row per thread
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;
    const uint32_t lane_base = uint32_t(quarter * 32) << 16;
    const float sc = prm.scale;
    for (int it = 0; it < n_it; ++it) {
      const int q0 = (entry_of(it) >> 2) * kTile;
      const bool valid = q0 + r < rec.len;
      float* dst_row = prm.dq_accum + ((int64_t(rec.ds) + q0 + r) * prm.Hq + head_of(it)) * D;
      mbar_wait(bar(B_DQ_FULL), it & 1, wctx);
      tc_fence_after();
#pragma unroll
      for (int ch = 0; ch < D / 32; ++ch) {
        uint32_t v[32];
        tmem_ld32(tmem + lane_base + kColDP + ch * 32, v);
        tc_wait_ld();
        if (valid) {
#pragma unroll
          for (int i = 0; i < 8; ++i)
            red_add_v4(dst_row + ch * 32 + 4 * i, __uint_as_float(v[4 * i]) * sc, __uint_as_float(v[4 * i + 1]) * sc,
                       __uint_as_float(v[4 * i + 2]) * sc, __uint_as_float(v[4 * i + 3]) * sc);
        }
      }
      tc_fence_before();
      mbar_arrive(bar(B_DQ_EMPTY));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, kBwdTmemCols);
  }
}

// delta[h][t] = sum_c dO[t,h,c] * O[t,h,c]; one 16-byte load per thread and tensor.
template <int D>
__global__ void __launch_bounds__(256)
psa_bwd_delta_kernel(const __nv_bfloat16* __restrict__ d_o, const __nv_bfloat16* __restrict__ o,
                     float* __restrict__ delta, int64_t n_rows /* T*Hq */, int32_t T, int32_t Hq) {
  constexpr int kLanes = D / 8;  // threads per (t, h) row
  const int64_t gid = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t row = gid / kLanes;
  const int part = int(gid % kLanes);
  float acc = 0.f;
  if (row < n_rows) {
    const uint4 a = reinterpret_cast<const uint4*>(d_o + row * D)[part];
    const uint4 b = reinterpret_cast<const uint4*>(o + row * D)[part];
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc = fmaf(__uint_as_float(aw[i] << 16), __uint_as_float(bw[i] << 16), acc);
      acc = fmaf(__uint_as_float(aw[i] & 0xffff0000u), __uint_as_float(bw[i] & 0xffff0000u), acc);
    }
  }
#pragma unroll
  for (int off = kLanes / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  if (row < n_rows && part == 0) {
    const int64_t t = row / Hq;
    const int h = int(row % Hq);
    delta[int64_t(h) * T + t] = acc;
  }
}

__global__ void __launch_bounds__(256)
psa_bwd_convert_kernel(const float4* __restrict__ acc, uint2* __restrict__ dq, int64_t n_vec4) {
  const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < n_vec4) {
    const float4 a = acc[i];
    uint2 w;
    w.x = pack_bf16x2(a.x, a.y);
    w.y = pack_bf16x2(a.z, a.w);
    dq[i] = w;
  }
}

template <int D>
psa_status_t launch_bwd_t(const psa_plan_t* plan, const void* d_o, const void* q, const void* k, const void* v,
                          const void* o, const float* lse, void* dq, void* dk, void* dv, void* workspace,
                          int32_t* device_status, cudaStream_t stream) {
  using L = BwdSmem<D>;
  const int64_t T = plan->T;
  const BwdWorkspace ws = bwd_workspace_layout(T, plan->Hq, D);
  char* wsp = static_cast<char*>(workspace);
  float* dq_accum = reinterpret_cast<float*>(wsp + ws.dq_accum_off);
  float* delta = reinterpret_cast<float*>(wsp + ws.delta_off);

  CUtensorMap tm_q, tm_k, tm_v, tm_do;
  if (!make_tile_map_bf16(&tm_q, q, T, plan->Hq, D) || !make_tile_map_bf16(&tm_k, k, T, plan->Hkv, D) ||
      !make_tile_map_bf16(&tm_v, v, T, plan->Hkv, D) || !make_tile_map_bf16(&tm_do, d_o, T, plan->Hq, D))
    return PSA_ERR_CUDA;
  if (cudaFuncSetAttribute(psa_bwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kRequest) != cudaSuccess)
    return PSA_ERR_CUDA;

  const int64_t n_rows = T * plan->Hq;
  if (cudaMemsetAsync(dq_accum, 0, size_t(n_rows) * D * sizeof(float), stream) != cudaSuccess) return PSA_ERR_CUDA;
  {
    const int64_t threads = n_rows * (D / 8);
    psa_bwd_delta_kernel<D><<<unsigned((threads + 255) / 256), 256, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(d_o), static_cast<const __nv_bfloat16*>(o), delta, n_rows, plan->T,
        plan->Hq);
  }
  BwdParams prm;
  prm.tiles = plan->d_kv_tiles;
  prm.entries = plan->d_bwd_entries;
  prm.lse = lse;
  prm.delta = delta;
  prm.dq_accum = dq_accum;
  prm.dk = static_cast<__nv_bfloat16*>(dk);
  prm.dv = static_cast<__nv_bfloat16*>(dv);
  prm.status = device_status;
  prm.T = plan->T;
  prm.Hq = plan->Hq;
  prm.Hkv = plan->Hkv;
  prm.scale = plan->scale;
  prm.scale_log2 = plan->scale * kLog2e;
  const unsigned grid = unsigned(plan->kv_tiles.size()) * unsigned(plan->Hkv);
  {
    ProfileScope prof(1, stream);
    psa_bwd_kernel<D><<<grid, kBwdThreads, L::kRequest, stream>>>(tm_q, tm_k, tm_v, tm_do, prm);
  }
  {
    const int64_t n_vec4 = n_rows * D / 4;
    psa_bwd_convert_kernel<<<unsigned((n_vec4 + 255) / 256), 256, 0, stream>>>(
        reinterpret_cast<const float4*>(dq_accum), static_cast<uint2*>(dq), n_vec4);
  }
  return check_last_cuda_error("psa_bwd launch");
}

}  // namespace

psa_status_t launch_bwd(const psa_plan_t* plan, const void* d_o, const void* q, const void* k, const void* v,
                        const void* o, const float* lse, void* dq, void* dk, void* dv, void* workspace,
                        int32_t* device_status, void* stream) {
  if (plan->d == 128)
    return launch_bwd_t<128>(plan, d_o, q, k, v, o, lse, dq, dk, dv, workspace, device_status, cudaStream_t(stream));
  return launch_bwd_t<64>(plan, d_o, q, k, v, o, lse, dq, dk, dv, workspace, device_status, cudaStream_t(stream));
}

}  // namespace psa
