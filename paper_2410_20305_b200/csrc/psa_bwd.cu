// psa_bwd: exact gradient of psa_fwd under the prefix-sharing mask with packing
// (Algorithm 3; Section 3.1).  Probabilities are recomputed from lse.
//
//   1. preprocess:  delta[h][t] = dO[t,h,:] . O[t,h,:]   (fp32), dq_accum = 0   (one kernel);
//      then, only for a pack that holds rejected rows with fewer than 32 visible keys outside
//      their sample's first query tile (prompts shorter than 32 tokens), a small kernel that
//      recomputes delta of those rows exactly
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
// Warp roles of the main kernel (512 threads = 4 warpgroups, one CTA per SM):
//   warp 0        TMA producer: K, V once; Q double-buffered, dO single-buffered per iteration
//   warp 1        UMMA issuer (tcgen05, all five products); warps 2, 3 idle
//   warps 4..11   workers: one thread per (key row, half of the 128 query columns);
//                 P^T -> TMEM (bf16, over S^T) for dV;  dS^T -> TMEM (bf16, over dP^T) for dK and
//                 -> shared memory (bf16, 128-byte swizzle) for dQ
//   warps 12..15  dQ drain: TMEM -> registers (columns released at once) -> shared-memory staging
//                 -> TMA reduce-add (cp.reduce.async.bulk.tensor, fp32) into dq_accum
// Registers are moved between the warpgroups with setmaxnreg (the drain holds a whole dQ row).
// TMEM columns: [0,128) S^T / P^T, [128,256) dP^T / dS^T / dQ, [256,256+D) dV, [384,384+D) dK.
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

constexpr int kBwdThreads = 512;   // 16 warps = 4 warpgroups, see the role table above
constexpr uint32_t kBwdTmemCols = 512;
constexpr uint32_t kColS = 0, kColDP = 128, kColDV = 256, kColDK = 384;
constexpr float kLog2e = 1.4426950408889634f;

struct BwdParams {
  const TileRec* tiles;     // key tiles
  const int32_t* entries;   // (query tile << 2) | (precise << 1) | needs_mask
  const int32_t* cta_map;   // per CTA: (key tile record, kv head)
  const float* lse;         // [Hq, T]
  const float* delta;       // [Hq, T]
  float* dq_accum;          // [T, Hq, D] fp32
  void* dk;                 // [T, Hkv, D], bf16 or (f32_out) fp32
  void* dv;
  int32_t* status;
  int32_t T, Hq, Hkv;
  int32_t f32_out;          // gradients leave as fp32: dk, dv from the accumulators, dq = dq_accum
  float scale, scale_log2;
};

template <int D>
struct BwdSmem {
  static constexpr int kSub = D / 64;
  static constexpr int kTileBytes = kTile * D * 2;      // K, V, Q, dO tiles
  static constexpr int kSubBytes = kTile * 128;
  static constexpr int kDsBytes = kTile * kTile * 2;    // dS^T tile, 128 x 128 bf16
  static constexpr int kStageBytes = kTile * 32 * 4;    // dQ staging: 128 rows x 32 fp32 columns
  static constexpr int kK = 0, kV = kTileBytes, kQ = 2 * kTileBytes /* 2 stages */, kDO = 4 * kTileBytes;
  static constexpr int kDQS = 5 * kTileBytes;           // 2 staging buffers
  static constexpr int kDS = kDQS + 2 * kStageBytes;
  static constexpr int kBars = kDS + kDsBytes;          // 16 mbarriers
  static constexpr int kTmemSlot = kBars + 128;
  static constexpr int kAbort = kTmemSlot + 4;
  static constexpr int kLse = kBars + 256;              // [2][128] floats
  static constexpr int kDelta = kLse + 1024;            // [2][128] floats
  static constexpr int kEnt = kDelta + 1024;            // first kEntCap entries of the tile's list
  static constexpr int kEntCap = 128;
  static constexpr int kBytes = kEnt + kEntCap * 4;
  // More than half an SM's shared memory: exactly one CTA per SM, so the
  // 512-column TMEM allocation never has to wait for a neighbour.
  static constexpr int kRequest = kBytes > 120 * 1024 ? kBytes : 120 * 1024;
};

enum {
  B_KV_FULL = 0, B_Q_FULL0, B_Q_FULL1, B_Q_EMPTY0, B_Q_EMPTY1, B_DO_FULL, B_DO_EMPTY,
  B_S_FULL, B_DP_FULL, B_P_FULL, B_DS_FULL, B_DS_EMPTY, B_DQ_FULL, B_DQ_EMPTY, B_DONE, B_COUNT
};


template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
psa_bwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
               const __grid_constant__ CUtensorMap tm_dq, const __grid_constant__ CUtensorMap tm_dk,
               const __grid_constant__ CUtensorMap tm_dv, const BwdParams prm) {
  using L = BwdSmem<D>;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  const uint32_t sK = base + L::kK, sV = base + L::kV, sDS = base + L::kDS;
  auto sQ = [&](int st) { return base + L::kQ + st * L::kTileBytes; };
  const uint32_t sDO = base + L::kDO;
  int32_t* s_ent = reinterpret_cast<int32_t*>(smem_raw + L::kEnt);
  auto bar = [&](int i) { return base + L::kBars + 8u * i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_raw + L::kTmemSlot);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_raw + L::kAbort);
  float* s_lse = reinterpret_cast<float*>(smem_raw + L::kLse);
  float* s_delta = reinterpret_cast<float*>(smem_raw + L::kDelta);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile_idx = prm.cta_map[2 * blockIdx.x];
  const int hk = prm.cta_map[2 * blockIdx.x + 1];
  const int g = prm.Hq / prm.Hkv;
  const TileRec rec = prm.tiles[tile_idx];
  const int32_t* ent = prm.entries + rec.list_off;
  const int n_list = rec.list_cnt;
  const int n_it = n_list * g;
  const WaitCtx wctx{abort_flag, prm.status, kWaitLimitClocks};

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    // The swizzled tiles need a 1024-byte aligned base; report instead of computing garbage.
    if (base & 1023u) {
      *abort_flag = 1;
      if (prm.status) atomicOr(prm.status, PSA_DEVSTAT_WAIT_EXPIRED);
    }
    for (int i = 0; i < B_COUNT; ++i) {
      mbar_init(bar(i), (i == B_P_FULL || i == B_DS_FULL) ? 256 : (i == B_DQ_EMPTY ? 128 : 1));
    }
    fence_mbar_init();
    // The K and V tiles are requested right away: their flight overlaps the TMEM allocation and
    // the CTA-wide barrier below.
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    mbar_expect_tx(bar(B_KV_FULL), 2 * L::kTileBytes);
    for (int s = 0; s < L::kSub; ++s) tma_load_3d(sK + s * L::kSubBytes, &tm_k, s * 64, hk, rec.row0, bar(B_KV_FULL));
    for (int s = 0; s < L::kSub; ++s) tma_load_3d(sV + s * L::kSubBytes, &tm_v, s * 64, hk, rec.row0, bar(B_KV_FULL));
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_do);
    // ... and so are Q and dO of the first iteration (head hk * g, first entry of the list).
    if (n_it > 0) {
      const int qrow0 = rec.ds + (ent[0] >> 2) * kTile;
      mbar_expect_tx(bar(B_Q_FULL0), L::kTileBytes);
      for (int s = 0; s < L::kSub; ++s) tma_load_3d(sQ(0) + s * L::kSubBytes, &tm_q, s * 64, hk * g, qrow0, bar(B_Q_FULL0));
      mbar_expect_tx(bar(B_DO_FULL), L::kTileBytes);
      for (int s = 0; s < L::kSub; ++s) tma_load_3d(sDO + s * L::kSubBytes, &tm_do, s * 64, hk * g, qrow0, bar(B_DO_FULL));
    }
    tma_prefetch_desc(&tm_dq);
  }
  // The list is read by every role in every iteration: keep its head in shared memory.
  if (int(threadIdx.x) < n_list && int(threadIdx.x) < L::kEntCap) s_ent[threadIdx.x] = ent[threadIdx.x];
  if (warp == 0) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kBwdTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // Iteration it -> (query head of the group, entry of the list).
  auto head_of = [&](int it) { return hk * g + it / n_list; };
  auto entry_of = [&](int it) {
    const int li = it % n_list;
    return li < L::kEntCap ? s_ent[li] : ent[li];
  };

  // Each warpgroup changes its register budget as its first action, inside its own branch, so
  // that everything the branch executes afterwards is compiled for that budget.
  if (warp < 4) {
  setmaxnreg_dec<72>();
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      for (int it = 1; it < n_it; ++it) {   // iteration 0 was requested before the CTA-wide barrier
        const int st = it & 1;
        const int h = head_of(it);
        const int qrow = rec.ds + (entry_of(it) >> 2) * kTile;
        if (it >= 2) mbar_wait(bar(B_Q_EMPTY0 + st), ((it >> 1) - 1) & 1, wctx);
        mbar_expect_tx(bar(B_Q_FULL0 + st), L::kTileBytes);
        for (int s = 0; s < L::kSub; ++s) tma_load_3d(sQ(st) + s * L::kSubBytes, &tm_q, s * 64, h, qrow, bar(B_Q_FULL0 + st));
        mbar_wait(bar(B_DO_EMPTY), (it - 1) & 1, wctx);   // dV of the previous iteration has read dO
        mbar_expect_tx(bar(B_DO_FULL), L::kTileBytes);
        for (int s = 0; s < L::kSub; ++s) tma_load_3d(sDO + s * L::kSubBytes, &tm_do, s * 64, h, qrow, bar(B_DO_FULL));
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ UMMA issuer
    // The whole warp runs this loop with warp-uniform operands; one elected lane issues.
    {
      const uint32_t issuer = elect_one();
      constexpr uint32_t idesc_st = umma_idesc_bf16(kTile, kTile, false, false);  // K/V and Q/dO, all K-major
      constexpr uint32_t idesc_dv = umma_idesc_bf16(kTile, D, false, true);       // P^T (TMEM) x dO (MN-major)
      constexpr uint32_t idesc_dk = umma_idesc_bf16(kTile, D, false, true);       // dS^T (K-major) x Q (MN-major)
      constexpr uint32_t idesc_dq = umma_idesc_bf16(kTile, D, true, true);        // dS (MN-major) x K (MN-major)
      // Low descriptor words of every operand view (K-major: _k, MN-major: _mn); a K step of 16
      // elements advances a K-major operand by 32 bytes inside its 64-element sub-tile and an
      // MN-major operand by 16 rows (2048 bytes).
      const uint32_t k_k = smem_desc_lo(sK, 16), v_k = smem_desc_lo(sV, 16), do_k = smem_desc_lo(sDO, 16);
      const uint32_t q0_k = smem_desc_lo(sQ(0), 16), q1_k = smem_desc_lo(sQ(1), 16);
      const uint32_t ds_mn = smem_desc_lo(sDS, 16384);
      const uint32_t do_mn = smem_desc_lo(sDO, L::kSubBytes), k_mn = smem_desc_lo(sK, L::kSubBytes);
      const uint32_t q0_mn = smem_desc_lo(sQ(0), L::kSubBytes), q1_mn = smem_desc_lo(sQ(1), L::kSubBytes);
      mbar_wait(bar(B_KV_FULL), 0, wctx);
      uint32_t ds_ph = 0;  // running parity of B_DS_FULL (it completes twice in a PRECISE iteration)
      // S^T = K Q^T of iteration `it`.  Its columns hold P^T of the previous iteration; the dV
      // product that reads it is always issued earlier by this thread and UMMAs execute in issue order.
      auto issue_s = [&](int it) {
        const int st = it & 1, ph = (it >> 1) & 1;
        mbar_wait(bar(B_Q_FULL0 + st), ph, wctx);
        tc_fence_after();
        const uint32_t q_lo = st ? q1_k : q0_k;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = ((kk >> 2) * L::kSubBytes + (kk & 3) * 32) >> 4;
          umma_ss_w(tmem + kColS, k_k + off, q_lo + off, idesc_st, kk > 0, issuer);
        }
        umma_commit_w(bar(B_S_FULL), issuer);
      };
      issue_s(0);
      for (int it = 0; it < n_it; ++it) {
        const int st = it & 1;
        // PRECISE tiles carry P^T and dS^T as two bf16 terms each.
        const int n_terms = (entry_of(it) & 2) ? 2 : 1;
        // dP^T = V dO^T into the columns the previous dQ occupied: wait until it was read out.
        // (This commit also covers the previous iteration's dK / dQ products, so a completed
        // dP^T tells the compute warps that the dS buffer is free again.)
        mbar_wait(bar(B_DO_FULL), it & 1, wctx);
        if (it > 0) mbar_wait(bar(B_DQ_EMPTY), (it - 1) & 1, wctx);
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = ((kk >> 2) * L::kSubBytes + (kk & 3) * 32) >> 4;
          umma_ss_w(tmem + kColDP, v_k + off, do_k + off, idesc_st, kk > 0, issuer);
        }
        umma_commit_w(bar(B_DP_FULL), issuer);
        // dV += P^T dO   (reduction over the 128 query rows, 16 per instruction)
        mbar_wait(bar(B_P_FULL), it & 1, wctx);
        tc_fence_after();
        // P^T of query columns [64 h, 64 h + 64) sits in S-region columns [64 h, 64 h + 32), the
        // second term of a PRECISE tile in [64 h + 32, 64 h + 64); 16 queries = 8 columns.
        for (int term = 0; term < n_terms; ++term) {
#pragma unroll
          for (int kk = 0; kk < kTile / 16; ++kk)
            umma_ts_w(tmem + kColDV, tmem + kColS + (kk >> 2) * 64 + term * 32 + (kk & 3) * 8,
                       do_mn + kk * (2048 >> 4), idesc_dv, (it > 0) || (kk > 0) || (term > 0), issuer);
        }
        umma_commit_w(bar(B_DO_EMPTY), issuer);
        // The next S^T goes in now, so that the compute warps can start on it while the dK / dQ
        // products of this iteration run.
        if (it + 1 < n_it) issue_s(it + 1);
        // dK += dS^T Q ; dQ = dS K.  dS^T reaches dK from TMEM (the workers leave it, as bf16 pairs
        // and with the second term of a PRECISE tile beside it, in the columns of dP^T they have
        // read) and dQ from the shared-memory buffer, whose two PRECISE terms pass through it one
        // after the other.  dK goes first: dQ's accumulator overwrites those columns.
        mbar_wait(bar(B_DS_FULL), ds_ph, wctx);
        ds_ph ^= 1;
        tc_fence_after();
        for (int term = 0; term < n_terms; ++term) {
#pragma unroll
          for (int kk = 0; kk < kTile / 16; ++kk)
            umma_ts_w(tmem + kColDK, tmem + kColDP + (kk >> 2) * 64 + term * 32 + (kk & 3) * 8,
                      (st ? q1_mn : q0_mn) + kk * (2048 >> 4), idesc_dk, (it > 0) || (kk > 0) || (term > 0), issuer);
        }
        umma_commit_w(bar(B_Q_EMPTY0 + st), issuer);
        for (int term = 0; term < n_terms; ++term) {
          if (term > 0) {
            umma_commit_w(bar(B_DS_EMPTY), issuer);
            mbar_wait(bar(B_DS_FULL), ds_ph, wctx);
            ds_ph ^= 1;
            tc_fence_after();
          }
#pragma unroll
          for (int kk = 0; kk < kTile / 16; ++kk)
            umma_ss_w(tmem + kColDP, ds_mn + kk * (2048 >> 4), k_mn + kk * (2048 >> 4), idesc_dq,
                       (kk > 0) || (term > 0), issuer);
        }
        umma_commit_w(bar(B_DQ_FULL), issuer);
      }
      umma_commit_w(bar(B_DONE), issuer);   // every product, the last dK included, has completed
    }
    __syncwarp();
  }  // warps 2, 3 of the first warpgroup are idle
  } else if (warp < 12) {
    // ------------------------------------------------------------ workers: warps 4..11
    // Thread = one key row (TMEM lane) and one half of the 128 query columns: warps 4..7 take
    // columns [0,64), warps 8..11 columns [64,128).
    setmaxnreg_inc<144>();
    constexpr int DH = D / 2;                           // dV / dK columns per worker in the epilogue
    const int quarter = warp & 3;
    const int half = (warp - 4) >> 2;
    const int r = quarter * 32 + lane;
    const uint32_t lane_base = uint32_t(quarter * 32) << 16;
    const int wt = threadIdx.x - 128;                   // 0..255 among the workers
    const int c0 = half * 64;                           // first query column of this thread
    const bool leader = wt == 0;
    const int kv_local = rec.local0 + r;
    const bool kv_valid = kv_local < rec.len;
    // Queries allowed to see this key: [kv_local, qend).
    const int qend = (kv_local >= rec.cs && kv_local < rec.rs) ? rec.rs : rec.len;
    const float cl = prm.scale_log2;

    // Per-column statistics of the iteration's query tile: workers 0..127 fetch lse * log2e,
    // workers 128..255 fetch delta, each for column (wt & 127).
    auto load_stat = [&](int it) {
      const int64_t qrow = int64_t(rec.ds) + (entry_of(it) >> 2) * kTile + (wt & 127);
      float x = 0.f;
      if (qrow < prm.T && PSA_IN_BOUNDS(int64_t(head_of(it)) * prm.T + qrow, int64_t(prm.Hq) * prm.T, prm.status)) {
        const int64_t idx = int64_t(head_of(it)) * prm.T + qrow;
        x = wt < 128 ? prm.lse[idx] * kLog2e : prm.delta[idx];
      }
      return x;
    };
    auto store_stat = [&](int st, float x) { (wt < 128 ? s_lse : s_delta)[st * kTile + (wt & 127)] = x; };
    store_stat(0, load_stat(0));
    named_bar_sync(1, 256);

    uint32_t dse_ph = 0;  // running parity of B_DS_EMPTY

    // One iteration = one (query head, query tile).  Two instantiations: PRECISE tiles carry
    // P^T and dS^T as two bf16 terms (and recompute delta exactly for a sample's first query
    // tile); keeping that out of the common instantiation keeps its register use down.
    auto iteration = [&](int it, auto precise_tag) {
      constexpr bool kPrecise = decltype(precise_tag)::value;
      const int st = it & 1;
      const int e = entry_of(it);
      const int q0 = (e >> 2) * kTile;
      float next_stat = 0.f;
      if (it + 1 < n_it) next_stat = load_stat(it + 1);

      mbar_wait(bar(B_S_FULL), it & 1, wctx);
      tc_fence_after();
      float p[64];
      {
        uint32_t sv[64];   // both loads in flight, one wait
        tmem_ld64_wait(tmem + lane_base + kColS + c0, sv);
        const float4* l4 = reinterpret_cast<const float4*>(s_lse + st * kTile + c0);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float4 l = l4[i];
          p[4 * i + 0] = ex2_approx(fmaf(__uint_as_float(sv[4 * i + 0]), cl, -l.x));
          p[4 * i + 1] = ex2_approx(fmaf(__uint_as_float(sv[4 * i + 1]), cl, -l.y));
          p[4 * i + 2] = ex2_approx(fmaf(__uint_as_float(sv[4 * i + 2]), cl, -l.z));
          p[4 * i + 3] = ex2_approx(fmaf(__uint_as_float(sv[4 * i + 3]), cl, -l.w));
        }
      }
      if (e & 1) {
        const int lo = kv_local - q0 - c0;                   // first allowed column (causal), relative to c0
        const int hi = qend - q0 - c0;                       // one past the last allowed column
        const uint32_t span = hi > lo ? uint32_t(hi - lo) : 0u;
#pragma unroll
        for (int i = 0; i < 64; ++i) p[i] = (uint32_t(i - lo) < span) ? p[i] : 0.f;
      }
      {
        // bf16 pairs: this half's 64 probabilities go to the first 32 of the 64 S^T columns this
        // thread has just read (never into the other half's columns: the thread of the other
        // half may not have read its S^T yet); the second term of a PRECISE tile to the last 32.
        uint32_t v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = pack_bf16x2(p[2 * i], p[2 * i + 1]);
        tmem_st32(tmem + lane_base + kColS + half * 64, v);
        if constexpr (kPrecise) {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = pack_bf16x2_residual(p[2 * i], p[2 * i + 1], v[i]);
          tmem_st32(tmem + lane_base + kColS + half * 64 + 32, v);
        }
      }
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar(B_P_FULL));

      // dS^T = P^T * (dP^T - delta) -> shared memory.  The buffer is free: dP^T of this
      // iteration was issued, and so completed, after the previous iteration's dK / dQ products.
      mbar_wait(bar(B_DP_FULL), it & 1, wctx);
      tc_fence_after();
      if constexpr (kPrecise) {
        if ((e >> 2) == 0) {
          // Rows of a sample's first query tile see only this key tile, and they are the rows
          // with few keys, where delta = dO . O computed from the bf16-rounded O is the largest
          // error left.  Recompute it exactly here:  delta_i = sum_j P_ij dP_ij  (fp32).
          // Column sums over the 128 key rows: transpose-reduce inside each warp, then add the
          // four warps of each half through the (still unused) dS buffer.
          float* scratch = reinterpret_cast<float*>(smem_raw + L::kDS);
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            uint32_t v[32];
            tmem_ld32_wait(tmem + lane_base + kColDP + c0 + j * 32, v);
            float t[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) t[i] = p[j * 32 + i] * __uint_as_float(v[i]);
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
            scratch[quarter * kTile + c0 + j * 32 + lane] = t[0];   // lane l holds column c0 + 32 j + l
          }
          named_bar_sync(1, 256);
          if (wt < kTile)
            s_delta[st * kTile + wt] = scratch[wt] + scratch[kTile + wt] + scratch[2 * kTile + wt] + scratch[3 * kTile + wt];
          named_bar_sync(1, 256);
        }
      }
      const float4* d4 = reinterpret_cast<const float4*>(s_delta + st * kTile + c0);
      uint32_t ds_lo[kPrecise ? 32 : 1];  // second bf16 term of dS^T
      // Row r of this half's 128 x 64 bf16 sub-tile: eight 16-byte chunks, each stored at chunk
      // index XOR (r & 7)  (128-byte swizzle).
      const uint32_t row_addr = sDS + half * 16384 + r * 128;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        uint32_t v[32];
        tmem_ld32_wait(tmem + lane_base + kColDP + c0 + j * 32, v);
        uint32_t w[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float4 dl = d4[j * 8 + i];
          const float a0 = p[j * 32 + 4 * i + 0] * (__uint_as_float(v[4 * i + 0]) - dl.x);
          const float a1 = p[j * 32 + 4 * i + 1] * (__uint_as_float(v[4 * i + 1]) - dl.y);
          const float a2 = p[j * 32 + 4 * i + 2] * (__uint_as_float(v[4 * i + 2]) - dl.z);
          const float a3 = p[j * 32 + 4 * i + 3] * (__uint_as_float(v[4 * i + 3]) - dl.w);
          w[2 * i] = pack_bf16x2(a0, a1);
          w[2 * i + 1] = pack_bf16x2(a2, a3);
          if constexpr (kPrecise) {
            ds_lo[j * 16 + 2 * i] = pack_bf16x2_residual(a0, a1, w[2 * i]);
            ds_lo[j * 16 + 2 * i + 1] = pack_bf16x2_residual(a2, a3, w[2 * i + 1]);
          }
        }
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
          const uint32_t chunk = uint32_t(j * 4 + c4) ^ uint32_t(r & 7);
          st_shared_v4(row_addr + chunk * 16, w[4 * c4], w[4 * c4 + 1], w[4 * c4 + 2], w[4 * c4 + 3]);
        }
        // The same values for dK, which takes dS^T from TMEM: over the first 32 of this thread's 64
        // dP^T columns, all of which it has read by now (chunk 0 before the first store).
        tmem_st16(tmem + lane_base + kColDP + half * 64 + j * 16, w);
      }
      if constexpr (kPrecise) {
        // second term of dS^T for dK: the other 32 of the thread's own columns
#pragma unroll
        for (int j = 0; j < 2; ++j)
          tmem_st16(tmem + lane_base + kColDP + half * 64 + 32 + j * 16,
                    reinterpret_cast<const uint32_t(&)[16]>(ds_lo[j * 16]));
      }
      tc_wait_st();
      fence_proxy_async_smem();
      tc_fence_before();
      mbar_arrive(bar(B_DS_FULL));
      if constexpr (kPrecise) {
        // second term: same buffer, once the products of the first term have read it
        mbar_wait(bar(B_DS_EMPTY), dse_ph, wctx);
        dse_ph ^= 1;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            const uint32_t chunk = uint32_t(j * 4 + c4) ^ uint32_t(r & 7);
            st_shared_v4(row_addr + chunk * 16, ds_lo[j * 16 + 4 * c4], ds_lo[j * 16 + 4 * c4 + 1],
                         ds_lo[j * 16 + 4 * c4 + 2], ds_lo[j * 16 + 4 * c4 + 3]);
          }
        }
        fence_proxy_async_smem();
        mbar_arrive(bar(B_DS_FULL));
      }

      store_stat(st ^ 1, next_stat);
      named_bar_sync(1, 256);
    };
    for (int it = 0; it < n_it; ++it) {
      if (entry_of(it) & 2) iteration(it, std::true_type{});
      else iteration(it, std::false_type{});
    }
    mbar_wait(bar(B_DONE), 0, wctx);
    tc_fence_after();

    // ---- epilogue: this half's columns of dV and dK (scaled) -> bf16, or fp32 as they are
    if (prm.f32_out) {
      // fp32 outputs: the accumulators leave unrounded, one row per thread.
      const int64_t row = int64_t(rec.row0) + r;
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        const float mul = which ? prm.scale : 1.f;
        float* dst_row = static_cast<float*>(which ? prm.dk : prm.dv) + (row * prm.Hkv + hk) * D + half * DH;
#pragma unroll
        for (int ch = 0; ch < DH / 32; ++ch) {
          uint32_t v[32];
          tmem_ld32_wait(tmem + lane_base + (which ? kColDK : kColDV) + half * DH + ch * 32, v);
          if (kv_valid && PSA_IN_BOUNDS((row * prm.Hkv + hk) * D + half * DH + ch * 32 + 31, int64_t(prm.T) * prm.Hkv * D,
                                        prm.status)) {
            float4* dst = reinterpret_cast<float4*>(dst_row + ch * 32);
#pragma unroll
            for (int i = 0; i < 8; ++i)
              dst[i] = make_float4(__uint_as_float(v[4 * i + 0]) * mul, __uint_as_float(v[4 * i + 1]) * mul,
                                   __uint_as_float(v[4 * i + 2]) * mul, __uint_as_float(v[4 * i + 3]) * mul);
          }
        }
      }
    } else if (rec.len - rec.local0 >= kTile) {
      // Full tile: rows go through shared memory (the K and V buffers are free now) in the
      // 128-byte-swizzled layout of the tensor maps, and two TMA stores per tensor write them
      // out coalesced.  (A ragged last tile must not touch the rows of the next sample, which the
      // box would cover: it takes the per-thread path below.)
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        const float mul = which ? prm.scale : 1.f;
        const uint32_t tile = which ? sK : sV;     // dK leaves through the K buffer, dV through V's
#pragma unroll
        for (int ch = 0; ch < DH / 32; ++ch) {
          uint32_t v[32];
          tmem_ld32_wait(tmem + lane_base + (which ? kColDK : kColDV) + half * DH + ch * 32, v);
          // 64-column sub-tile of this thread's columns, then the 16-byte chunk inside its row
          const int col0 = half * DH + ch * 32;
          const uint32_t row_addr = tile + (col0 >> 6) * L::kSubBytes + r * 128;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint32_t chunk = uint32_t(((col0 & 63) >> 3) + i) ^ uint32_t(r & 7);
            st_shared_v4(row_addr + chunk * 16,
                         pack_bf16x2(__uint_as_float(v[8 * i + 0]) * mul, __uint_as_float(v[8 * i + 1]) * mul),
                         pack_bf16x2(__uint_as_float(v[8 * i + 2]) * mul, __uint_as_float(v[8 * i + 3]) * mul),
                         pack_bf16x2(__uint_as_float(v[8 * i + 4]) * mul, __uint_as_float(v[8 * i + 5]) * mul),
                         pack_bf16x2(__uint_as_float(v[8 * i + 6]) * mul, __uint_as_float(v[8 * i + 7]) * mul));
          }
        }
      }
      fence_proxy_async_smem();
      named_bar_sync(1, 256);
      if (leader) {
        for (int s = 0; s < L::kSub; ++s) {
          tma_store_3d(&tm_dv, sV + s * L::kSubBytes, s * 64, hk, rec.row0);
          tma_store_3d(&tm_dk, sK + s * L::kSubBytes, s * 64, hk, rec.row0);
        }
        tma_commit_group();
        tma_wait_group_read<0>();   // shared memory must outlive the stores' reads
      }
    } else {
    const int64_t row = int64_t(rec.row0) + r;
    __nv_bfloat16* dv_row = static_cast<__nv_bfloat16*>(prm.dv) + (row * prm.Hkv + hk) * D + half * DH;
    __nv_bfloat16* dk_row = static_cast<__nv_bfloat16*>(prm.dk) + (row * prm.Hkv + hk) * D + half * DH;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      const float mul = which ? prm.scale : 1.f;
      __nv_bfloat16* dst_row = which ? dk_row : dv_row;
#pragma unroll
      for (int ch = 0; ch < DH / 32; ++ch) {
        uint32_t v[32];
        tmem_ld32_wait(tmem + lane_base + (which ? kColDK : kColDV) + half * DH + ch * 32, v);
        if (kv_valid && PSA_IN_BOUNDS((row * prm.Hkv + hk) * D + half * DH + ch * 32 + 31, int64_t(prm.T) * prm.Hkv * D,
                                      prm.status)) {
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
    }
  } else {
    // ------------------------------------------------------------ dQ drain: warps 12..15, one query row per thread
    setmaxnreg_inc<152>();
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;
    const uint32_t lane_base = uint32_t(quarter * 32) << 16;
    const bool leader = threadIdx.x == 384;
    const float sc = prm.scale;
    const uint32_t stage0 = base + L::kDQS;
    for (int it = 0; it < n_it; ++it) {
      const int q0 = (entry_of(it) >> 2) * kTile;
      const int h = head_of(it);
      mbar_wait(bar(B_DQ_FULL), it & 1, wctx);
      tc_fence_after();
      // Pull the whole row out of TMEM first and release the columns at once: the next dP^T
      // is waiting for them.  Staging and reducing then proceed from registers, at the pace
      // the reduce-adds are absorbed by L2.
      uint32_t v[D];
#pragma unroll
      for (int ch = 0; ch < D / 64; ++ch)
        tmem_ld64_wait(tmem + lane_base + kColDP + ch * 64, reinterpret_cast<uint32_t(&)[64]>(v[ch * 64]));
      tc_fence_before();
      mbar_arrive(bar(B_DQ_EMPTY));
#pragma unroll
      for (int ch = 0; ch < D / 32; ++ch) {
        const uint32_t stage = stage0 + (ch & 1) * L::kStageBytes;
        // The reduce issued two chunks ago read this staging buffer: wait until it has.
        if (leader) tma_wait_group_read<1>();
        named_bar_sync(2, 128);
        // Row r, 128 bytes, eight 16-byte chunks at index XOR (r & 7): the 128-byte swizzle the
        // tensor map of dq_accum expects.  Rows past the sample's end hold exact zeros (their dS
        // columns are masked), so adding them is harmless; rows past T are clipped by the TMA.
        const uint32_t row_addr = stage + r * 128;
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) {
          const uint32_t chunk = uint32_t(c4) ^ uint32_t(r & 7);
          st_shared_v4(row_addr + chunk * 16, __float_as_uint(__uint_as_float(v[ch * 32 + 4 * c4]) * sc),
                       __float_as_uint(__uint_as_float(v[ch * 32 + 4 * c4 + 1]) * sc),
                       __float_as_uint(__uint_as_float(v[ch * 32 + 4 * c4 + 2]) * sc),
                       __float_as_uint(__uint_as_float(v[ch * 32 + 4 * c4 + 3]) * sc));
        }
        fence_proxy_async_smem();
        named_bar_sync(2, 128);
        if (leader) {
          tma_reduce_add_3d(&tm_dq, stage, ch * 32, h, rec.ds + q0);
          tma_commit_group();
        }
      }
    }
    if (leader) tma_wait_group_read<0>();   // shared memory must outlive the last reduce's reads (the adds
                                            // themselves complete before the kernel does)
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, kBwdTmemCols);
  }
}

// delta[h][t] = sum_c dO[t,h,c] * O[t,h,c]; one 16-byte load per thread and tensor.  The kernel also
// clears the fp32 dq accumulator (same element mapping), which saves a separate pass over it.
template <int D>
__global__ void __launch_bounds__(256)
psa_bwd_delta_kernel(const __nv_bfloat16* __restrict__ d_o, const __nv_bfloat16* __restrict__ o,
                     float* __restrict__ delta, float* __restrict__ dq_accum, int64_t n_rows /* T*Hq */, int32_t T,
                     int32_t Hq, int32_t* status) {
  constexpr int kLanes = D / 8;  // threads per (t, h) row
  const int64_t gid = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t row = gid / kLanes;
  const int part = int(gid % kLanes);
  float acc = 0.f;
  if (row < n_rows) {
    const uint4 a = reinterpret_cast<const uint4*>(d_o + row * D)[part];
    const uint4 b = reinterpret_cast<const uint4*>(o + row * D)[part];
    // the same thread clears the eight accumulator elements that belong to its eight inputs
    float4* z = reinterpret_cast<float4*>(dq_accum + row * D + part * 8);
    z[0] = make_float4(0.f, 0.f, 0.f, 0.f);
    z[1] = make_float4(0.f, 0.f, 0.f, 0.f);
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
    if (PSA_IN_BOUNDS(int64_t(h) * T + t, int64_t(Hq) * T, status)) delta[int64_t(h) * T + t] = acc;
  }
}

// Exact delta for the rejected rows of short-prompt samples that see fewer than kFewKeys keys and
// lie outside their sample's first query tile (the main kernel recomputes delta of first-tile
// rows itself):  delta_i = sum_j P_ij dP_ij  over the row's visible keys, P_ij = exp(scale q_i.k_j
// - lse_i), dP_ij = dO_i.v_j, in fp32.  For such rows delta = dO.O taken from the bf16-rounded O is
// the largest error left in dQ and dK.  One warp per (row, query head), one key per lane.
template <int D>
__global__ void __launch_bounds__(128)
psa_bwd_delta_few_keys_kernel(const FewKeyRow* __restrict__ rows, const __nv_bfloat16* __restrict__ q,
                              const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
                              const __nv_bfloat16* __restrict__ d_o, const float* __restrict__ lse,
                              float* __restrict__ delta, int32_t T, int32_t Hq, int32_t Hkv, float scale_log2,
                              int32_t* status) {
  const FewKeyRow rec = rows[blockIdx.x];
  const int h = blockIdx.y * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (h >= Hq) return;
  const int hk = h / (Hq / Hkv);
  const int n_keys = rec.n_prompt + (rec.row - rec.rs_row + 1);   // < kFewKeys = 32
  float term = 0.f;
  const int64_t key = lane < rec.n_prompt ? rec.ds + lane : rec.rs_row + (lane - rec.n_prompt);
  if (lane < n_keys && PSA_IN_BOUNDS(key, T, status) && PSA_IN_BOUNDS(rec.row, T, status)) {
    const uint4* q4 = reinterpret_cast<const uint4*>(q + (int64_t(rec.row) * Hq + h) * D);
    const uint4* g4 = reinterpret_cast<const uint4*>(d_o + (int64_t(rec.row) * Hq + h) * D);
    const uint4* k4 = reinterpret_cast<const uint4*>(k + (key * Hkv + hk) * D);
    const uint4* v4 = reinterpret_cast<const uint4*>(v + (key * Hkv + hk) * D);
    float s = 0.f, dp = 0.f;
    auto dot8 = [](const uint4& a, const uint4& b, float acc) {
      const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        acc = fmaf(__uint_as_float(aw[i] << 16), __uint_as_float(bw[i] << 16), acc);
        acc = fmaf(__uint_as_float(aw[i] & 0xffff0000u), __uint_as_float(bw[i] & 0xffff0000u), acc);
      }
      return acc;
    };
#pragma unroll 4
    for (int c = 0; c < D / 8; ++c) {
      s = dot8(q4[c], k4[c], s);
      dp = dot8(g4[c], v4[c], dp);
    }
    term = ex2_approx(fmaf(s, scale_log2, -lse[int64_t(h) * T + rec.row] * kLog2e)) * dp;
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) term += __shfl_xor_sync(0xffffffffu, term, off);
  if (lane == 0 && PSA_IN_BOUNDS(rec.row, T, status)) delta[int64_t(h) * T + rec.row] = term;
}

// dq = bf16(dq_accum).  Four independent 16-byte loads in flight per thread and streaming (evict-first)
// accesses: the pass runs at the copy bandwidth (one load per thread left it 20 % short of it).
__global__ void __launch_bounds__(256)
psa_bwd_convert_kernel(const float4* __restrict__ acc, uint2* __restrict__ dq, int64_t n_vec4) {
  const int64_t base = (int64_t(blockIdx.x) * blockDim.x) * 4 + threadIdx.x;
  float4 a[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int64_t i = base + u * 256;
    if (i < n_vec4) a[u] = __ldcs(acc + i);
  }
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int64_t i = base + u * 256;
    if (i < n_vec4) {
      uint2 w;
      w.x = pack_bf16x2(a[u].x, a[u].y);
      w.y = pack_bf16x2(a[u].z, a[u].w);
      __stcs(dq + i, w);
    }
  }
}

template <int D>
psa_status_t launch_bwd_t(const psa_plan_t* plan, const void* d_o, const void* q, const void* k, const void* v,
                          const void* o, const float* lse, void* dq, void* dk, void* dv, void* workspace,
                          bool f32_out, int32_t* device_status, cudaStream_t stream) {
  using L = BwdSmem<D>;
  const int64_t T = plan->T;
  const BwdWorkspace ws = bwd_workspace_layout(T, plan->Hq, D);
  char* wsp = static_cast<char*>(workspace);
  // With fp32 outputs the caller's dq is the accumulator itself and nothing is converted.
  float* dq_accum = f32_out ? static_cast<float*>(dq) : reinterpret_cast<float*>(wsp + ws.dq_accum_off);
  float* delta = reinterpret_cast<float*>(wsp + ws.delta_off);

  CUtensorMap tm_q, tm_k, tm_v, tm_do, tm_dq, tm_dk, tm_dv;
  if (!make_tile_map_bf16(&tm_q, q, T, plan->Hq, D) || !make_tile_map_bf16(&tm_k, k, T, plan->Hkv, D) ||
      !make_tile_map_bf16(&tm_v, v, T, plan->Hkv, D) || !make_tile_map_bf16(&tm_do, d_o, T, plan->Hq, D) ||
      !make_tile_map(&tm_dq, dq_accum, T, plan->Hq, D, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, 32, 128) ||
      // (with fp32 outputs dk and dv leave through per-thread stores; their maps are built but not used)
      !make_tile_map_bf16(&tm_dk, dk, T, plan->Hkv, D) || !make_tile_map_bf16(&tm_dv, dv, T, plan->Hkv, D))
    return PSA_ERR_CUDA;
  if (cudaFuncSetAttribute(psa_bwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kRequest) != cudaSuccess)
    return PSA_ERR_CUDA;

  const int64_t n_rows = T * plan->Hq;
  {
    ProfileScope prof(3, stream);
    const int64_t threads = n_rows * (D / 8);
    psa_bwd_delta_kernel<D><<<unsigned((threads + 255) / 256), 256, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(d_o), static_cast<const __nv_bfloat16*>(o), delta, dq_accum, n_rows, plan->T,
        plan->Hq, device_status);
  }
  if (!plan->few_key_rows.empty())
    psa_bwd_delta_few_keys_kernel<D><<<dim3(unsigned(plan->few_key_rows.size()), unsigned((plan->Hq + 3) / 4)), 128, 0, stream>>>(
        plan->d_few_key_rows, static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k),
        static_cast<const __nv_bfloat16*>(v), static_cast<const __nv_bfloat16*>(d_o), lse, delta, plan->T, plan->Hq,
        plan->Hkv, plan->scale * kLog2e, device_status);
  BwdParams prm;
  prm.tiles = plan->d_kv_tiles;
  prm.entries = plan->d_bwd_entries;
  prm.cta_map = plan->d_bwd_cta_map;
  prm.lse = lse;
  prm.delta = delta;
  prm.dq_accum = dq_accum;
  prm.dk = dk;
  prm.dv = dv;
  prm.f32_out = f32_out ? 1 : 0;
  prm.status = device_status;
  prm.T = plan->T;
  prm.Hq = plan->Hq;
  prm.Hkv = plan->Hkv;
  prm.scale = plan->scale;
  prm.scale_log2 = plan->scale * kLog2e;
  const unsigned grid = unsigned(plan->kv_tiles.size()) * unsigned(plan->Hkv);
  {
    ProfileScope prof(1, stream);
    psa_bwd_kernel<D><<<grid, kBwdThreads, L::kRequest, stream>>>(tm_q, tm_k, tm_v, tm_do, tm_dq, tm_dk, tm_dv, prm);
  }
  if (!f32_out) {
    ProfileScope prof(4, stream);
    const int64_t n_vec4 = n_rows * D / 4;
    psa_bwd_convert_kernel<<<unsigned((n_vec4 + 1023) / 1024), 256, 0, stream>>>(
        reinterpret_cast<const float4*>(dq_accum), static_cast<uint2*>(dq), n_vec4);
  }
  return check_last_cuda_error("psa_bwd launch");
}

}  // namespace

psa_status_t launch_bwd(const psa_plan_t* plan, const void* d_o, const void* q, const void* k, const void* v,
                        const void* o, const float* lse, void* dq, void* dk, void* dv, void* workspace,
                        bool f32_out, int32_t* device_status, void* stream) {
  if (plan->d == 128)
    return launch_bwd_t<128>(plan, d_o, q, k, v, o, lse, dq, dk, dv, workspace, f32_out, device_status,
                             cudaStream_t(stream));
  return launch_bwd_t<64>(plan, d_o, q, k, v, o, lse, dq, dk, dv, workspace, f32_out, device_status,
                          cudaStream_t(stream));
}

}  // namespace psa

