// psa_fwd: attention forward under the prefix-sharing mask with packing
// (Algorithm 3; Section 3.1), one CTA per (query tile, query head).
//
// Warp roles (384 threads = 3 warpgroups):
//   warp 0       TMA producer: Q once, then K_j and V_j of every live key tile
//   warp 1       UMMA issuer:  S = Q K_j^T  and  O += P V_j  (tcgen05, accumulators in TMEM)
//   warps 2, 3   idle (they complete the first warpgroup, which gives its registers away)
//   warps 4..11  softmax: two threads per query row, one for each half of the 128 key columns.
//                S is read from TMEM, masked in registers when the tile is PARTIAL, turned into
//                P = exp2(S*c - m*c) in fp32 and written back to TMEM as bf16 (over the thread's
//                own S columns) for the second UMMA.  The two halves of a row exchange their
//                maxima through shared memory.
// A CTA takes two work items (query tile, query head), one after the other: items 2 b and 2 b + 1 of the list
// (longest first; usually the same query tile and two heads of one kv head).  Barrier parities run on over both
// items; the second item's Q and first K tile are requested as soon as the first item's last score product has
// read them, i.e. they arrive while the first item's last softmax, P V and output store are still going on, and
// the barrier initialisation, the TMEM allocation and the exit are paid once for two items.
// Two CTAs share an SM (100 KB of shared memory and 256 TMEM columns each for head_dim 128), so
// one CTA's softmax overlaps the other's UMMAs, and with eight softmax warps per CTA every SM
// sub-partition has two warps feeding its exponential unit even when only one CTA is in that phase.
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

constexpr int kFwdThreads = 384;
constexpr int kSoftmaxThreads = 256;
// Register split of the 80 per thread the launch bound allows: the first warpgroup (producer,
// issuer) gives registers to the two softmax warpgroups.
constexpr int kRegsWg0 = 32, kRegsSoftmax = 104;
constexpr uint32_t kTmemCols = 256;   // S: columns [0,128), O: columns [128, 128+D)
constexpr uint32_t kColS = 0, kColO = 128;

struct FwdParams {
  const TileRec* tiles;
  const int32_t* entries;
  __nv_bfloat16* o;
  float* lse;
  int32_t* status;
  int32_t T, Hq, Hkv;
  int32_t n_items;   // query tiles x query heads
  float scale_log2;  // softmax_scale * log2(e)
};

// What a role needs to know about one work item; both items of the CTA are kept in shared memory.
struct FwdItem {
  TileRec rec;
  int32_t h, hk, n_it, pad;
};
static_assert(sizeof(FwdItem) == 48, "FwdItem is 12 int32");

template <int D>
struct FwdSmem {
  static constexpr int kSub = D / 64;                 // 64-column (128-byte) sub-tiles per row
  static constexpr int kTileBytes = kTile * D * 2;    // one Q / K / V tile
  static constexpr int kSubBytes = kTile * 128;       // one sub-tile: 128 rows x 128 bytes
  static constexpr int kQ = 0, kK = kTileBytes, kV = 2 * kTileBytes;
  static constexpr int kBars = 3 * kTileBytes;        // 9 mbarriers
  static constexpr int kTmemSlot = kBars + 72;
  static constexpr int kAbort = kTmemSlot + 4;
  static constexpr int kItems = kBars + 128;          // FwdItem [2]
  static constexpr int kEnt = kItems + 128;           // first kEntCap entries of each item's list
  static constexpr int kEntCap = 128;
  static constexpr int kXchg = kEnt + 2 * kEntCap * 4;  // float [2 parities][2 halves][128 rows]
  static constexpr int kBytes = kXchg + 2 * 2 * kTile * 4;
  // Request enough that at most two CTAs fit on an SM: their TMEM allocations
  // (256 columns each) then always succeed without waiting.
  static constexpr int kRequest = (kBytes + 1024 > 100 * 1024) ? kBytes + 1024 : 100 * 1024;
};

enum { BAR_Q_FULL = 0, BAR_K_FULL, BAR_V_FULL, BAR_K_EMPTY, BAR_V_EMPTY, BAR_S_FULL, BAR_P_FULL, BAR_O_FULL,
       BAR_STAGE_FREE };   // the output staging (the V buffer) of the first item has been read by its TMA stores

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 2)
psa_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
               const FwdParams prm) {
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
  // The CTA's work items: 2 b and 2 b + 1 of the list (longest first, so the CTAs stay sorted by length and the
  // short ones still fill the tail of the launch); the last CTA of an odd count has one item.
  const int idx0 = 2 * int(blockIdx.x), idx1 = idx0 + 1;
  const int n_items = idx1 < prm.n_items ? 2 : 1;
  FwdItem* s_item = reinterpret_cast<FwdItem*>(gen_base + L::kItems);
  int32_t* s_ent_all = reinterpret_cast<int32_t*>(gen_base + L::kEnt);
  const WaitCtx wctx{abort_flag, prm.status, kWaitLimitClocks};
  // Every role reads the list entry of every iteration: the head of each item's list is kept in shared memory.
  struct ItemView {
    TileRec rec;
    int h, hk, n_it;
    const int32_t* ent_g;
    const int32_t* s_ent;
    __device__ __forceinline__ int ent(int it) const { return it < L::kEntCap ? s_ent[it] : ent_g[it]; }
  };
  auto view = [&](int item) {
    const FwdItem im = s_item[item];
    return ItemView{im.rec, im.h, im.hk, im.n_it, prm.entries + im.rec.list_off, s_ent_all + item * L::kEntCap};
  };

  if (threadIdx.x == 32 && n_items == 2) {   // the second item's record, while thread 0 requests the first tiles
    const int h1 = idx1 % prm.Hq;
    const TileRec r1 = prm.tiles[idx1 / prm.Hq];
    s_item[1] = FwdItem{r1, h1, h1 / (prm.Hq / prm.Hkv), r1.list_cnt, 0};
  }
  if (threadIdx.x >= 128 && threadIdx.x < 128 + L::kEntCap && n_items == 2) {
    const TileRec r1 = prm.tiles[idx1 / prm.Hq];
    const int i = int(threadIdx.x) - 128;
    if (i < r1.list_cnt) s_ent_all[L::kEntCap + i] = prm.entries[r1.list_off + i];
  }
  const int h = idx0 % prm.Hq;
  const int hk = h / (prm.Hq / prm.Hkv);
  const TileRec rec = prm.tiles[idx0 / prm.Hq];
  const int32_t* ent_g = prm.entries + rec.list_off;
  const int n_it = rec.list_cnt;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    s_item[0] = FwdItem{rec, h, hk, n_it, 0};
    mbar_init(bar(BAR_STAGE_FREE), 1);
    mbar_init(bar(BAR_Q_FULL), 1);
    mbar_init(bar(BAR_K_FULL), 1);
    mbar_init(bar(BAR_V_FULL), 1);
    mbar_init(bar(BAR_K_EMPTY), 1);
    mbar_init(bar(BAR_V_EMPTY), 1);
    mbar_init(bar(BAR_S_FULL), 1);
    mbar_init(bar(BAR_P_FULL), kSoftmaxThreads);
    mbar_init(bar(BAR_O_FULL), 1);
    fence_mbar_init();
    // Q and the first K, V tiles are requested right away: their flight overlaps the TMEM
    // allocation and the CTA-wide barrier below.  (This thread is also the producer.)
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    mbar_expect_tx(bar(BAR_Q_FULL), L::kTileBytes);
    for (int s = 0; s < L::kSub; ++s) tma_load_3d(sQ + s * L::kSubBytes, &tm_q, s * 64, h, rec.row0, bar(BAR_Q_FULL));
    if (n_it > 0) {
      const int krow = rec.ds + (ent_g[0] >> 2) * kTile;
      mbar_expect_tx(bar(BAR_K_FULL), L::kTileBytes);
      for (int s = 0; s < L::kSub; ++s) tma_load_3d(sK + s * L::kSubBytes, &tm_k, s * 64, hk, krow, bar(BAR_K_FULL));
      mbar_expect_tx(bar(BAR_V_FULL), L::kTileBytes);
      for (int s = 0; s < L::kSub; ++s) tma_load_3d(sV + s * L::kSubBytes, &tm_v, s * 64, hk, krow, bar(BAR_V_FULL));
    }
    tma_prefetch_desc(&tm_o);
  }
  if (int(threadIdx.x) < n_it && int(threadIdx.x) < L::kEntCap) s_ent_all[threadIdx.x] = ent_g[threadIdx.x];
  if (warp == 0) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp < 4) {
   setmaxnreg_dec<kRegsWg0>();
   if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int g = 0;   // iteration count over both items: the parity of every per-iteration barrier
      for (int item = 0; item < n_items; ++item) {
        const ItemView w = view(item);
        for (int it = 0; it < w.n_it; ++it, ++g) {
          if (g == 0) continue;   // requested before the CTA-wide barrier
          const int krow = w.rec.ds + (w.ent(it) >> 2) * kTile;
          mbar_wait(bar(BAR_K_EMPTY), (g - 1) & 1, wctx);
          if (it == 0) {
            // First tile of the second item.  The first item's last score product has completed, so
            // its Q is no longer needed either.
            mbar_expect_tx(bar(BAR_Q_FULL), L::kTileBytes);
            for (int s = 0; s < L::kSub; ++s) tma_load_3d(sQ + s * L::kSubBytes, &tm_q, s * 64, w.h, w.rec.row0, bar(BAR_Q_FULL));
          }
          mbar_expect_tx(bar(BAR_K_FULL), L::kTileBytes);
          for (int s = 0; s < L::kSub; ++s) tma_load_3d(sK + s * L::kSubBytes, &tm_k, s * 64, w.hk, krow, bar(BAR_K_FULL));
          mbar_wait(bar(BAR_V_EMPTY), (g - 1) & 1, wctx);
          // The first item's output leaves through the V buffer: its TMA stores must have read it.
          if (it == 0) mbar_wait(bar(BAR_STAGE_FREE), 0, wctx);
          mbar_expect_tx(bar(BAR_V_FULL), L::kTileBytes);
          for (int s = 0; s < L::kSub; ++s) tma_load_3d(sV + s * L::kSubBytes, &tm_v, s * 64, w.hk, krow, bar(BAR_V_FULL));
        }
      }
    }
    __syncwarp();
   } else if (warp == 1) {
    // ------------------------------------------------------------ UMMA issuer
    // The whole warp runs this loop with warp-uniform operands; one elected lane issues.
    {
      const uint32_t issuer = elect_one();
      constexpr uint32_t idesc_s = umma_idesc_bf16(kTile, kTile, false, false);  // Q, K both K-major
      constexpr uint32_t idesc_o = umma_idesc_bf16(kTile, D, false, true);       // P (TMEM), V MN-major
      // Low descriptor words (start address + LBO); the high word is a constant.
      const uint32_t q_k = smem_desc_lo(sQ, 16), k_k = smem_desc_lo(sK, 16), v_mn = smem_desc_lo(sV, L::kSubBytes);
      int g = 0;   // iteration count over both items
      for (int item = 0; item < n_items; ++item) {
      const ItemView w = view(item);
      mbar_wait(bar(BAR_Q_FULL), item & 1, wctx);
      for (int it = 0; it < w.n_it; ++it, ++g) {
        mbar_wait(bar(BAR_K_FULL), g & 1, wctx);
        // The S columns are also where P_{it-1} lives.  UMMAs issued by one thread execute in
        // issue order, so this S = Q K^T cannot overwrite P before the previous P V has read it.
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = ((kk >> 2) * L::kSubBytes + (kk & 3) * 32) >> 4;
          umma_ss_w(tmem + kColS, q_k + off, k_k + off, idesc_s, kk > 0, issuer);
        }
        umma_commit_w(bar(BAR_K_EMPTY), issuer);
        umma_commit_w(bar(BAR_S_FULL), issuer);
        mbar_wait(bar(BAR_V_FULL), g & 1, wctx);
        mbar_wait(bar(BAR_P_FULL), g & 1, wctx);
        tc_fence_after();
        // P of key half hf lies in columns [64 hf, 64 hf + 32) of the S region (two bf16 per column);
        // PRECISE tiles carry a second bf16 term in columns [64 hf + 32, 64 hf + 64).
        const int n_terms = (w.ent(it) & 2) ? 2 : 1;
        for (int term = 0; term < n_terms; ++term) {
#pragma unroll
          for (int kk = 0; kk < kTile / 16; ++kk) {
            // A: 16 keys of P = 8 TMEM columns (two bf16 per column).  B: 16 key rows of V.
            umma_ts_w(tmem + kColO, tmem + kColS + (kk >> 2) * 64 + term * 32 + (kk & 3) * 8, v_mn + kk * (2048 >> 4), idesc_o,
                       (it > 0) || (kk > 0) || (term > 0), issuer);
          }
        }
        umma_commit_w(bar(BAR_V_EMPTY), issuer);
        umma_commit_w(bar(BAR_O_FULL), issuer);
      }
      }
    }
    __syncwarp();
   }
  } else {
    // ------------------------------------------------------------ softmax, two threads per row
    setmaxnreg_inc<kRegsSoftmax>();
    const int quarter = warp & 3;                 // TMEM lanes this warp may touch
    const int hfz = (warp - 4) >> 2;              // which half of the key columns this thread owns
    const int r = quarter * 32 + lane;            // row within the tile
    const uint32_t lane_base = uint32_t(quarter * 32) << 16;
    const uint32_t col_s = kColS + 64u * hfz;     // this thread's 64 S columns; its P goes over them
    const float c = prm.scale_log2;
    float* xchg = reinterpret_cast<float*>(gen_base + L::kXchg);
    // Barrier of the two warps that share a row quarter (ids 1..4, immediate so that the kernel
    // is known to use five barriers, not all sixteen).
    auto pair_sync = [&]() {
      switch (quarter) {
        case 0: asm volatile("bar.sync 1, 64;" ::: "memory"); break;
        case 1: asm volatile("bar.sync 2, 64;" ::: "memory"); break;
        case 2: asm volatile("bar.sync 3, 64;" ::: "memory"); break;
        default: asm volatile("bar.sync 4, 64;" ::: "memory"); break;
      }
    };

    int gbase = 0;       // iterations of the items before this one: barrier parities run on over both items
    uint32_t xs = 0;     // uses of the exchange slots so far (they alternate with every use)
    for (int item = 0; item < n_items; ++item) {
    const ItemView w = view(item);
    const TileRec& rec = w.rec;
    const int h = w.h, n_it = w.n_it;
    const int q_local = rec.local0 + r;
    const bool row_valid = q_local < rec.len;
    float m_run = -INFINITY, l_run = 0.f;         // l_run: this thread's half of the row sum
    for (int it = 0; it < n_it; ++it, ++xs) {
      const int g = gbase + it;
      const int e = w.ent(it);
      const int k0 = (e >> 2) * kTile;
      const bool precise = (e & 2) != 0;
      mbar_wait(bar(BAR_S_FULL), g & 1, wctx);
      tc_fence_after();
      // Allowed keys of this row in a PARTIAL tile, relative to the tile: [0, a) and [b, b + span).
      int a = kTile, b = 0;
      uint32_t span = 0;
      if (e & 1) {
        if (q_local < rec.rs) { a = q_local + 1 - k0; }
        else { a = rec.cs - k0; b = rec.rs - k0; span = uint32_t(q_local + 1 - rec.rs); }
      }
      // Warp-uniform class of this warp's two 32-column chunks: 0 = every lane allows every column
      // (no masking), 1 = mixed (mask per element), 2 = no lane allows any column (skipped: no load,
      // no exponential).  On a causal diagonal tile this skips 3/8 of the exponentials.
      uint32_t cls = 0;
      if (e & 1) {
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
          const int lo = hfz * 64 + sub * 32, hi = lo + 32;
          const bool all_ok = (hi <= a) || (lo >= b && uint32_t(hi - b) <= span);
          const bool none_ok = (lo >= a) && (span == 0u || hi <= b || (lo >= b && uint32_t(lo - b) >= span));
          const uint32_t cc = __all_sync(0xffffffffu, all_ok) ? 0u : (__all_sync(0xffffffffu, none_ok) ? 2u : 1u);
          cls |= cc << (2 * sub);
        }
      }
      auto chunk_class = [&](int sub) { return (cls >> (2 * sub)) & 3u; };
      // The thread's scores are read from TMEM twice, 32 at a time (first for the row maximum,
      // then for the exponentials), which keeps the live registers small.
      auto load_chunk = [&](int sub, float (&x)[32]) {
        uint32_t v[32];
        tmem_ld32_wait(tmem + lane_base + col_s + sub * 32, v);
        if (chunk_class(sub) == 1u) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int col = hfz * 64 + sub * 32 + i;
            const bool ok = (col < a) || (uint32_t(col - b) < span);
            x[i] = ok ? __uint_as_float(v[i]) : -INFINITY;
          }
        } else {   // class 0; callers never use the values of a class-2 chunk
#pragma unroll
          for (int i = 0; i < 32; ++i) x[i] = __uint_as_float(v[i]);
        }
      };
      // Fast path (every tile but the first of a list and the PRECISE ones): one pass.  The
      // exponentials are taken against the running maximum; P stays in registers until the two
      // threads of the row have agreed that the running maximum still holds (it nearly always
      // does, see the 2^8 rule below).  If it does not, nothing has been written yet and the
      // two-pass path below redoes the tile.
      bool fast_done = false;
      if (it == 0 && !precise && cls == 0u) {
        // First tile of a list, nothing masked: there is no accumulator to rescale yet, so the
        // scores can stay in registers across the exchange of the maxima (one load instead of three).
        uint32_t v[64];
        tmem_ld64_wait(tmem + lane_base + col_s, v);
        float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < 64; i += 8) {
          m4[0] = max3(m4[0], __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
          m4[1] = max3(m4[1], __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
          m4[2] = max3(m4[2], __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
          m4[3] = max3(m4[3], __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
        }
        float mxf = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        {
          float* slot = xchg + (xs & 1) * 2 * kTile;
          slot[hfz * kTile + r] = mxf;
          pair_sync();
          mxf = fmaxf(mxf, slot[(hfz ^ 1) * kTile + r]);
        }
        m_run = mxf;
        const float mc0 = (m_run == -INFINITY) ? 0.f : m_run * c;
        const uint64_t c2 = pack_f32x2(c, c), mc2 = pack_f32x2(-mc0, -mc0);
        uint64_t sum2[2] = {0ull, 0ull};
        uint32_t pk[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float t0, t1;
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1])), c2, mc2), t0, t1);
          const float p0 = ex2_approx(t0), p1 = ex2_approx(t1);
          sum2[i & 1] = add_f32x2(sum2[i & 1], pack_f32x2(p0, p1));
          pk[i] = pack_bf16x2(p0, p1);
        }
        tmem_st32(tmem + lane_base + col_s, pk);
        float a0, a1, b0, b1;
        unpack_f32x2(sum2[0], a0, a1);
        unpack_f32x2(sum2[1], b0, b1);
        l_run = (a0 + a1) + (b0 + b1);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar(BAR_P_FULL));
        continue;
      }
      if (it > 0 && !precise) {
        uint32_t pk[32];
        uint64_t sum2[2] = {0ull, 0ull};
        const float mc0 = (m_run == -INFINITY) ? 0.f : m_run * c;
        const uint64_t c2 = pack_f32x2(c, c), mc2 = pack_f32x2(-mc0, -mc0);
        if (cls == 0u) {
          // Nothing masked (every FULL tile): all 64 columns with one load and one wait.  Every
          // wait exposes the TMEM latency, which the two warps per sub-partition do not hide.
          uint32_t v[64];
          tmem_ld64_wait(tmem + lane_base + col_s, v);
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            float t0, t1;
            unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1])), c2, mc2), t0, t1);
            const float p0 = ex2_approx(t0), p1 = ex2_approx(t1);
            sum2[i & 1] = add_f32x2(sum2[i & 1], pack_f32x2(p0, p1));
            pk[i] = pack_bf16x2(p0, p1);
          }
        } else
        // PARTIAL tiles, 16 columns at a time: P of the whole tile (32 registers) stays live next to them
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          const uint32_t cc = chunk_class(ch >> 1);
          if (cc == 2u) {
#pragma unroll
            for (int i = 0; i < 8; ++i) pk[8 * ch + i] = 0u;
            continue;
          }
          uint32_t v[16];
          tmem_ld16_wait(tmem + lane_base + col_s + ch * 16, v);
          float x[16];
          if (cc == 1u) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const int col = hfz * 64 + ch * 16 + i;
              const bool ok = (col < a) || (uint32_t(col - b) < span);
              x[i] = ok ? __uint_as_float(v[i]) : -INFINITY;
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) x[i] = __uint_as_float(v[i]);
          }
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float t0, t1;
            unpack_f32x2(fma_f32x2(pack_f32x2(x[2 * i], x[2 * i + 1]), c2, mc2), t0, t1);
            const float p0 = ex2_approx(t0), p1 = ex2_approx(t1);
            sum2[i & 1] = add_f32x2(sum2[i & 1], pack_f32x2(p0, p1));
            pk[8 * ch + i] = pack_bf16x2(p0, p1);
          }
        }
        // The running maximum still holds if no probability of the tile exceeds 2^8 against it.  The
        // row sum, which is needed anyway, bounds them all: above 256 (or not a number) the tile goes to
        // the two-pass path.  So does every tile of a row whose running maximum is still -inf, unless the
        // whole tile is masked for the warp: exponentials taken against "no maximum yet" may all have
        // underflowed to 0, which a row sum cannot tell from "nothing to add".
        float a0, a1, b0, b1;
        unpack_f32x2(sum2[0], a0, a1);
        unpack_f32x2(sum2[1], b0, b1);
        const float sumf = (a0 + a1) + (b0 + b1);
        bool redo = !(sumf <= 256.f) || (m_run == -INFINITY && cls != 0xAu);
        {
          // both threads of a row must take the same path
          float* slot = xchg + (xs & 1) * 2 * kTile;
          slot[hfz * kTile + r] = redo ? 1.f : 0.f;
          pair_sync();
          redo = redo || slot[(hfz ^ 1) * kTile + r] != 0.f;
        }
        if (!__any_sync(0xffffffffu, redo)) {
          // the 16 values of chunk ch go to columns [8 ch, 8 ch + 8) of the thread's own 64
          tmem_st32(tmem + lane_base + col_s, pk);
          l_run += sumf;
          tc_wait_st();
          tc_fence_before();
          mbar_arrive(bar(BAR_P_FULL));
          fast_done = true;
        }
      }
      if (fast_done) continue;
      float mx;
      {
        float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four independent chains
        if (cls == 0u) {
          // nothing masked (every FULL tile): both chunks with one wait
          uint32_t v[64];
          tmem_ld64_wait(tmem + lane_base + col_s, v);
#pragma unroll
          for (int i = 0; i < 64; i += 8) {
            m4[0] = max3(m4[0], __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
            m4[1] = max3(m4[1], __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
            m4[2] = max3(m4[2], __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
            m4[3] = max3(m4[3], __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
          }
        } else
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
          if (chunk_class(sub) == 2u) continue;
          float x[32];
          load_chunk(sub, x);
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            m4[0] = max3(m4[0], x[i], x[i + 1]);
            m4[1] = max3(m4[1], x[i + 2], x[i + 3]);
            m4[2] = max3(m4[2], x[i + 4], x[i + 5]);
            m4[3] = max3(m4[3], x[i + 6], x[i + 7]);
          }
        }
        mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
      }
      // Row maximum over both halves: the two threads of a row trade maxima through shared memory
      // (slots alternate with the iteration parity, so a slot is rewritten only after the partner
      // has passed the next barrier, hence read it).
      {
        float* slot = xchg + (xs & 1) * 2 * kTile;
        slot[hfz * kTile + r] = mx;
        pair_sync();
        mx = fmaxf(mx, slot[(hfz ^ 1) * kTile + r]);
      }
      const float m_new = fmaxf(m_run, mx);
      // Keep a stale maximum while it is within 2^8 of the true one: P stays <= 256
      // and the accumulator needs no rescaling.  (-inf) - (-inf) is NaN -> false.
      // Both threads of a row see the same maxima, hence take the same decision.
      const bool grow = (m_new - m_run) * c > 8.0f;
      float alpha = 1.f;
      if (grow) {
        alpha = ex2_approx((m_run - m_new) * c);   // m_run = -inf -> 0
        m_run = m_new;
        l_run *= alpha;
      }
      if (it > 0 && __any_sync(0xffffffffu, grow)) {
        mbar_wait(bar(BAR_O_FULL), (g - 1) & 1, wctx);
        tc_fence_after();
        // Each thread rescales its half of the accumulator's columns.
#pragma unroll
        for (int ch = 0; ch < D / 64; ++ch) {
          uint32_t v[32];
          const uint32_t col = kColO + hfz * (D / 2) + ch * 32;
          tmem_ld32_wait(tmem + lane_base + col, v);
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
          tmem_st32(tmem + lane_base + col, v);
        }
      }
      const float mc = (m_run == -INFINITY) ? 0.f : m_run * c;
      float s4[4] = {0.f, 0.f, 0.f, 0.f};
      uint64_t sum2[2] = {0ull, 0ull};                 // two packed pairs of partial row sums
      const uint64_t c2 = pack_f32x2(c, c), mc2 = pack_f32x2(-mc, -mc);
      if (!precise) {
        // P -> bf16 over the thread's own S columns: the 32 values of chunk sub go to columns
        // [16 sub, 16 sub + 16) of them, which never reaches a column that is still to be read.
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
          uint32_t v[16];
          if (chunk_class(sub) == 2u) {
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = 0u;
          } else {
            float x[32];
            load_chunk(sub, x);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              // two scores per instruction for the scale-and-shift and for the row sum
              float t0, t1;
              unpack_f32x2(fma_f32x2(pack_f32x2(x[2 * i], x[2 * i + 1]), c2, mc2), t0, t1);
              const float p0 = ex2_approx(t0), p1 = ex2_approx(t1);
              sum2[i & 1] = add_f32x2(sum2[i & 1], pack_f32x2(p0, p1));
              v[i] = pack_bf16x2(p0, p1);
            }
          }
          tmem_st16(tmem + lane_base + col_s + sub * 16, v);
        }
      } else {
        // PRECISE tiles also store the rounding residual as a second bf16 term in columns
        // [32,64) of the thread's own: all 64 scores are taken into registers before anything
        // is written.
        float x0[32], x1[32];
        load_chunk(0, x0);
        load_chunk(1, x1);
        if (chunk_class(0) == 2u) {
#pragma unroll
          for (int i = 0; i < 32; ++i) x0[i] = -INFINITY;
        }
        if (chunk_class(1) == 2u) {
#pragma unroll
          for (int i = 0; i < 32; ++i) x1[i] = -INFINITY;
        }
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
          uint32_t v[16], vr[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float p0 = ex2_approx(fmaf(sub ? x1[2 * i] : x0[2 * i], c, -mc));
            const float p1 = ex2_approx(fmaf(sub ? x1[2 * i + 1] : x0[2 * i + 1], c, -mc));
            s4[i & 1] += p0;
            s4[2 + (i & 1)] += p1;
            v[i] = pack_bf16x2(p0, p1);
            vr[i] = pack_bf16x2_residual(p0, p1, v[i]);
          }
          tmem_st16(tmem + lane_base + col_s + sub * 16, v);
          tmem_st16(tmem + lane_base + col_s + 32 + sub * 16, vr);
        }
      }
      {
        float a0, a1, b0, b1;
        unpack_f32x2(sum2[0], a0, a1);
        unpack_f32x2(sum2[1], b0, b1);
        s4[0] += a0 + a1;
        s4[2] += b0 + b1;
      }
      const float sum = (s4[0] + s4[1]) + (s4[2] + s4[3]);
      l_run += sum;
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar(BAR_P_FULL));
    }

    // ---- epilogue: O / l -> bf16, lse.  The two halves of the row sum meet in shared memory.
    {
      float* slot = xchg + (xs & 1) * 2 * kTile;
      ++xs;
      slot[hfz * kTile + r] = l_run;
      pair_sync();
      l_run += slot[(hfz ^ 1) * kTile + r];
    }
    if (n_it > 0) {
      mbar_wait(bar(BAR_O_FULL), (gbase + n_it - 1) & 1, wctx);
      tc_fence_after();
    }
    const float inv_l = 1.f / l_run;
    const int64_t row = int64_t(rec.row0) + r;
    __nv_bfloat16* orow = prm.o + (row * prm.Hq + h) * D + hfz * (D / 2);
    // A full tile leaves through shared memory (the V buffer is free now) in the 128-byte-swizzled
    // layout of the tensor map and one TMA store per 64-column sub-tile writes it out coalesced.
    // (A ragged last tile must not touch the rows of the next sample, which the box would cover:
    // it takes the per-thread stores.)
    const bool full_tile = rec.len - rec.local0 >= kTile;
#pragma unroll
    for (int ch = 0; ch < D / 64; ++ch) {
      uint32_t v[32];
      tmem_ld32_wait(tmem + lane_base + kColO + hfz * (D / 2) + ch * 32, v);
      if (full_tile) {
        const int col0 = hfz * (D / 2) + ch * 32;
        const uint32_t row_addr = sV + (col0 >> 6) * L::kSubBytes + r * 128;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t chunk = uint32_t(((col0 & 63) >> 3) + i) ^ uint32_t(r & 7);
          st_shared_v4(row_addr + chunk * 16,
                       pack_bf16x2(__uint_as_float(v[8 * i + 0]) * inv_l, __uint_as_float(v[8 * i + 1]) * inv_l),
                       pack_bf16x2(__uint_as_float(v[8 * i + 2]) * inv_l, __uint_as_float(v[8 * i + 3]) * inv_l),
                       pack_bf16x2(__uint_as_float(v[8 * i + 4]) * inv_l, __uint_as_float(v[8 * i + 5]) * inv_l),
                       pack_bf16x2(__uint_as_float(v[8 * i + 6]) * inv_l, __uint_as_float(v[8 * i + 7]) * inv_l));
        }
      } else if (row_valid && PSA_IN_BOUNDS((row * prm.Hq + h) * D + hfz * (D / 2) + ch * 32 + 31,
                                             int64_t(prm.T) * prm.Hq * D, prm.status)) {
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
    if (row_valid && hfz == 0 && PSA_IN_BOUNDS(int64_t(h) * prm.T + row, int64_t(prm.Hq) * prm.T, prm.status)) {
      const float mc = (m_run == -INFINITY) ? 0.f : m_run * c;
      prm.lse[int64_t(h) * prm.T + row] = (mc + log2f(l_run)) * 0.6931471805599453f;
    }
    if (full_tile) {
      fence_proxy_async_smem();
      asm volatile("bar.sync 5, 256;" ::: "memory");   // the eight softmax warps
      if (threadIdx.x == 128) {
        for (int s = 0; s < L::kSub; ++s) tma_store_3d(&tm_o, sV + s * L::kSubBytes, s * 64, h, rec.row0);
        tma_commit_group();
        tma_wait_group_read<0>();   // shared memory must outlive the stores' reads
      }
    }
    // The V buffer may be refilled (by the next item's first V tile) once the stores have read it.
    if (threadIdx.x == 128 && item == 0) mbar_arrive(bar(BAR_STAGE_FREE));
    gbase += n_it;
    }   // items
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
  CUtensorMap tm_q, tm_k, tm_v, tm_o;
  if (!make_tile_map_bf16(&tm_q, q, plan->T, plan->Hq, D) || !make_tile_map_bf16(&tm_k, k, plan->T, plan->Hkv, D) ||
      !make_tile_map_bf16(&tm_v, v, plan->T, plan->Hkv, D) || !make_tile_map_bf16(&tm_o, o, plan->T, plan->Hq, D))
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
  prm.n_items = int32_t(plan->q_tiles.size()) * plan->Hq;
  prm.scale_log2 = plan->scale * 1.4426950408889634f;
  const unsigned grid = unsigned(prm.n_items + 1) / 2u;   // two work items per CTA
  {
    ProfileScope prof(0, stream);
    psa_fwd_kernel<D><<<grid, kFwdThreads, L::kRequest, stream>>>(tm_q, tm_k, tm_v, tm_o, prm);
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

