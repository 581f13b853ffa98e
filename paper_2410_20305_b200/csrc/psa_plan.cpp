// Host planner: block-sparsity tile map of the prefix-sharing mask with packing
// (Algorithm 3), built once per step and reused by every layer (Section 3.1).
//
// Tiles are 128 x 128 and aligned to each sample's first token, so that within a
// sample query tile i and key tile j cover local rows [128 i, 128 i + 128) and
// [128 j, 128 j + 128).  In local coordinates (cs = P, rs = P + C, len = P+C+R)
// the mask is:  kv <= q  and not (q >= rs and cs <= kv < rs).
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <numeric>
#include <queue>
#include <utility>
#include <vector>

#include "psa_internal.h"

namespace psa {

BwdWorkspace bwd_workspace_layout(int64_t T, int Hq, int d) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  BwdWorkspace w{};
  int64_t Tpad = (T + kTile - 1) / kTile * kTile + kTile;
  w.dq_accum_off = 0;
  w.dq_accum_bytes = up(size_t(T) * Hq * d * sizeof(float));
  w.delta_off = w.dq_accum_off + w.dq_accum_bytes;
  w.delta_bytes = up(size_t(Hq) * Tpad * sizeof(float));
  w.total = w.delta_off + w.delta_bytes;
  return w;
}

namespace {

// Classification of tile pair (i, j) of one sample.  Returns 0 = dropped,
// 1 = live and full, 2 = live and needs masking.  `bwd` also requires the rows
// past the sample's end (ragged last query tile) to be masked.
int classify(int i, int j, int len, int cs, int rs, bool bwd) {
  if (j > i) return 0;
  const int q0 = i * kTile, q1 = std::min(q0 + kTile, len);  // valid query rows
  const int k0 = j * kTile, k1 = std::min(k0 + kTile, len);  // valid key rows
  if (j == i) return 2;  // the diagonal tile always holds the row's own key
  // j < i: causality holds for every pair.  Forbidden rectangle: q >= rs, cs <= kv < rs.
  const bool rows_all_rejected = q0 >= rs;
  const bool rows_some_rejected = q1 > rs;        // q1 - 1 >= rs
  const bool keys_all_chosen = k0 >= cs && k1 <= rs;
  const bool keys_some_chosen = k1 > cs && k0 < rs;
  if (rows_all_rejected && keys_all_chosen) return 0;
  bool partial = rows_some_rejected && keys_some_chosen;
  if (bwd && q0 + kTile > len) partial = true;
  return partial ? 2 : 1;
}

// A query tile is PRECISE when one of its rows sees fewer than 128 keys.  Such rows
// have large probabilities, whose bf16 rounding dominates the error of dK and dV;
// the kernels carry P and dS of these tiles as a sum of two bf16 terms.
bool precise_rows(int i, int len, int cs, int rs) {
  if (i == 0) return true;                          // row 0 sees one key
  const int q0 = i * kTile, q1 = std::min(q0 + kTile, len);
  const int q = std::max(q0, rs);                   // first rejected row of the tile, if any
  return q < q1 && cs + (q - rs + 1) < kTile;       // it sees the prompt and q - rs + 1 own keys
}

}  // namespace
}  // namespace psa

using psa::kTile;
using psa::TileRec;

extern "C" const char* psa_status_string(psa_status_t s) {
  switch (s) {
    case PSA_OK: return "ok";
    case PSA_ERR_INVALID_ARG: return "invalid argument";
    case PSA_ERR_INCONSISTENT_LENGTHS: return "cu_seqlens inconsistent with prefix/chosen/rejected lengths";
    case PSA_ERR_UNSUPPORTED: return "unsupported configuration";
    case PSA_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
    case PSA_ERR_CUDA: return "CUDA call failed";
    case PSA_ERR_DEVICE_STATUS: return "kernel reported bad data";
    case PSA_ERR_TIMEOUT: return "bounded device wait expired";
  }
  return "unknown status";
}

extern "C" psa_status_t psa_plan(const int32_t* cu_seqlens, const int32_t* prefix_len,
                                 const int32_t* chosen_len, const int32_t* rejected_len,
                                 int32_t n_samples, int32_t n_q_heads, int32_t n_kv_heads,
                                 int32_t head_dim, float softmax_scale, int32_t flags,
                                 void* stream, psa_plan_t** out) {
  if (!out) return PSA_ERR_INVALID_ARG;
  *out = nullptr;
  if (n_samples < 0 || !cu_seqlens) return PSA_ERR_INVALID_ARG;
  if (n_samples > 0 && (!prefix_len || !chosen_len || !rejected_len)) return PSA_ERR_INVALID_ARG;
  if (n_q_heads <= 0 || n_kv_heads <= 0) return PSA_ERR_INVALID_ARG;
  if (flags & ~PSA_PLAN_HOST_ONLY) return PSA_ERR_INVALID_ARG;
  if (n_q_heads % n_kv_heads != 0) return PSA_ERR_UNSUPPORTED;
  if (head_dim != 64 && head_dim != 128) return PSA_ERR_UNSUPPORTED;
  if (cu_seqlens[0] != 0) return PSA_ERR_INCONSISTENT_LENGTHS;
  for (int s = 0; s < n_samples; ++s) {
    if (prefix_len[s] < 0 || chosen_len[s] < 0 || rejected_len[s] < 0) return PSA_ERR_INVALID_ARG;
    int64_t tot = int64_t(prefix_len[s]) + chosen_len[s] + rejected_len[s];
    if (int64_t(cu_seqlens[s + 1]) - cu_seqlens[s] != tot) return PSA_ERR_INCONSISTENT_LENGTHS;
  }
  // Row indices, and row*heads products used for grid sizes, stay in int32.
  if (int64_t(cu_seqlens[n_samples]) > (int64_t(1) << 30)) return PSA_ERR_UNSUPPORTED;

  psa_plan_t* p = new (std::nothrow) psa_plan_t;
  if (!p) return PSA_ERR_INVALID_ARG;
  p->n_samples = n_samples;
  p->T = cu_seqlens[n_samples];
  p->Hq = n_q_heads;
  p->Hkv = n_kv_heads;
  p->d = head_dim;
  p->scale = softmax_scale > 0.f ? softmax_scale : 1.0f / std::sqrt(float(head_dim));

  for (int s = 0; s < n_samples; ++s) {
    const int P = prefix_len[s], C = chosen_len[s], R = rejected_len[s];
    const int len = P + C + R, cs = P, rs = P + C, ds = cu_seqlens[s];
    p->useful_pairs += int64_t(P + C) * (P + C + 1) / 2 + int64_t(R) * P + int64_t(R) * (R + 1) / 2;
    const int nt = (len + kTile - 1) / kTile;
    for (int i = 0; i < nt; ++i) {  // forward: query tile i, its key tiles in ascending order
      TileRec r{ds + i * kTile, ds, i * kTile, len, cs, rs, int32_t(p->fwd_entries.size()), 0};
      for (int j = 0; j <= i; ++j) {
        int c = psa::classify(i, j, len, cs, rs, false);
        if (!c) continue;
        p->fwd_entries.push_back((j << 2) | (int(psa::precise_rows(i, len, cs, rs)) << 1) | (c == 2));
        ++r.list_cnt;
        ++p->live_tiles;
        p->partial_tiles += (c == 2);
      }
      p->q_tiles.push_back(r);
    }
    for (int j = 0; j < nt; ++j) {  // transposed: key tile j, its query tiles in ascending order
      TileRec r{ds + j * kTile, ds, j * kTile, len, cs, rs, int32_t(p->bwd_entries.size()), 0};
      for (int i = j; i < nt; ++i) {
        int c = psa::classify(i, j, len, cs, rs, true);
        if (!c) continue;
        p->bwd_entries.push_back((i << 2) | (int(psa::precise_rows(i, len, cs, rs)) << 1) | (c == 2));
        ++r.list_cnt;
      }
      p->kv_tiles.push_back(r);
    }
    // Rejected rows past the first query tile that see fewer than kFewKeys keys (only a sample
    // with a prompt shorter than that has any).
    for (int q = std::max(rs, kTile); q < len && P + (q - rs + 1) < psa::kFewKeys; ++q)
      p->few_key_rows.push_back(psa::FewKeyRow{ds + q, ds, P, ds + rs});
  }
  // Longest list first: the hardware hands out CTAs in index order, so the long
  // work items start early and the short ones fill the tail.
  auto longest_first = [](const TileRec& a, const TileRec& b) { return a.list_cnt > b.list_cnt; };
  std::stable_sort(p->q_tiles.begin(), p->q_tiles.end(), longest_first);
  std::stable_sort(p->kv_tiles.begin(), p->kv_tiles.end(), longest_first);
  p->bwd_workspace_bytes = psa::bwd_workspace_layout(p->T, p->Hq, p->d).total;
  // Backward CTA order.  Every CTA adds its dQ contributions into the fp32 accumulator rows of
  // its sample and query-head group, so CTAs that share those rows are launched together: the
  // rows then stay in L2 while they are being updated.  Samples with the most work first, then
  // kv head, then the sample's key tiles, longest list first.
  {
    std::vector<int64_t> work(n_samples, 0);
    std::vector<std::vector<int32_t>> tiles_of(n_samples);
    std::vector<int32_t> sample_of_start(n_samples);
    for (size_t t = 0; t < p->kv_tiles.size(); ++t) {
      // the sample is found from its start row (cu_seqlens is increasing over non-empty samples)
      const int32_t ds = p->kv_tiles[t].ds;
      int s = int(std::upper_bound(cu_seqlens, cu_seqlens + n_samples + 1, ds) - cu_seqlens) - 1;
      while (s + 1 < n_samples && cu_seqlens[s + 1] == ds) ++s;   // skip zero-length samples
      work[s] += p->kv_tiles[t].list_cnt;
      tiles_of[s].push_back(int32_t(t));                          // already longest first
    }
    std::vector<int> order(n_samples);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return work[a] > work[b]; });
    std::vector<std::pair<int32_t, int32_t>> ctas;   // (key tile record, kv head)
    ctas.reserve(p->kv_tiles.size() * n_kv_heads);
    int64_t total_work = 0;
    for (int s : order)
      for (int hk = 0; hk < n_kv_heads; ++hk)
        for (int32_t t : tiles_of[s]) {
          ctas.emplace_back(t, hk);
          total_work += p->kv_tiles[t].list_cnt;
        }
    // The grouped order can leave a ragged tail (its makespan over 148 SMs is 8 % above the mean
    // on the Llama-3-8B-shaped pack).  Alternative: hand out the last 30 % of the work longest
    // first.  That evens out the finish but gives up the L2 locality of the tail, so it is taken
    // only when a list-scheduling simulation says it shortens the makespan by more than 5 %.
    {
      int n_sm = 148;
      if (!(flags & PSA_PLAN_HOST_ONLY)) {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
          n_sm = v;
      }
      auto makespan = [&](const std::vector<std::pair<int32_t, int32_t>>& order_) {
        std::priority_queue<int64_t, std::vector<int64_t>, std::greater<int64_t>> sm;
        for (int i = 0; i < n_sm; ++i) sm.push(0);
        int64_t end = 0;
        for (const auto& c : order_) {
          const int64_t t = sm.top() + p->kv_tiles[c.first].list_cnt;
          sm.pop();
          sm.push(t);
          end = std::max(end, t);
        }
        return end;
      };
      std::vector<std::pair<int32_t, int32_t>> hybrid = ctas;
      int64_t acc = 0;
      size_t split = 0;
      while (split < hybrid.size() && acc * 10 < total_work * 7) acc += p->kv_tiles[hybrid[split++].first].list_cnt;
      std::stable_sort(hybrid.begin() + split, hybrid.end(), [&](const auto& a, const auto& b) {
        return p->kv_tiles[a.first].list_cnt > p->kv_tiles[b.first].list_cnt;
      });
      if (makespan(ctas) * 100 > makespan(hybrid) * 105) ctas.swap(hybrid);
    }
    p->bwd_cta_map.reserve(ctas.size() * 2);
    for (const auto& c : ctas) {
      p->bwd_cta_map.push_back(c.first);
      p->bwd_cta_map.push_back(c.second);
    }
  }

  if (!(flags & PSA_PLAN_HOST_ONLY)) {
    psa_status_t st = psa_plan_upload(p, stream);
    if (st != PSA_OK) {
      delete p;
      return st;
    }
  }
  *out = p;
  return PSA_OK;
}

namespace {
// Process-wide cache of plan blobs.  An entry is a device allocation, a pinned staging buffer of
// the same size and two events: `copied` (the last upload has been read out of the staging buffer)
// and `last_use` (every kernel that read the device blob under its previous owner has finished).
struct BlobEntry {
  int device = -1;
  void* dptr = nullptr;
  void* hptr = nullptr;
  size_t capacity = 0;
  cudaEvent_t copied = nullptr, last_use = nullptr;
  bool last_use_valid = false;
};
constexpr size_t kBlobCacheMax = 16;
std::mutex g_blob_mutex;
std::vector<BlobEntry> g_blob_cache;

void free_entry(BlobEntry& e) {
  if (e.dptr) cudaFree(e.dptr);
  if (e.hptr) cudaFreeHost(e.hptr);
  if (e.copied) cudaEventDestroy(e.copied);
  if (e.last_use) cudaEventDestroy(e.last_use);
  e = BlobEntry{};
}

bool take_entry(int device, size_t bytes, BlobEntry* out) {
  {
    std::lock_guard<std::mutex> lock(g_blob_mutex);
    int best = -1;
    for (size_t i = 0; i < g_blob_cache.size(); ++i) {
      const BlobEntry& e = g_blob_cache[i];
      if (e.device == device && e.capacity >= bytes && (best < 0 || e.capacity < g_blob_cache[best].capacity))
        best = int(i);
    }
    if (best >= 0) {
      *out = g_blob_cache[best];
      g_blob_cache.erase(g_blob_cache.begin() + best);
      return true;
    }
  }
  BlobEntry e;
  e.device = device;
  e.capacity = (bytes + 65535) / 65536 * 65536;   // round up so that plans of similar size share entries
  if (cudaMalloc(&e.dptr, e.capacity) != cudaSuccess || cudaMallocHost(&e.hptr, e.capacity) != cudaSuccess ||
      cudaEventCreateWithFlags(&e.copied, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&e.last_use, cudaEventDisableTiming) != cudaSuccess) {
    free_entry(e);
    return false;
  }
  *out = e;
  return true;
}

void give_entry(BlobEntry e) {
  {
    std::lock_guard<std::mutex> lock(g_blob_mutex);
    if (g_blob_cache.size() < kBlobCacheMax) {
      g_blob_cache.push_back(e);
      return;
    }
  }
  if (e.last_use_valid) cudaEventSynchronize(e.last_use);
  free_entry(e);
}
}  // namespace

extern "C" psa_status_t psa_plan_upload(psa_plan_t* p, void* stream) {
  if (!p) return PSA_ERR_INVALID_ARG;
  if (p->d_blob) return PSA_OK;
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  const size_t b0 = up(p->q_tiles.size() * sizeof(TileRec));
  const size_t b1 = up(p->kv_tiles.size() * sizeof(TileRec));
  const size_t b2 = up(p->fwd_entries.size() * sizeof(int32_t));
  const size_t b3 = up(p->bwd_entries.size() * sizeof(int32_t));
  const size_t b4 = up(p->bwd_cta_map.size() * sizeof(int32_t));
  const size_t b5 = up(p->few_key_rows.size() * sizeof(psa::FewKeyRow));
  const size_t total = b0 + b1 + b2 + b3 + b4 + b5 + 256;
  if (cudaGetDevice(&p->device) != cudaSuccess) return PSA_ERR_CUDA;
  BlobEntry e;
  if (!take_entry(p->device, total, &e)) return PSA_ERR_CUDA;
  const cudaStream_t st = cudaStream_t(stream);
  // The staging buffer may still be feeding the previous owner's upload (not in steady state: that
  // copy was enqueued a whole step ago), and the device blob may still be read by the previous
  // owner's kernels: the new upload is ordered after them on the device, without a host wait.
  bool ok = cudaEventSynchronize(e.copied) == cudaSuccess;
  if (ok && e.last_use_valid) ok = cudaStreamWaitEvent(st, e.last_use, 0) == cudaSuccess;
  if (ok) {
    char* host = static_cast<char*>(e.hptr);
    std::memcpy(host, p->q_tiles.data(), p->q_tiles.size() * sizeof(TileRec));
    std::memcpy(host + b0, p->kv_tiles.data(), p->kv_tiles.size() * sizeof(TileRec));
    std::memcpy(host + b0 + b1, p->fwd_entries.data(), p->fwd_entries.size() * sizeof(int32_t));
    std::memcpy(host + b0 + b1 + b2, p->bwd_entries.data(), p->bwd_entries.size() * sizeof(int32_t));
    std::memcpy(host + b0 + b1 + b2 + b3, p->bwd_cta_map.data(), p->bwd_cta_map.size() * sizeof(int32_t));
    std::memcpy(host + b0 + b1 + b2 + b3 + b4, p->few_key_rows.data(), p->few_key_rows.size() * sizeof(psa::FewKeyRow));
    ok = cudaMemcpyAsync(e.dptr, e.hptr, total, cudaMemcpyHostToDevice, st) == cudaSuccess &&
         cudaEventRecord(e.copied, st) == cudaSuccess;
  }
  if (!ok) {
    cudaDeviceSynchronize();
    free_entry(e);
    return PSA_ERR_CUDA;
  }
  char* b = static_cast<char*>(e.dptr);
  p->d_blob = e.dptr;
  p->h_stage = e.hptr;
  p->blob_capacity = e.capacity;
  p->ev_copied = e.copied;
  p->ev_last_use = e.last_use;
  p->used_streams.clear();
  p->used_streams.push_back(stream);   // the upload itself
  p->d_q_tiles = reinterpret_cast<const TileRec*>(b);
  p->d_kv_tiles = reinterpret_cast<const TileRec*>(b + b0);
  p->d_fwd_entries = reinterpret_cast<const int32_t*>(b + b0 + b1);
  p->d_bwd_entries = reinterpret_cast<const int32_t*>(b + b0 + b1 + b2);
  p->d_bwd_cta_map = reinterpret_cast<const int32_t*>(b + b0 + b1 + b2 + b3);
  p->d_few_key_rows = reinterpret_cast<const psa::FewKeyRow*>(b + b0 + b1 + b2 + b3 + b4);
  return PSA_OK;
}

namespace psa {
void note_plan_use(const psa_plan_t* plan, void* stream) {
  std::lock_guard<std::mutex> lock(plan->used_mutex);
  for (void* s : plan->used_streams)
    if (s == stream) return;
  // used_streams[0] is the upload's stream; any other stream has to see the uploaded blob first
  if (plan->ev_copied) cudaStreamWaitEvent(cudaStream_t(stream), cudaEvent_t(plan->ev_copied), 0);
  plan->used_streams.push_back(stream);
}
}  // namespace psa

extern "C" psa_status_t psa_plan_destroy(psa_plan_t* p) {
  if (!p) return PSA_OK;
  psa_status_t st = PSA_OK;
  if (p->d_blob) {
    // Hand the blob back.  Its next owner must not overwrite it before the kernels enqueued under
    // this plan have run: one event, recorded in turn on every stream that used the plan (each
    // stream first waits for the previous recording, so the last recording covers them all).
    BlobEntry e;
    e.device = p->device;
    e.dptr = p->d_blob;
    e.hptr = p->h_stage;
    e.capacity = p->blob_capacity;
    e.copied = cudaEvent_t(p->ev_copied);
    e.last_use = cudaEvent_t(p->ev_last_use);
    int cur = -1;
    bool ok = cudaGetDevice(&cur) == cudaSuccess && (cur == p->device || cudaSetDevice(p->device) == cudaSuccess);
    bool first = true;
    for (void* s : p->used_streams) {
      if (!ok) break;
      if (!first) ok = cudaStreamWaitEvent(cudaStream_t(s), e.last_use, 0) == cudaSuccess;
      if (ok) ok = cudaEventRecord(e.last_use, cudaStream_t(s)) == cudaSuccess;
      first = false;
    }
    if (!ok) {   // a stream is gone or the context is in trouble: fall back to a full wait
      cudaGetLastError();
      if (cudaDeviceSynchronize() != cudaSuccess) st = PSA_ERR_CUDA;
      e.last_use_valid = false;
    } else {
      e.last_use_valid = true;
    }
    if (cur >= 0 && cur != p->device) cudaSetDevice(cur);
    give_entry(e);
  }
  delete p;
  return st;
}

extern "C" psa_status_t psa_plan_stats(const psa_plan_t* p, int64_t* total_tokens, int64_t* useful_pairs,
                                       int64_t* live_tiles, int64_t* partial_tiles,
                                       size_t* bwd_workspace_bytes) {
  if (!p) return PSA_ERR_INVALID_ARG;
  if (total_tokens) *total_tokens = p->T;
  if (useful_pairs) *useful_pairs = p->useful_pairs;
  if (live_tiles) *live_tiles = p->live_tiles;
  if (partial_tiles) *partial_tiles = p->partial_tiles;
  if (bwd_workspace_bytes) *bwd_workspace_bytes = p->bwd_workspace_bytes;
  return PSA_OK;
}

extern "C" psa_status_t psa_plan_counts(const psa_plan_t* p, int32_t direction, int32_t* n_tiles,
                                        int32_t* n_entries) {
  if (!p || (direction != 0 && direction != 1)) return PSA_ERR_INVALID_ARG;
  const auto& tiles = direction ? p->kv_tiles : p->q_tiles;
  const auto& entries = direction ? p->bwd_entries : p->fwd_entries;
  if (n_tiles) *n_tiles = int32_t(tiles.size());
  if (n_entries) *n_entries = int32_t(entries.size());
  return PSA_OK;
}

extern "C" psa_status_t psa_plan_export(const psa_plan_t* p, int32_t direction, int32_t* tiles,
                                        int32_t* entries) {
  if (!p || (direction != 0 && direction != 1) || !tiles || !entries) return PSA_ERR_INVALID_ARG;
  const auto& t = direction ? p->kv_tiles : p->q_tiles;
  const auto& e = direction ? p->bwd_entries : p->fwd_entries;
  if (!t.empty()) std::memcpy(tiles, t.data(), t.size() * sizeof(TileRec));
  if (!e.empty()) std::memcpy(entries, e.data(), e.size() * sizeof(int32_t));
  return PSA_OK;
}

// First-fit-decreasing packing (Section 3.2 / 4.3.2).  The "first bin with room" query is
// answered by a max segment tree over the bins' free space: O(n log n) for n units.
extern "C" psa_status_t psa_pack_ffd(const int32_t* unit_len, int32_t n_units, int32_t capacity,
                                     int32_t* bin_of_unit, int32_t* n_bins) {
  if (n_units < 0 || capacity <= 0 || !n_bins || (n_units > 0 && (!unit_len || !bin_of_unit)))
    return PSA_ERR_INVALID_ARG;
  for (int i = 0; i < n_units; ++i) {
    if (unit_len[i] < 0) return PSA_ERR_INVALID_ARG;
    if (unit_len[i] > capacity) return PSA_ERR_UNSUPPORTED;
  }
  std::vector<int32_t> order(n_units);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return unit_len[a] > unit_len[b]; });
  int leaves = 1;
  while (leaves < std::max(n_units, 1)) leaves <<= 1;
  std::vector<int32_t> tree(2 * leaves, 0);   // free space of bin b at tree[leaves + b]; unopened bins hold 0
  int32_t opened = 0;
  auto update = [&](int b, int32_t v) {
    int node = leaves + b;
    tree[node] = v;
    for (node >>= 1; node >= 1; node >>= 1) tree[node] = std::max(tree[2 * node], tree[2 * node + 1]);
  };
  for (int32_t u : order) {
    const int32_t len = unit_len[u];
    int b;
    if (opened > 0 && tree[1] >= len) {
      int node = 1;
      while (node < leaves) node = tree[2 * node] >= len ? 2 * node : 2 * node + 1;   // leftmost bin with room
      b = node - leaves;
    } else {
      b = opened++;
      update(b, capacity);
    }
    update(b, tree[leaves + b] - len);
    bin_of_unit[u] = b;
  }
  *n_bins = opened;
  return PSA_OK;
}
