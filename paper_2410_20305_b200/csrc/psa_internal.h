// Internal definitions shared by the host planner and the kernel launchers.
#pragma once
#include <cstdint>
#include <mutex>
#include <vector>

#include "psa.h"

namespace psa {

constexpr int kTile = 128;  // query-tile and key-tile edge, in tokens

// One record per query tile (forward map) or per key tile (transposed map).
// All positions except row0 / ds are relative to the sample start.
struct TileRec {
  int32_t row0;      // packed-row index of the tile's first row
  int32_t ds;        // packed-row index of the sample's first token
  int32_t local0;    // row0 - ds
  int32_t len;       // sample length P + C + R
  int32_t cs;        // chosen start  = P
  int32_t rs;        // rejected start = P + C
  int32_t list_off;  // first entry of this tile's list
  int32_t list_cnt;  // number of live partner tiles
};
static_assert(sizeof(TileRec) == 32, "TileRec is 8 int32");

// A rejected-response row that lies outside its sample's first query tile and sees fewer than
// kFewKeys keys (a sample with a very short prompt).  Its visible keys are the packed rows
// [ds, ds + n_prompt) and [rs_row, row].  The backward pass recomputes delta of these rows exactly.
constexpr int kFewKeys = 32;
struct FewKeyRow {
  int32_t row;       // packed-row index of the query row
  int32_t ds;        // packed-row index of the sample's first token
  int32_t n_prompt;  // prompt length P
  int32_t rs_row;    // packed-row index of the first rejected token
};
static_assert(sizeof(FewKeyRow) == 16, "FewKeyRow is 4 int32");

}  // namespace psa

struct psa_plan {
  int32_t n_samples = 0, T = 0, Hq = 0, Hkv = 0, d = 0;
  float scale = 0.f;
  int64_t useful_pairs = 0, live_tiles = 0, partial_tiles = 0;
  size_t bwd_workspace_bytes = 0;
  std::vector<psa::TileRec> q_tiles, kv_tiles;   // sorted, longest list first
  std::vector<int32_t> fwd_entries, bwd_entries;
  // Launch order of the backward CTAs: pairs (index into kv_tiles, kv head).
  std::vector<int32_t> bwd_cta_map;
  std::vector<psa::FewKeyRow> few_key_rows;
  // device copy (one allocation, taken from and returned to a small process-wide cache so that a
  // plan per step costs no cudaMalloc / cudaFree and no host synchronisation)
  int device = -1;
  void* d_blob = nullptr;
  void* h_stage = nullptr;        // pinned staging buffer the blob was uploaded from
  size_t blob_capacity = 0;
  void* ev_copied = nullptr;      // cudaEvent_t: the upload has left the staging buffer
  void* ev_last_use = nullptr;    // cudaEvent_t: recorded at destroy on the streams that used the plan
  mutable std::vector<void*> used_streams;   // streams that launched kernels reading the blob
  mutable std::mutex used_mutex;             // launches from several host threads may share a plan
  const psa::TileRec* d_q_tiles = nullptr;
  const psa::TileRec* d_kv_tiles = nullptr;
  const int32_t* d_fwd_entries = nullptr;
  const int32_t* d_bwd_entries = nullptr;
  const int32_t* d_bwd_cta_map = nullptr;
  const psa::FewKeyRow* d_few_key_rows = nullptr;
};

namespace psa {
// Called before kernels that read the plan's device blob are enqueued on `stream`: remembers the
// stream (psa_plan_destroy orders the blob's next owner behind it) and, the first time a stream
// other than the upload's is used, makes it wait for the upload (which is asynchronous).
void note_plan_use(const psa_plan_t* plan, void* stream);

// True when the current CUDA device is the one the plan's device blob was uploaded to.
bool plan_on_current_device(const psa_plan_t* plan);

// Returns PSA_OK if no CUDA error is pending, else PSA_ERR_CUDA; with PSA_DEBUG set in the
// environment the CUDA error string is written to stderr.
psa_status_t check_last_cuda_error(const char* where);

// Optional event pairs recorded around one kernel (see psa_profile_events).
struct ProfileEvents { void* start; void* stop; };
extern ProfileEvents g_profile[5];
struct ProfileScope {  // records start now and stop at scope exit, if registered
  ProfileEvents ev; void* stream;
  ProfileScope(int which, void* s);
  ~ProfileScope();
};

// Workspace layout of psa_bwd (byte offsets, each 256-aligned).
struct BwdWorkspace {
  size_t dq_accum_off, dq_accum_bytes;  // fp32 [T, Hq, d]
  size_t delta_off, delta_bytes;        // fp32 [Hq, Tpad]  D_i = dO_i . O_i
  size_t total;
};
BwdWorkspace bwd_workspace_layout(int64_t T, int Hq, int d);

psa_status_t launch_fwd(const psa_plan_t* plan, const void* q, const void* k, const void* v, void* o,
                        float* lse, int32_t* device_status, void* stream);
psa_status_t launch_bwd(const psa_plan_t* plan, const void* d_o, const void* q, const void* k,
                        const void* v, const void* o, const float* lse, void* dq, void* dk, void* dv,
                        void* workspace, bool f32_out, int32_t* device_status, void* stream);
}  // namespace psa
