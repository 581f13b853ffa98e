// Host-side helpers around the kernels: the label layout of the log-prob gather on the shared
// layout (Section 2.1, Section 3.2) and the packer's output in the form psa_plan consumes
// (Section 3.2, Section 4.3.2).  No CUDA call is made here.
#include <algorithm>
#include <numeric>
#include <vector>

#include "psa.h"

// In the shared layout [prompt | chosen | rejected] the logits row of a token predicts the next
// token of that token's own context:
//   rows cs-1 .. rs-2 predict the chosen tokens cs .. rs-1 (row cs-1 is the last prompt row);
//   rows rs .. de-2 predict the rejected tokens rs+1 .. de-1;
//   the first rejected token follows the PROMPT, so it is predicted by row cs-1 as well: that row
//   carries a second label, which travels in the fork list;
//   the last chosen row and the last rejected row predict nothing.
// With an empty prompt the first token of each response has no predicting row and is skipped.
extern "C" psa_status_t psa_logp_labels(const int32_t* token_ids, const int32_t* cu_seqlens,
                                        const int32_t* prefix_len, const int32_t* chosen_len,
                                        const int32_t* rejected_len, int32_t n_samples, int32_t* targets,
                                        int32_t* segment_ids, int32_t* fork_rows, int32_t* fork_targets,
                                        int32_t* fork_segments, int32_t* n_forks) {
  if (n_samples < 0 || !cu_seqlens || !n_forks) return PSA_ERR_INVALID_ARG;
  if (n_samples > 0 && (!prefix_len || !chosen_len || !rejected_len || !fork_rows || !fork_targets || !fork_segments))
    return PSA_ERR_INVALID_ARG;
  if (cu_seqlens[0] != 0) return PSA_ERR_INCONSISTENT_LENGTHS;
  for (int s = 0; s < n_samples; ++s) {
    if (prefix_len[s] < 0 || chosen_len[s] < 0 || rejected_len[s] < 0) return PSA_ERR_INVALID_ARG;
    if (int64_t(cu_seqlens[s + 1]) - cu_seqlens[s] != int64_t(prefix_len[s]) + chosen_len[s] + rejected_len[s])
      return PSA_ERR_INCONSISTENT_LENGTHS;
  }
  const int32_t T = cu_seqlens[n_samples];
  if (T > 0 && (!token_ids || !targets || !segment_ids)) return PSA_ERR_INVALID_ARG;
  for (int32_t t = 0; t < T; ++t) {
    targets[t] = 0;
    segment_ids[t] = -1;
  }
  int32_t nf = 0;
  for (int s = 0; s < n_samples; ++s) {
    const int32_t ds = cu_seqlens[s], cs = ds + prefix_len[s], rs = cs + chosen_len[s], de = rs + rejected_len[s];
    for (int32_t t = std::max(cs - 1, ds); t < rs - 1; ++t) {   // chosen tokens after their predecessors
      targets[t] = token_ids[t + 1];
      segment_ids[t] = 2 * s;
    }
    if (rejected_len[s] >= 1 && prefix_len[s] >= 1) {           // first rejected token: the last prompt row again
      fork_rows[nf] = cs - 1;
      fork_targets[nf] = token_ids[rs];
      fork_segments[nf] = 2 * s + 1;
      ++nf;
    }
    for (int32_t t = rs; t < de - 1; ++t) {                     // the other rejected tokens
      targets[t] = token_ids[t + 1];
      segment_ids[t] = 2 * s + 1;
    }
  }
  *n_forks = nf;
  return PSA_OK;
}

extern "C" psa_status_t psa_pack_ffd_emit(const int32_t* prefix_len, const int32_t* chosen_len,
                                          const int32_t* rejected_len, int32_t n_units, int32_t capacity,
                                          int32_t paired, int32_t* bin_of_unit, int32_t* n_packs,
                                          int32_t* pack_sample_offset, int32_t* sample_unit,
                                          int32_t* out_prefix_len, int32_t* out_chosen_len,
                                          int32_t* out_rejected_len, int32_t* out_cu_seqlens) {
  if (n_units < 0 || capacity <= 0 || !n_packs || !pack_sample_offset || !out_cu_seqlens) return PSA_ERR_INVALID_ARG;
  if (n_units > 0 && (!prefix_len || !chosen_len || !rejected_len || !bin_of_unit || !sample_unit || !out_prefix_len ||
                      !out_chosen_len || !out_rejected_len))
    return PSA_ERR_INVALID_ARG;
  std::vector<int32_t> unit_len(n_units);
  for (int i = 0; i < n_units; ++i) {
    if (prefix_len[i] < 0 || chosen_len[i] < 0 || rejected_len[i] < 0) return PSA_ERR_INVALID_ARG;
    // the packing unit is the prompt with both responses; the paired layout repeats the prompt
    const int64_t len = int64_t(paired ? 2 : 1) * prefix_len[i] + chosen_len[i] + rejected_len[i];
    if (len > capacity) return PSA_ERR_UNSUPPORTED;
    unit_len[i] = int32_t(len);
  }
  int32_t bins = 0;
  const psa_status_t st = psa_pack_ffd(unit_len.data(), n_units, capacity, bin_of_unit, &bins);
  if (st != PSA_OK) return st;
  // Units of a pack in the order the packer placed them: longest first, ties by index.
  std::vector<int32_t> order(n_units);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
    return bin_of_unit[a] != bin_of_unit[b] ? bin_of_unit[a] < bin_of_unit[b] : unit_len[a] > unit_len[b];
  });
  const int per_unit = paired ? 2 : 1;
  int32_t m = 0;       // samples written so far
  int32_t cur = -1;    // pack being written
  int32_t row = 0;     // tokens of the current pack so far
  for (int32_t u : order) {
    const int32_t b = bin_of_unit[u];
    while (cur < b) {  // open pack cur + 1: its sample range and its own cu_seqlens array start here
      ++cur;
      pack_sample_offset[cur] = m;
      row = 0;
      out_cu_seqlens[m + cur] = 0;
    }
    for (int half = 0; half < per_unit; ++half) {
      const int32_t P = prefix_len[u];
      const int32_t C = paired ? (half == 0 ? chosen_len[u] : rejected_len[u]) : chosen_len[u];
      const int32_t R = paired ? 0 : rejected_len[u];
      sample_unit[m] = u;
      out_prefix_len[m] = P;
      out_chosen_len[m] = C;
      out_rejected_len[m] = R;
      row += P + C + R;
      out_cu_seqlens[m + cur + 1] = row;
      ++m;
    }
  }
  pack_sample_offset[bins] = m;
  *n_packs = bins;
  return PSA_OK;
}
