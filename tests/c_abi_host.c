/* A C caller of libpsa's host-side entry points: shows that include/psa.h is plain C and that the
 * library can be used without Python.  Built and run by tests/test_c_abi_from_c.py (no GPU needed:
 * the plan is built with PSA_PLAN_HOST_ONLY).  Expected values are hand-derived in the comments. */
#include <stdio.h>
#include <string.h>

#include "psa.h"

#define CHECK(cond)                                                        \
  do {                                                                     \
    if (!(cond)) {                                                         \
      printf("FAILED line %d: %s\n", __LINE__, #cond);                     \
      return 1;                                                            \
    }                                                                      \
  } while (0)

int main(void) {
  /* the tiny configuration: A = 256/64/96, B = 128/80/48 -> 109,648 unmasked pairs per head */
  const int32_t cu[3] = {0, 416, 672}, P[2] = {256, 128}, C[2] = {64, 80}, R[2] = {96, 48};
  psa_plan_t* plan = NULL;
  CHECK(psa_plan(cu, P, C, R, 2, 4, 4, 64, 0.0f, PSA_PLAN_HOST_ONLY, NULL, &plan) == PSA_OK);
  int64_t T = 0, pairs = 0, live = 0, partial = 0;
  size_t ws = 0;
  CHECK(psa_plan_stats(plan, &T, &pairs, &live, &partial, &ws) == PSA_OK);
  CHECK(T == 672 && pairs == 109648 && live > 0 && partial > 0 && ws > 0);
  /* sample A has 4 tiles, sample B has 2: query-tile records 6; A's tile 3 (rows 384..415, all rejected)
     drops key tile 2 (keys 256..383: chosen keys 256..319 and rejected keys 320..383 -> kept, it holds
     rejected keys), so nothing is dropped there; lists are 1+2+3+4 and 1+2 = 13 entries */
  int32_t n_tiles = 0, n_entries = 0;
  CHECK(psa_plan_counts(plan, 0, &n_tiles, &n_entries) == PSA_OK);
  CHECK(n_tiles == 6 && n_entries == 13 && n_entries == live);
  /* a launch on a plan without a device copy is refused before any pointer is touched */
  CHECK(psa_fwd(plan, cu, cu, cu, (void*)cu, (float*)cu, NULL, NULL) == PSA_ERR_INVALID_ARG);
  CHECK(psa_plan_destroy(plan) == PSA_OK);
  /* inconsistent lengths are reported as such */
  const int32_t bad_cu[3] = {0, 400, 672};
  CHECK(psa_plan(bad_cu, P, C, R, 2, 4, 4, 64, 0.0f, PSA_PLAN_HOST_ONLY, NULL, &plan) == PSA_ERR_INCONSISTENT_LENGTHS);
  CHECK(strcmp(psa_status_string(PSA_OK), "ok") == 0);
  CHECK(psa_check_device_status(0) == PSA_OK && psa_check_device_status(PSA_DEVSTAT_WAIT_EXPIRED) == PSA_ERR_TIMEOUT);

  /* position ids: samples (2,2,3) and (0,1,2): rejected tokens restart right after the prompt */
  const int32_t cu2[3] = {0, 7, 10}, P2[2] = {2, 0}, C2[2] = {2, 1}, R2[2] = {3, 2};
  int32_t pos[10];
  const int32_t want_pos[10] = {0, 1, 2, 3, 2, 3, 4, 0, 0, 1};
  CHECK(psa_position_ids(cu2, P2, C2, R2, 2, pos) == PSA_OK);
  CHECK(memcmp(pos, want_pos, sizeof pos) == 0);

  /* labels on the same pack, tokens 100..109: sample 0 (rows 0..6): the last prompt row 1 scores the first
     chosen token (row 2) and, through the fork list, the first rejected token (row 4); chosen row 2 scores
     token 3; rejected rows 4, 5 score tokens 5, 6; rows 0, 3, 6 score nothing.  Sample 1 has no prompt:
     the first tokens of its responses have no scoring row; rejected row 8 scores token 9. */
  int32_t tok[10], targets[10], seg[10], fr[2], ft[2], fs[2], nf = -1;
  for (int i = 0; i < 10; ++i) tok[i] = 100 + i;
  CHECK(psa_logp_labels(tok, cu2, P2, C2, R2, 2, targets, seg, fr, ft, fs, &nf) == PSA_OK);
  const int32_t want_seg[10] = {-1, 0, 0, -1, 1, 1, -1, -1, 3, -1};
  CHECK(memcmp(seg, want_seg, sizeof seg) == 0);
  CHECK(targets[1] == 102 && targets[2] == 103 && targets[4] == 105 && targets[5] == 106 && targets[8] == 109);
  CHECK(nf == 1 && fr[0] == 1 && ft[0] == 104 && fs[0] == 1);

  /* packing: units (P,C,R) of lengths 7, 3, 5, 4 into packs of 10 -> [7, 3] and [5, 4] */
  const int32_t uP[4] = {4, 1, 3, 2}, uC[4] = {2, 1, 2, 1}, uR[4] = {1, 1, 0, 1};
  int32_t bin[4], n_packs = 0, off[5], unit[4], oP[4], oC[4], oR[4], ocu[8];
  CHECK(psa_pack_ffd_emit(uP, uC, uR, 4, 10, 0, bin, &n_packs, off, unit, oP, oC, oR, ocu) == PSA_OK);
  CHECK(n_packs == 2 && off[0] == 0 && off[1] == 2 && off[2] == 4);
  CHECK(bin[0] == 0 && bin[1] == 0 && bin[2] == 1 && bin[3] == 1);
  CHECK(unit[0] == 0 && unit[1] == 1 && unit[2] == 2 && unit[3] == 3);
  CHECK(ocu[0] == 0 && ocu[1] == 7 && ocu[2] == 10 && ocu[3] == 0 && ocu[4] == 5 && ocu[5] == 9);
  /* each emitted pack goes straight into psa_plan */
  for (int b = 0; b < n_packs; ++b) {
    CHECK(psa_plan(ocu + off[b] + b, oP + off[b], oC + off[b], oR + off[b], off[b + 1] - off[b], 8, 2, 128, 0.0f,
                   PSA_PLAN_HOST_ONLY, NULL, &plan) == PSA_OK);
    CHECK(psa_plan_stats(plan, &T, NULL, NULL, NULL, NULL) == PSA_OK && T == (b == 0 ? 10 : 9));
    CHECK(psa_plan_destroy(plan) == PSA_OK);
  }
  printf("C_ABI_OK\n");
  return 0;
}
