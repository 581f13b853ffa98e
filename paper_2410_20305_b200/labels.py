"""Host-side label layout for the per-response log-prob gather (Section 2.1,
Section 3.2: responses are recovered at loss time from their boundaries).

In the shared layout [prompt | chosen | rejected] the logits row of a token
predicts the NEXT token of that token's own context:

* rows cs-1 .. rs-2 predict the chosen tokens cs .. rs-1 (row cs-1 is the
  last prompt row);
* rows rs .. de-2 predict the rejected tokens rs+1 .. de-1;
* the first rejected token (position rs) follows the PROMPT, not the last
  chosen token, so it is predicted by row cs-1 as well.  That row therefore
  carries two labels; the second one travels in a short "fork" list.
* the last chosen row (rs-1) and the last rejected row (de-1) predict nothing.

With an empty prompt the first token of each response has no predicting row
and is skipped, as in the paired format.
"""
from __future__ import annotations

import numpy as np


def logp_labels(token_ids, cu_seqlens, prefix_len, chosen_len, rejected_len):
    """Returns (targets int32 [T], segment_ids int32 [T], fork_rows, fork_targets,
    fork_segments int32 [n_forks]).  Response ids: 2s = chosen, 2s+1 = rejected,
    -1 = row not scored."""
    tok = np.asarray(token_ids, dtype=np.int64)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    n = len(cu) - 1
    T = int(cu[n])
    targets = np.zeros(T, dtype=np.int32)
    segment_ids = np.full(T, -1, dtype=np.int32)
    fork_rows, fork_targets, fork_segments = [], [], []
    for s in range(n):
        P, C, R = int(prefix_len[s]), int(chosen_len[s]), int(rejected_len[s])
        ds = int(cu[s]); cs = ds + P; rs = cs + C; de = rs + R
        lo = max(cs - 1, ds)
        # chosen: rows [max(cs-1, ds), rs-2] predict token row+1
        for t in range(lo, rs - 1):
            targets[t] = tok[t + 1]
            segment_ids[t] = 2 * s
        # rejected, first token: predicted by the last prompt row (fork)
        if R >= 1 and P >= 1:
            fork_rows.append(cs - 1)
            fork_targets.append(int(tok[rs]))
            fork_segments.append(2 * s + 1)
        # rejected, remaining tokens: rows [rs, de-2]
        for t in range(rs, de - 1):
            targets[t] = tok[t + 1]
            segment_ids[t] = 2 * s + 1
    as_i32 = lambda a: np.asarray(a, dtype=np.int32)
    return targets, segment_ids, as_i32(fork_rows), as_i32(fork_targets), as_i32(fork_segments)
