"""Label layout for the per-response log-prob gather (Section 2.1, Section 3.2): the binding of
the library's psa_logp_labels.  The index work itself (which logits row scores which token on the
shared layout, and the fork list for the first rejected token) is done inside the library."""
from __future__ import annotations

from .binding import psa_logp_labels


def logp_labels(token_ids, cu_seqlens, prefix_len, chosen_len, rejected_len):
    """Returns (targets int32 [T], segment_ids int32 [T], fork_rows, fork_targets,
    fork_segments int32 [n_forks]).  Response ids: 2s = chosen, 2s+1 = rejected,
    -1 = row not scored."""
    return psa_logp_labels(token_ids, cu_seqlens, prefix_len, chosen_len, rejected_len)
