"""CPU oracle for prefix-shared attention and the per-response log-prob gather.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this module;
it is used by the tests, by the smoke check and by the benchmark's CPU-baseline
leg.  It shares no code with the CUDA library and imports nothing from the
package.

Everything is the plain textbook definition in float64 with an explicit dense
boolean mask: no tiling, no online softmax, no block map.  A BLAS matmul is the
only library primitive used as a step.

Paper passages each function follows:

* ``token_roles`` / ``prefix_sharing_mask_packed``: Algorithm 3 ("Prefix
  Sharing Mask with Packing"): causal AND same-document AND NOT(rejected query
  looking at a chosen key), from dense per-token arrays (sample id and
  prompt / chosen / rejected role of every token, Section 3.2).
* ``prefix_sharing_mask_single``: Algorithm 1 ("Prefix Sharing Mask").
* ``paired_packing_mask``: Algorithm 2 ("Attention Mask for Packing w/o Prefix
  Sharing"): causal AND same per-token response id.
* ``attention_fwd`` / ``attention_bwd``: Section 3.1: the attention computed
  under the mask is ordinary softmax attention; the backward is its exact
  gradient.
* ``dpo_logp`` / ``paired_response_logps``: Section 2.1: the total log
  probability of each completion given the prompt, recovered per response
  from the packed row with the response boundaries (Section 3.2).
* ``ideal_token_speedup`` / ``ideal_attention_speedup``: the two footnotes of
  Section 4.2 (2(p+c)/(p+2c) and 2(p+c)^2/(2(p+c)^2-p^2)).
* ``ffd_pack`` / ``ffd_pack_layout``: Section 3.2 and Section 4.3.2 (first-fit-decreasing
  packing of prompt-plus-both-responses units; the lay-out of every pack).
* ``attention_layer_fwd`` / ``attention_layer_bwd``: the full attention layer of the
  Section 4.2 micro-benchmark (projections, rotary embedding on the shared layout's
  position ids of Section 3.1, attention, output projection) and its gradient.
* ``dpo_loss`` / ``dpo_logp_grad``: Eq. 1 (Section 2.1).  The equation is printed as a
  ratio of logs; it is read as the DPO loss of its cited source,
  -log sigmoid(beta * [(lp_theta(chosen) - lp_ref(chosen)) - (lp_theta(rejected) - lp_ref(rejected))]),
  averaged over the samples; its gradient with respect to the logits follows from
  d log softmax(x)[y] / dx = onehot(y) - softmax(x).

Parity pins (tests/test_oracle_*.py): the paired-format equivalence claimed in
Section 3.1 checked against torch's own scaled_dot_product_attention and
autograd in float64, hand-derived mask fixtures, closed forms for q = 0,
finite differences, torch.log_softmax for the gather.  No function here is
"parity unpinned".
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------
# Masks
# --------------------------------------------------------------------------

PROMPT, CHOSEN, REJECTED = 0, 1, 2


def token_roles(cu_seqlens, prefix_len, chosen_len, rejected_len):
    """Per-token description of one packed row: which sample a token belongs to and whether it
    is a prompt, chosen or rejected token.  (Algorithm 3 carries the same information as a
    document id and two start indices per token, Section 3.2.)  Returns (sample_of, role),
    each int64 [T]."""
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    n = len(cu) - 1
    T = int(cu[n])
    sample_of = np.empty(T, dtype=np.int64)
    role = np.empty(T, dtype=np.int64)
    for s in range(n):
        P, C, R = int(prefix_len[s]), int(chosen_len[s]), int(rejected_len[s])
        lo, hi = int(cu[s]), int(cu[s + 1])
        if hi - lo != P + C + R:
            raise ValueError("sample %d: cu_seqlens span %d != P+C+R = %d" % (s, hi - lo, P + C + R))
        sample_of[lo:hi] = s
        role[lo:lo + P] = PROMPT
        role[lo + P:lo + P + C] = CHOSEN
        role[lo + P + C:hi] = REJECTED
    return sample_of, role


def prefix_sharing_mask_packed(sample_of, role):
    """The mask of Algorithm 3 over every (query, key) pair of the packed row: a query sees a
    key iff the key is not after it, both belong to the same sample, and it is not the case
    that the query is a rejected token while the key is a chosen token."""
    T = len(role)
    pos = np.arange(T, dtype=np.int64)
    not_later = pos[None, :] <= pos[:, None]                       # [query, key]
    same_sample = sample_of[:, None] == sample_of[None, :]
    rejected_sees_chosen = (role[:, None] == REJECTED) & (role[None, :] == CHOSEN)
    return not_later & same_sample & ~rejected_sees_chosen


def prefix_sharing_mask_single(L, chosen_start, rejected_start):
    """Algorithm 1: one unpacked sample of length L whose chosen response starts at
    chosen_start and whose rejected response starts at rejected_start."""
    pos = np.arange(L, dtype=np.int64)
    role = np.where(pos < chosen_start, PROMPT, np.where(pos < rejected_start, CHOSEN, REJECTED))
    return prefix_sharing_mask_packed(np.zeros(L, dtype=np.int64), role)


def paired_packing_mask(response_ids):
    """Algorithm 2 (the paired baseline layout, packed): a query sees the keys of its own
    sequence that are not after it; `response_ids` names the sequence of every token."""
    ids = np.asarray(response_ids, dtype=np.int64)
    pos = np.arange(len(ids), dtype=np.int64)
    return (pos[None, :] <= pos[:, None]) & (ids[:, None] == ids[None, :])


def packed_mask(cu_seqlens, prefix_len, chosen_len, rejected_len):
    """Convenience: Algorithm 3's mask straight from the per-sample lengths."""
    return prefix_sharing_mask_packed(*token_roles(cu_seqlens, prefix_len, chosen_len, rejected_len))


def useful_pairs(prefix_len, chosen_len, rejected_len):
    """Number of unmasked (q, kv) pairs per head, counted from the lengths:
    the causal triangle over prompt+chosen, plus for the rejected rows the
    prompt rectangle and their own causal triangle."""
    U = 0
    for P, C, R in zip(prefix_len, chosen_len, rejected_len):
        P, C, R = int(P), int(C), int(R)
        U += (P + C) * (P + C + 1) // 2 + R * P + R * (R + 1) // 2
    return U


def ideal_token_speedup(p, c):
    """Footnote of Section 4.2.1: paired tokens / shared tokens = 2(p+c)/(p+2c)."""
    return 2.0 * (p + c) / (p + 2.0 * c)


def ideal_attention_speedup(p, c):
    """Footnote of Section 4.2.2: 2(p+c)^2 / (2(p+c)^2 - p^2)."""
    return 2.0 * (p + c) ** 2 / (2.0 * (p + c) ** 2 - p ** 2)


# --------------------------------------------------------------------------
# Attention, forward and backward, dense mask, float64
# --------------------------------------------------------------------------

def _as_f64(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def attention_fwd(q, k, v, mask, softmax_scale=None):
    """Masked softmax attention.

    q [T, Hq, d]; k, v [T, Hkv, d]; mask bool [T, T] (True = may attend).
    Query head h reads kv head h // (Hq // Hkv).
    Returns o [T, Hq, d] and lse [Hq, T] = log sum_j exp(scale * q_i . k_j)
    over the allowed j (natural log).  Every row must allow at least one key.
    """
    q, k, v = _as_f64(q), _as_f64(k), _as_f64(v)
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    g = Hq // Hkv
    scale = (1.0 / np.sqrt(d)) if softmax_scale is None else float(softmax_scale)
    o = np.empty((T, Hq, d), dtype=np.float64)
    lse = np.empty((Hq, T), dtype=np.float64)
    for h in range(Hq):
        kh = k[:, h // g, :]
        vh = v[:, h // g, :]
        S = scale * (q[:, h, :] @ kh.T)
        S = np.where(mask, S, -np.inf)
        m = S.max(axis=1)
        E = np.exp(S - m[:, None])
        l = E.sum(axis=1)
        lse[h] = m + np.log(l)
        P = E / l[:, None]
        o[:, h, :] = P @ vh
    return o, lse


def attention_bwd(q, k, v, d_o, mask, softmax_scale=None):
    """Exact gradient of attention_fwd for the loss sum(o * d_o).

    Returns dq [T, Hq, d], dk, dv [T, Hkv, d]; dk, dv are summed over the
    query heads that share a kv head.
        P   = softmax(S) on the allowed pairs
        dV  = P^T dO           dP = dO V^T
        D_i = dO_i . o_i       dS = P * (dP - D)
        dQ  = scale * dS K     dK = scale * dS^T Q
    """
    q, k, v, d_o = _as_f64(q), _as_f64(k), _as_f64(v), _as_f64(d_o)
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    g = Hq // Hkv
    scale = (1.0 / np.sqrt(d)) if softmax_scale is None else float(softmax_scale)
    dq = np.zeros((T, Hq, d), dtype=np.float64)
    dk = np.zeros((T, Hkv, d), dtype=np.float64)
    dv = np.zeros((T, Hkv, d), dtype=np.float64)
    for h in range(Hq):
        kh = k[:, h // g, :]
        vh = v[:, h // g, :]
        qh = q[:, h, :]
        doh = d_o[:, h, :]
        S = scale * (qh @ kh.T)
        S = np.where(mask, S, -np.inf)
        m = S.max(axis=1)
        E = np.exp(S - m[:, None])
        P = E / E.sum(axis=1)[:, None]
        oh = P @ vh
        Dvec = (doh * oh).sum(axis=1)
        dP = doh @ vh.T
        dS = P * (dP - Dvec[:, None])
        dq[:, h, :] = scale * (dS @ kh)
        dk[:, h // g, :] += scale * (dS.T @ qh)
        dv[:, h // g, :] += P.T @ doh
    return dq, dk, dv


def attention_rows(q, k, v, mask_rows, rows, softmax_scale=None):
    """attention_fwd restricted to the query rows `rows` (for sampled checks at
    sizes where the full T x T problem is too slow).  mask_rows is the
    corresponding [len(rows), T] slice of the dense mask."""
    q, k, v = _as_f64(q), _as_f64(k), _as_f64(v)
    T, Hq, d = q.shape
    g = Hq // k.shape[1]
    scale = (1.0 / np.sqrt(d)) if softmax_scale is None else float(softmax_scale)
    rows = np.asarray(rows, dtype=np.int64)
    o = np.empty((len(rows), Hq, d), dtype=np.float64)
    lse = np.empty((Hq, len(rows)), dtype=np.float64)
    for h in range(Hq):
        S = scale * (q[rows, h, :] @ k[:, h // g, :].T)
        S = np.where(mask_rows, S, -np.inf)
        m = S.max(axis=1)
        E = np.exp(S - m[:, None])
        l = E.sum(axis=1)
        lse[h] = m + np.log(l)
        o[:, h, :] = (E / l[:, None]) @ v[:, h // g, :]
    return o, lse


def attention_bwd_sampled(q, k, v, d_o, o, lse, mask, rows, cols, softmax_scale=None):
    """attention_bwd restricted to the query rows `rows` (dq) and the key positions `cols` (dk, dv),
    for checks at sizes where the dense T x T gradient is too slow.  `o` [T, Hq, d] and `lse` [Hq, T]
    are the results of this oracle's own forward for ALL rows (attention_fwd, or attention_rows
    called chunk by chunk); `mask` is the dense [T, T] mask.  Same definition as attention_bwd,
    written per row i and per column j:
        P_ij = exp(S_ij - lse_i)   D_i = dO_i . o_i   dS_ij = P_ij (dO_i . v_j - D_i)
        dq_i = scale sum_j dS_ij k_j      dk_j = scale sum_i dS_ij q_i      dv_j = sum_i P_ij dO_i
    (dk, dv summed over the query heads of the kv head).  Returns
    (dq_rows [len(rows), Hq, d], dk_cols [len(cols), Hkv, d], dv_cols [len(cols), Hkv, d])."""
    q, k, v, d_o, o = _as_f64(q), _as_f64(k), _as_f64(v), _as_f64(d_o), _as_f64(o)
    lse = np.asarray(lse, dtype=np.float64)
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    g = Hq // Hkv
    scale = (1.0 / np.sqrt(d)) if softmax_scale is None else float(softmax_scale)
    rows = np.asarray(rows, dtype=np.int64)
    cols = np.asarray(cols, dtype=np.int64)
    Dvec = (d_o * o).sum(axis=2)                       # [T, Hq]
    dq_rows = np.zeros((len(rows), Hq, d), dtype=np.float64)
    dk_cols = np.zeros((len(cols), Hkv, d), dtype=np.float64)
    dv_cols = np.zeros((len(cols), Hkv, d), dtype=np.float64)
    for h in range(Hq):
        kh, vh, qh, doh = k[:, h // g, :], v[:, h // g, :], q[:, h, :], d_o[:, h, :]
        # rows: everything of row i
        S = scale * (qh[rows] @ kh.T)
        P = np.where(mask[rows], np.exp(S - lse[h, rows][:, None]), 0.0)
        dS = P * (doh[rows] @ vh.T - Dvec[rows, h][:, None])
        dq_rows[:, h, :] = scale * (dS @ kh)
        # columns: everything of key j
        S = scale * (qh @ kh[cols].T)                   # [T, len(cols)]
        P = np.where(mask[:, cols], np.exp(S - lse[h][:, None]), 0.0)
        dS = P * (doh @ vh[cols].T - Dvec[:, h][:, None])
        dk_cols[:, h // g, :] += scale * (dS.T @ qh)
        dv_cols[:, h // g, :] += P.T @ doh
    return dq_rows, dk_cols, dv_cols


# --------------------------------------------------------------------------
# Per-response summed log-probabilities
# --------------------------------------------------------------------------

def row_logprob(logits_row, target):
    """log softmax(logits_row)[target] in float64."""
    x = np.asarray(logits_row, dtype=np.float64)
    m = x.max()
    return float(x[int(target)] - (m + np.log(np.exp(x - m).sum())))


def dpo_logp(logits, targets, segment_ids, n_segments,
             fork_rows=(), fork_targets=(), fork_segments=()):
    """out[g] = sum of log softmax(logits[t])[y] over every scored (t, y) whose
    response id is g.

    Row t scores targets[t] for response segment_ids[t] (skipped when the id is
    negative).  The fork list adds second labels: row fork_rows[f] also scores
    fork_targets[f] for response fork_segments[f].  In the shared layout this
    is the last prompt row, whose next token is both the first chosen and the
    first rejected token.
    """
    logits = np.asarray(logits, dtype=np.float64)
    out = np.zeros(int(n_segments), dtype=np.float64)
    for t in range(logits.shape[0]):
        g = int(segment_ids[t])
        if g >= 0:
            out[g] += row_logprob(logits[t], targets[t])
    for r, y, g in zip(fork_rows, fork_targets, fork_segments):
        if int(g) >= 0:
            out[int(g)] += row_logprob(logits[int(r)], y)
    return out


def paired_response_logps(logits_fn, token_ids, cu_seqlens, prefix_len, chosen_len, rejected_len):
    """The paired-format definition of Section 2.1, written out.

    For every sample build the two ordinary sequences [prompt | chosen] and
    [prompt | rejected]; position i of a sequence predicts token i+1; the
    response's log-prob is the sum over its own tokens.  `logits_fn(rows)`
    returns the logits of the given packed-row indices (so that a paired
    sequence can be assembled by copying rows of the shared layout).
    Returns float64 [2n]: entry 2s = chosen, 2s+1 = rejected.
    """
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    tok = np.asarray(token_ids, dtype=np.int64)
    n = len(cu) - 1
    out = np.zeros(2 * n, dtype=np.float64)
    for s in range(n):
        P, C, R = int(prefix_len[s]), int(chosen_len[s]), int(rejected_len[s])
        ds = int(cu[s])
        prompt = np.arange(ds, ds + P)
        for which, resp in ((0, np.arange(ds + P, ds + P + C)),
                            (1, np.arange(ds + P + C, ds + P + C + R))):
            seq = np.concatenate([prompt, resp])
            lg = np.asarray(logits_fn(seq), dtype=np.float64)
            for i in range(len(seq) - 1):
                nxt = i + 1
                if nxt >= P:
                    out[2 * s + which] += row_logprob(lg[i], tok[seq[nxt]])
    return out


# --------------------------------------------------------------------------
# DPO loss (Eq. 1) and its gradient back into the logits
# --------------------------------------------------------------------------

def dpo_loss(policy_logps, ref_logps, beta):
    """Mean over the n samples of  -log sigmoid(beta * margin_s),
    margin_s = (pol[2s] - ref[2s]) - (pol[2s+1] - ref[2s+1])   (entry 2s = chosen, 2s+1 = rejected).
    Returns (loss, coef) with coef[g] = d loss / d policy_logps[g]."""
    pol = np.asarray(policy_logps, dtype=np.float64)
    ref = np.asarray(ref_logps, dtype=np.float64)
    n = len(pol) // 2
    margin = (pol[0::2] - ref[0::2]) - (pol[1::2] - ref[1::2])
    z = float(beta) * margin
    # -log sigmoid(z) = log(1 + exp(-z)), evaluated without overflow
    loss_s = np.maximum(-z, 0.0) + np.log1p(np.exp(-np.abs(z)))
    sig_neg = np.exp(-np.maximum(z, 0.0)) / (1.0 + np.exp(-np.abs(z)))      # sigmoid(-z)
    coef = np.zeros(2 * n, dtype=np.float64)
    coef[0::2] = -float(beta) * sig_neg / n
    coef[1::2] = +float(beta) * sig_neg / n
    return float(loss_s.mean()), coef


def simpo_loss(policy_logps, lengths, beta, gamma):
    """Length-normalised, reference-free variant of the paired loss (SimPO, one of the paired
    preference methods Section 1 names as served by the same layout): mean over the n samples of
        -log sigmoid(beta * (pol[2s] / len[2s] - pol[2s+1] / len[2s+1]) - gamma).
    `lengths[g]` is the number of scored tokens of response g.  Returns (loss, coef) with
    coef[g] = d loss / d policy_logps[g]."""
    pol = np.asarray(policy_logps, dtype=np.float64)
    ln = np.asarray(lengths, dtype=np.float64)
    n = len(pol) // 2
    z = float(beta) * (pol[0::2] / ln[0::2] - pol[1::2] / ln[1::2]) - float(gamma)
    loss_s = np.maximum(-z, 0.0) + np.log1p(np.exp(-np.abs(z)))
    sig_neg = np.exp(-np.maximum(z, 0.0)) / (1.0 + np.exp(-np.abs(z)))      # sigmoid(-z)
    coef = np.zeros(2 * n, dtype=np.float64)
    coef[0::2] = -float(beta) * sig_neg / (n * ln[0::2])
    coef[1::2] = +float(beta) * sig_neg / (n * ln[1::2])
    return float(loss_s.mean()), coef


def orpo_loss(policy_logps, lengths, lam):
    """Odds-ratio variant of the paired loss (ORPO, named in Section 1 beside DPO and SimPO): with
    a_g = pol[g] / len[g] (mean token log-prob, < 0), P_g = exp(a_g) and log-odds
    lo_g = a_g - log(1 - P_g), mean over the n samples of
        -a_{2s}  +  lam * -log sigmoid(lo_{2s} - lo_{2s+1})
    (the first term is the supervised loss on the chosen response).  Returns (loss, coef) with
    coef[g] = d loss / d policy_logps[g]."""
    pol = np.asarray(policy_logps, dtype=np.float64)
    ln = np.asarray(lengths, dtype=np.float64)
    n = len(pol) // 2
    a = pol / ln
    one_minus_p = -np.expm1(a)                          # 1 - exp(a), accurate near a = 0
    lo = a - np.log(one_minus_p)
    z = lo[0::2] - lo[1::2]
    nls = np.maximum(-z, 0.0) + np.log1p(np.exp(-np.abs(z)))             # -log sigmoid(z)
    sig_neg = np.exp(-np.maximum(z, 0.0)) / (1.0 + np.exp(-np.abs(z)))   # sigmoid(-z)
    loss = float((-a[0::2] + float(lam) * nls).mean())
    dlo_da = 1.0 / one_minus_p                          # d lo / d a
    coef = np.zeros(2 * n, dtype=np.float64)
    coef[0::2] = (-1.0 - float(lam) * sig_neg * dlo_da[0::2]) / (n * ln[0::2])
    coef[1::2] = (+float(lam) * sig_neg * dlo_da[1::2]) / (n * ln[1::2])
    return loss, coef


def dpo_logp_grad(logits, targets, segment_ids, coef, fork_rows=(), fork_targets=(), fork_segments=()):
    """d(sum_g coef[g] * out[g]) / d logits for out = dpo_logp(...): every scored (row t, label y,
    response g) contributes coef[g] * (onehot(y) - softmax(logits[t])) to row t; rows that score
    nothing get zeros."""
    x = np.asarray(logits, dtype=np.float64)
    d = np.zeros_like(x)
    def add(t, y, g):
        if g < 0:
            return
        m = x[t].max()
        p = np.exp(x[t] - m)
        p /= p.sum()
        d[t] -= coef[g] * p
        d[t, int(y)] += coef[g]
    for t in range(x.shape[0]):
        add(t, targets[t], int(segment_ids[t]))
    for r, y, g in zip(fork_rows, fork_targets, fork_segments):
        add(int(r), y, int(g))
    return d


# --------------------------------------------------------------------------
# Packing of prefix-shared units (Section 3.2, Section 4.3.2: first-fit-decreasing)
# --------------------------------------------------------------------------

def ffd_pack(unit_lengths, capacity):
    """First-fit-decreasing bin packing, the textbook algorithm: take the units from the
    longest to the shortest (ties: lower index first) and put each into the first bin, in order
    of creation, that still has room; open a new bin if none has.  Returns bin_of_unit
    (list of bin indices).  A unit longer than the capacity is an error."""
    order = sorted(range(len(unit_lengths)), key=lambda i: (-int(unit_lengths[i]), i))
    free, bin_of = [], [None] * len(unit_lengths)
    for i in order:
        L = int(unit_lengths[i])
        if L > capacity:
            raise ValueError("unit %d of length %d exceeds the capacity %d" % (i, L, capacity))
        for b in range(len(free)):
            if free[b] >= L:
                free[b] -= L
                bin_of[i] = b
                break
        else:
            free.append(capacity - L)
            bin_of[i] = len(free) - 1
    return bin_of


def ffd_pack_layout(prefix_len, chosen_len, rejected_len, capacity, paired=False):
    """The packs a first-fit-decreasing sampler hands to the attention layers (Section 3.2: the
    packing unit is the prompt with both responses; Section 4.3.2).  Units are packed by
    ffd_pack over their lengths, P + C + R in the shared layout and 2P + C + R in the paired
    baseline layout, where a unit is laid out as two sequences (P, C, 0) and (P, R, 0) next to
    each other.  Inside a pack the units stand in the order they were placed (longest first,
    ties by index).  Returns a list of packs, each a dict with cu_seqlens (starting at 0),
    prefix_len, chosen_len, rejected_len and units (source unit of every sample)."""
    n = len(prefix_len)
    unit_len = [(2 if paired else 1) * int(prefix_len[i]) + int(chosen_len[i]) + int(rejected_len[i]) for i in range(n)]
    bin_of = ffd_pack(unit_len, capacity)
    packs = [dict(cu_seqlens=[0], prefix_len=[], chosen_len=[], rejected_len=[], units=[])
             for _ in range(max(bin_of, default=-1) + 1)]
    for i in sorted(range(n), key=lambda i: (-unit_len[i], i)):
        pk = packs[bin_of[i]]
        P, C, R = int(prefix_len[i]), int(chosen_len[i]), int(rejected_len[i])
        for (p, c, r) in ([(P, C, 0), (P, R, 0)] if paired else [(P, C, R)]):
            pk["prefix_len"].append(p)
            pk["chosen_len"].append(c)
            pk["rejected_len"].append(r)
            pk["units"].append(i)
            pk["cu_seqlens"].append(pk["cu_seqlens"][-1] + p + c + r)
    return packs


def optimal_bin_count(unit_lengths, capacity):
    """Fewest bins that hold all units, by exhaustive search (tiny inputs only)."""
    items = sorted((int(x) for x in unit_lengths), reverse=True)
    best = [len(items)]
    def place(k, free):
        if len(free) >= best[0]:
            return
        if k == len(items):
            best[0] = len(free)
            return
        seen = set()
        for b in range(len(free)):
            if free[b] >= items[k] and free[b] not in seen:
                seen.add(free[b])
                free[b] -= items[k]
                place(k + 1, free)
                free[b] += items[k]
        free.append(capacity - items[k])
        place(k + 1, free)
        free.pop()
    place(0, [])
    return best[0]


# --------------------------------------------------------------------------
# Position ids of the shared layout (Section 3.1) and rotary embedding
# --------------------------------------------------------------------------

def position_ids(cu_seqlens, prefix_len, chosen_len, rejected_len):
    """Section 3.1: positions are set so that each response sees the positions it would have
    in the paired format: prompt and chosen tokens count on from the sample start, the
    rejected tokens restart right after the prompt (position P + j for the j-th rejected token)."""
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    pos = np.zeros(int(cu[-1]), dtype=np.int64)
    for s in range(len(cu) - 1):
        P, C, R = int(prefix_len[s]), int(chosen_len[s]), int(rejected_len[s])
        ds = int(cu[s])
        pos[ds:ds + P + C] = np.arange(P + C)
        pos[ds + P + C:ds + P + C + R] = P + np.arange(R)
    return pos


def rope(x, pos, theta=10000.0):
    """Rotary position embedding, "rotate-half" convention (the one Llama-family models use):
    with x = [x1 | x2] split at d/2 and angle_i = pos * theta^(-2i/d),
        y1 = x1 cos - x2 sin,   y2 = x2 cos + x1 sin.
    x [T, H, d] float64, pos [T]."""
    x = np.asarray(x, dtype=np.float64)
    T, H, d = x.shape
    inv_freq = float(theta) ** (-np.arange(0, d, 2, dtype=np.float64) / d)      # [d/2]
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv_freq[None, :]        # [T, d/2]
    cos, sin = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., : d // 2], x[..., d // 2:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


# --------------------------------------------------------------------------
# One attention layer on the shared layout (Section 4.2: the full attention-layer benchmark)
# --------------------------------------------------------------------------

def attention_layer_fwd(x, wq, wk, wv, wo, pos, mask, n_q_heads, n_kv_heads, theta=10000.0, softmax_scale=None):
    """Query / key / value projections, rotary embedding with the shared layout's position ids,
    attention under the mask, output projection, all in float64:
        q = rope(x wq), k = rope(x wk), v = x wv, o = attention(q, k, v), out = o wo.
    x [T, hidden]; wq [hidden, Hq d]; wk, wv [hidden, Hkv d]; wo [Hq d, hidden].
    Returns (out [T, hidden], cache) where cache holds what the backward needs."""
    x, wq, wk, wv, wo = (_as_f64(a) for a in (x, wq, wk, wv, wo))
    T = x.shape[0]
    d = wq.shape[1] // n_q_heads
    q = rope((x @ wq).reshape(T, n_q_heads, d), pos, theta)
    k = rope((x @ wk).reshape(T, n_kv_heads, d), pos, theta)
    v = (x @ wv).reshape(T, n_kv_heads, d)
    o, lse = attention_fwd(q, k, v, mask, softmax_scale)
    out = o.reshape(T, n_q_heads * d) @ wo
    return out, dict(q=q, k=k, v=v, o=o, lse=lse)


def attention_layer_bwd(x, wq, wk, wv, wo, pos, mask, n_q_heads, n_kv_heads, d_out, theta=10000.0,
                        softmax_scale=None):
    """Gradient of sum(out * d_out) for attention_layer_fwd with respect to x and the four weight
    matrices.  The rotary embedding is a rotation per position, so a gradient passes back
    through it by the inverse rotation (the same formula with the negated position).
    Returns dict(dx, dwq, dwk, dwv, dwo)."""
    x, wq, wk, wv, wo, d_out = (_as_f64(a) for a in (x, wq, wk, wv, wo, d_out))
    T = x.shape[0]
    d = wq.shape[1] // n_q_heads
    out, c = attention_layer_fwd(x, wq, wk, wv, wo, pos, mask, n_q_heads, n_kv_heads, theta, softmax_scale)
    o2 = c["o"].reshape(T, n_q_heads * d)
    dwo = o2.T @ d_out
    d_o = (d_out @ wo.T).reshape(T, n_q_heads, d)
    dq, dk, dv = attention_bwd(c["q"], c["k"], c["v"], d_o, mask, softmax_scale)
    neg = -np.asarray(pos, dtype=np.float64)
    dq2 = rope(dq, neg, theta).reshape(T, -1)
    dk2 = rope(dk, neg, theta).reshape(T, -1)
    dv2 = dv.reshape(T, -1)
    return dict(dx=dq2 @ wq.T + dk2 @ wk.T + dv2 @ wv.T, dwq=x.T @ dq2, dwk=x.T @ dk2, dwv=x.T @ dv2, dwo=dwo)
