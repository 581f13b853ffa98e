"""Pins for the oracle's attention forward and backward.

The main pin is the equivalence the paper states in Section 3.1: attention in
the shared layout equals ordinary causal attention on [prompt|chosen] and on
[prompt|rejected].  The ordinary causal attention and its gradient come from
torch (scaled_dot_product_attention + autograd, float64, CPU), an independent
library routine.
"""
import numpy as np
import pytest
import torch

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import workloads as wl


def _torch_causal(q, k, v, d_o, scale):
    """q,k,v,d_o: [L,H,d] float64 numpy (MHA).  Returns o, lse, dq, dk, dv."""
    tq, tk, tv = (torch.tensor(x).permute(1, 0, 2).contiguous().requires_grad_(True) for x in (q, k, v))
    o = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=scale)
    o.backward(torch.tensor(d_o).permute(1, 0, 2))
    L = q.shape[0]
    s = torch.einsum("hqd,hkd->hqk", tq.detach(), tk.detach()) * scale
    s = s.masked_fill(~torch.tril(torch.ones(L, L, dtype=torch.bool)), float("-inf"))
    lse = torch.logsumexp(s, dim=-1)
    back = lambda t: t.permute(1, 0, 2).numpy()
    return back(o.detach()), lse.numpy(), back(tq.grad), back(tk.grad), back(tv.grad)


def _expand_kv(x, g):
    return np.repeat(x, g, axis=1)


def _check_invariant(pack, seed, tol=1e-11):
    q, k, v, d_o = (wl.to_f64(t) for t in wl.attention_inputs(pack, seed))
    Hq, Hkv, d = pack.n_q_heads, pack.n_kv_heads, pack.head_dim
    g = Hq // Hkv
    scale = 1.0 / np.sqrt(d)
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    o, lse = orc.attention_fwd(q, k, v, mask, scale)
    dq, dk, dv = orc.attention_bwd(q, k, v, d_o, mask, scale)
    worst = 0.0
    for s in range(pack.n_samples):
        ds = int(pack.cu_seqlens[s]); P = int(pack.prefix_len[s]); C = int(pack.chosen_len[s]); R = int(pack.rejected_len[s])
        ia = np.arange(ds, ds + P + C)
        ib = np.concatenate([np.arange(ds, ds + P), np.arange(ds + P + C, ds + P + C + R)])
        exp_dq = np.zeros((P + C + R, Hq, d)); exp_dk = np.zeros((P + C + R, Hkv, d)); exp_dv = np.zeros_like(exp_dk)
        for idx, zero_prompt in ((ia, False), (ib, True)):
            if len(idx) == 0:
                continue
            dd = d_o[idx].copy()
            if zero_prompt:
                dd[:P] = 0.0          # the prompt rows' outputs belong to the [prompt|chosen] run
            ro, rl, rdq, rdk, rdv = _torch_causal(q[idx], _expand_kv(k[idx], g), _expand_kv(v[idx], g), dd, scale)
            rows = slice(P, None) if zero_prompt else slice(None)
            worst = max(worst, np.abs(o[idx][rows] - ro[rows]).max(initial=0.0))
            worst = max(worst, np.abs(lse[:, idx][:, rows] - rl[:, rows]).max(initial=0.0))
            exp_dq[idx - ds] += rdq
            exp_dk[idx - ds] += rdk.reshape(len(idx), Hkv, g, d).sum(axis=2)
            exp_dv[idx - ds] += rdv.reshape(len(idx), Hkv, g, d).sum(axis=2)
        sl = slice(ds, ds + P + C + R)
        worst = max(worst, np.abs(dq[sl] - exp_dq).max(), np.abs(dk[sl] - exp_dk).max(), np.abs(dv[sl] - exp_dv).max())
    assert worst < tol, worst


def test_paired_format_equivalence_tiny_config():
    _check_invariant(wl.config_pack(0), seed=0)


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_paired_format_equivalence_random_gqa(seed):
    _check_invariant(wl.random_pack(seed, 3, 24, 4, 2, 16), seed)


def test_paired_format_equivalence_degenerate_lengths():
    pack = wl.pack_from_lengths("deg", [(0, 5, 4), (6, 0, 3), (4, 7, 0), (1, 1, 1), (3, 0, 0)], 2, 1, 8)
    _check_invariant(pack, seed=7)


def test_zero_query_closed_form():
    """q = 0: every allowed key has the same weight, so lse = ln(count) and o is
    the mean of the allowed v rows."""
    pack = wl.random_pack(21, 3, 15, 2, 1, 8)
    q, k, v, _ = (wl.to_f64(t) for t in wl.attention_inputs(pack, 5))
    q[:] = 0.0
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    o, lse = orc.attention_fwd(q, k, v, mask)
    for s in range(pack.n_samples):
        ds = int(pack.cu_seqlens[s]); P = int(pack.prefix_len[s]); C = int(pack.chosen_len[s])
        cs, rs = ds + P, ds + P + C
        for t in range(ds, int(pack.cu_seqlens[s + 1])):
            keys = list(range(ds, t + 1)) if t < rs else list(range(ds, cs)) + list(range(rs, t + 1))
            assert np.allclose(lse[:, t], np.log(len(keys)), atol=1e-13)
            assert np.allclose(o[t, :, :], v[keys, 0, :].mean(axis=0)[None, :], atol=1e-13)


def test_first_row_of_each_sample():
    pack = wl.random_pack(22, 3, 10, 2, 2, 8, allow_zero=False)
    q, k, v, _ = (wl.to_f64(t) for t in wl.attention_inputs(pack, 6))
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    scale = 0.3
    o, lse = orc.attention_fwd(q, k, v, mask, scale)
    for s in range(pack.n_samples):
        t = int(pack.cu_seqlens[s])
        assert np.allclose(o[t], v[t], atol=1e-14)
        assert np.allclose(lse[:, t], scale * (q[t] * k[t]).sum(-1), atol=1e-13)


def test_backward_finite_differences():
    pack = wl.pack_from_lengths("fd", [(3, 2, 2), (2, 3, 1)], 2, 1, 4)
    q, k, v, d_o = (wl.to_f64(t) for t in wl.attention_inputs(pack, 9))
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    scale = 0.5
    dq, dk, dv = orc.attention_bwd(q, k, v, d_o, mask, scale)
    loss = lambda a, b, c: float((orc.attention_fwd(a, b, c, mask, scale)[0] * d_o).sum())
    eps = 1e-6
    rng = np.random.default_rng(0)
    for name, x, gx in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(12):
            idx = tuple(int(rng.integers(0, n)) for n in x.shape)
            xp = x.copy(); xm = x.copy()
            xp[idx] += eps; xm[idx] -= eps
            args_p = {"q": (xp, k, v), "k": (q, xp, v), "v": (q, k, xp)}[name]
            args_m = {"q": (xm, k, v), "k": (q, xm, v), "v": (q, k, xm)}[name]
            fd = (loss(*args_p) - loss(*args_m)) / (2 * eps)
            assert abs(fd - gx[idx]) < 1e-7, (name, idx, fd, gx[idx])


def test_swapping_chosen_and_rejected_permutes_outputs():
    """Which response is called chosen must not matter to either response."""
    P, C, R, H, d = 6, 4, 5, 2, 8
    a = wl.pack_from_lengths("a", [(P, C, R)], H, H, d)
    b = wl.pack_from_lengths("b", [(P, R, C)], H, H, d)
    q, k, v, d_o = (wl.to_f64(t) for t in wl.attention_inputs(a, 4))
    perm = np.concatenate([np.arange(P), np.arange(P + C, P + C + R), np.arange(P, P + C)])
    ma = orc.packed_mask(a.cu_seqlens, a.prefix_len, a.chosen_len, a.rejected_len)
    mb = orc.packed_mask(b.cu_seqlens, b.prefix_len, b.chosen_len, b.rejected_len)
    oa, la = orc.attention_fwd(q, k, v, ma)
    ob, lb = orc.attention_fwd(q[perm], k[perm], v[perm], mb)
    assert np.allclose(oa[perm], ob, atol=1e-13) and np.allclose(la[:, perm], lb, atol=1e-13)
    ga = orc.attention_bwd(q, k, v, d_o, ma)
    gb = orc.attention_bwd(q[perm], k[perm], v[perm], d_o[perm], mb)
    for x, y in zip(ga, gb):
        assert np.allclose(x[perm], y, atol=1e-12)


def test_packing_is_independent_per_sample_and_rows_variant():
    pack = wl.random_pack(31, 3, 14, 4, 2, 8)
    q, k, v, d_o = (wl.to_f64(t) for t in wl.attention_inputs(pack, 8))
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    o, lse = orc.attention_fwd(q, k, v, mask)
    dq, dk, dv = orc.attention_bwd(q, k, v, d_o, mask)
    for s in range(pack.n_samples):
        lo, hi = int(pack.cu_seqlens[s]), int(pack.cu_seqlens[s + 1])
        m1 = orc.packed_mask([0, hi - lo], pack.prefix_len[s:s + 1], pack.chosen_len[s:s + 1], pack.rejected_len[s:s + 1])
        o1, l1 = orc.attention_fwd(q[lo:hi], k[lo:hi], v[lo:hi], m1)
        g1 = orc.attention_bwd(q[lo:hi], k[lo:hi], v[lo:hi], d_o[lo:hi], m1)
        assert np.allclose(o[lo:hi], o1, atol=1e-13) and np.allclose(lse[:, lo:hi], l1, atol=1e-13)
        for x, y in zip((dq, dk, dv), g1):
            assert np.allclose(x[lo:hi], y, atol=1e-12)
    rows = np.array([0, 3, pack.total_tokens - 1])
    o2, l2 = orc.attention_rows(q, k, v, mask[rows], rows)
    assert np.allclose(o2, o[rows], atol=1e-14) and np.allclose(l2, lse[:, rows], atol=1e-14)


def test_sampled_gradient_equals_the_dense_gradient_on_its_rows_and_columns():
    # attention_bwd_sampled is the per-row / per-column form of attention_bwd: same numbers
    pack = wl.pack_from_lengths("s", [(70, 33, 21), (5, 0, 40), (64, 64, 0)], 4, 2, 16)
    q, k, v, d_o = (wl.to_f64(t) for t in wl.attention_inputs(pack, 12))
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    o, lse = orc.attention_fwd(q, k, v, mask)
    dq, dk, dv = orc.attention_bwd(q, k, v, d_o, mask)
    T = pack.total_tokens
    rows = np.array([0, 1, 69, 70, 102, 103, 123, 124, 128, 168, 169, T - 1])
    cols = np.array([0, 5, 69, 70, 100, 110, 124, 125, 160, 232, T - 1])
    # the forward for all rows, chunk by chunk, is the forward
    parts = [orc.attention_rows(q, k, v, mask[r0:r0 + 50], np.arange(r0, min(T, r0 + 50))) for r0 in range(0, T, 50)]
    o2 = np.concatenate([p[0] for p in parts], axis=0)
    lse2 = np.concatenate([p[1] for p in parts], axis=1)
    assert np.abs(o2 - o).max() < 1e-14 and np.abs(lse2 - lse).max() < 1e-13
    sq, sk, sv = orc.attention_bwd_sampled(q, k, v, d_o, o2, lse2, mask, rows, cols)
    assert np.abs(sq - dq[rows]).max() < 1e-13
    assert np.abs(sk - dk[cols]).max() < 1e-13 and np.abs(sv - dv[cols]).max() < 1e-13


def test_sampled_backward_needs_the_forward_only_on_the_rows_that_see_the_sampled_keys():
    """The full-size GPU tests call attention_bwd_sampled with o and lse filled in only on the
    sampled query rows and on the rows that see a sampled key (zeros elsewhere): the result must
    be the dense gradient at those rows and key positions."""
    pack = wl.pack_from_lengths("s", [(37, 21, 30)], 4, 2, 16)
    q, k, v, d_o = (wl.to_f64(t) for t in wl.attention_inputs(pack, 12))
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    dq, dk, dv = orc.attention_bwd(q, k, v, d_o, mask)
    rows = np.array([0, 5, 36, 37, 57, 58, 87])
    cols = np.array([50, 57, 80, 87])                      # tails of the chosen and of the rejected response
    need = np.unique(np.concatenate([rows, np.nonzero(mask[:, cols].any(axis=1))[0]]))
    assert len(need) < pack.total_tokens - 20              # far from all rows
    o, lse = np.zeros_like(q), np.zeros((4, pack.total_tokens))
    o[need], lse[:, need] = orc.attention_rows(q, k, v, mask[need], need)
    sdq, sdk, sdv = orc.attention_bwd_sampled(q, k, v, d_o, o, lse, mask, rows, cols)
    assert np.allclose(sdq, dq[rows], atol=1e-12)
    assert np.allclose(sdk, dk[cols], atol=1e-12) and np.allclose(sdv, dv[cols], atol=1e-12)
