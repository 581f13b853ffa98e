"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The dense oracle cannot do a 16k-32k token pack for 32 heads in seconds.  Attention never
crosses a sample boundary (the oracle's own tests pin that), so the oracle is run sample by
sample: (1) on whole samples for one kv-head group, every element; (2) over the whole pack
and all heads on sampled outputs it can compute one by one: forward rows of every sample
(random rows, every prompt / chosen / rejected boundary, tile edges), and on the longest
sample, where the tile lists are longest, gradients of sampled query rows and of key
positions in the tails of the responses (the oracle's per-row / per-column form).
"""
import numpy as np
import pytest
import torch

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import binding as B
from paper_2410_20305_b200 import workloads as wl
from paper_2410_20305_b200.labels import logp_labels

from gpu_util import TOL_LOGP, TOL_LSE, TOL_O, device_plan, grad_errors, max_abs, read_status

pytestmark = pytest.mark.gpu
VOCAB = 128256


def _sample_views(pack, s, tensors, heads, kv_heads):
    lo, hi = int(pack.cu_seqlens[s]), int(pack.cu_seqlens[s + 1])
    q, k, v, d_o = tensors
    f = wl.to_f64
    return lo, hi, f(q[lo:hi, heads]), f(k[lo:hi, kv_heads]), f(v[lo:hi, kv_heads]), f(d_o[lo:hi, heads])


@pytest.mark.parametrize("workload", [1, 2, 3, 4])
def test_attention_on_the_bench_packs(workload):
    pack = wl.config_pack(workload)
    Hq, Hkv, d = pack.n_q_heads, pack.n_kv_heads, pack.head_dim
    g = Hq // Hkv
    q, k, v, d_o = wl.attention_inputs(pack, 2000 + workload)
    plan = device_plan(pack)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    qd, kd, vd, dod = q.cuda(), k.cuda(), v.cuda(), d_o.cuda()
    o, lse = B.psa_fwd(plan, qd, kd, vd, status=status)
    dq, dk, dv = B.psa_bwd(plan, dod, qd, kd, vd, o, lse, status=status)
    fq, fk, fv = B.psa_bwd_f32(plan, dod, qd, kd, vd, o, lse, status=status)
    assert read_status(status) == 0
    o, lse, dq, dk, dv, fq, fk, fv = (t.cpu() for t in (o, lse, dq, dk, dv, fq, fk, fv))
    del qd, kd, vd, dod

    lens = pack.cu_seqlens[1:] - pack.cu_seqlens[:-1]
    rng = np.random.default_rng(workload)

    # ---- (1) whole samples, one kv-head group each, every element (dense oracle)
    small = [s for s in np.argsort(lens) if lens[s] <= 3000]
    picks = sorted({int(small[0]), int(small[-1]), int(rng.choice(small))})
    for s in picks:
        hk = int(rng.integers(0, Hkv))
        hs = slice(hk * g, hk * g + g)
        lo, hi, sq, sk, sv, sdo = _sample_views(pack, s, (q, k, v, d_o), hs, slice(hk, hk + 1))
        P, C, R = (int(x[s]) for x in (pack.prefix_len, pack.chosen_len, pack.rejected_len))
        mask = orc.packed_mask([0, hi - lo], [P], [C], [R])
        ro, rl = orc.attention_fwd(sq, sk, sv, mask)
        rdq, rdk, rdv = orc.attention_bwd(sq, sk, sv, sdo, mask)
        eo, el = max_abs(o[lo:hi, hs], ro), max_abs(lse[hs, lo:hi], rl)
        assert eo <= TOL_O and el <= TOL_LSE, (workload, s, eo, el)
        for name, got, got32, ref in (("dq", dq[lo:hi, hs], fq[lo:hi, hs], rdq),
                                      ("dk", dk[lo:hi, hk:hk + 1], fk[lo:hi, hk:hk + 1], rdk),
                                      ("dv", dv[lo:hi, hk:hk + 1], fv[lo:hi, hk:hk + 1], rdv)):
            raw, raw_small, excess = grad_errors(got, ref)
            assert raw_small <= TOL_O and excess <= TOL_O, (workload, s, name, raw, raw_small, excess)
            raw32 = max_abs(got32, ref)          # fp32 outputs: the gate as stated, raw, on every element
            print("workload %d sample %d %s: raw max abs error bf16 out %.4f, fp32 out %.4f" % (workload, s, name, raw, raw32))
            assert raw32 <= TOL_O, (workload, s, name, raw32)

    # ---- (2) sampled over the WHOLE pack and ALL heads: forward rows (random rows of every sample and
    # every boundary row), and on the longest sample gradients of sampled rows (dq) and of key positions
    # in the tails of the two responses (dk, dv), where the oracle needs only the rows that see them.
    all_q, all_kv = slice(0, Hq), slice(0, Hkv)
    longest = int(np.argmax(lens))
    for s in range(pack.n_samples):
        lo, hi, sq, sk, sv, sdo = _sample_views(pack, s, (q, k, v, d_o), all_q, all_kv)
        L = hi - lo
        P, C, R = (int(x[s]) for x in (pack.prefix_len, pack.chosen_len, pack.rejected_len))
        edge = [0, 1, 127, 128, P - 1, P, P + C - 1, P + C, L - 1, (L - 1) // 128 * 128, (L - 1) // 128 * 128 - 1]
        rows = np.unique(np.clip(np.concatenate([edge, rng.integers(0, L, 14 if s != longest else 40)]), 0, L - 1))
        mask = orc.packed_mask([0, L], [P], [C], [R])
        cols = np.zeros(0, dtype=np.int64)
        need = rows
        if s == longest:
            tail = lambda a, b: np.unique(np.clip(np.concatenate([[b - 1, max(a, b - 64)], rng.integers(max(a, b - 64), max(b, a + 1), 6)]), a, max(a, b - 1)))
            cols = np.unique(np.concatenate([tail(P, P + C) if C else [], tail(P + C, L) if R else []]).astype(np.int64))
            need = np.unique(np.concatenate([rows, np.nonzero(mask[:, cols].any(axis=1))[0]]))
        ro, rl = orc.attention_rows(sq, sk, sv, mask[need], need)
        at = np.searchsorted(need, rows)
        eo, el = max_abs(o[lo:hi][rows], ro[at]), max_abs(lse[:, lo:hi][:, rows], rl[:, at])
        assert eo <= TOL_O and el <= TOL_LSE, (workload, s, "sampled rows", eo, el)
        if s != longest:
            continue
        full_o = np.zeros((L, Hq, d)); full_l = np.zeros((Hq, L))
        full_o[need], full_l[:, need] = ro, rl
        rdq, rdk, rdv = orc.attention_bwd_sampled(sq, sk, sv, sdo, full_o, full_l, mask, rows, cols)
        for name, got, got32, ref in (("dq", dq[lo:hi][rows], fq[lo:hi][rows], rdq), ("dk", dk[lo:hi][cols], fk[lo:hi][cols], rdk),
                                      ("dv", dv[lo:hi][cols], fv[lo:hi][cols], rdv)):
            raw, raw_small, excess = grad_errors(got, ref)
            raw32 = max_abs(got32, ref)
            print("workload %d longest sample (%d tokens) %s, all heads, sampled: raw bf16 out %.4f, fp32 out %.4f"
                  % (workload, L, name, raw, raw32))
            assert raw_small <= TOL_O and excess <= TOL_O and raw32 <= TOL_O, (workload, name, raw, raw_small, excess, raw32)

    # ---- (2b) the short-many pack is small enough for the dense oracle on every sample and ALL heads:
    # every element of every output of the whole pack
    if workload == 4:
        worst = {}
        for s in range(pack.n_samples):
            lo, hi, sq, sk, sv, sdo = _sample_views(pack, s, (q, k, v, d_o), all_q, all_kv)
            P, C, R = (int(x[s]) for x in (pack.prefix_len, pack.chosen_len, pack.rejected_len))
            mask = orc.packed_mask([0, hi - lo], [P], [C], [R])
            ro, rl = orc.attention_fwd(sq, sk, sv, mask)
            rdq, rdk, rdv = orc.attention_bwd(sq, sk, sv, sdo, mask)
            assert max_abs(o[lo:hi], ro) <= TOL_O and max_abs(lse[:, lo:hi], rl) <= TOL_LSE, (s, "whole pack")
            for name, got, got32, ref in (("dq", dq[lo:hi], fq[lo:hi], rdq), ("dk", dk[lo:hi], fk[lo:hi], rdk),
                                          ("dv", dv[lo:hi], fv[lo:hi], rdv)):
                raw, raw_small, excess = grad_errors(got, ref)
                raw32 = max_abs(got32, ref)
                worst[name] = max(worst.get(name, 0.0), raw32)
                assert raw_small <= TOL_O and excess <= TOL_O and raw32 <= TOL_O, (s, name, raw, raw_small, excess, raw32)
        print("workload 4, whole pack, all heads, every element: worst raw error of the fp32 gradients", worst)

    # ---- (3) properties that hold at any size: finite everywhere, lse >= the row's own score
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    assert all(torch.isfinite(t.float()).all() for t in (dq, dk, dv, fq, fk, fv))
    own = (q.float() * k.float().repeat_interleave(g, dim=1)).sum(-1).t() * d ** -0.5     # [Hq, T]
    assert (lse + 1e-3 >= own).all()


def test_paired_layout_of_a_bench_pack():
    """The unshared baseline layout (Algorithm 2) through the same kernels."""
    pack = wl.config_pack(4).paired()
    q, k, v, d_o = wl.attention_inputs(pack, 77)
    plan = device_plan(pack)
    o, lse = B.psa_fwd(plan, q.cuda(), k.cuda(), v.cuda())
    dq, dk, dv = B.psa_bwd(plan, d_o.cuda(), q.cuda(), k.cuda(), v.cuda(), o, lse)
    s, hk, g = 3, 2, 4
    lo, hi = int(pack.cu_seqlens[s]), int(pack.cu_seqlens[s + 1])
    hs = slice(hk * g, hk * g + g)
    rid = np.zeros(hi - lo, dtype=np.int64)
    mask = orc.paired_packing_mask(rid)           # one causal sequence
    f = wl.to_f64
    ro, rl = orc.attention_fwd(f(q[lo:hi, hs]), f(k[lo:hi, hk:hk + 1]), f(v[lo:hi, hk:hk + 1]), mask)
    rdq, rdk, rdv = orc.attention_bwd(f(q[lo:hi, hs]), f(k[lo:hi, hk:hk + 1]), f(v[lo:hi, hk:hk + 1]), f(d_o[lo:hi, hs]), mask)
    assert max_abs(o.cpu()[lo:hi, hs], ro) <= TOL_O and max_abs(lse.cpu()[hs, lo:hi], rl) <= TOL_LSE
    for got, ref in ((dq.cpu()[lo:hi, hs], rdq), (dk.cpu()[lo:hi, hk:hk + 1], rdk), (dv.cpu()[lo:hi, hk:hk + 1], rdv)):
        raw, raw_small, excess = grad_errors(got, ref)
        assert raw_small <= TOL_O and excess <= TOL_O, (raw, raw_small, excess)


def test_dpo_logp_at_full_vocab_on_the_multi_turn_pack():
    pack = wl.config_pack(3)
    T = pack.total_tokens
    gen = torch.Generator(device="cuda").manual_seed(5)
    logits = torch.empty((T, VOCAB), dtype=torch.bfloat16, device="cuda")
    for lo in range(0, T, 2048):
        hi = min(T, lo + 2048)
        logits[lo:hi] = (torch.randn((hi - lo, VOCAB), generator=gen, device="cuda") * 3.0 ** 0.5).to(torch.bfloat16)
    tok = torch.randint(0, VOCAB, (T,), generator=gen, device="cuda", dtype=torch.int32).cpu().numpy()
    targets, seg, fr, ft, fs = logp_labels(tok, pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    dev = lambda a: torch.as_tensor(np.asarray(a, dtype=np.int32)).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = B.dpo_logp(logits, dev(targets), dev(seg), 2 * pack.n_samples, dev(fr), dev(ft), dev(fs), status=status)
    assert read_status(status) == 0
    out = out.cpu().double().numpy()
    # every response: token count x (about -ln V - 1.5) is the right order of magnitude
    n_tok = np.bincount(np.concatenate([seg[seg >= 0], fs]), minlength=2 * pack.n_samples)
    assert np.all(out < 0) and np.allclose(out / n_tok, -(np.log(VOCAB) + 1.5), atol=0.5)
    # four responses recomputed by the oracle from the rows they score
    for gseg in (0, 1, 2 * pack.n_samples - 1, pack.n_samples):
        rows = np.nonzero(seg == gseg)[0]
        forks = [i for i in range(len(fr)) if fs[i] == gseg]
        want = 0.0
        for chunk in np.array_split(rows, max(1, len(rows) // 64)):
            x = wl.to_f64(logits[torch.as_tensor(chunk).cuda()])
            want += sum(orc.row_logprob(x[i], targets[t]) for i, t in enumerate(chunk))
        for i in forks:
            want += orc.row_logprob(wl.to_f64(logits[int(fr[i])]), ft[i])
        assert abs(out[gseg] - want) <= TOL_LOGP * abs(want), (gseg, out[gseg], want)
