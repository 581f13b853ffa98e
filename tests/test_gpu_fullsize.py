"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The dense oracle cannot do a 16k-32k token pack for 32 heads in seconds, so whole samples
of the pack are checked instead: attention never crosses a sample boundary (the oracle's
own tests pin that), hence the oracle run on one sample alone, for one kv-head group,
must reproduce the GPU's outputs on that sample's rows and heads.
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


@pytest.mark.parametrize("workload", [1, 2, 3, 4])
def test_attention_on_whole_samples_of_the_bench_packs(workload):
    pack = wl.config_pack(workload)
    Hq, Hkv, d = pack.n_q_heads, pack.n_kv_heads, pack.head_dim
    g = Hq // Hkv
    q, k, v, d_o = wl.attention_inputs(pack, 2000 + workload)
    plan = device_plan(pack)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    qd, kd, vd, dod = q.cuda(), k.cuda(), v.cuda(), d_o.cuda()
    o, lse = B.psa_fwd(plan, qd, kd, vd, status=status)
    dq, dk, dv = B.psa_bwd(plan, dod, qd, kd, vd, o, lse, status=status)
    assert read_status(status) == 0
    o, lse, dq, dk, dv = (t.cpu() for t in (o, lse, dq, dk, dv))

    lens = pack.cu_seqlens[1:] - pack.cu_seqlens[:-1]
    rng = np.random.default_rng(workload)
    small = [s for s in np.argsort(lens) if lens[s] <= 3000]
    picks = sorted({int(small[0]), int(small[-1]), int(rng.choice(small))})
    for s in picks:
        hk = int(rng.integers(0, Hkv))
        lo, hi = int(pack.cu_seqlens[s]), int(pack.cu_seqlens[s + 1])
        hs = slice(hk * g, hk * g + g)
        P, C, R = (int(x[s]) for x in (pack.prefix_len, pack.chosen_len, pack.rejected_len))
        mask = orc.packed_mask([0, hi - lo], [P], [C], [R])
        f = wl.to_f64
        sq, sk, sv, sdo = f(q[lo:hi, hs]), f(k[lo:hi, hk:hk + 1]), f(v[lo:hi, hk:hk + 1]), f(d_o[lo:hi, hs])
        ro, rl = orc.attention_fwd(sq, sk, sv, mask)
        rdq, rdk, rdv = orc.attention_bwd(sq, sk, sv, sdo, mask)
        eo, el = max_abs(o[lo:hi, hs], ro), max_abs(lse[hs, lo:hi], rl)
        assert eo <= TOL_O and el <= TOL_LSE, (workload, s, eo, el)
        for name, got, ref in (("dq", dq[lo:hi, hs], rdq), ("dk", dk[lo:hi, hk:hk + 1], rdk), ("dv", dv[lo:hi, hk:hk + 1], rdv)):
            raw, raw_small, excess = grad_errors(got, ref)
            assert raw_small <= TOL_O and excess <= TOL_O, (workload, s, name, raw, raw_small, excess)
    # properties that hold at any size: finite everywhere, lse >= the row's own score
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    assert all(torch.isfinite(t.float()).all() for t in (dq, dk, dv))
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
