"""Pins for the oracle's DPO loss (Eq. 1) and its gradient into the logits."""
import numpy as np
import torch

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import workloads as wl
from paper_2410_20305_b200.labels import logp_labels


def test_loss_closed_forms():
    # equal policy and reference: margin 0 -> loss = ln 2, gradient = -/+ beta / (2 n)
    pol = np.array([-3.0, -5.0, -1.0, -2.0]); ref = pol.copy()
    loss, coef = orc.dpo_loss(pol, ref, beta=0.1)
    assert abs(loss - np.log(2.0)) < 1e-15
    assert np.allclose(coef, [-0.025, 0.025, -0.025, 0.025], atol=1e-16)
    # a very large positive margin: loss -> 0, gradient -> 0; very negative: loss -> -beta*margin
    loss, coef = orc.dpo_loss([1000.0, 0.0], [0.0, 0.0], beta=1.0)
    assert loss < 1e-300 and abs(coef).max() < 1e-300
    loss, coef = orc.dpo_loss([-1000.0, 0.0], [0.0, 0.0], beta=0.5)
    assert abs(loss - 500.0) < 1e-9 and np.allclose(coef, [-0.5, 0.5])


def test_loss_matches_torch_logsigmoid_and_autograd():
    rng = np.random.default_rng(0)
    pol = rng.normal(-40, 10, size=12); ref = rng.normal(-40, 10, size=12)
    tp = torch.tensor(pol, requires_grad=True)
    margin = (tp[0::2] - torch.tensor(ref[0::2])) - (tp[1::2] - torch.tensor(ref[1::2]))
    tl = -torch.nn.functional.logsigmoid(0.3 * margin).mean()
    tl.backward()
    loss, coef = orc.dpo_loss(pol, ref, 0.3)
    assert abs(loss - tl.item()) < 1e-13 and np.allclose(coef, tp.grad.numpy(), atol=1e-15)


def test_logit_gradient_matches_torch_autograd_through_the_whole_chain():
    pack = wl.pack_from_lengths("g", [(4, 3, 2), (0, 2, 3), (3, 0, 2), (2, 2, 0), (1, 1, 1)], 1, 1, 8)
    T, V = pack.total_tokens, 23
    x, tok = wl.logits_and_tokens(T, V, seed=4, std=1.3)
    targets, seg, fr, ft, fs = logp_labels(tok.numpy(), pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    n_seg = 2 * pack.n_samples
    ref_lp = np.random.default_rng(1).normal(-8, 2, size=n_seg)
    tx = x.double().clone().requires_grad_(True)
    lsm = torch.log_softmax(tx, dim=-1)
    out = torch.zeros(n_seg, dtype=torch.float64)
    for t in range(T):
        if seg[t] >= 0:
            out[seg[t]] = out[seg[t]] + lsm[t, int(targets[t])]
    for r, y, g in zip(fr, ft, fs):
        out[g] = out[g] + lsm[int(r), int(y)]
    margin = (out[0::2] - torch.tensor(ref_lp[0::2])) - (out[1::2] - torch.tensor(ref_lp[1::2]))
    (-torch.nn.functional.logsigmoid(0.25 * margin).mean()).backward()
    lp = orc.dpo_logp(wl.to_f64(x), targets, seg, n_seg, fr, ft, fs)
    assert np.allclose(lp, out.detach().numpy(), atol=1e-12)
    loss, coef = orc.dpo_loss(lp, ref_lp, 0.25)
    got = orc.dpo_logp_grad(wl.to_f64(x), targets, seg, coef, fr, ft, fs)
    assert np.allclose(got, tx.grad.numpy(), atol=1e-14)
    # rows that score nothing have zero gradient; every row's gradient sums to zero
    dead = (seg < 0) & ~np.isin(np.arange(T), fr)
    assert (got[dead] == 0).all() and np.abs(got.sum(axis=1)).max() < 1e-14


def test_logit_gradient_finite_differences():
    x = np.random.default_rng(2).normal(size=(5, 7))
    targets = np.array([1, 6, 0, 3, 2]); seg = np.array([0, 0, -1, 1, 1])
    coef = np.array([0.7, -0.4])
    g = orc.dpo_logp_grad(x, targets, seg, coef, [1], [4], [1])
    f = lambda z: float(coef @ orc.dpo_logp(z, targets, seg, 2, [1], [4], [1]))
    eps = 1e-6
    for idx in [(0, 1), (1, 4), (1, 6), (2, 3), (4, 0)]:
        zp = x.copy(); zm = x.copy(); zp[idx] += eps; zm[idx] -= eps
        assert abs((f(zp) - f(zm)) / (2 * eps) - g[idx]) < 1e-8


def test_simpo_loss_closed_forms_and_reduction_to_dpo():
    # equal length-normalised log-probs, gamma 0: loss = ln 2; with gamma: -log sigmoid(-gamma)
    pol = np.array([-6.0, -9.0, -1.0, -2.0]); ln = np.array([2, 3, 5, 10])
    loss, coef = orc.simpo_loss(pol, ln, beta=2.0, gamma=0.0)
    assert abs(loss - np.log(2.0)) < 1e-15
    assert np.allclose(coef, [-2.0 / (2 * 2 * 2), 2.0 / (2 * 2 * 3), -2.0 / (2 * 2 * 5), 2.0 / (2 * 2 * 10)], atol=1e-16)
    loss, _ = orc.simpo_loss(pol, ln, beta=2.0, gamma=0.7)
    assert abs(loss - np.log1p(np.exp(0.7))) < 1e-15
    # unit lengths, zero reference, gamma 0: the DPO loss of Eq. 1 (pinned above on its own)
    rng = np.random.default_rng(3)
    pol = rng.normal(-30, 8, size=10)
    l1, c1 = orc.simpo_loss(pol, np.ones(10), 0.4, 0.0)
    l2, c2 = orc.dpo_loss(pol, np.zeros(10), 0.4)
    assert abs(l1 - l2) < 1e-15 and np.allclose(c1, c2, atol=1e-16)


def test_simpo_loss_matches_torch_autograd():
    rng = np.random.default_rng(5)
    pol = rng.normal(-60, 20, size=14); ln = rng.integers(1, 90, size=14)
    tp = torch.tensor(pol, requires_grad=True)
    tl_ = torch.tensor(ln, dtype=torch.float64)
    z = 2.5 * (tp[0::2] / tl_[0::2] - tp[1::2] / tl_[1::2]) - 1.2
    tl = -torch.nn.functional.logsigmoid(z).mean()
    tl.backward()
    loss, coef = orc.simpo_loss(pol, ln, 2.5, 1.2)
    assert abs(loss - tl.item()) < 1e-13 and np.allclose(coef, tp.grad.numpy(), atol=1e-15)


def test_orpo_loss_closed_form_and_torch_autograd():
    # equal mean log-probs: the odds ratio is 1, loss = -a + lam * ln 2
    loss, _ = orc.orpo_loss([-6.0, -9.0], [3, 4.5], 0.25)
    assert abs(loss - (2.0 + 0.25 * np.log(2.0))) < 1e-14
    rng = np.random.default_rng(8)
    ln = rng.integers(2, 60, size=16)
    pol = -rng.uniform(0.05, 3.0, size=16) * ln
    tp = torch.tensor(pol, requires_grad=True)
    a = tp / torch.tensor(ln, dtype=torch.float64)
    lo = a - torch.log1p(-torch.exp(a))
    tl = (-a[0::2] - 0.7 * torch.nn.functional.logsigmoid(lo[0::2] - lo[1::2])).mean()
    tl.backward()
    loss, coef = orc.orpo_loss(pol, ln, 0.7)
    assert abs(loss - tl.item()) < 1e-12 and np.allclose(coef, tp.grad.numpy(), rtol=1e-11, atol=1e-14)
