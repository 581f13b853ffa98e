"""dpo_loss and dpo_logp_bwd on the GPU against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import binding as B
from paper_2410_20305_b200 import workloads as wl
from paper_2410_20305_b200.labels import logp_labels

from gpu_util import read_status

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.as_tensor(np.asarray(a, dtype=np.int32)).cuda()


def test_dpo_loss_values_and_coefficients():
    rng = np.random.default_rng(3)
    for n in (1, 7, 300):
        pol = rng.normal(-60, 25, size=2 * n).astype(np.float32)
        ref = rng.normal(-60, 25, size=2 * n).astype(np.float32)
        loss, coef = B.dpo_loss(torch.tensor(pol).cuda(), torch.tensor(ref).cuda(), 0.1)
        want_loss, want_coef = orc.dpo_loss(pol.astype(np.float64), ref.astype(np.float64), 0.1)
        assert abs(loss.item() - want_loss) <= 1e-5 * max(1.0, abs(want_loss))
        assert np.allclose(coef.cpu().numpy(), want_coef, rtol=1e-4, atol=1e-8)


@pytest.mark.parametrize("dtype,vocab", [(torch.float32, 1024), (torch.bfloat16, 128256), (torch.bfloat16, 50257 + 7)])
def test_logit_gradient_matches_oracle(dtype, vocab):
    pack = wl.pack_from_lengths("g", [(20, 9, 13), (0, 5, 4), (7, 0, 3), (3, 4, 0), (1, 1, 1)], 1, 1, 64)
    T = pack.total_tokens
    stride = (vocab + 7) // 8 * 8
    x, tok = wl.logits_and_tokens(T, stride, 9, 3.0 ** 0.5, dtype)
    tok = tok % vocab
    targets, seg, fr, ft, fs = logp_labels(tok.numpy(), pack.cu_seqlens, pack.prefix_len, pack.chosen_len,
                                           pack.rejected_len)
    n_seg = 2 * pack.n_samples
    xd = x.cuda()[:, :vocab]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lp = B.dpo_logp(xd, _dev(targets), _dev(seg), n_seg, _dev(fr), _dev(ft), _dev(fs), status=status)
    ref_lp = torch.tensor(np.random.default_rng(5).normal(-30, 5, size=n_seg), dtype=torch.float32).cuda()
    loss, coef = B.dpo_loss(lp, ref_lp, 0.2)
    d = torch.full_like(x.cuda(), 7.0)[:, :vocab]
    B.dpo_logp_bwd(xd, _dev(targets), _dev(seg), coef, _dev(fr), _dev(ft), _dev(fs), dlogits=d, status=status)
    assert read_status(status) == 0
    x64 = wl.to_f64(x)[:, :vocab]
    want_lp = orc.dpo_logp(x64, targets, seg, n_seg, fr, ft, fs)
    want_loss, want_coef = orc.dpo_loss(want_lp, ref_lp.cpu().double().numpy(), 0.2)
    want = orc.dpo_logp_grad(x64, targets, seg, want_coef, fr, ft, fs)
    got = d.cpu().double().numpy()
    assert abs(loss.item() - want_loss) <= 1e-4 * max(1.0, abs(want_loss))
    # |d| <= |coef| <= beta / n; fp32 arithmetic, bf16 output rounding for bf16 logits
    tol = 1e-6 if dtype == torch.float32 else 2.0 ** -8 * np.abs(want).max() + 1e-7
    assert np.abs(got - want).max() <= tol, (np.abs(got - want).max(), tol)
    dead = (seg < 0) & ~np.isin(np.arange(T), fr)
    assert (got[dead] == 0).all()
    if stride > vocab:   # padding columns of the strided rows are not touched
        full = torch.full_like(x.cuda(), 7.0)
        B.dpo_logp_bwd(xd, _dev(targets), _dev(seg), coef, _dev(fr), _dev(ft), _dev(fs), dlogits=full[:, :vocab])
        torch.cuda.synchronize()
        assert (full[:, vocab:] == 7.0).all()


def test_same_token_scored_twice_by_the_fork_row():
    x, _ = wl.logits_and_tokens(3, 64, 1, 1.0, torch.float32)
    targets = np.array([5, 9, 0], dtype=np.int32); seg = np.array([0, -1, -1], dtype=np.int32)
    fr, ft, fs = np.array([0], np.int32), np.array([5], np.int32), np.array([1], np.int32)   # same token 5
    coef = torch.tensor([0.3, -0.8], dtype=torch.float32).cuda()
    d = B.dpo_logp_bwd(x.cuda(), _dev(targets), _dev(seg), coef, _dev(fr), _dev(ft), _dev(fs))
    want = orc.dpo_logp_grad(wl.to_f64(x), targets, seg, [0.3, -0.8], fr, ft, fs)
    assert np.abs(d.cpu().double().numpy() - want).max() <= 1e-6


def test_simpo_loss_matches_oracle_and_feeds_the_gradient():
    rng = np.random.default_rng(11)
    n = 37
    pol = rng.normal(-80, 30, size=2 * n).astype(np.float32)
    ln = rng.integers(1, 120, size=2 * n).astype(np.int32)
    loss, coef = B.simpo_loss(torch.tensor(pol).cuda(), torch.tensor(ln).cuda(), 2.5, 1.4)
    rl, rc = orc.simpo_loss(pol.astype(np.float64), ln, 2.5, 1.4)
    assert abs(loss.item() - rl) <= 1e-5 * max(1.0, abs(rl))
    assert np.abs(coef.cpu().numpy().astype(np.float64) - rc).max() <= 1e-6 * np.abs(rc).max() + 1e-9
    # a length below one is reported, never divided by
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ln[5] = 0
    loss2, coef2 = B.simpo_loss(torch.tensor(pol).cuda(), torch.tensor(ln).cuda(), 2.5, 1.4, status=status)
    assert status.item() != 0 and torch.isfinite(loss2).all() and torch.isfinite(coef2).all()
    assert coef2[4].item() == 0.0 and coef2[5].item() == 0.0


def test_orpo_loss_matches_oracle():
    rng = np.random.default_rng(13)
    n = 41
    ln = rng.integers(2, 200, size=2 * n).astype(np.int32)
    pol = (-rng.uniform(0.05, 4.0, size=2 * n) * ln).astype(np.float32)
    loss, coef = B.orpo_loss(torch.tensor(pol).cuda(), torch.tensor(ln).cuda(), 0.3)
    rl, rc = orc.orpo_loss(pol.astype(np.float64), ln, 0.3)
    assert abs(loss.item() - rl) <= 1e-5 * max(1.0, abs(rl))
    assert np.abs(coef.cpu().numpy().astype(np.float64) - rc).max() <= 2e-5 * np.abs(rc).max()
