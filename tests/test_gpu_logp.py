"""dpo_logp on the GPU against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import binding as B
from paper_2410_20305_b200 import workloads as wl
from paper_2410_20305_b200.labels import logp_labels

from gpu_util import TOL_LOGP, read_status

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.as_tensor(np.asarray(a, dtype=np.int32)).cuda()


def _run(pack, vocab, seed, std, dtype):
    T = pack.total_tokens
    x, tok = wl.logits_and_tokens(T, vocab, seed, std, dtype)
    targets, seg, fr, ft, fs = logp_labels(tok.numpy(), pack.cu_seqlens, pack.prefix_len, pack.chosen_len,
                                           pack.rejected_len)
    n_seg = 2 * pack.n_samples
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = B.dpo_logp(x.cuda(), _dev(targets), _dev(seg), n_seg, _dev(fr), _dev(ft), _dev(fs), status=status)
    assert read_status(status) == 0
    want = orc.dpo_logp(wl.to_f64(x), targets, seg, n_seg, fr, ft, fs)
    got = out.cpu().double().numpy()
    live = np.abs(want) > 0
    assert (got[~live] == 0).all()
    rel = np.abs(got[live] - want[live]) / np.abs(want[live])
    return float(rel.max(initial=0.0))


def test_tiny_config_fp32_logits():
    assert _run(wl.config_pack(0), 1024, 0, 2.0 ** 0.5, torch.float32) <= TOL_LOGP
    assert _run(wl.config_pack(0), 1024, 1, 2.0, torch.float32) <= TOL_LOGP


@pytest.mark.parametrize("vocab", [128256, 32000, 1000, 8, 50257 + 7])
def test_bf16_logits_ragged_vocab(vocab):
    pack = wl.pack_from_lengths("lp", [(20, 9, 13), (0, 5, 4), (7, 0, 3), (3, 4, 0), (1, 1, 1)], 1, 1, 64)
    if vocab % 8:
        # rows must start 16-byte aligned: pad the row stride, keep the vocab ragged
        T = pack.total_tokens
        stride = (vocab + 7) // 8 * 8
        x, tok = wl.logits_and_tokens(T, stride, 3, 3.0 ** 0.5, torch.bfloat16)
        tok = tok % vocab
        targets, seg, fr, ft, fs = logp_labels(tok.numpy(), pack.cu_seqlens, pack.prefix_len, pack.chosen_len,
                                               pack.rejected_len)
        out = B.dpo_logp(x.cuda()[:, :vocab], _dev(targets), _dev(seg), 10, _dev(fr), _dev(ft), _dev(fs))
        want = orc.dpo_logp(wl.to_f64(x)[:, :vocab], targets, seg, 10, fr, ft, fs)
        got = out.cpu().double().numpy()
        live = np.abs(want) > 0
        assert (np.abs(got[live] - want[live]) / np.abs(want[live])).max() <= TOL_LOGP
    else:
        assert _run(pack, vocab, 3, 3.0 ** 0.5, torch.bfloat16) <= TOL_LOGP


def test_plain_gather_without_forks_and_dead_rows():
    x, tok = wl.logits_and_tokens(300, 4096, 5, 1.7, torch.bfloat16)
    seg = np.random.default_rng(1).integers(-1, 7, size=300).astype(np.int32)
    out = B.dpo_logp(x.cuda(), tok.cuda(), _dev(seg), 7)
    want = orc.dpo_logp(wl.to_f64(x), tok.numpy(), seg, 7)
    assert (np.abs(out.cpu().double().numpy() - want) / np.abs(want)).max() <= TOL_LOGP


def test_bad_labels_set_status_bits_and_are_skipped():
    x, tok = wl.logits_and_tokens(6, 64, 5, 1.0, torch.float32)
    targets = np.array([1, 64, 3, -5, 2, 7], dtype=np.int32)      # rows 1 and 3 are out of range
    seg = np.array([0, 0, 1, 1, 9, -1], dtype=np.int32)            # row 4 names a segment >= n_segments
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = B.dpo_logp(x.cuda(), _dev(targets), _dev(seg), 2, status=status)
    assert read_status(status) == (B.PSA_DEVSTAT_BAD_TARGET | B.PSA_DEVSTAT_BAD_SEGMENT)
    want = [orc.row_logprob(wl.to_f64(x)[0], 1), orc.row_logprob(wl.to_f64(x)[2], 3)]
    assert np.allclose(out.cpu().numpy(), want, rtol=1e-4)


def test_zero_rows_and_zero_segments():
    x = torch.empty((0, 128), dtype=torch.float32, device="cuda")
    e = torch.empty(0, dtype=torch.int32, device="cuda")
    out = B.dpo_logp(x, e, e, 3)
    assert (out.cpu() == 0).all()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("vocab", [1, 3, 7, 129])
def test_single_row_of_any_width(vocab, dtype):
    """One row has no stride, so a vocabulary that is not a multiple of 16 bytes is accepted; the
    ragged tail of the row is handled by scalar loads."""
    x, tok = wl.logits_and_tokens(1, vocab, 11, 2.0, dtype)
    seg = np.zeros(1, dtype=np.int32)
    coef = torch.tensor([0.75], dtype=torch.float32, device="cuda")
    out = B.dpo_logp(x.cuda(), tok.cuda(), _dev(seg), 1)
    want = orc.dpo_logp(wl.to_f64(x), tok.numpy(), seg, 1)
    assert abs(out.item() - want[0]) <= TOL_LOGP * max(1.0, abs(want[0]))
    grad = B.dpo_logp_bwd(x.cuda(), tok.cuda(), _dev(seg), coef)
    ref = orc.dpo_logp_grad(wl.to_f64(x), tok.numpy(), seg, [0.75])
    assert np.abs(grad.cpu().double().numpy() - ref).max() <= (2e-6 if dtype == torch.float32 else 2.0 ** -8)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_rows_that_begin_with_a_block_of_minus_infinity(dtype):
    """Banned or padded vocabulary entries are -inf.  A thread whose first chunk of the row is all
    -inf must carry "nothing yet", not a NaN, into the rest of the row; the gradient sweep too."""
    n_rows, vocab = 6, 4096
    x, tok = wl.logits_and_tokens(n_rows, vocab, 21, 2.0, dtype)
    x[0, :1024] = -float("inf")            # every thread's first chunk (and more)
    x[1, :32] = -float("inf")              # exactly one thread's first chunk
    x[2, 100:2100] = -float("inf")         # a block in the middle
    x[3, vocab - 700:] = -float("inf")     # the tail
    x[4, ::2] = -float("inf")              # every other entry
    tok = tok.clone()
    tok[0], tok[1], tok[2], tok[3], tok[4] = 2000, 40, 50, 7, 1
    seg = np.arange(n_rows, dtype=np.int32)
    out = B.dpo_logp(x.cuda(), tok.cuda(), _dev(seg), n_rows)
    want = orc.dpo_logp(wl.to_f64(x), tok.numpy(), seg, n_rows)
    got = out.cpu().double().numpy()
    assert np.isfinite(got).all()
    assert (np.abs(got - want) / np.abs(want)).max() <= TOL_LOGP
    coef = torch.linspace(0.1, 0.6, n_rows, dtype=torch.float32).cuda()
    grad = B.dpo_logp_bwd(x.cuda(), tok.cuda(), _dev(seg), coef).cpu().double().numpy()
    ref = orc.dpo_logp_grad(wl.to_f64(x), tok.numpy(), seg, coef.cpu().double().numpy())
    assert np.isfinite(grad).all()
    assert np.abs(grad - ref).max() <= (2e-6 if dtype == torch.float32 else 2.0 ** -8)
