"""Pins for the oracle's per-response log-prob gather."""
import numpy as np
import torch

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import workloads as wl
from paper_2410_20305_b200.labels import logp_labels


def test_matches_torch_log_softmax_gather():
    x, tok = wl.logits_and_tokens(40, 97, seed=3, std=2.0 ** 0.5)
    seg = np.random.default_rng(0).integers(-1, 6, size=40).astype(np.int32)
    got = orc.dpo_logp(wl.to_f64(x), tok.numpy(), seg, 6)
    lp = torch.log_softmax(x.double(), dim=-1).gather(1, tok.long()[:, None])[:, 0].numpy()
    want = np.zeros(6)
    for t in range(40):
        if seg[t] >= 0:
            want[seg[t]] += lp[t]
    assert np.allclose(got, want, rtol=1e-13, atol=1e-12)


def test_constant_logits_give_minus_n_log_v():
    V, rows = 50, 12
    x = np.full((rows, V), 3.25)
    seg = np.array([0] * 5 + [-1] * 3 + [1] * 4, dtype=np.int32)
    out = orc.dpo_logp(x, np.zeros(rows, dtype=np.int32), seg, 2, [6], [7], [1])
    assert np.allclose(out, [-5 * np.log(V), -5 * np.log(V)], rtol=1e-14)


def test_shared_layout_labels_reproduce_paired_definition():
    """Section 2.1: the log-probs must be those of the paired format.  The
    paired sequences are assembled by copying logits rows of the shared layout
    (valid because a row's logits depend only on its own context)."""
    pack = wl.pack_from_lengths("lp", [(5, 3, 4), (1, 1, 1), (0, 3, 2), (4, 0, 2), (3, 2, 0), (2, 1, 5)], 1, 1, 8)
    T, V = pack.total_tokens, 31
    x, tok = wl.logits_and_tokens(T, V, seed=11, std=1.5)
    x64 = wl.to_f64(x)
    targets, seg, fr, ft, fs = logp_labels(tok.numpy(), pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    got = orc.dpo_logp(x64, targets, seg, 2 * pack.n_samples, fr, ft, fs)
    want = orc.paired_response_logps(lambda rows: x64[rows], tok.numpy(), pack.cu_seqlens,
                                     pack.prefix_len, pack.chosen_len, pack.rejected_len)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-12)
    # the last chosen row never scores the first rejected token
    for s in range(pack.n_samples):
        rs = pack.cu_seqlens[s] + pack.prefix_len[s] + pack.chosen_len[s]
        if pack.chosen_len[s] > 0:
            assert seg[rs - 1] == -1 or pack.chosen_len[s] == 0


def test_number_of_scored_tokens():
    pack = wl.config_pack(4)
    tok = np.zeros(pack.total_tokens, dtype=np.int32)
    targets, seg, fr, ft, fs = logp_labels(tok, pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    assert int((seg >= 0).sum()) + len(fr) == int(pack.chosen_len.sum() + pack.rejected_len.sum())
