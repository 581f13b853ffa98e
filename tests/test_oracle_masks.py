"""Pins for the oracle's masks: hand-derived fixtures, closed forms, brute force."""
import os

import numpy as np
import pytest

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _load(name):
    return np.loadtxt(os.path.join(GOLDEN, name), dtype=np.int64, comments="#")


def test_alg1_hand_fixture():
    want = _load("mask_alg1_p2_c2_r2.txt").astype(bool)
    got = orc.prefix_sharing_mask_single(6, 2, 4)
    assert (got == want).all()


def test_alg3_hand_fixture():
    want = _load("mask_alg3_two_samples.txt").astype(bool)
    got = orc.packed_mask([0, 3, 8], [1, 2], [1, 1], [1, 2])
    assert (got == want).all()


def test_alg2_hand_fixture():
    want = _load("mask_alg2_paired.txt").astype(bool)
    got = orc.paired_packing_mask([0, 0, 0, 1, 1, 1, 1])
    assert (got == want).all()


def test_alg3_reduces_to_alg1_for_one_document():
    for P, C, R in [(5, 3, 4), (1, 1, 1), (0, 4, 2), (7, 0, 3), (6, 2, 0)]:
        L = P + C + R
        a3 = orc.packed_mask([0, L], [P], [C], [R])
        a1 = orc.prefix_sharing_mask_single(L, P, P + C)
        assert (a3 == a1).all()


def test_alg3_with_no_rejected_is_alg2_on_paired_layout():
    pack = wl.random_pack(3, 4, 12, 1, 1, 8, allow_zero=False)
    pp = pack.paired()
    a3 = orc.packed_mask(pp.cu_seqlens, pp.prefix_len, pp.chosen_len, pp.rejected_len)
    rid = np.concatenate([np.full(pp.cu_seqlens[i + 1] - pp.cu_seqlens[i], i) for i in range(pp.n_samples)])
    assert (a3 == orc.paired_packing_mask(rid)).all()


def test_brute_force_python_loops():
    """The vectorised predicate against a literal triple loop with the sample
    structure spelled out in words: same sample, causal, and a rejected query
    never sees a chosen key."""
    pack = wl.random_pack(11, 3, 9, 1, 1, 8)
    got = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    T = pack.total_tokens
    kind, samp = [], []
    for s in range(pack.n_samples):
        kind += ["p"] * pack.prefix_len[s] + ["c"] * pack.chosen_len[s] + ["r"] * pack.rejected_len[s]
        samp += [s] * (pack.prefix_len[s] + pack.chosen_len[s] + pack.rejected_len[s])
    for q in range(T):
        for kv in range(T):
            want = samp[q] == samp[kv] and kv <= q and not (kind[q] == "r" and kind[kv] == "c")
            assert bool(got[q, kv]) == want, (q, kv)


def test_row_interval_form():
    """A different statement of the same mask, from the sample boundaries alone: a prompt or
    chosen row q sees the keys [sample start, q]; a rejected row sees the prompt
    [sample start, chosen start) and its own response [rejected start, q]."""
    pack = wl.random_pack(17, 4, 14, 1, 1, 8)
    got = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    want = np.zeros_like(got)
    for s in range(pack.n_samples):
        ds = int(pack.cu_seqlens[s]); cs = ds + int(pack.prefix_len[s]); rs = cs + int(pack.chosen_len[s])
        for q in range(ds, int(pack.cu_seqlens[s + 1])):
            if q < rs:
                want[q, ds:q + 1] = True
            else:
                want[q, ds:cs] = True
                want[q, rs:q + 1] = True
    assert (got == want).all()


def test_tiny_mask_count_matches_closed_form():
    rows = _load("tiny_mask_count.txt")
    pack = wl.config_pack(0)
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    assert int(mask.sum()) == int(rows[:, 3].sum()) == 109648
    for s, (P, C, R, cnt) in enumerate(rows):
        lo, hi = pack.cu_seqlens[s], pack.cu_seqlens[s + 1]
        assert (pack.prefix_len[s], pack.chosen_len[s], pack.rejected_len[s]) == (P, C, R)
        assert int(mask[lo:hi, lo:hi].sum()) == cnt
    assert orc.useful_pairs(pack.prefix_len, pack.chosen_len, pack.rejected_len) == 109648


def test_every_row_sees_itself_and_counts():
    pack = wl.random_pack(5, 5, 20, 1, 1, 8)
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    assert mask.diagonal().all()
    assert int(mask.sum()) == orc.useful_pairs(pack.prefix_len, pack.chosen_len, pack.rejected_len)
    # per-row counts: prompt/chosen rows see q-ds+1 keys, rejected rows see P + q-rs+1
    for s in range(pack.n_samples):
        ds = int(pack.cu_seqlens[s]); P = int(pack.prefix_len[s]); C = int(pack.chosen_len[s])
        rs = ds + P + C
        for q in range(ds, int(pack.cu_seqlens[s + 1])):
            want = q - ds + 1 if q < rs else P + q - rs + 1
            assert int(mask[q].sum()) == want


def test_ideal_speedup_footnotes():
    for p, c, tn, td, an, ad in _load("ideal_speedups.txt"):
        assert orc.ideal_token_speedup(p, c) == pytest.approx(tn / td, rel=1e-14)
        assert orc.ideal_attention_speedup(p, c) == pytest.approx(an / ad, rel=1e-14)
        # the same ratios come out of the token and pair counters when C = R = c
        shared_tokens = p + 2 * c
        paired_tokens = 2 * (p + c)
        assert paired_tokens / shared_tokens == pytest.approx(tn / td, rel=1e-14)
        # pairs, not counting the diagonal's +1 terms (the footnote's idealisation):
        # 2*U - (number of rows) turns n(n+1)/2 triangles into n^2/2-style counts
        U_shared = 2 * orc.useful_pairs([p], [c], [c]) - shared_tokens
        U_paired = 2 * orc.useful_pairs([p, p], [c, c], [0, 0]) - paired_tokens
        assert U_paired / U_shared == pytest.approx(an / ad, rel=1e-14)
