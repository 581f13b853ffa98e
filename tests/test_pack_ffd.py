"""First-fit-decreasing packer (host): the library against the textbook algorithm written out in
the oracle, the oracle against exhaustive search on tiny inputs, and the packing gain of prefix
sharing (Section 3.2: shorter units pack better) on synthetic lengths."""
import numpy as np
import pytest

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import binding as B


def test_oracle_ffd_hand_example():
    # capacity 10, units 7 5 4 3 3 2 -> sorted the same; bins: [7,3] [5,4] [3,2]
    assert orc.ffd_pack([7, 5, 4, 3, 3, 2], 10) == [0, 1, 1, 0, 2, 2]
    # ties keep the lower index first; unsorted input
    assert orc.ffd_pack([2, 9, 2, 9], 11) == [0, 0, 1, 1]


def test_oracle_ffd_within_the_classical_bound_of_the_optimum():
    rng = np.random.default_rng(0)
    for _ in range(40):
        n = int(rng.integers(1, 9))
        lens = rng.integers(1, 11, size=n)
        cap = 10
        bins = orc.ffd_pack(lens, cap)
        used = max(bins) + 1
        opt = orc.optimal_bin_count(lens, cap)
        assert opt <= used <= (11 * opt + 6) // 9 + 1      # FFD <= 11/9 OPT + 6/9
        for b in range(used):
            assert sum(int(l) for l, bb in zip(lens, bins) if bb == b) <= cap


@pytest.mark.parametrize("seed", range(5))
def test_library_matches_oracle(seed):
    rng = np.random.default_rng(seed)
    lens = rng.integers(0, 4000, size=int(rng.integers(1, 400)))
    cap = 16384
    got, n_bins = B.psa_pack_ffd(lens, cap)
    want = orc.ffd_pack(lens, cap)
    assert list(got) == want and n_bins == max(want) + 1


def test_library_edge_cases():
    bins, n = B.psa_pack_ffd([], 100)
    assert len(bins) == 0 and n == 0
    bins, n = B.psa_pack_ffd([100, 100, 1], 100)
    assert list(bins) == [0, 1, 2] and n == 3
    with pytest.raises(B.PsaError) as e:
        B.psa_pack_ffd([5, 101], 100)
    assert e.value.code == 3
    with pytest.raises(B.PsaError) as e:
        B.psa_pack_ffd([5, -1], 100)
    assert e.value.code == 1


def test_shared_units_need_fewer_packs_than_paired_units():
    rng = np.random.default_rng(7)
    P = rng.integers(1024, 3073, size=300); Cc = rng.integers(32, 129, size=300); R = rng.integers(32, 129, size=300)
    cap = 16384
    _, shared = B.psa_pack_ffd(P + Cc + R, cap)
    _, paired = B.psa_pack_ffd(2 * P + Cc + R, cap)
    tokens_ratio = (2 * P + Cc + R).sum() / (P + Cc + R).sum()
    assert paired / shared == pytest.approx(tokens_ratio, rel=0.05)   # long prompts: about 1.9x


def test_oracle_pack_layout_hand_example():
    # units (P, C, R): 0 -> (4, 2, 1) = 7, 1 -> (1, 1, 1) = 3, 2 -> (3, 2, 0) = 5, 3 -> (2, 1, 1) = 4; capacity 10.
    # Longest first: 7, 5, 4, 3 -> packs [7, 3] and [5, 4].
    packs = orc.ffd_pack_layout([4, 1, 3, 2], [2, 1, 2, 1], [1, 1, 0, 1], 10)
    assert len(packs) == 2
    assert packs[0] == dict(cu_seqlens=[0, 7, 10], prefix_len=[4, 1], chosen_len=[2, 1], rejected_len=[1, 1], units=[0, 1])
    assert packs[1] == dict(cu_seqlens=[0, 5, 9], prefix_len=[3, 2], chosen_len=[2, 1], rejected_len=[0, 1], units=[2, 3])
    # paired layout, capacity 12: unit lengths 2P + C + R = 11, 4, 8, 6 -> packs [11], [8, 4], [6]
    packs = orc.ffd_pack_layout([4, 1, 3, 2], [2, 1, 2, 1], [1, 1, 0, 1], 12, paired=True)
    assert [p["units"] for p in packs] == [[0, 0], [2, 2, 1, 1], [3, 3]]
    assert packs[1] == dict(cu_seqlens=[0, 5, 8, 10, 12], prefix_len=[3, 3, 1, 1], chosen_len=[2, 0, 1, 1],
                            rejected_len=[0, 0, 0, 0], units=[2, 2, 1, 1])


@pytest.mark.parametrize("paired", [False, True])
def test_oracle_pack_layout_properties(paired):
    rng = np.random.default_rng(5)
    P = rng.integers(0, 300, size=60); Cc = rng.integers(0, 120, size=60); R = rng.integers(0, 120, size=60)
    cap = 1024
    packs = orc.ffd_pack_layout(P, Cc, R, cap, paired=paired)
    seen = []
    for pk in packs:
        cu = np.asarray(pk["cu_seqlens"])
        assert cu[0] == 0 and cu[-1] <= cap
        assert list(np.diff(cu)) == [p + c + r for p, c, r in zip(pk["prefix_len"], pk["chosen_len"], pk["rejected_len"])]
        seen += pk["units"]
        for j, u in enumerate(pk["units"]):     # every sample carries its unit's lengths
            assert pk["prefix_len"][j] == P[u]
            if paired:
                assert pk["rejected_len"][j] == 0 and pk["chosen_len"][j] in (Cc[u], R[u])
            else:
                assert (pk["chosen_len"][j], pk["rejected_len"][j]) == (Cc[u], R[u])
    assert sorted(seen) == sorted(list(range(60)) * (2 if paired else 1))
    # the number of useful pairs is that of the units, whatever the packing
    total = sum(orc.useful_pairs(pk["prefix_len"], pk["chosen_len"], pk["rejected_len"]) for pk in packs)
    want = orc.useful_pairs(np.repeat(P, 2), np.stack([Cc, R], 1).reshape(-1), np.zeros(120, int)) if paired \
        else orc.useful_pairs(P, Cc, R)
    assert total == want


@pytest.mark.parametrize("paired", [False, True])
@pytest.mark.parametrize("seed", range(3))
def test_library_pack_layout_matches_oracle_and_feeds_the_planner(seed, paired):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(1, 200))
    P = rng.integers(0, 3000, size=n); Cc = rng.integers(0, 900, size=n); R = rng.integers(0, 900, size=n)
    cap = 16384
    bins, packs = B.psa_pack_ffd_emit(P, Cc, R, cap, paired=paired)
    want = orc.ffd_pack_layout(P, Cc, R, cap, paired=paired)
    assert len(packs) == len(want)
    for got, ref in zip(packs, want):
        for key in ("cu_seqlens", "prefix_len", "chosen_len", "rejected_len", "units"):
            assert list(got[key]) == list(ref[key]), key
    assert list(bins) == orc.ffd_pack([(2 if paired else 1) * int(p) + int(c) + int(r) for p, c, r in zip(P, Cc, R)], cap)
    # every pack goes straight into psa_plan
    for got in packs[:4]:
        if got["cu_seqlens"][-1] == 0:
            continue
        plan = B.psa_plan(got["cu_seqlens"], got["prefix_len"], got["chosen_len"], got["rejected_len"], 8, 2, 128,
                          host_only=True)
        assert plan.total_tokens == int(got["cu_seqlens"][-1])
        assert plan.useful_pairs == orc.useful_pairs(got["prefix_len"], got["chosen_len"], got["rejected_len"])


def test_library_pack_layout_edge_cases():
    bins, packs = B.psa_pack_ffd_emit([], [], [], 100)
    assert len(bins) == 0 and packs == []
    with pytest.raises(B.PsaError) as e:
        B.psa_pack_ffd_emit([60], [30], [30], 100)          # 120 > 100
    assert e.value.code == 3
    with pytest.raises(B.PsaError) as e:
        B.psa_pack_ffd_emit([40], [10], [10], 90, paired=True)   # 2 * 40 + 20 = 100 > 90
    assert e.value.code == 3
