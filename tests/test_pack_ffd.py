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
