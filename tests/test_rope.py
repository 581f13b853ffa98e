"""Position ids (host) and the rotary-embedding kernel (GPU) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import binding as B
from paper_2410_20305_b200 import workloads as wl


def test_position_ids_match_oracle_and_validate():
    for seed in range(4):
        pack = wl.random_pack(200 + seed, 5, 300, 1, 1, 64)
        got = B.psa_position_ids(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
        want = orc.position_ids(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
        assert (got == want).all()
    with pytest.raises(B.PsaError) as e:
        B.psa_position_ids([0, 9], [4], [3], [3])
    assert e.value.code == 2


@pytest.mark.gpu
@pytest.mark.parametrize("H,d,theta", [(32, 128, 500000.0), (8, 128, 10000.0), (4, 64, 10000.0), (3, 16, 10000.0)])
def test_rope_kernel_matches_oracle(H, d, theta):
    pack = wl.config_pack(4)
    T = pack.total_tokens
    x = wl.bf16_normal((T, H, d), 5)
    pos = B.psa_position_ids(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    y = B.psa_rope(x.cuda(), torch.as_tensor(pos).cuda(), theta)
    want = orc.rope(wl.to_f64(x), pos, theta)
    got = y.cpu().double().numpy()
    # bf16 output (half an ulp = 2^-9 relative) plus fp32 sin / cos of angles up to ~700 rad
    assert np.abs(got - want).max() <= 2.0 ** -8 * np.abs(want).max()
    assert np.abs(got - want).mean() <= 2e-3
    # in place gives the same bits
    z = x.cuda().clone()
    B.psa_rope(z, torch.as_tensor(pos).cuda(), theta, out=z)
    assert torch.equal(z, y)
