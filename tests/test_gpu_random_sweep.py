"""A seeded sweep of small random packs through psa_fwd and psa_bwd against the oracle: lengths drawn
around the tile edge (120-136), prompts of 0-2 tokens, long prompts with 0-2 chosen tokens, parts that
are whole multiples of 128 or empty, one to four samples per pack, six head shapes.  Each family of
lengths hits another corner of the plan (tile classes, PRECISE marking, the few-key rows of short
prompts, ragged last tiles)."""
import numpy as np
import pytest
import torch

from paper_2410_20305_b200 import binding as B
from paper_2410_20305_b200 import workloads as wl

from gpu_util import TOL_LSE, TOL_O, device_plan, grad_errors, max_abs, oracle_bwd, oracle_fwd, read_status

pytestmark = pytest.mark.gpu

SHAPES = [(128, 4, 1), (128, 8, 2), (128, 2, 2), (64, 4, 2), (64, 3, 3), (128, 6, 3)]


def _draw_lengths(rng):
    mode = int(rng.integers(0, 5))
    if mode == 0:
        l = tuple(int(rng.integers(0, 300)) for _ in range(3))
    elif mode == 1:
        l = tuple(int(rng.integers(120, 136)) for _ in range(3))
    elif mode == 2:
        l = (int(rng.integers(0, 3)), int(rng.integers(0, 260)), int(rng.integers(0, 260)))
    elif mode == 3:
        l = (int(rng.integers(200, 520)), int(rng.integers(0, 3)), int(rng.integers(0, 140)))
    else:
        l = tuple(128 * int(rng.integers(0, 3)) for _ in range(3))
    return l if sum(l) > 0 else (1, 0, 0)


@pytest.mark.parametrize("chunk", range(4))
def test_random_packs(chunk):
    rng = np.random.default_rng(500 + chunk)
    for case in range(12):
        d, hq, hkv = SHAPES[(chunk * 12 + case) % len(SHAPES)]
        lens = [_draw_lengths(rng) for _ in range(int(rng.integers(1, 5)))]
        pack = wl.pack_from_lengths("sweep", lens, hq, hkv, d)
        q, k, v, d_o = wl.attention_inputs(pack, int(rng.integers(0, 1 << 30)))
        plan = device_plan(pack)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
        o, lse = B.psa_fwd(plan, qd, kd, vd, status=status)
        dq, dk, dv = B.psa_bwd(plan, d_o.cuda(), qd, kd, vd, o, lse, status=status)
        assert read_status(status) == 0, lens
        ro, rl = oracle_fwd(pack, q, k, v)
        rdq, rdk, rdv = oracle_bwd(pack, q, k, v, d_o)
        assert max_abs(lse, rl) <= TOL_LSE, lens
        # o takes the gradients' reading here: a row with one or two keys has o close to a v row, and
        # |v| >= 4 (where half a bf16 ulp is 0.0156) does occur among this many short rows
        for name, got, ref in (("o", o, ro), ("dq", dq, rdq), ("dk", dk, rdk), ("dv", dv, rdv)):
            raw, raw_small, excess = grad_errors(got, ref)
            assert raw_small <= TOL_O and excess <= TOL_O, (name, lens, (d, hq, hkv), raw, raw_small, excess)
