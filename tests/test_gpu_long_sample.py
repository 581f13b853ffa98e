"""One sample of 16.7k tokens: 131 tiles, so that tile lists are longer than the part the kernels
keep in shared memory (128 entries) and the rest is read from global memory.  The forward is
checked on every row (the oracle's forward called chunk by chunk), the gradients on sampled rows
(dq) and key positions (dk, dv) with the oracle's per-row / per-column form."""
import numpy as np
import pytest
import torch

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import binding as B
from paper_2410_20305_b200 import workloads as wl

from gpu_util import TOL_LSE, TOL_O, device_plan, grad_errors, max_abs, read_status

pytestmark = pytest.mark.gpu


def test_sample_longer_than_the_cached_part_of_the_tile_lists():
    P, C, R = 15000, 1000, 700
    pack = wl.pack_from_lengths("verylong", [(P, C, R)], 2, 1, 64)
    T = pack.total_tokens
    assert (T + 127) // 128 > 128
    q, k, v, d_o = wl.attention_inputs(pack, 3)
    plan = device_plan(pack)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    qd, kd, vd, dod = q.cuda(), k.cuda(), v.cuda(), d_o.cuda()
    o, lse = B.psa_fwd(plan, qd, kd, vd, status=status)
    dq, dk, dv = B.psa_bwd(plan, dod, qd, kd, vd, o, lse, status=status)
    assert read_status(status) == 0
    o, lse, dq, dk, dv = (t.cpu() for t in (o, lse, dq, dk, dv))

    f = wl.to_f64
    fq, fk, fv, fdo = f(q), f(k), f(v), f(d_o)
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    ro = np.empty((T, 2, 64)); rl = np.empty((2, T))
    for r0 in range(0, T, 1024):
        rows = np.arange(r0, min(T, r0 + 1024))
        ro[rows], rl[:, rows] = orc.attention_rows(fq, fk, fv, mask[rows], rows)
    assert max_abs(o, ro) <= TOL_O and max_abs(lse, rl) <= TOL_LSE

    rng = np.random.default_rng(7)
    edge = [0, 1, 127, 128, P - 1, P, P + C - 1, P + C, T - 129, T - 128, T - 1, 128 * 128 - 1, 128 * 128, 128 * 129]
    rows = np.unique(np.concatenate([edge, rng.integers(0, T, 40)]))
    cols = np.unique(np.concatenate([edge, rng.integers(0, T, 40)]))
    rdq, rdk, rdv = orc.attention_bwd_sampled(fq, fk, fv, fdo, ro, rl, mask, rows, cols)
    for name, got, ref in (("dq", dq[rows], rdq), ("dk", dk[cols], rdk), ("dv", dv[cols], rdv)):
        raw, raw_small, excess = grad_errors(got, ref)
        assert raw_small <= TOL_O and excess <= TOL_O, (name, raw, raw_small, excess)
