"""The gradient gate as stated: max abs error 1e-2 on dq, dk, dv against the fp64 oracle, raw,
on every element.  psa_bwd_f32 writes the kernels' fp32 accumulators out as they are, so the
rounding of the OUTPUT to bf16 (half an ulp is 0.0156 in [4, 8), more than the gate) is out of
the comparison; everything else (bf16 operands of the tensor-core products, fp32 accumulation)
is the same computation psa_bwd runs.  The bf16-output tests in test_gpu_bwd.py print their raw
maxima beside the reading they gate on."""
import numpy as np
import pytest
import torch

from paper_2410_20305_b200 import binding as B
from paper_2410_20305_b200 import workloads as wl

from gpu_util import TOL_O, device_plan, max_abs, oracle_bwd, read_status

pytestmark = pytest.mark.gpu


def run_bwd_f32(pack, seed):
    q, k, v, d_o = wl.attention_inputs(pack, seed)
    plan = device_plan(pack)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    qd, kd, vd, dod = q.cuda(), k.cuda(), v.cuda(), d_o.cuda()
    o, lse = B.psa_fwd(plan, qd, kd, vd, status=status)
    T = pack.total_tokens
    pad = lambda t: torch.full((T + 2,) + tuple(t.shape[1:]), 3.0, dtype=torch.float32, device="cuda")
    dq_buf, dk_buf, dv_buf = pad(q), pad(k), pad(v)
    dq, dk, dv = B.psa_bwd_f32(plan, dod, qd, kd, vd, o, lse, dq=dq_buf[:T], dk=dk_buf[:T], dv=dv_buf[:T], status=status)
    assert read_status(status) == 0
    for buf in (dq_buf, dk_buf, dv_buf):
        assert (buf[T:] == 3.0).all(), "wrote past the last token"
    rdq, rdk, rdv = oracle_bwd(pack, q, k, v, d_o)
    err = {"dq": max_abs(dq, rdq), "dk": max_abs(dk, rdk), "dv": max_abs(dv, rdv)}
    print("fp32 gradients, raw max abs error %s seed %d: dq %.4f dk %.4f dv %.4f" % (pack.name, seed, err["dq"], err["dk"], err["dv"]))
    assert max(err.values()) <= TOL_O, (pack.name, seed, err)
    # the bf16 entry point is the same computation rounded once more
    bq, bk, bv = B.psa_bwd(plan, dod, qd, kd, vd, o, lse)
    assert (bk.float() - dk.to(torch.bfloat16).float()).abs().max().item() == 0.0
    assert (bv.float() - dv.to(torch.bfloat16).float()).abs().max().item() == 0.0
    return err


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_tiny_config_raw_gate(seed):
    run_bwd_f32(wl.config_pack(0), seed)


@pytest.mark.parametrize("d,hq,hkv", [(128, 4, 1), (128, 8, 8), (64, 8, 2), (64, 1, 1)])
def test_random_ragged_gqa_packs_raw_gate(d, hq, hkv):
    for seed in range(3):
        run_bwd_f32(wl.random_pack(40 + seed, 4, 330, hq, hkv, d), seed)


def test_degenerate_lengths_raw_gate():
    lengths = [(0, 70, 200), (300, 0, 45), (129, 255, 0), (1, 0, 0), (1, 1, 1), (128, 128, 128), (0, 0, 5)]
    run_bwd_f32(wl.pack_from_lengths("deg", lengths, 4, 2, 128), 5)


def test_long_sample_raw_gate():
    run_bwd_f32(wl.pack_from_lengths("long", [(1500, 300, 421), (700, 90, 33)], 4, 2, 128), 9)
