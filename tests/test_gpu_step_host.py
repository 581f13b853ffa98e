"""psa_step_host (host buffers in, host buffers out) against psa_fwd + psa_bwd on device
tensors, and against the fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2410_20305_b200 import binding as B
from paper_2410_20305_b200 import workloads as wl

from gpu_util import TOL_LSE, TOL_O, device_plan, grad_errors, max_abs, oracle_bwd, oracle_fwd, read_status

pytestmark = pytest.mark.gpu


def _host_step(pack, seed, pinned):
    q, k, v, d_o = wl.attention_inputs(pack, seed)
    plan = device_plan(pack, 0.0)
    host = lambda t: t.pin_memory() if pinned else t.clone()
    hq, hk, hv, hdo = host(q), host(k), host(v), host(d_o)
    T, Hq = pack.total_tokens, pack.n_q_heads
    h_o, h_dq = host(torch.zeros_like(q)), host(torch.zeros_like(q))
    h_dk, h_dv = host(torch.zeros_like(k)), host(torch.zeros_like(k))
    h_lse = host(torch.zeros((Hq, T), dtype=torch.float32))
    n = B.psa_step_host_arena_bytes(plan)
    assert n >= 4 * q.numel() * 2 + 4 * k.numel() * 2 + plan.bwd_workspace_bytes
    arena = torch.empty(n, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.Stream()
    B.psa_step_host(plan, hq, hk, hv, hdo, h_o, h_lse, h_dq, h_dk, h_dv, arena, status=status,
                    stream=stream.cuda_stream)
    stream.synchronize()
    assert read_status(status) == 0
    return plan, (q, k, v, d_o), (h_o, h_lse, h_dq, h_dk, h_dv)


@pytest.mark.parametrize("pinned", [True, False])
def test_step_host_matches_device_calls_and_oracle(pinned):
    pack = wl.random_pack(5, 3, 300, 4, 2, 128)
    plan, (q, k, v, d_o), (h_o, h_lse, h_dq, h_dk, h_dv) = _host_step(pack, 3, pinned)
    dq_, dk_, dv_, do_ = q.cuda(), k.cuda(), v.cuda(), d_o.cuda()
    o, lse = B.psa_fwd(plan, dq_, dk_, dv_)
    gq, gk, gv = B.psa_bwd(plan, do_, dq_, dk_, dv_, o, lse)
    torch.cuda.synchronize()
    # same kernels on the same data: everything with a fixed summation order is bit-identical
    assert torch.equal(h_o, o.cpu()) and torch.equal(h_lse, lse.cpu())
    assert torch.equal(h_dk, gk.cpu()) and torch.equal(h_dv, gv.cpu())
    # dq is summed over key tiles with unordered fp32 adds before its rounding to bf16
    assert max_abs(h_dq, gq.float().cpu().numpy().astype(np.float64)) <= 0.0625
    ro, rl = oracle_fwd(pack, q, k, v, None)
    assert max_abs(h_o, ro) <= TOL_O and max_abs(h_lse, rl) <= TOL_LSE
    rdq, rdk, rdv = oracle_bwd(pack, q, k, v, d_o, None)
    for got, ref in ((h_dq, rdq), (h_dk, rdk), (h_dv, rdv)):
        _, raw_small, excess = grad_errors(got, ref)   # the gate of the psa_bwd parity tests
        assert raw_small <= TOL_O and excess <= TOL_O, (raw_small, excess)


def test_step_host_rejects_small_arena_and_null():
    pack = wl.config_pack(0)
    plan = device_plan(pack, 0.0)
    q, k, v, d_o = wl.attention_inputs(pack, 0)
    T, Hq = pack.total_tokens, pack.n_q_heads
    outs = [torch.zeros_like(q), torch.zeros((Hq, T), dtype=torch.float32), torch.zeros_like(q),
            torch.zeros_like(k), torch.zeros_like(k)]
    small = torch.empty(B.psa_step_host_arena_bytes(plan) - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.PsaError) as e:
        B.psa_step_host(plan, q, k, v, d_o, *outs, small)
    assert e.value.code == 1
