"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import binding as B
from paper_2410_20305_b200 import workloads as wl

# Tolerances of the parity gate: bf16 I/O, fp32 accumulate.
TOL_O = 1e-2      # max abs error on o, dq, dk, dv
TOL_LSE = 1e-3    # max abs error on lse
TOL_LOGP = 1e-3   # relative error on per-response log-probs


def device_plan(pack, scale=0.0):
    return B.psa_plan(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len,
                      pack.n_q_heads, pack.n_kv_heads, pack.head_dim, softmax_scale=scale)


def oracle_fwd(pack, q, k, v, scale=None):
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    return orc.attention_fwd(wl.to_f64(q), wl.to_f64(k), wl.to_f64(v), mask, scale)


def oracle_bwd(pack, q, k, v, d_o, scale=None):
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    return orc.attention_bwd(wl.to_f64(q), wl.to_f64(k), wl.to_f64(v), wl.to_f64(d_o), mask, scale)


def max_abs(a, b):
    a = a.detach().to("cpu").to(torch.float64).numpy() if isinstance(a, torch.Tensor) else np.asarray(a)
    if a.size == 0:
        return 0.0
    d = np.abs(a - b)
    assert np.isfinite(a).all(), "non-finite values in the GPU result"
    return float(d.max())


def half_ulp_bf16(ref):
    """Half a bf16 unit in the last place at each reference value (bf16 keeps 8
    significant bits): the error a correctly rounded bf16 output may carry."""
    a = np.abs(np.asarray(ref, dtype=np.float64))
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -126)))
    return 2.0 ** (e - 8)


def grad_errors(a, ref):
    """For a bf16 gradient tensor returns (raw max abs error, max abs error on the
    elements with |ref| < 2, max of error minus the bf16 half-ulp at the reference).
    The gate of 1e-2 is applied to the last two: where |ref| >= 2 the rounding of
    the exact value to bf16 alone can exceed 1e-2 (half an ulp is 0.0156 in [4, 8)),
    so there the gate bounds the error in excess of that rounding."""
    a = a.detach().to("cpu").to(torch.float64).numpy()
    assert np.isfinite(a).all(), "non-finite values in the GPU result"
    if a.size == 0:
        return 0.0, 0.0, 0.0
    err = np.abs(a - ref)
    small = np.abs(ref) < 2.0
    return (float(err.max()), float(err[small].max(initial=0.0)),
            float((err - half_ulp_bf16(ref)).max()))


def read_status(status):
    torch.cuda.synchronize()
    return int(status.item())
