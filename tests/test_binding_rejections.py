"""Host-side rejections that need no GPU: tensors whose shape does not match the plan (the
kernels size their tensor maps and grids from the plan alone, so such a call must never reach
them), plans without a device copy, and the reading of the device status word."""
import numpy as np
import pytest
import torch

from paper_2410_20305_b200 import binding as B
from paper_2410_20305_b200 import workloads as wl


def host_plan(pack):
    return B.psa_plan(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len,
                      pack.n_q_heads, pack.n_kv_heads, pack.head_dim, host_only=True)


def tensors(pack, T=None):
    T = pack.total_tokens if T is None else T
    bf = lambda h: torch.zeros((T, h, pack.head_dim), dtype=torch.bfloat16)
    return {"q": bf(pack.n_q_heads), "k": bf(pack.n_kv_heads), "v": bf(pack.n_kv_heads), "o": bf(pack.n_q_heads),
            "d_o": bf(pack.n_q_heads), "lse": torch.zeros((pack.n_q_heads, T), dtype=torch.float32)}


@pytest.mark.parametrize("wrong", ["q", "k", "o", "d_o", "lse", "dq", "dk", "dv"])
def test_backward_wrappers_refuse_tensors_of_another_pack(wrong):
    pack = wl.config_pack(0)
    plan = host_plan(pack)
    for fn in (B.psa_bwd, B.psa_bwd_f32, B.psa_bwd_static_scratch):
        t = tensors(pack)
        small = tensors(pack, pack.total_tokens - 1)
        gdt = torch.float32 if fn is B.psa_bwd_f32 else torch.bfloat16
        grads = {"dq": torch.zeros_like(t["q"], dtype=gdt), "dk": torch.zeros_like(t["k"], dtype=gdt),
                 "dv": torch.zeros_like(t["v"], dtype=gdt)}
        if wrong in grads:
            grads[wrong] = grads[wrong][:-1].contiguous()
        else:
            t[wrong] = small[wrong]
        with pytest.raises(ValueError, match=wrong + ":"):
            fn(plan, t["d_o"], t["q"], t["k"], t["v"], t["o"], t["lse"], grads["dq"], grads["dk"], grads["dv"])


def test_forward_and_step_host_refuse_wrong_shapes_and_dtypes():
    pack = wl.config_pack(0)
    plan = host_plan(pack)
    t = tensors(pack)
    with pytest.raises(ValueError, match="k:"):
        B.psa_fwd(plan, t["q"], t["k"][:, :1].contiguous(), t["v"])
    with pytest.raises(ValueError, match="q: dtype"):
        B.psa_fwd(plan, t["q"].float(), t["k"], t["v"])
    with pytest.raises(ValueError, match="CUDA"):
        B.psa_fwd(plan, t["q"], t["k"], t["v"])          # right shapes, but host tensors
    arena = torch.zeros(16, dtype=torch.uint8)
    with pytest.raises(ValueError, match="h_dk:"):
        B.psa_step_host(plan, t["q"], t["k"], t["v"], t["d_o"], t["o"], t["lse"], t["q"].clone(),
                        t["k"][:-1].contiguous(), t["v"].clone(), arena)


def test_calls_on_a_plan_without_device_copy_return_invalid_arg():
    pack = wl.config_pack(0)
    plan = host_plan(pack)
    lib = B.load_library()
    buf = np.zeros(64, dtype=np.uint8).ctypes.data     # never dereferenced: the plan is refused first
    assert lib.psa_fwd(plan._h, buf, buf, buf, buf, buf, None, None) == 1
    assert lib.psa_bwd(plan._h, buf, buf, buf, buf, buf, buf, buf, buf, buf, buf, None, None) == 1
    assert lib.psa_bwd_f32(plan._h, buf, buf, buf, buf, buf, buf, buf, buf, buf, buf, None, None) == 1
    assert lib.psa_bwd_static_scratch(plan._h, buf, buf, buf, buf, buf, buf, buf, buf, buf, None, None) == 1


def test_device_status_word_maps_to_status_codes():
    assert B.psa_check_device_status(0) == 0
    assert B.psa_check_device_status(B.PSA_DEVSTAT_WAIT_EXPIRED) == 7
    assert B.psa_check_device_status(B.PSA_DEVSTAT_WAIT_EXPIRED | B.PSA_DEVSTAT_BAD_TARGET) == 7
    assert B.psa_check_device_status(B.PSA_DEVSTAT_BAD_TARGET) == 6
    assert B.psa_check_device_status(B.PSA_DEVSTAT_BAD_SEGMENT) == 6
    lib = B.load_library()
    assert lib.psa_selftest_wait_expiry(None, 1000, None, None) == 1     # refused before any launch
