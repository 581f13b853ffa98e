"""Run by tests/test_gpu_debug_library.py in a process of its own with PSA_DEBUG_LIB=1, so that the
binding loads libpsa_debug.so (checked global indices).  Runs small packs through every attention entry
point and the gather, compares with the oracle, and requires that no index check fired."""
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from paper_2410_20305_b200 import binding as B            # noqa: E402
from paper_2410_20305_b200 import workloads as wl         # noqa: E402
from paper_2410_20305_b200.labels import logp_labels      # noqa: E402
from oracle import psa_oracle as orc                      # noqa: E402
from gpu_util import TOL_LSE, TOL_O, device_plan, max_abs, oracle_bwd, oracle_fwd   # noqa: E402


def main():
    lib = B.load_library()
    assert os.path.basename(lib._name) == "libpsa_debug.so", lib._name
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    result = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.psa_selftest_bounds(status, result)
    torch.cuda.synchronize()
    assert int(result.item()) == 1 and int(status.item()) == B.PSA_DEVSTAT_OUT_OF_BOUNDS, (result.item(), status.item())
    status.zero_()
    packs = [wl.config_pack(0), wl.random_pack(41, 4, 330, 8, 2, 128), wl.random_pack(42, 4, 330, 4, 4, 64),
             wl.pack_from_lengths("deg", [(0, 70, 200), (300, 0, 45), (129, 255, 0), (1, 0, 0), (1, 1, 1), (128, 128, 128), (0, 0, 5)], 4, 2, 128),
             wl.pack_from_lengths("short-prompt", [(2, 150, 190), (0, 140, 170)], 4, 2, 128)]
    for i, pack in enumerate(packs):
        q, k, v, d_o = wl.attention_inputs(pack, 50 + i)
        plan = device_plan(pack)
        qd, kd, vd, dod = q.cuda(), k.cuda(), v.cuda(), d_o.cuda()
        o, lse = B.psa_fwd(plan, qd, kd, vd, status=status)
        B.psa_bwd(plan, dod, qd, kd, vd, o, lse, status=status)
        dq, dk, dv = B.psa_bwd_f32(plan, dod, qd, kd, vd, o, lse, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0, (pack.name, int(status.item()))
        ro, rl = oracle_fwd(pack, q, k, v)
        rdq, rdk, rdv = oracle_bwd(pack, q, k, v, d_o)
        assert max_abs(lse, rl) <= TOL_LSE and max_abs(o, ro) <= 1.6e-2, pack.name     # (o: bf16 output, few-key rows)
        assert max(max_abs(dq, rdq), max_abs(dk, rdk), max_abs(dv, rdv)) <= TOL_O, pack.name
    pack = packs[0]
    x, tok = wl.logits_and_tokens(pack.total_tokens, 1024, 0, 2.0 ** 0.5)
    targets, seg, fr, ft, fs = logp_labels(tok.numpy(), pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    dev = lambda a: torch.as_tensor(np.asarray(a, dtype=np.int32)).cuda()
    lp = B.dpo_logp(x.cuda(), dev(targets), dev(seg), 2 * pack.n_samples, dev(fr), dev(ft), dev(fs), status=status)
    torch.cuda.synchronize()
    want = orc.dpo_logp(wl.to_f64(x), targets, seg, 2 * pack.n_samples, fr, ft, fs)
    assert int(status.item()) == 0 and np.allclose(lp.cpu().double().numpy(), want, rtol=1e-3)
    print("DEBUG_LIBRARY_OK")


if __name__ == "__main__":
    main()
