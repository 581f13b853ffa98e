"""The attention layer as composed in paper_2410_20305_b200/layer.py (library GEMMs for the
projections; psa_rope, psa_fwd, psa_bwd for the rest) against the oracle's float64 layer.
Every stage rounds its result to bf16 (2^-9 relative), so the comparison is relative to the
largest magnitude of each output: 2 % covers the six roundings on the longest path
(projection, rotation, attention, its gradient, inverse rotation, projection)."""
import numpy as np
import pytest
import torch

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import workloads as wl
from paper_2410_20305_b200.layer import AttentionLayer

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("d,hq,hkv", [(64, 4, 2), (128, 4, 1)])
def test_layer_forward_and_backward_match_the_oracle(d, hq, hkv):
    pack = wl.pack_from_lengths("layer", [(150, 60, 90), (0, 40, 70), (200, 33, 0), (31, 129, 5)], hq, hkv, d)
    T, hid = pack.total_tokens, hq * d
    bf = lambda shape, seed, std: wl.bf16_normal(shape, seed, std)
    x, d_out = bf((T, hid), 1, 1.0), bf((T, hid), 2, 1.0)
    std = hid ** -0.5        # unit-variance q, k, v and outputs
    wq, wk, wv, wo = bf((hid, hq * d), 3, std), bf((hid, hkv * d), 4, std), bf((hid, hkv * d), 5, std), bf((hq * d, hid), 6, std)
    layer = AttentionLayer((pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len), hq, hkv, d, "cuda")
    dev = [t.cuda() for t in (x, wq, wk, wv, wo)]
    out, saved = layer.forward(*dev)
    grads = layer.backward(*dev, saved, d_out.cuda())
    torch.cuda.synchronize()

    f = wl.to_f64
    pos = orc.position_ids(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    rout, _ = orc.attention_layer_fwd(f(x), f(wq), f(wk), f(wv), f(wo), pos, mask, hq, hkv)
    rg = orc.attention_layer_bwd(f(x), f(wq), f(wk), f(wv), f(wo), pos, mask, hq, hkv, f(d_out))
    for name, got, ref in [("out", out, rout)] + [(n, g, rg[n]) for n, g in zip(("dx", "dwq", "dwk", "dwv", "dwo"), grads)]:
        got = f(got)
        assert np.isfinite(got).all()
        rel = np.abs(got - ref).max() / np.abs(ref).max()
        print("layer %s: max error / max magnitude = %.4f" % (name, rel))
        assert rel <= 2e-2, (name, rel)
