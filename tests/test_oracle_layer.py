"""Pin for the oracle's attention layer (projections, rotary embedding on the shared layout's
position ids, attention under the prefix-sharing mask, output projection) and its gradient:
the same layer written with library routines (torch matmul, the transformers library's rotary
embedding, torch's scaled_dot_product_attention with a boolean mask) in float64, differentiated
by autograd."""
import numpy as np
import torch

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import workloads as wl


def test_attention_layer_and_gradient_match_library_routines_and_autograd():
    from transformers.models.llama.modeling_llama import apply_rotary_pos_emb
    pack = wl.pack_from_lengths("layer", [(5, 4, 3), (0, 2, 6), (7, 3, 0)], 4, 2, 8)
    T, Hq, Hkv, d, hid, theta = pack.total_tokens, 4, 2, 8, 24, 10000.0
    rng = np.random.default_rng(3)
    x = rng.normal(size=(T, hid)); d_out = rng.normal(size=(T, hid))
    wq, wk, wv = rng.normal(size=(hid, Hq * d)) * 0.3, rng.normal(size=(hid, Hkv * d)) * 0.3, rng.normal(size=(hid, Hkv * d)) * 0.3
    wo = rng.normal(size=(Hq * d, hid)) * 0.3
    pos = orc.position_ids(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)

    out, _ = orc.attention_layer_fwd(x, wq, wk, wv, wo, pos, mask, Hq, Hkv, theta)
    grads = orc.attention_layer_bwd(x, wq, wk, wv, wo, pos, mask, Hq, Hkv, d_out, theta)

    tx, twq, twk, twv, two = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (x, wq, wk, wv, wo))
    inv_freq = theta ** (-torch.arange(0, d, 2, dtype=torch.float64) / d)
    ang = torch.tensor(pos, dtype=torch.float64)[:, None] * inv_freq[None, :]
    emb = torch.cat([ang, ang], dim=-1)[None]
    tq = (tx @ twq).view(T, Hq, d).permute(1, 0, 2)[None]
    tk = (tx @ twk).view(T, Hkv, d).permute(1, 0, 2)[None]
    tv = (tx @ twv).view(T, Hkv, d).permute(1, 0, 2)[None]
    tq, tk = apply_rotary_pos_emb(tq, tk, emb.cos(), emb.sin())
    g = Hq // Hkv
    to = torch.nn.functional.scaled_dot_product_attention(
        tq, tk.repeat_interleave(g, dim=1), tv.repeat_interleave(g, dim=1), attn_mask=torch.tensor(mask)[None, None])
    tout = to[0].permute(1, 0, 2).reshape(T, Hq * d) @ two
    (tout * torch.tensor(d_out)).sum().backward()

    assert np.allclose(out, tout.detach().numpy(), atol=1e-11)
    for name, t in (("dx", tx), ("dwq", twq), ("dwk", twk), ("dwv", twv), ("dwo", two)):
        assert np.allclose(grads[name], t.grad.numpy(), atol=1e-10), name
