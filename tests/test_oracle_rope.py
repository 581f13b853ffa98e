"""Pins for the oracle's position ids (Section 3.1) and rotary embedding."""
import numpy as np
import torch

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import workloads as wl


def test_position_ids_hand_example():
    # samples (P,C,R) = (2,2,3) and (0,1,2): rejected tokens restart right after the prompt
    got = orc.position_ids([0, 7, 10], [2, 0], [2, 1], [3, 2])
    assert list(got) == [0, 1, 2, 3, 2, 3, 4, 0, 0, 1]


def test_rope_matches_the_transformers_library_routine():
    from transformers.models.llama.modeling_llama import apply_rotary_pos_emb
    T, H, d, theta = 37, 3, 16, 500000.0
    x = np.random.default_rng(0).normal(size=(T, H, d))
    pos = np.random.default_rng(1).integers(0, 5000, size=T)
    inv_freq = theta ** (-torch.arange(0, d, 2, dtype=torch.float64) / d)
    ang = torch.tensor(pos, dtype=torch.float64)[:, None] * inv_freq[None, :]
    emb = torch.cat([ang, ang], dim=-1)[None]                       # [1, T, d]
    tq = torch.tensor(x).permute(1, 0, 2)[None]                     # [1, H, T, d]
    want, _ = apply_rotary_pos_emb(tq, tq, emb.cos(), emb.sin())
    got = orc.rope(x, pos, theta)
    assert np.allclose(got, want[0].permute(1, 0, 2).numpy(), atol=1e-12)


def test_rope_is_a_rotation_and_depends_on_relative_position_only():
    T, H, d = 9, 2, 8
    rng = np.random.default_rng(2)
    q, k = rng.normal(size=(T, H, d)), rng.normal(size=(T, H, d))
    pos = rng.integers(0, 1000, size=T)
    rq, rk = orc.rope(q, pos), orc.rope(k, pos)
    assert np.allclose(np.linalg.norm(rq, axis=-1), np.linalg.norm(q, axis=-1))
    assert np.allclose(orc.rope(q, np.zeros(T)), q)
    shifted_q, shifted_k = orc.rope(q, pos + 123), orc.rope(k, pos + 123)
    s0 = np.einsum("ihd,jhd->hij", rq, rk)
    s1 = np.einsum("ihd,jhd->hij", shifted_q, shifted_k)
    assert np.allclose(s0, s1, atol=1e-9)


def test_shared_layout_with_reset_positions_equals_the_paired_format():
    """Rotary embedding with the shared layout's position ids, then attention under the shared
    mask, gives each response exactly what the paired format gives it."""
    pack = wl.pack_from_lengths("r", [(5, 4, 3), (2, 3, 4)], 2, 1, 8)
    q, k, v, _ = (wl.to_f64(t) for t in wl.attention_inputs(pack, 3))
    pos = orc.position_ids(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    o, _ = orc.attention_fwd(orc.rope(q, pos), orc.rope(k, pos), v, mask)
    for s in range(pack.n_samples):
        ds, P, C, R = int(pack.cu_seqlens[s]), int(pack.prefix_len[s]), int(pack.chosen_len[s]), int(pack.rejected_len[s])
        for idx in (np.arange(ds, ds + P + C), np.concatenate([np.arange(ds, ds + P), np.arange(ds + P + C, ds + P + C + R)])):
            L = len(idx)
            causal = np.tril(np.ones((L, L), dtype=bool))
            ordinary = np.arange(L)                                  # plain positions of an ordinary sequence
            ro, _ = orc.attention_fwd(orc.rope(q[idx], ordinary), orc.rope(k[idx], ordinary), v[idx], causal)
            assert np.allclose(o[idx][P:], ro[P:], atol=1e-12)
