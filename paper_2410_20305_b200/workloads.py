"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no arithmetic of the method: only sample-length draws, the
packing of those samples into one row, and random tensors.  Both the CUDA
path's tests and the CPU oracle's tests read their inputs from here so that
the two sides see identical bits.

The paper measures on public preference datasets (Section 4.3, Tables 1-2);
those are not available, so the length distributions below stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch


@dataclass
class Pack:
    """One packed row of prefix-shared samples."""
    name: str
    cu_seqlens: np.ndarray      # int32 [n+1]
    prefix_len: np.ndarray      # int32 [n]
    chosen_len: np.ndarray      # int32 [n]
    rejected_len: np.ndarray    # int32 [n]
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    pack_len: int               # the fixed packing length the row was filled towards

    @property
    def n_samples(self) -> int:
        return len(self.prefix_len)

    @property
    def total_tokens(self) -> int:
        return int(self.cu_seqlens[-1])

    def paired(self) -> "Pack":
        """The same samples in the unshared paired layout: 2n causal sequences
        [prompt | chosen] and [prompt | rejected] (rejected_len = 0)."""
        P = np.repeat(self.prefix_len, 2)
        C = np.stack([self.chosen_len, self.rejected_len], axis=1).reshape(-1)
        R = np.zeros_like(P)
        cu = np.zeros(len(P) + 1, dtype=np.int32)
        cu[1:] = np.cumsum(P + C)
        return Pack(self.name + "-paired", cu, P.astype(np.int32), C.astype(np.int32),
                    R.astype(np.int32), self.n_q_heads, self.n_kv_heads, self.head_dim,
                    self.pack_len * 2)


def pack_from_lengths(name, lengths, n_q_heads, n_kv_heads, head_dim, pack_len=0) -> Pack:
    P = np.array([l[0] for l in lengths], dtype=np.int32)
    C = np.array([l[1] for l in lengths], dtype=np.int32)
    R = np.array([l[2] for l in lengths], dtype=np.int32)
    cu = np.zeros(len(lengths) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(P + C + R)
    return Pack(name, cu, P, C, R, n_q_heads, n_kv_heads, head_dim, pack_len or int(cu[-1]))


def _lognormal_clipped(rng, median, sigma, lo, hi):
    return int(np.clip(np.round(rng.lognormal(np.log(median), sigma)), lo, hi))


def _fill(rng, draw, pack_len):
    """Draw samples in order; stop at the first one that does not fit."""
    out, used = [], 0
    while True:
        p, c, r = draw(rng)
        if used + p + c + r > pack_len:
            break
        out.append((p, c, r))
        used += p + c + r
    return out


CONFIG_NAMES = ("tiny", "llama3-8b", "long-prompt", "multi-turn", "short-many")


def _length_recipe(index: int):
    """(draw, pack_len) of workload 1..4: draw(rng) -> (P, C, R)."""
    if index == 1:
        draw = lambda g: (_lognormal_clipped(g, 600, 1.0, 64, 4096),
                          _lognormal_clipped(g, 250, 1.0, 16, 1024),
                          _lognormal_clipped(g, 250, 1.0, 16, 1024))
        pack_len = 16384
    elif index == 2:
        draw = lambda g: (int(g.integers(1024, 3073)), int(g.integers(32, 129)), int(g.integers(32, 129)))
        pack_len = 16384
    elif index == 3:
        draw = lambda g: (int(g.integers(200, 4001)), int(g.integers(100, 801)), int(g.integers(100, 801)))
        pack_len = 32768
    elif index == 4:
        draw = lambda g: (int(g.integers(64, 257)), int(g.integers(64, 257)), int(g.integers(64, 257)))
        pack_len = 8192
    else:
        raise ValueError("config index 1..4")
    return draw, pack_len


def config_pack(index: int, seed: int | None = None) -> Pack:
    """Workload `index` (0..4).  Lengths are drawn from
    numpy.random.default_rng(1000 + index) unless a seed is given."""
    rng = np.random.default_rng(1000 + index if seed is None else seed)
    if index == 0:
        return pack_from_lengths("tiny", [(256, 64, 96), (128, 80, 48)], 4, 4, 64)
    draw, pack_len = _length_recipe(index)
    return pack_from_lengths(CONFIG_NAMES[index], _fill(rng, draw, pack_len), 32, 8, 128, pack_len)


def sample_lengths(index: int, n: int, seed: int):
    """n samples (P, C, R) of workload 1..4's length distribution, and its pack length."""
    draw, pack_len = _length_recipe(index)
    rng = np.random.default_rng(seed)
    return [draw(rng) for _ in range(n)], pack_len


def random_pack(seed, n_samples, max_len, n_q_heads, n_kv_heads, head_dim, allow_zero=True) -> Pack:
    """Small ragged packs for parity tests: odd lengths, occasional zero-length
    prompt / chosen / rejected parts."""
    rng = np.random.default_rng(seed)
    lengths = []
    for _ in range(n_samples):
        while True:
            p, c, r = (int(rng.integers(0 if allow_zero else 1, max_len + 1)) for _ in range(3))
            if allow_zero and rng.random() < 0.15:
                which = int(rng.integers(0, 3))
                p, c, r = (0 if which == 0 else p), (0 if which == 1 else c), (0 if which == 2 else r)
            if p + c + r >= 1:
                break
        lengths.append((p, c, r))
    return pack_from_lengths("random-%d" % seed, lengths, n_q_heads, n_kv_heads, head_dim)


def bf16_normal(shape, seed, std=1.0, device="cpu") -> torch.Tensor:
    """N(0, std^2) rounded to bf16; generated on the CPU so the bits do not
    depend on the device, then moved."""
    g = torch.Generator(device="cpu").manual_seed(int(seed))
    x = torch.randn(shape, generator=g, dtype=torch.float32) * std
    return x.to(torch.bfloat16).to(device)


def attention_inputs(pack: Pack, seed: int, std: float = 1.0, device="cpu"):
    """q [T,Hq,d], k, v [T,Hkv,d], d_o [T,Hq,d], all bf16."""
    T, Hq, Hkv, d = pack.total_tokens, pack.n_q_heads, pack.n_kv_heads, pack.head_dim
    q = bf16_normal((T, Hq, d), seed * 4 + 0, std, device)
    k = bf16_normal((T, Hkv, d), seed * 4 + 1, std, device)
    v = bf16_normal((T, Hkv, d), seed * 4 + 2, std, device)
    d_o = bf16_normal((T, Hq, d), seed * 4 + 3, std, device)
    return q, k, v, d_o


def to_f64(x: torch.Tensor) -> np.ndarray:
    """Exact upcast of a (bf16/fp32) tensor to a float64 numpy array."""
    return x.detach().to("cpu").to(torch.float64).numpy()


def logits_and_tokens(n_rows, vocab, seed, std, dtype=torch.float32, device="cpu"):
    """Random logits [n_rows, vocab] ~ N(0, std^2) in `dtype`, and uniform random
    token ids int32 [n_rows]."""
    g = torch.Generator(device="cpu").manual_seed(int(seed))
    x = (torch.randn((n_rows, vocab), generator=g, dtype=torch.float32) * std).to(dtype).to(device)
    tok = torch.randint(0, vocab, (n_rows,), generator=g, dtype=torch.int32)
    return x, tok
