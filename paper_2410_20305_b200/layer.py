"""One attention layer on the shared layout (Section 4.2: the full attention-layer benchmark):
query / key / value projections, rotary embedding on the position ids of Section 3.1,
psa_fwd, output projection, and the backward of all of it.

The projections are library GEMMs (torch.matmul, i.e. cuBLAS); the rotary embedding, the
attention and its backward are this library's kernels.  A composition for the layer-level
measurement and its parity test, not a kernel of its own.
"""
from __future__ import annotations

from . import binding as B


class AttentionLayer:
    """Holds a plan, the position ids and the scratch of one pack; `forward` and `backward`
    run the layer for bf16 CUDA inputs x [T, hidden] and weights wq [hidden, Hq d],
    wk, wv [hidden, Hkv d], wo [Hq d, hidden]."""

    def __init__(self, pack_lengths, n_q_heads, n_kv_heads, head_dim, device, rope_theta=10000.0):
        import torch
        cu, P, C, R = pack_lengths
        self.plan = B.psa_plan(cu, P, C, R, n_q_heads, n_kv_heads, head_dim)
        self.pos = torch.as_tensor(B.psa_position_ids(cu, P, C, R)).to(device)
        self.neg = -self.pos
        self.ws = torch.empty(max(self.plan.bwd_workspace_bytes, 256), dtype=torch.uint8, device=device)
        self.theta = float(rope_theta)
        self.Hq, self.Hkv, self.d = n_q_heads, n_kv_heads, head_dim

    def forward(self, x, wq, wk, wv, wo):
        T = x.shape[0]
        q = (x @ wq).view(T, self.Hq, self.d)
        k = (x @ wk).view(T, self.Hkv, self.d)
        v = (x @ wv).view(T, self.Hkv, self.d)
        B.psa_rope(q, self.pos, self.theta, out=q)
        B.psa_rope(k, self.pos, self.theta, out=k)
        o, lse = B.psa_fwd(self.plan, q, k, v)
        out = o.view(T, self.Hq * self.d) @ wo
        return out, (q, k, v, o, lse)

    def backward(self, x, wq, wk, wv, wo, saved, d_out):
        """Returns (dx, dwq, dwk, dwv, dwo) for the loss sum(out * d_out)."""
        q, k, v, o, lse = saved
        T = x.shape[0]
        d_o = (d_out @ wo.t()).view(T, self.Hq, self.d)
        dwo = o.view(T, self.Hq * self.d).t() @ d_out
        dq, dk, dv = B.psa_bwd(self.plan, d_o, q, k, v, o, lse, workspace=self.ws)
        # the gradient of a rotation is the inverse rotation
        B.psa_rope(dq, self.neg, self.theta, out=dq)
        B.psa_rope(dk, self.neg, self.theta, out=dk)
        dq2, dk2, dv2 = dq.view(T, -1), dk.view(T, -1), dv.view(T, -1)
        dx = dq2 @ wq.t() + dk2 @ wk.t() + dv2 @ wv.t()
        return dx, x.t() @ dq2, x.t() @ dk2, x.t() @ dv2, dwo
