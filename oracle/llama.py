"""Decoder attention layer (prefill): RMSNorm -> fused QKV linear -> head split/transpose ->
RoPE -> causal attention -> head merge -> output linear.  Every layout operator is
materialised.  Test infrastructure only."""
from __future__ import annotations

import numpy as np

from . import layout, ops


def causal_attention(q, k, v):
    """q,k,v [H,S,D] -> [H,S,D]; position i attends to j <= i; scores scaled by D^-1/2."""
    H, S, D = q.shape
    out = np.empty_like(q)
    allowed = np.tril(np.ones((S, S), dtype=bool))
    for h in range(H):
        kt = layout.transpose(k[h], (1, 0))
        sc = (q[h] @ kt) * (float(D) ** -0.5)
        sc = np.where(allowed, sc, -np.inf)
        out[h] = ops.softmax(sc) @ v[h]
    return out


def attn_layer(x, p, *, heads, head_dim, eps=1e-5, theta=10000.0, add_residual=False, keep=None):
    """x [B,S,hidden] fp64 -> [B,S,hidden]."""
    B, S, hidden = x.shape
    outs = []
    for b in range(B):
        xn = ops.rmsnorm(x[b], p["rms_g"], eps)                                   # L1
        qkv = ops.linear(xn, p["w_qkv"])                                          # L2 [S,3*hidden]
        t = layout.transpose(layout.reshape(qkv, (S, 3, heads, head_dim)), (1, 2, 0, 3))  # L3
        q, k, v = t[0], t[1], t[2]                                                # [H,S,D] each
        q = ops.rope(q, theta)                                                    # L4
        k = ops.rope(k, theta)
        o = causal_attention(q, k, v)                                             # L5
        om = layout.reshape(layout.transpose(o, (1, 0, 2)), (S, hidden))          # L6
        out = ops.linear(om, p["w_o"])                                            # L7
        if add_residual:
            out = out + x[b]
        if keep is not None and b == 0:
            keep.update(xn=xn, qkv=qkv, q=q, k=k, v=v, o=o, om=om)
        outs.append(out)
    return np.stack(outs)
