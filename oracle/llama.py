"""Decoder attention layer: RMSNorm -> fused QKV linear -> head split/transpose -> RoPE -> causal
attention -> head merge -> output linear, as a prefill over S positions (`attn_layer`) and as one
decode step against a key/value cache (`decode_step`).  Every layout operator (and the cache's
Concat) is materialised.  Test infrastructure only."""
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


def attn_layer(x, p, *, heads, head_dim, eps=1e-5, theta=10000.0, add_residual=False, keep=None, rotary_dim=None):
    """x [B,S,hidden] fp64 -> [B,S,hidden].  rotary_dim: rotate only the first rotary_dim features of each head."""
    B, S, hidden = x.shape
    outs = []
    for b in range(B):
        xn = ops.rmsnorm(x[b], p["rms_g"], eps)                                   # L1
        qkv = ops.linear(xn, p["w_qkv"])                                          # L2 [S,3*hidden]
        t = layout.transpose(layout.reshape(qkv, (S, 3, heads, head_dim)), (1, 2, 0, 3))  # L3
        q, k, v = t[0], t[1], t[2]                                                # [H,S,D] each
        if rotary_dim is None:
            q = ops.rope(q, theta)                                                # L4
            k = ops.rope(k, theta)
        else:
            q = ops.rope_partial(q, theta, rotary_dim)
            k = ops.rope_partial(k, theta, rotary_dim)
        o = causal_attention(q, k, v)                                             # L5
        om = layout.reshape(layout.transpose(o, (1, 0, 2)), (S, hidden))          # L6
        out = ops.linear(om, p["w_o"])                                            # L7
        if add_residual:
            out = out + x[b]
        if keep is not None and b == 0:
            keep.update(xn=xn, qkv=qkv, q=q, k=k, v=v, o=o, om=om)
        outs.append(out)
    return np.stack(outs)


def decode_step(x, k_cache, v_cache, p, *, heads, head_dim, eps=1e-5, theta=10000.0, add_residual=False, rotary_dim=None):
    """One decode step of the same layer for B independent sequences that all hold `pos` cached
    positions.  x [B,hidden]; k_cache, v_cache [B,pos,H,D] (keys already rotated, as the prefill left
    them).  Returns (y [B,hidden], k_new [B,H,D], v_new [B,H,D]): the new token sits at position
    `pos`, its rotated key and its value are appended to the cache (Concat along the sequence axis)
    and its query attends to all pos+1 positions (the causal mask of the last row is all-true)."""
    B, hidden = x.shape
    pos = k_cache.shape[1]
    ys, kn, vn = [], [], []
    for b in range(B):
        xn = ops.rmsnorm(x[b:b + 1], p["rms_g"], eps)                              # [1,hidden]
        qkv = ops.linear(xn, p["w_qkv"])                                           # [1,3*hidden]
        t = layout.transpose(layout.reshape(qkv, (1, 3, heads, head_dim)), (1, 2, 0, 3))   # [3,H,1,D]
        if rotary_dim is None:
            q = ops.rope_at(t[0], pos, theta)
            k = ops.rope_at(t[1], pos, theta)
        else:
            q = ops.rope_partial(t[0], theta, rotary_dim, pos=pos)
            k = ops.rope_partial(t[1], theta, rotary_dim, pos=pos)
        v = t[2]
        K = np.concatenate([layout.transpose(k_cache[b], (1, 0, 2)), k], axis=1)   # [H,pos+1,D]
        V = np.concatenate([layout.transpose(v_cache[b], (1, 0, 2)), v], axis=1)
        o = np.empty((heads, 1, head_dim), dtype=np.float64)
        for h in range(heads):
            sc = (q[h] @ layout.transpose(K[h], (1, 0))) * (float(head_dim) ** -0.5)   # [1,pos+1]
            o[h] = ops.softmax(sc) @ V[h]
        om = layout.reshape(layout.transpose(o, (1, 0, 2)), (1, hidden))
        out = ops.linear(om, p["w_o"])
        if add_residual:
            out = out + x[b:b + 1]
        ys.append(out[0]); kn.append(k[:, 0]); vn.append(v[:, 0])
    return np.stack(ys), np.stack(kn), np.stack(vn)
