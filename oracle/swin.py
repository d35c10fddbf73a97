"""One Swin Transformer block, every operator of the unoptimised graph executed in order
and every layout operator materialised.  Test infrastructure only.

Step numbers S1..S17 name the operators of the chain: LayerNorm, cyclic shift, window
partition, QKV linear, head split, K transpose, scores, relative-position bias,
shifted-window mask, softmax, P.V, head merge, window reverse, reverse shift, proj linear,
residual, then the MLP half (LayerNorm, fc1, GELU, fc2, residual).
"""
from __future__ import annotations

import numpy as np

from . import layout, ops


def window_attention(q, k, v, bias_table, ws, mask=None, keep=None):
    """q,k,v [nW,nH,T,d] -> [nW,nH,T,d].  scores = d^-1/2 q k^T + bias[idx] (+ mask), softmax, P v."""
    nW, nH, T, d = q.shape
    kt = layout.transpose(k, (0, 1, 3, 2))                               # S6: K^T materialised
    scores = (q @ kt) * (float(d) ** -0.5)                               # S7
    idx = ops.rel_pos_index(ws)                                          # [T,T]
    bias = layout.transpose(bias_table[idx.reshape(-1)].reshape(T, T, nH), (2, 0, 1))
    scores = scores + bias[None]                                         # S8
    if mask is not None:                                                 # S9
        nWin = mask.shape[0]
        scores = scores + np.tile(mask, (nW // nWin, 1, 1))[:, None, :, :]
    p = ops.softmax(scores)                                              # S10
    if keep is not None:
        keep["scores"] = scores
        keep["p"] = p
    return p @ v                                                         # S11


def swin_block(x, p, *, heads, window, shift, mlp_ratio, eps=1e-5, keep=None):
    """x [B,H,W,C] fp64, p = dict of fp64 parameters ([out,in] weights).  Returns y (attention
    half only when mlp_ratio == 0).  `keep`, if a dict, receives intermediates."""
    B, H, W, C = x.shape
    ws, s = window, shift
    xn = ops.layernorm(x, p["ln1_g"], p["ln1_b"], eps)                   # S1
    xs = layout.cyclic_shift(xn, s) if s > 0 else xn                     # S2
    xw = layout.window_partition(xs, ws)                                 # S3  [nW,T,C]
    qkv = ops.linear(xw, p["w_qkv"], p["b_qkv"])                         # S4  [nW,T,3C]
    q, k, v = layout.head_split(qkv, heads)                              # S5
    mask = ops.shifted_window_mask(H, W, ws, s) if s > 0 else None
    o = window_attention(q, k, v, p["rel_bias_table"], ws, mask, keep)   # S6-S11
    om = layout.head_merge(o)                                            # S12 [nW,T,C]
    orev = layout.window_reverse(om, ws, B, H, W)                        # S13a
    ouns = layout.cyclic_unshift(orev, s) if s > 0 else orev             # S13b
    pr = ops.linear(ouns, p["w_proj"], p["b_proj"])                      # S13c
    y = x + pr                                                           # S13d
    if keep is not None:
        keep.update(xn=xn, xw=xw, qkv=qkv, q=q, k=k, v=v, o=o, om=om, y=y)
    if mlp_ratio == 0:
        return y
    yn = ops.layernorm(y, p["ln2_g"], p["ln2_b"], eps)                   # S14
    h = ops.gelu(ops.linear(yn, p["w_fc1"], p["b_fc1"]))                 # S15
    z = y + ops.linear(h, p["w_fc2"], p["b_fc2"])                        # S16, S17
    if keep is not None:
        keep.update(yn=yn, h=h)
    return z


def patch_merging(x, gamma, beta, w, eps=1e-5):
    """Swin patch merging between stages: [B,H,W,C] -> [B, H/2*W/2, 2C]: the 2x2 neighbourhood gathered to 4C
    channels (Slice x4 + Concat), LayerNorm over 4C, linear 4C -> 2C without bias (w [2C,4C])."""
    return ops.linear(ops.layernorm(layout.patch_merge_gather(x), gamma, beta, eps), w)
