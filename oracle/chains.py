"""Operator chains: a list of layout operators applied one after another, each
materialised, followed by a consumer.  Test infrastructure only.

An operator is a dict: {"op": "reshape", "shape": [...]}, {"op": "transpose", "perm": [...]},
{"op": "roll", "shift": s, "axis": a}, {"op": "slice", "start": [...], "extent": [...]},
{"op": "window_partition", "window": ws}, {"op": "window_reverse", "window": ws, "B":.., "H":.., "W":..},
{"op": "depth_to_space", "block": b}, {"op": "space_to_depth", "block": b}.
"""
from __future__ import annotations

import numpy as np

from . import layout, ops


def apply_layout_chain(x: np.ndarray, chain) -> np.ndarray:
    y = x
    for o in chain:
        kind = o["op"]
        if kind == "reshape":
            y = layout.reshape(y, o["shape"])
        elif kind == "transpose":
            y = layout.transpose(y, o["perm"])
        elif kind == "roll":
            y = layout.roll(y, o["shift"], o["axis"])
        elif kind == "slice":
            y = layout.slice_(y, o["start"], o["extent"])
        elif kind == "window_partition":
            y = layout.window_partition(y, o["window"])
        elif kind == "window_reverse":
            y = layout.window_reverse(y, o["window"], o["B"], o["H"], o["W"])
        elif kind == "depth_to_space":
            y = layout.depth_to_space(y, o["block"])
        elif kind == "space_to_depth":
            y = layout.space_to_depth(y, o["block"])
        else:
            raise ValueError(f"not a layout operator: {kind}")
    return y


def source_offsets(shape, chain) -> np.ndarray:
    """For every element of the chain's output (in its row-major order) the linear offset
    of the input element it came from: push arange through the materialised operators.
    This is what an eliminated chain's composed index map must reproduce."""
    n = int(np.prod(shape))
    ids = np.arange(n, dtype=np.int64).reshape(shape)
    return apply_layout_chain(ids, chain)


def chain_2a_scores(xq: np.ndarray, xk: np.ndarray, heads: int) -> np.ndarray:
    """[B,S,H*D] x2 -> reshape [B,S,H,D] -> transpose (0,2,1,3) -> scores[b,h,i,j] = sum_e Q K."""
    B, S, HD = xq.shape
    D = HD // heads
    ch = [{"op": "reshape", "shape": (B, S, heads, D)}, {"op": "transpose", "perm": (0, 2, 1, 3)}]
    q = apply_layout_chain(xq, ch)
    k = apply_layout_chain(xk, ch)
    return q @ layout.transpose(k, (0, 1, 3, 2))


def chain_2b_gemm(x: np.ndarray, w: np.ndarray) -> np.ndarray:
    """NCHW -> transpose (0,2,3,1) -> reshape [B*H*W, C] -> out = A w^T."""
    B, C, H, W = x.shape
    a = apply_layout_chain(x, [{"op": "transpose", "perm": (0, 2, 3, 1)}, {"op": "reshape", "shape": (B * H * W, C)}])
    return a @ w.T


def fanout(x: np.ndarray, w_p: np.ndarray, w_a: np.ndarray, w_b: np.ndarray, B: int, S: int):
    """A producer with two consumers of different reduction dimensions (Section 3.2.2, "Global"):
    P = x w_p^T as [B, S, N];  YA = P w_a^T aggregates along N;  YB[b] = P[b]^T w_b^T aggregates along S.
    The layout of P is the implementation's business: the results do not depend on it.  Returns (YA [B*S, Na], YB [B, N, Nb])."""
    P = ops.linear(x, w_p)                               # [B*S, N]
    ya = ops.linear(P, w_a)
    P3 = layout.reshape(P, (B, S, P.shape[1]))
    yb = np.stack([layout.transpose(P3[b], (1, 0)) @ w_b.T for b in range(B)])
    return ya, yb
