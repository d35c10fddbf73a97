"""Compute operators as their plain definitions, fp64.  Test infrastructure only."""
from __future__ import annotations

import math

import numpy as np
from scipy.special import erf as _erf   # library primitive; pinned against math.erf and Phi(1)


def layernorm(x: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float) -> np.ndarray:
    """LayerNorm over the last dim (Table 3, ILD & Variable): biased variance,
    y = (x - mean) / sqrt(var + eps) * gamma + beta."""
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * gamma + beta


def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """y = x * g / sqrt(mean(x^2) + eps) over the last dim."""
    ms = (x * x).mean(axis=-1, keepdims=True)
    return x * g / np.sqrt(ms + eps)


def linear(x: np.ndarray, w: np.ndarray, b=None) -> np.ndarray:
    """MatMul (Table 3): y[.., n] = sum_k x[.., k] * w[n, k] (+ b[n]).  The reduction
    dimension k is the contiguous one of both operands (Section 3.2.2)."""
    y = x @ w.T
    if b is not None:
        y = y + b
    return y


def gelu(u: np.ndarray) -> np.ndarray:
    """Exact (erf) GELU: u/2 * (1 + erf(u / sqrt 2))."""
    return 0.5 * u * (1.0 + _erf(u / math.sqrt(2.0)))


def softmax(s: np.ndarray) -> np.ndarray:
    """Softmax over the last dim with max subtraction (Table 3, ILD & Variable)."""
    m = s.max(axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / e.sum(axis=-1, keepdims=True)


def rel_pos_index(ws: int) -> np.ndarray:
    """[T,T] index into the relative-position bias table of (2ws-1)^2 rows:
    token t sits at (y,x) = (t div ws, t mod ws);
    idx(i,j) = (y_i - y_j + ws - 1) * (2ws - 1) + (x_i - x_j + ws - 1)."""
    T = ws * ws
    idx = np.zeros((T, T), dtype=np.int64)
    for i in range(T):
        for j in range(T):
            yi, xi = divmod(i, ws)
            yj, xj = divmod(j, ws)
            idx[i, j] = (yi - yj + ws - 1) * (2 * ws - 1) + (xi - xj + ws - 1)
    return idx


def shifted_window_mask(H: int, W: int, ws: int, s: int) -> np.ndarray:
    """[nWh*nWw, T, T] additive mask (0 or -100) of the shifted-window block.

    Region labels live in SHIFTED coordinates: r(u,N) = 0 for u < N-ws, 1 for
    N-ws <= u < N-s, 2 otherwise; label = 3 r(h',H) + r(w',W).  The label image is window
    partitioned like a [1,H,W,1] tensor; two tokens of a window may attend to each other
    iff their labels are equal."""
    from . import layout

    def r(u, n):
        return 0 if u < n - ws else (1 if u < n - s else 2)

    lab = np.zeros((1, H, W, 1), dtype=np.float64)
    for h in range(H):
        for w in range(W):
            lab[0, h, w, 0] = 3 * r(h, H) + r(w, W)
    lab_w = layout.window_partition(lab, ws)[:, :, 0]          # [nWin, T]
    eq = lab_w[:, :, None] == lab_w[:, None, :]
    return np.where(eq, 0.0, -100.0)


def rope(x: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding on [.., S, D] (position = index along the second-to-last dim),
    half-split pairing: for i in [0, D/2): f_i = theta^(-2i/D), phi = p * f_i,
    (x_i, x_{i+D/2}) <- (x_i cos phi - x_{i+D/2} sin phi, x_{i+D/2} cos phi + x_i sin phi)."""
    S, D = x.shape[-2], x.shape[-1]
    half = D // 2
    f = np.array([theta ** (-(2.0 * i) / D) for i in range(half)], dtype=np.float64)
    phi = np.arange(S, dtype=np.float64)[:, None] * f[None, :]
    c, sn = np.cos(phi), np.sin(phi)
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * sn, b * c + a * sn], axis=-1)


def rope_at(x: np.ndarray, pos: int, theta: float) -> np.ndarray:
    """Rotary embedding of vectors [.., D] that all sit at one position `pos` (the decode step of a
    decoder layer): same pairing and frequencies as `rope`, angle phi_i = pos * theta^(-2i/D)."""
    D = x.shape[-1]
    half = D // 2
    out = np.empty_like(x)
    for i in range(half):
        phi = float(pos) * theta ** (-(2.0 * i) / D)
        c, sn = np.cos(phi), np.sin(phi)
        out[..., i] = x[..., i] * c - x[..., i + half] * sn
        out[..., i + half] = x[..., i + half] * c + x[..., i] * sn
    return out


def rope_partial(x: np.ndarray, theta: float, rotary_dim: int, pos=None) -> np.ndarray:
    """Partial rotary embedding (GPT-NeoX / Pythia style): the first `rotary_dim` = R features of a head rotate in
    pairs (i, i + R/2) at frequencies theta^(-2i/R); features R.. pass through unchanged.  x [.., S, D]
    with position = index along the second-to-last dim, or, when `pos` is given, x [.., D] all at that position."""
    R = rotary_dim
    out = x.copy()
    for i in range(R // 2):
        f = theta ** (-(2.0 * i) / R)
        if pos is None:
            phi = np.arange(x.shape[-2], dtype=np.float64) * f          # [S], broadcasts over leading dims
        else:
            phi = float(pos) * f
        c, sn = np.cos(phi), np.sin(phi)
        a, b = x[..., i], x[..., i + R // 2]
        out[..., i] = a * c - b * sn
        out[..., i + R // 2] = b * c + a * sn
    return out
