"""Layout operators, each materialised into a fresh C-contiguous buffer.

Test infrastructure only (see the package docstring).  Tensors are row-major: the last
dimension is contiguous, the 1-D buffer model in which Reshape is metadata-only
(Section 2.3, "GPU texture memory" discussion of 1-D buffers; Section 3.2.1 background).
"""
from __future__ import annotations

import numpy as np


def reshape(x: np.ndarray, shape) -> np.ndarray:
    """Reshape (Section 3.2.1 background): same elements in the same linear order,
    prod(shape) == prod(x.shape).  y.flat[i] = x.flat[i]."""
    shape = tuple(int(s) for s in shape)
    if int(np.prod(shape)) != x.size:
        raise ValueError("reshape: element count changes")
    flat = np.ascontiguousarray(x).reshape(-1).copy()
    return flat.reshape(shape)


def transpose(x: np.ndarray, perm) -> np.ndarray:
    """Transpose (Section 3.2.1 background; ONNX/NumPy perm convention):
    y.shape[k] = x.shape[perm[k]] and y[j_0..j_{n-1}] = x[i_0..i_{n-1}] with i_{perm[k]} = j_k."""
    perm = tuple(int(p) for p in perm)
    if sorted(perm) != list(range(x.ndim)):
        raise ValueError("transpose: perm is not a permutation")
    return np.ascontiguousarray(np.transpose(x, perm)).copy()


def inverse_perm(perm):
    inv = [0] * len(perm)
    for k, p in enumerate(perm):
        inv[p] = k
    return tuple(inv)


def roll(x: np.ndarray, shift: int, axis: int) -> np.ndarray:
    """Cyclic shift along one axis (a Slice/Gather-class operator, Table 3):
    y[.., j, ..] = x[.., (j - shift) mod N, ..] with the non-negative mod."""
    n = x.shape[axis]
    src = (np.arange(n) - int(shift)) % n
    return np.ascontiguousarray(np.take(x, src, axis=axis)).copy()


def slice_(x: np.ndarray, start, extent) -> np.ndarray:
    """Slice (Table 3, ILI & Fixed): y[j] = x[start + j] for 0 <= j < extent, per dim."""
    idx = tuple(slice(int(s), int(s) + int(e)) for s, e in zip(start, extent))
    return np.ascontiguousarray(x[idx]).copy()


def window_partition(x: np.ndarray, ws: int) -> np.ndarray:
    """[B,H,W,C] -> [B*(H/ws)*(W/ws), ws*ws, C] as Reshape -> Transpose -> Reshape."""
    B, H, W, C = x.shape
    if H % ws or W % ws:
        raise ValueError("window must divide H and W")
    y = reshape(x, (B, H // ws, ws, W // ws, ws, C))
    y = transpose(y, (0, 1, 3, 2, 4, 5))
    return reshape(y, (B * (H // ws) * (W // ws), ws * ws, C))


def window_reverse(xw: np.ndarray, ws: int, B: int, H: int, W: int) -> np.ndarray:
    """[B*(H/ws)*(W/ws), ws*ws, C] -> [B,H,W,C] as Reshape -> Transpose -> Reshape."""
    C = xw.shape[-1]
    y = reshape(xw, (B, H // ws, W // ws, ws, ws, C))
    y = transpose(y, (0, 1, 3, 2, 4, 5))
    return reshape(y, (B, H, W, C))


def cyclic_shift(x: np.ndarray, s: int) -> np.ndarray:
    """Forward shifted-window displacement: roll by -s along H, then by -s along W, so
    y[b,h,w,:] = x[b,(h+s) mod H,(w+s) mod W,:].  Two materialised rolls."""
    return roll(roll(x, -s, 1), -s, 2)


def cyclic_unshift(x: np.ndarray, s: int) -> np.ndarray:
    """Inverse displacement: roll by +s along H and W."""
    return roll(roll(x, s, 1), s, 2)


def head_split(qkv: np.ndarray, heads: int):
    """[nW,T,3C] -> reshape [nW,T,3,nH,d] -> transpose (2,0,3,1,4) -> q,k,v each [nW,nH,T,d]."""
    nW, T, C3 = qkv.shape
    C = C3 // 3
    d = C // heads
    y = reshape(qkv, (nW, T, 3, heads, d))
    y = transpose(y, (2, 0, 3, 1, 4))
    return (slice_(y, (0, 0, 0, 0, 0), (1, nW, heads, T, d))[0],
            slice_(y, (1, 0, 0, 0, 0), (1, nW, heads, T, d))[0],
            slice_(y, (2, 0, 0, 0, 0), (1, nW, heads, T, d))[0])


def head_merge(o: np.ndarray) -> np.ndarray:
    """[nW,nH,T,d] -> transpose (0,2,1,3) -> reshape [nW,T,nH*d]."""
    nW, nH, T, d = o.shape
    return reshape(transpose(o, (0, 2, 1, 3)), (nW, T, nH * d))


def depth_to_space(x: np.ndarray, b: int) -> np.ndarray:
    """[N, C*b*b, H, W] -> [N, C, H*b, W*b], depth-column-row order (the DtoS operator of Table 3, with
    the ONNX DepthToSpace "DCR" element order): out[n, c, h*b+i, w*b+j] = x[n, (i*b+j)*C + c, h, w].
    Written as the definition: one strided assignment per (i, j) block offset."""
    N, Cb, H, W = x.shape
    assert Cb % (b * b) == 0
    C = Cb // (b * b)
    out = np.empty((N, C, H * b, W * b), dtype=x.dtype)
    for i in range(b):
        for j in range(b):
            out[:, :, i::b, j::b] = x[:, (i * b + j) * C:(i * b + j + 1) * C]
    return out


def space_to_depth(x: np.ndarray, b: int) -> np.ndarray:
    """[N, C, H, W] -> [N, C*b*b, H/b, W/b] (the StoD operator of Table 3, ONNX SpaceToDepth order):
    out[n, (i*b+j)*C + c, h, w] = x[n, c, h*b+i, w*b+j]."""
    N, C, H, W = x.shape
    assert H % b == 0 and W % b == 0
    out = np.empty((N, C * b * b, H // b, W // b), dtype=x.dtype)
    for i in range(b):
        for j in range(b):
            out[:, (i * b + j) * C:(i * b + j + 1) * C] = x[:, :, i::b, j::b]
    return out


def patch_merge_gather(x: np.ndarray) -> np.ndarray:
    """Swin patch merging, layout part: [B,H,W,C] -> [B, H/2*W/2, 4C], the channel-wise Concat of the four
    Slices x[:, 0::2, 0::2], x[:, 1::2, 0::2], x[:, 0::2, 1::2], x[:, 1::2, 1::2] (in that order)."""
    B, H, W, C = x.shape
    assert H % 2 == 0 and W % 2 == 0
    parts = [x[:, 0::2, 0::2], x[:, 1::2, 0::2], x[:, 0::2, 1::2], x[:, 1::2, 1::2]]
    return np.concatenate(parts, axis=-1).reshape(B, (H // 2) * (W // 2), 4 * C)
