"""Pins for the oracle's layout operators: the paper's worked example, brute-force loops,
closed forms and invariants.  CPU only."""
import itertools
import os

import numpy as np
import pytest

from oracle import chains, layout

HERE = os.path.dirname(os.path.abspath(__file__))
rng = np.random.default_rng(7)


def test_paper_example_5x5x5_reshape_transpose():
    # Section 2.2: 5x5x5 -> Reshape 5x25 -> Transpose 25x5
    x = np.arange(125, dtype=np.float64).reshape(5, 5, 5)
    y = layout.transpose(layout.reshape(x, (5, 25)), (1, 0))
    assert y.shape == (25, 5)
    for a, b, c in itertools.product(range(5), repeat=3):
        assert y[5 * b + c, a] == x[a, b, c]
    with open(os.path.join(HERE, "golden", "reshape_transpose_5x5x5.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            a, b, c, r, col = (int(t) for t in line.split())
            assert y[r, col] == x[a, b, c]


def test_reshape_keeps_linear_order():
    x = rng.standard_normal((4, 6, 5))
    y = layout.reshape(x, (8, 15))
    assert [y.flat[i] for i in range(120)] == [x.flat[i] for i in range(120)]
    with pytest.raises(ValueError):
        layout.reshape(x, (7, 17))


def test_transpose_bruteforce_and_inverse():
    x = rng.standard_normal((2, 3, 4, 5))
    for perm in [(0, 2, 1, 3), (3, 1, 0, 2), (1, 0, 3, 2), (2, 3, 0, 1)]:
        y = layout.transpose(x, perm)
        assert y.shape == tuple(x.shape[p] for p in perm)
        for j in itertools.product(*[range(n) for n in y.shape]):
            i = [0] * 4
            for k in range(4):
                i[perm[k]] = j[k]
            assert y[j] == x[tuple(i)]
        assert np.array_equal(layout.transpose(y, layout.inverse_perm(perm)), x)
    m = rng.standard_normal((3, 7))
    t = layout.transpose(m, (1, 0))
    assert all(t[j, i] == m[i, j] for i in range(3) for j in range(7))


def test_roll_pins():
    assert layout.roll(np.array([0, 1, 2, 3]), -1, 0).tolist() == [1, 2, 3, 0]
    assert layout.roll(np.array([0, 1, 2, 3]), 1, 0).tolist() == [3, 0, 1, 2]
    x = rng.standard_normal((3, 8, 6, 2))
    for s in (1, 2, 5):
        assert np.array_equal(layout.roll(layout.roll(x, s, 1), -s, 1), x)
        assert np.array_equal(layout.cyclic_unshift(layout.cyclic_shift(x, s), s), x)
    assert np.array_equal(layout.roll(layout.roll(x, 2, 1), 3, 1), layout.roll(x, 5, 1))
    assert np.array_equal(layout.roll(x, 8, 1), x)
    y = layout.cyclic_shift(x, 3)
    for b, h, w in itertools.product(range(3), range(8), range(6)):
        assert np.array_equal(y[b, h, w], x[b, (h + 3) % 8, (w + 3) % 6])


def test_slice_bruteforce():
    x = rng.standard_normal((4, 5, 6))
    y = layout.slice_(x, (1, 0, 2), (2, 5, 3))
    for j in itertools.product(range(2), range(5), range(3)):
        assert y[j] == x[1 + j[0], j[1], 2 + j[2]]


@pytest.mark.parametrize("H,W,ws,s", [(8, 8, 4, 2), (14, 14, 7, 3), (21, 14, 7, 3), (56, 56, 7, 3)])
def test_window_partition_closed_form_and_bijection(H, W, ws, s):
    B, C = 2, 3
    x = np.arange(B * H * W * C, dtype=np.float64).reshape(B, H, W, C)
    xw = layout.window_partition(layout.cyclic_shift(x, s), ws)
    nWh, nWw = H // ws, W // ws
    assert xw.shape == (B * nWh * nWw, ws * ws, C)
    # closed form: window n = b*nWh*nWw + wy*nWw + wx, token t = ty*ws + tx
    #   <- pixel ((wy*ws+ty+s) mod H, (wx*ws+tx+s) mod W) of image b
    for b, wy, wx, ty, tx in itertools.product(range(B), range(nWh), range(nWw), range(ws), range(ws)):
        n = b * nWh * nWw + wy * nWw + wx
        t = ty * ws + tx
        assert np.array_equal(xw[n, t], x[b, (wy * ws + ty + s) % H, (wx * ws + tx + s) % W])
    assert sorted(xw.reshape(-1).tolist()) == list(range(B * H * W * C))  # every source hit once
    assert np.array_equal(layout.window_reverse(layout.window_partition(x, ws), ws, B, H, W), x)
    w_ = rng.standard_normal((B * nWh * nWw, ws * ws, C))
    assert np.array_equal(layout.window_partition(layout.window_reverse(w_, ws, B, H, W), ws), w_)


def test_head_split_merge_closed_form():
    nW, T, heads, d = 3, 5, 2, 4
    C = heads * d
    qkv = rng.standard_normal((nW, T, 3 * C))
    q, k, v = layout.head_split(qkv, heads)
    for which, t in enumerate((q, k, v)):
        for n, h, i, e in itertools.product(range(nW), range(heads), range(T), range(d)):
            assert t[n, h, i, e] == qkv[n, i, which * C + h * d + e]
    m = layout.head_merge(q)
    for n, h, i, e in itertools.product(range(nW), range(heads), range(T), range(d)):
        assert m[n, i, h * d + e] == q[n, h, i, e]


def test_chain_source_offsets_match_closed_forms():
    # chain 2a: [B,S,H*D] -> reshape -> transpose(0,2,1,3): (b,h,s,e) <- b*S*HD + s*HD + h*D + e
    B, S, H, D = 2, 5, 3, 4
    off = chains.source_offsets((B, S, H * D), [{"op": "reshape", "shape": (B, S, H, D)},
                                                {"op": "transpose", "perm": (0, 2, 1, 3)}])
    for b, h, s, e in itertools.product(range(B), range(H), range(S), range(D)):
        assert off[b, h, s, e] == b * S * H * D + s * H * D + h * D + e
    # chain 2b: NCHW -> NHWC -> [B*HW, C]: (m = b*HW + hw, c) <- b*C*HW + c*HW + hw
    B, C, Hh, Ww = 2, 3, 4, 5
    off = chains.source_offsets((B, C, Hh, Ww), [{"op": "transpose", "perm": (0, 2, 3, 1)},
                                                 {"op": "reshape", "shape": (B * Hh * Ww, C)}])
    for b, hw, c in itertools.product(range(B), range(Hh * Ww), range(C)):
        assert off[b * Hh * Ww + hw, c] == b * C * Hh * Ww + c * Hh * Ww + hw


@pytest.mark.parametrize("N,C,H,W,b", [(1, 1, 2, 3, 2), (2, 3, 2, 2, 2), (1, 2, 1, 2, 3)])
def test_depth_to_space_and_space_to_depth_bruteforce(N, C, H, W, b):
    """Element by element against the index definition, and the two operators invert each other."""
    x = rng.standard_normal((N, C * b * b, H, W))
    y = layout.depth_to_space(x, b)
    assert y.shape == (N, C, H * b, W * b)
    for n, c, h, w, i, j in itertools.product(range(N), range(C), range(H), range(W), range(b), range(b)):
        assert y[n, c, h * b + i, w * b + j] == x[n, (i * b + j) * C + c, h, w]
    assert np.array_equal(layout.space_to_depth(y, b), x)
    z = rng.standard_normal((N, C, H * b, W * b))
    s = layout.space_to_depth(z, b)
    assert s.shape == (N, C * b * b, H, W)
    for n, c, h, w, i, j in itertools.product(range(N), range(C), range(H), range(W), range(b), range(b)):
        assert s[n, (i * b + j) * C + c, h, w] == z[n, c, h * b + i, w * b + j]
    # block size 1 moves nothing
    assert np.array_equal(layout.depth_to_space(x, 1), x)


def test_depth_to_space_equals_its_reshape_transpose_form():
    """The textbook three-operator form: reshape [N,b,b,C,H,W] -> transpose (0,3,4,1,5,2) -> reshape."""
    N, C, H, W, b = 2, 3, 4, 5, 2
    x = rng.standard_normal((N, C * b * b, H, W))
    ref = x.reshape(N, b, b, C, H, W).transpose(0, 3, 4, 1, 5, 2).reshape(N, C, H * b, W * b)
    assert np.array_equal(layout.depth_to_space(x, b), ref)


def test_patch_merge_gather_bruteforce():
    """out[b, i*(W/2)+j, q*C + c] = x[b, 2i + q%2, 2j + q//2, c]: the four slices in the order
    (0,0), (1,0), (0,1), (1,1) of (row, column) offsets."""
    B, H, W, C = 2, 4, 6, 3
    x = rng.standard_normal((B, H, W, C))
    y = layout.patch_merge_gather(x)
    assert y.shape == (B, (H // 2) * (W // 2), 4 * C)
    for b, i, j, q, c in itertools.product(range(B), range(H // 2), range(W // 2), range(4), range(C)):
        assert y[b, i * (W // 2) + j, q * C + c] == x[b, 2 * i + q % 2, 2 * j + q // 2, c]
    # the same permutation as a reshape -> transpose -> reshape chain (what the planner composes)
    chain = [{"op": "reshape", "shape": [B, H // 2, 2, W // 2, 2, C]}, {"op": "transpose", "perm": [0, 1, 3, 4, 2, 5]},
             {"op": "reshape", "shape": [B, (H // 2) * (W // 2), 4 * C]}]
    assert np.array_equal(chains.apply_layout_chain(x, chain), y)
