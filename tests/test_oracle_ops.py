"""Pins for the oracle's compute operators and whole blocks: closed forms, invariants,
textbook special cases and brute force on tiny inputs.  CPU only."""
import itertools
import math

import numpy as np
import pytest

from oracle import layout, llama, ops, swin

rng = np.random.default_rng(11)


# ---------------------------------------------------------------- normalisation / linear
def test_layernorm_invariants():
    x = rng.standard_normal((6, 32)) * 3 + 1.5
    eps = 1e-5
    y = ops.layernorm(x, np.ones(32), np.zeros(32), eps)
    assert np.allclose(y.mean(-1), 0, atol=1e-12)
    var = x.var(-1)                                  # biased
    assert np.allclose(y.var(-1), var / (var + eps), rtol=1e-12)
    assert np.allclose(ops.layernorm(x + 7.0, np.ones(32), np.zeros(32), eps), y, atol=1e-9)
    g, b = rng.standard_normal(32), rng.standard_normal(32)
    assert np.allclose(ops.layernorm(x, g, b, eps), y * g + b, atol=1e-12)
    # brute force on one row
    r = x[0]
    mu = sum(r) / 32
    v = sum((t - mu) ** 2 for t in r) / 32
    assert np.allclose(y[0], [(t - mu) / math.sqrt(v + eps) for t in r], atol=1e-12)


def test_rmsnorm_invariants():
    x = rng.standard_normal((5, 64))
    y = ops.rmsnorm(x, np.ones(64), 1e-5)
    assert np.allclose(np.sqrt((y * y).mean(-1)), 1.0, atol=1e-4)
    assert np.allclose(ops.rmsnorm(3.0 * x, np.ones(64), 0.0), ops.rmsnorm(x, np.ones(64), 0.0), atol=1e-12)
    r = x[1]
    ms = sum(t * t for t in r) / 64
    g = rng.standard_normal(64)
    assert np.allclose(ops.rmsnorm(x, g, 1e-5)[1], [t * gg / math.sqrt(ms + 1e-5) for t, gg in zip(r, g)], atol=1e-12)


def test_linear_identity_and_bruteforce():
    x = rng.standard_normal((4, 6))
    assert np.array_equal(ops.linear(x, np.eye(6)), x)
    w, b = rng.standard_normal((3, 6)), rng.standard_normal(3)
    y = ops.linear(x, w, b)
    for m, n in itertools.product(range(4), range(3)):
        assert abs(y[m, n] - (sum(x[m, k] * w[n, k] for k in range(6)) + b[n])) < 1e-12


def test_gelu_pins():
    assert ops.gelu(np.array([0.0]))[0] == 0.0
    u = rng.standard_normal(50) * 3
    assert np.allclose(ops.gelu(u) - ops.gelu(-u), u, atol=1e-12)
    assert abs(ops.gelu(np.array([1.0]))[0] - 0.8413447460685429) < 1e-12     # Phi(1)
    assert abs(ops.gelu(np.array([-1.0]))[0] + 0.15865525393145707) < 1e-12
    assert np.allclose(ops.gelu(u), [0.5 * t * (1 + math.erf(t / math.sqrt(2))) for t in u], atol=1e-14)


def test_softmax_pins():
    s = rng.standard_normal((3, 4, 9)) * 5
    p = ops.softmax(s)
    assert np.allclose(p.sum(-1), 1.0, atol=1e-13)
    assert np.allclose(ops.softmax(s + 100.0), p, atol=1e-13)
    assert np.allclose(ops.softmax(np.full((2, 5), 3.3)), 0.2)
    r = s[0, 0]
    e = [math.exp(t - max(r)) for t in r]
    assert np.allclose(p[0, 0], [t / sum(e) for t in e], atol=1e-14)


# ---------------------------------------------------------------- bias / mask / rope
def test_rel_pos_index_pins():
    idx = ops.rel_pos_index(7)
    assert idx.min() == 0 and idx.max() == 168 and len(np.unique(idx)) == 169
    assert (np.diag(idx) == 84).all()
    ws = 7
    for i, j, k, l in [(0, 8, 10, 18), (3, 48, 0, 45), (20, 6, 34, 20)]:
        di = (i // ws - j // ws, i % ws - j % ws)
        dk = (k // ws - l // ws, k % ws - l % ws)
        assert (di == dk) == (idx[i, j] == idx[k, l])
    # equal displacement <=> equal index, exhaustively
    disp = {}
    for i in range(49):
        for j in range(49):
            key = (i // ws - j // ws, i % ws - j % ws)
            assert disp.setdefault(key, idx[i, j]) == idx[i, j]
    assert len(disp) == 169
    idx4 = ops.rel_pos_index(4)
    assert idx4.max() == 48 and (np.diag(idx4) == 24).all()


def test_rel_pos_index_orientation_hand_values():
    """The index is (y_i - y_j + ws - 1)(2ws - 1) + (x_i - x_j + ws - 1), i the query and j the key: the row part
    comes from the vertical displacement, and a key to the right of / below the query gives the smaller index.
    Values worked out by hand from token t = (t div ws, t mod ws); each fails if i and j or the two axes are swapped."""
    idx = ops.rel_pos_index(7)
    # token 0 = (0,0), 1 = (0,1), 7 = (1,0), 8 = (1,1), 48 = (6,6), 6 = (0,6), 42 = (6,0)
    assert idx[0, 1] == 6 * 13 + 5 == 83        # dy 0, dx -1
    assert idx[1, 0] == 6 * 13 + 7 == 85        # dy 0, dx +1
    assert idx[0, 7] == 5 * 13 + 6 == 71        # dy -1, dx 0
    assert idx[7, 0] == 7 * 13 + 6 == 97        # dy +1, dx 0
    assert idx[0, 8] == 5 * 13 + 5 == 70 and idx[8, 0] == 7 * 13 + 7 == 98
    assert idx[0, 48] == 0 and idx[48, 0] == 168
    assert idx[6, 42] == 0 * 13 + 12 == 12      # dy -6, dx +6
    assert idx[42, 6] == 12 * 13 + 0 == 156     # dy +6, dx -6
    idx4 = ops.rel_pos_index(4)                  # (dy + 3) * 7 + (dx + 3); token 4 = (1,0)
    assert idx4[0, 1] == 23 and idx4[1, 0] == 25 and idx4[0, 4] == 17 and idx4[4, 0] == 31
    assert idx4[0, 15] == 0 and idx4[15, 0] == 48 and idx4[3, 12] == 6 and idx4[12, 3] == 42


@pytest.mark.parametrize("H,W,ws,s,nontrivial", [(8, 8, 4, 2, 3), (14, 14, 7, 3, 3), (56, 56, 7, 3, 15), (21, 21, 7, 3, 5)])
def test_shift_mask_no_wrap_characterisation(H, W, ws, s, nontrivial):
    """Two tokens of one shifted window may attend iff, in ORIGINAL coordinates, they are
    not separated by the image seam: |dh| < ws and |dw| < ws."""
    mask = ops.shifted_window_mask(H, W, ws, s)
    nWh, nWw = H // ws, W // ws
    assert mask.shape == (nWh * nWw, ws * ws, ws * ws)
    assert set(np.unique(mask).tolist()) <= {0.0, -100.0}
    assert sum(1 for m in mask if (m != 0).any()) == nontrivial
    for wy, wx in itertools.product(range(nWh), range(nWw)):
        coords = [((wy * ws + ty + s) % H, (wx * ws + tx + s) % W) for ty in range(ws) for tx in range(ws)]
        m = mask[wy * nWw + wx]
        for i, (hi, wi) in enumerate(coords):
            for j, (hj, wj) in enumerate(coords):
                ok = abs(hi - hj) < ws and abs(wi - wj) < ws
                assert (m[i, j] == 0.0) == ok


def test_rope_pins():
    S, D = 9, 16
    q, k = rng.standard_normal((S, D)), rng.standard_normal((S, D))
    rq = ops.rope(q, 10000.0)
    assert np.allclose(rq[0], q[0])                                         # position 0 is identity
    half = D // 2
    assert np.allclose(rq[:, :half] ** 2 + rq[:, half:] ** 2, q[:, :half] ** 2 + q[:, half:] ** 2)
    # <RoPE(q,m), RoPE(k,n)> depends only on m - n: place the same vectors at other positions
    qq, kk = np.tile(q[0], (S, 1)), np.tile(k[0], (S, 1))
    a, b = ops.rope(qq, 10000.0), ops.rope(kk, 10000.0)
    assert abs(a[5] @ b[3] - a[7] @ b[5]) < 1e-12 and abs(a[2] @ b[2] - a[8] @ b[8]) < 1e-12
    # brute force of one element pair
    p, i = 4, 3
    phi = p * 10000.0 ** (-(2 * i) / D)
    assert abs(rq[p, i] - (q[p, i] * math.cos(phi) - q[p, i + half] * math.sin(phi))) < 1e-12
    assert abs(rq[p, i + half] - (q[p, i + half] * math.cos(phi) + q[p, i] * math.sin(phi))) < 1e-12


# ---------------------------------------------------------------- attention
def _attention_bruteforce(q, k, v, allowed):
    T, d = q.shape
    out = np.zeros((T, v.shape[1]))
    for i in range(T):
        sc = [sum(q[i, e] * k[j, e] for e in range(d)) / math.sqrt(d) if allowed(i, j) else None for j in range(T)]
        m = max(t for t in sc if t is not None)
        w = [math.exp(t - m) if t is not None else 0.0 for t in sc]
        for j in range(T):
            out[i] += w[j] / sum(w) * v[j]
    return out


def test_window_attention_reduces_to_plain_attention():
    # ws = H = W, no shift, zero bias table  =>  textbook multi-head attention over all tokens
    ws, heads, d = 3, 2, 4
    T = ws * ws
    q, k, v = (rng.standard_normal((1, heads, T, d)) for _ in range(3))
    o = swin.window_attention(q, k, v, np.zeros(((2 * ws - 1) ** 2, heads)), ws)
    for h in range(heads):
        assert np.allclose(o[0, h], _attention_bruteforce(q[0, h], k[0, h], v[0, h], lambda i, j: True), atol=1e-12)


def test_window_attention_bias_is_added_per_head():
    ws, heads, d = 2, 2, 4
    T = 4
    q = np.zeros((1, heads, T, d))
    k = np.zeros((1, heads, T, d))
    v = rng.standard_normal((1, heads, T, d))
    table = np.zeros((9, heads))
    table[4, 1] = 50.0            # centre of the table = zero displacement, head 1 only
    o = swin.window_attention(q, k, v, table, ws)
    assert np.allclose(o[0, 0], v[0, 0].mean(0, keepdims=True).repeat(T, 0))   # head 0 uniform
    assert np.allclose(o[0, 1], v[0, 1], atol=1e-12)                            # head 1: diagonal dominates


def test_window_attention_off_centre_bias_row():
    """A one-hot at an OFF-centre row of the table: ws = 2, tokens 0=(0,0) 1=(0,1) 2=(1,0) 3=(1,1); table row
    (dy+1)*3 + (dx+1) = 3 is the displacement dy = 0, dx = -1, i.e. query (y,0) looking at key (y,1): pairs
    (i,j) = (0,1) and (2,3).  With q = k = 0 those two queries copy the key's value, the others average."""
    ws, heads, d, T = 2, 1, 3, 4
    q = np.zeros((1, heads, T, d))
    k = np.zeros((1, heads, T, d))
    v = np.array([[1.0, 0.0, 0.0], [0.0, 2.0, 0.0], [0.0, 0.0, 3.0], [4.0, 4.0, 4.0]]).reshape(1, 1, T, d)
    table = np.zeros((9, heads))
    table[3, 0] = 60.0
    o = swin.window_attention(q, k, v, table, ws)[0, 0]
    mean = np.array([5.0 / 4, 6.0 / 4, 7.0 / 4])
    assert np.allclose(o[0], [0.0, 2.0, 0.0], atol=1e-12)       # token 0 -> value of token 1
    assert np.allclose(o[1], mean, atol=1e-12)                  # token 1: no key at dx = -1 from it: uniform
    assert np.allclose(o[2], [4.0, 4.0, 4.0], atol=1e-12)       # token 2 -> value of token 3
    assert np.allclose(o[3], mean, atol=1e-12)
    # a vertical displacement instead: row (−1+1)*3 + (0+1) = 1 is dy = -1, dx = 0: pairs (0,2) and (1,3)
    table = np.zeros((9, heads))
    table[1, 0] = 60.0
    o = swin.window_attention(q, k, v, table, ws)[0, 0]
    assert np.allclose(o[0], [0.0, 0.0, 3.0], atol=1e-12) and np.allclose(o[1], [4.0, 4.0, 4.0], atol=1e-12)
    assert np.allclose(o[2], mean, atol=1e-12) and np.allclose(o[3], mean, atol=1e-12)


def test_causal_attention_pins():
    H, S, D = 2, 7, 4
    q, k, v = (rng.standard_normal((H, S, D)) for _ in range(3))
    o = llama.causal_attention(q, k, v)
    assert np.allclose(o[:, 0], v[:, 0])
    for h in range(H):
        assert np.allclose(o[h], _attention_bruteforce(q[h], k[h], v[h], lambda i, j: j <= i), atol=1e-12)
    o0 = llama.causal_attention(np.zeros_like(q), k, v)
    for i in range(S):
        assert np.allclose(o0[:, i], v[:, : i + 1].mean(1))


# ---------------------------------------------------------------- whole blocks
def _params(C, heads, ws, mlp_ratio, scale=0.2):
    p = {"ln1_g": 1 + 0.1 * rng.standard_normal(C), "ln1_b": 0.1 * rng.standard_normal(C),
         "w_qkv": scale * rng.standard_normal((3 * C, C)), "b_qkv": 0.1 * rng.standard_normal(3 * C),
         "rel_bias_table": 0.3 * rng.standard_normal(((2 * ws - 1) ** 2, heads)),
         "w_proj": scale * rng.standard_normal((C, C)), "b_proj": 0.1 * rng.standard_normal(C)}
    if mlp_ratio:
        p.update({"ln2_g": 1 + 0.1 * rng.standard_normal(C), "ln2_b": 0.1 * rng.standard_normal(C),
                  "w_fc1": scale * rng.standard_normal((C * mlp_ratio, C)), "b_fc1": 0.1 * rng.standard_normal(C * mlp_ratio),
                  "w_fc2": scale * rng.standard_normal((C, C * mlp_ratio)), "b_fc2": 0.1 * rng.standard_normal(C)})
    return p


def test_swin_block_uniform_attention_closed_form():
    """w_q = w_k = 0 and a zero bias table make the softmax uniform over allowed keys, so
    each token's attention output is the mean of v over the tokens of its shifted window
    that are not across the seam -- computed here token by token in ORIGINAL coordinates,
    with no partition or roll code."""
    B, H, W, C, heads, ws, s = 2, 8, 8, 8, 2, 4, 2
    p = _params(C, heads, ws, 0)
    p["w_qkv"][: 2 * C] = 0.0
    p["b_qkv"][: 2 * C] = 0.0
    p["rel_bias_table"][:] = 0.0
    x = rng.standard_normal((B, H, W, C))
    y = swin.swin_block(x, p, heads=heads, window=ws, shift=s, mlp_ratio=0)
    xn = ops.layernorm(x, p["ln1_g"], p["ln1_b"], 1e-5)
    vfull = xn @ p["w_qkv"][2 * C:].T + p["b_qkv"][2 * C:]                 # [B,H,W,C]
    exp = np.zeros_like(x)
    for b, h, w in itertools.product(range(B), range(H), range(W)):
        # shifted coordinates decide the window; original coordinates decide the seam
        hs, wsft = (h - s) % H, (w - s) % W
        members = []
        for h2, w2 in itertools.product(range(H), range(W)):
            h2s, w2s = (h2 - s) % H, (w2 - s) % W
            if h2s // ws == hs // ws and w2s // ws == wsft // ws and abs(h2 - h) < ws and abs(w2 - w) < ws:
                members.append(vfull[b, h2, w2])
        exp[b, h, w] = x[b, h, w] + np.mean(members, axis=0) @ p["w_proj"].T + p["b_proj"]
    assert np.allclose(y, exp, atol=1e-10)


def test_swin_block_special_cases():
    B, H, W, C, heads, ws = 1, 8, 8, 8, 2, 4
    x = rng.standard_normal((B, H, W, C))
    p = _params(C, heads, ws, 2)
    # all linear weights and biases zero => y = x (both halves)
    z = {k: (np.zeros_like(v) if k.startswith(("w_", "b_")) else v) for k, v in p.items()}
    assert np.allclose(swin.swin_block(x, z, heads=heads, window=ws, shift=2, mlp_ratio=2), x)
    # a block is equivariant to a cyclic translation by a whole window when unshifted
    y0 = swin.swin_block(x, p, heads=heads, window=ws, shift=0, mlp_ratio=2)
    xt = layout.roll(layout.roll(x, ws, 1), ws, 2)
    yt = swin.swin_block(xt, p, heads=heads, window=ws, shift=0, mlp_ratio=2)
    assert np.allclose(layout.roll(layout.roll(y0, ws, 1), ws, 2), yt, atol=1e-12)
    # shift changes the result (the shifted path is not a no-op)
    y2 = swin.swin_block(x, p, heads=heads, window=ws, shift=2, mlp_ratio=2)
    assert np.abs(y2 - y0).max() > 1e-3
    # single window covering the image, no shift: block == plain MHA + MLP written directly
    ws2 = 8
    p2 = _params(C, heads, ws2, 2)
    p2["rel_bias_table"][:] = 0.0
    y = swin.swin_block(x, p2, heads=heads, window=ws2, shift=0, mlp_ratio=2)
    xn = ops.layernorm(x, p2["ln1_g"], p2["ln1_b"], 1e-5).reshape(H * W, C)
    qkv = xn @ p2["w_qkv"].T + p2["b_qkv"]
    d = C // heads
    att = np.zeros((H * W, C))
    for h in range(heads):
        q, k, v = (qkv[:, i * C + h * d: i * C + (h + 1) * d] for i in range(3))
        att[:, h * d:(h + 1) * d] = _attention_bruteforce(q, k, v, lambda i, j: True)
    y1 = x.reshape(H * W, C) + att @ p2["w_proj"].T + p2["b_proj"]
    yn = ops.layernorm(y1, p2["ln2_g"], p2["ln2_b"], 1e-5)
    zz = y1 + ops.gelu(yn @ p2["w_fc1"].T + p2["b_fc1"]) @ p2["w_fc2"].T + p2["b_fc2"]
    assert np.allclose(y.reshape(H * W, C), zz, atol=1e-10)


def test_attn_layer_against_direct_restatement():
    S, heads, D = 6, 2, 8
    hidden = heads * D
    x = rng.standard_normal((1, S, hidden))
    p = {"rms_g": 1 + 0.1 * rng.standard_normal(hidden), "w_qkv": 0.3 * rng.standard_normal((3 * hidden, hidden)),
         "w_o": 0.3 * rng.standard_normal((hidden, hidden))}
    y = llama.attn_layer(x, p, heads=heads, head_dim=D, add_residual=True)
    xn = x[0] * p["rms_g"] / np.sqrt((x[0] ** 2).mean(-1, keepdims=True) + 1e-5)
    qkv = xn @ p["w_qkv"].T
    att = np.zeros((S, hidden))
    for h in range(heads):
        q, k, v = (qkv[:, i * hidden + h * D: i * hidden + (h + 1) * D] for i in range(3))
        att[:, h * D:(h + 1) * D] = _attention_bruteforce(ops.rope(q, 10000.0), ops.rope(k, 10000.0), v, lambda i, j: j <= i)
    assert np.allclose(y[0], x[0] + att @ p["w_o"].T, atol=1e-10)
    # q = k = 0 => prefix means of v pass through w_o
    p0 = dict(p)
    p0["w_qkv"] = p["w_qkv"].copy()
    p0["w_qkv"][: 2 * hidden] = 0
    y0 = llama.attn_layer(x, p0, heads=heads, head_dim=D)
    v = (xn @ p["w_qkv"].T)[:, 2 * hidden:]
    pm = np.cumsum(v, 0) / np.arange(1, S + 1)[:, None]
    assert np.allclose(y0[0], pm @ p["w_o"].T, atol=1e-10)


def test_rope_at_pins():
    """One-position rotary: equals row `pos` of the sequence form, is the identity at position 0,
    and for D = 2 is the plane rotation by `pos` radians (frequency theta^0 = 1)."""
    x = rng.standard_normal((3, 5, 16))
    for pos in (0, 1, 4):
        assert np.allclose(ops.rope_at(x[:, pos], pos, 10000.0), ops.rope(x, 10000.0)[:, pos], atol=1e-13)
    assert np.allclose(ops.rope_at(x[:, 2], 0, 10000.0), x[:, 2])
    r = ops.rope_at(np.array([[1.0, 0.0]]), 3, 10000.0)
    assert np.allclose(r, [[np.cos(3.0), np.sin(3.0)]], atol=1e-15)


def test_decode_step_equals_the_last_row_of_the_prefill():
    """A decode step on the cache that a prefill of the first S-1 tokens leaves must give row S-1 of the
    prefill over all S tokens (causal attention: the earlier rows never see the last token), and the
    appended key / value must be that prefill's row S-1."""
    S, heads, D, B = 7, 2, 8, 2
    hidden = heads * D
    x = rng.standard_normal((B, S, hidden))
    p = {"rms_g": 1 + 0.1 * rng.standard_normal(hidden), "w_qkv": 0.3 * rng.standard_normal((3 * hidden, hidden)),
         "w_o": 0.3 * rng.standard_normal((hidden, hidden))}
    kc, vc, full, keeps = [], [], [], []
    for b in range(B):
        keep = {}
        full.append(llama.attn_layer(x[b:b + 1], p, heads=heads, head_dim=D, add_residual=True, keep=keep)[0])
        keeps.append(keep)
        kc.append(np.transpose(keep["k"][:, :S - 1], (1, 0, 2)))     # [S-1,H,D]
        vc.append(np.transpose(keep["v"][:, :S - 1], (1, 0, 2)))
    y, kn, vn = llama.decode_step(x[:, S - 1], np.stack(kc), np.stack(vc), p, heads=heads, head_dim=D, add_residual=True)
    for b in range(B):
        assert np.allclose(y[b], full[b][S - 1], atol=1e-11)
        assert np.allclose(kn[b], keeps[b]["k"][:, S - 1], atol=1e-12)
        assert np.allclose(vn[b], keeps[b]["v"][:, S - 1], atol=1e-12)


def test_decode_step_special_cases():
    """Empty cache: softmax over one position is 1, so y = w_o v_new (+ x).  q-weights zero: uniform
    attention, so the attended value is the mean of the cached and the new values."""
    heads, D, B, pos = 2, 4, 3, 5
    hidden = heads * D
    x = rng.standard_normal((B, hidden))
    p = {"rms_g": 1 + 0.1 * rng.standard_normal(hidden), "w_qkv": 0.3 * rng.standard_normal((3 * hidden, hidden)),
         "w_o": 0.3 * rng.standard_normal((hidden, hidden))}
    xn = x * p["rms_g"] / np.sqrt((x ** 2).mean(-1, keepdims=True) + 1e-5)
    v_new = (xn @ p["w_qkv"].T)[:, 2 * hidden:]
    empty = np.zeros((B, 0, heads, D))
    y, _, vn = llama.decode_step(x, empty, empty, p, heads=heads, head_dim=D)
    assert np.allclose(vn.reshape(B, hidden), v_new, atol=1e-12)
    assert np.allclose(y, v_new @ p["w_o"].T, atol=1e-11)
    p0 = dict(p)
    p0["w_qkv"] = p["w_qkv"].copy()
    p0["w_qkv"][:hidden] = 0
    kc, vc = rng.standard_normal((B, pos, heads, D)), rng.standard_normal((B, pos, heads, D))
    y0, _, _ = llama.decode_step(x, kc, vc, p0, heads=heads, head_dim=D, add_residual=True)
    mean_v = (vc.reshape(B, pos, hidden).sum(1) + v_new) / (pos + 1)
    assert np.allclose(y0, x + mean_v @ p["w_o"].T, atol=1e-11)


def test_patch_merging_against_direct_restatement():
    """Token (i, j) of the merged grid = LayerNorm over the 4C channels of its 2x2 neighbourhood, times w^T."""
    B, H, W, C = 1, 4, 4, 3
    x = rng.standard_normal((B, H, W, C))
    g, b = 1 + 0.1 * rng.standard_normal(4 * C), 0.1 * rng.standard_normal(4 * C)
    w = rng.standard_normal((2 * C, 4 * C))
    y = swin.patch_merging(x, g, b, w)
    assert y.shape == (B, 4, 2 * C)
    for i, j in itertools.product(range(2), range(2)):
        nb = np.concatenate([x[0, 2 * i, 2 * j], x[0, 2 * i + 1, 2 * j], x[0, 2 * i, 2 * j + 1], x[0, 2 * i + 1, 2 * j + 1]])
        nn = (nb - nb.mean()) / np.sqrt(nb.var() + 1e-5) * g + b
        assert np.allclose(y[0, i * 2 + j], w @ nn, atol=1e-12)
    # constant input: LayerNorm gives beta, so every token maps to w beta
    yc = swin.patch_merging(np.full((B, H, W, C), 2.5), g, b, w)
    assert np.allclose(yc, np.broadcast_to(w @ b, yc.shape), atol=1e-9)


def test_rope_partial_pins():
    """R = D is the full rotary embedding; for R < D the first R features equal the full embedding of a head of
    dimension R and the rest pass through; the one-position form equals the matching row of the sequence form;
    rotation preserves the norm of every pair."""
    x = rng.standard_normal((2, 6, 16))
    assert np.allclose(ops.rope_partial(x, 10000.0, 16), ops.rope(x, 10000.0), atol=1e-13)
    for R in (4, 8):
        y = ops.rope_partial(x, 10000.0, R)
        assert np.allclose(y[..., :R], ops.rope(x[..., :R], 10000.0), atol=1e-13)
        assert np.array_equal(y[..., R:], x[..., R:])
        assert np.allclose(y[..., :R // 2] ** 2 + y[..., R // 2:R] ** 2, x[..., :R // 2] ** 2 + x[..., R // 2:R] ** 2)
        for pos in (0, 3, 5):
            assert np.allclose(ops.rope_partial(x[:, pos], 10000.0, R, pos=pos), y[:, pos], atol=1e-13)


def test_partial_rotary_layer_and_decode_step_agree():
    """With a partial rotary dimension the decode step still reproduces the prefill's last row."""
    S, heads, D, R = 5, 2, 8, 4
    hidden = heads * D
    x = rng.standard_normal((1, S, hidden))
    p = {"rms_g": 1 + 0.1 * rng.standard_normal(hidden), "w_qkv": 0.3 * rng.standard_normal((3 * hidden, hidden)),
         "w_o": 0.3 * rng.standard_normal((hidden, hidden))}
    keep = {}
    full = llama.attn_layer(x, p, heads=heads, head_dim=D, keep=keep, rotary_dim=R)[0]
    assert not np.allclose(full, llama.attn_layer(x, p, heads=heads, head_dim=D)[0])          # it is a different layer
    kc = np.transpose(keep["k"][:, :S - 1], (1, 0, 2))[None]
    vc = np.transpose(keep["v"][:, :S - 1], (1, 0, 2))[None]
    y, kn, _ = llama.decode_step(x[:, S - 1], kc, vc, p, heads=heads, head_dim=D, rotary_dim=R)
    assert np.allclose(y[0], full[S - 1], atol=1e-11)
    assert np.allclose(kn[0], keep["k"][:, S - 1], atol=1e-12)
