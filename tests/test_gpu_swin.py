"""GPU parity of smartmem_swin_block against the fp64 oracle, both modes."""
import numpy as np
import pytest
import torch

from oracle import swin as oswin
from paper_2404_13528_b200 import binding as sm
from paper_2404_13528_b200 import synth
from tests.gpu_util import assert_close_bf16, assert_close_f32, check_status, stream, to_dev, to_host_f64

pytestmark = pytest.mark.gpu

PARAM_NAMES = ["ln1_g", "ln1_b", "w_qkv", "b_qkv", "rel_bias_table", "w_proj", "b_proj",
               "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2"]


def run_block(inp, dev, *, B, H, W, C, heads, window, shift, mlp_ratio, dtype, mode, x_dev=None):
    p = sm.SwinParams()
    p.dtype = sm.F32 if dtype == "f32" else sm.BF16
    p.B, p.H, p.W, p.C, p.heads, p.window, p.shift, p.mlp_ratio = B, H, W, C, heads, window, shift, mlp_ratio
    p.ln_eps = 1e-5
    for n in PARAM_NAMES:
        if n in dev:
            setattr(p, n, dev[n].data_ptr())
    x = dev["x"] if x_dev is None else x_dev
    y = torch.full_like(x, float("nan"))
    wsb = sm.smartmem_swin_block_workspace_bytes(p, mode)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    sm.smartmem_swin_block(p, x.data_ptr(), y.data_ptr(), ws.data_ptr(), wsb, mode, stream())
    check_status()
    return y


def oracle_block(inp, images, *, heads, window, shift, mlp_ratio, x=None):
    pf = {k: synth.to_f64(v) for k, v in inp.items() if k != "x"}
    xf = synth.to_f64(inp["x"] if x is None else x)[images]
    return oswin.swin_block(xf, pf, heads=heads, window=window, shift=shift, mlp_ratio=mlp_ratio)


def case(config_id, *, B, H, W, C, heads, window, shift, mlp_ratio, dtype, images=None, **kw):
    inp = synth.swin_inputs(config_id, B, H, W, C, heads, window, mlp_ratio, dtype, **kw)
    dev = {k: to_dev(v) for k, v in inp.items()}
    images = list(range(B)) if images is None else images
    ref = oracle_block(inp, images, heads=heads, window=window, shift=shift, mlp_ratio=mlp_ratio)
    outs = {}
    for mode in (sm.ELIMINATE, sm.ELIMINATE_UNFUSED, sm.EXPLICIT):
        y = run_block(inp, dev, B=B, H=H, W=W, C=C, heads=heads, window=window, shift=shift, mlp_ratio=mlp_ratio,
                      dtype=dtype, mode=mode)
        got = to_host_f64(y)[images]
        (assert_close_f32 if dtype == "f32" else assert_close_bf16)(got, ref, f"mode {mode}")
        outs[mode] = y
    # the kernel-by-kernel eliminated chain and the explicit chain run the same arithmetic in the same order: only
    # the data movement differs.  (ELIMINATE may fuse the attention half of a narrow block into one kernel, which
    # applies LayerNorm to the QKV accumulator instead of to the rows: same result within the tolerance, not bit for bit.)
    assert torch.equal(outs[sm.ELIMINATE_UNFUSED], outs[sm.EXPLICIT])


def test_config1_tiny_swin_fp32():
    """B=1, 8x8 tokens, C=32, 2 heads of 16, window 4, shift 2, attention half only."""
    cfg = dict(B=1, H=8, W=8, C=32, heads=2, window=4, shift=2, mlp_ratio=0, dtype="f32")
    case(1, perturbed_affine=False, zero_bias=True, **cfg)      # gamma = 1, beta = 0, b = 0 as stated
    case(1, perturbed_affine=True, zero_bias=False, **cfg)      # an indexing error in gamma/beta/bias would show


def test_fp32_with_mlp_and_no_shift():
    case(11, B=2, H=8, W=12, C=32, heads=2, window=4, shift=0, mlp_ratio=2, dtype="f32")
    case(12, B=1, H=14, W=14, C=64, heads=2, window=7, shift=3, mlp_ratio=4, dtype="f32")


@pytest.mark.parametrize("cfg", [
    dict(B=2, H=14, W=14, C=64, heads=2, window=7, shift=3, mlp_ratio=4),
    dict(B=3, H=14, W=21, C=96, heads=3, window=7, shift=0, mlp_ratio=4),
    dict(B=1, H=8, W=8, C=32, heads=2, window=4, shift=2, mlp_ratio=0),       # head_dim 16, T = 16
    dict(B=2, H=16, W=16, C=64, heads=2, window=8, shift=5, mlp_ratio=2),     # T = 64 exactly
    dict(B=5, H=7, W=7, C=32, heads=1, window=7, shift=0, mlp_ratio=1),       # one window per image, ragged M
    dict(B=5, H=7, W=7, C=96, heads=3, window=7, shift=0, mlp_ratio=0),       # fused attention half: odd window count (a half pair)
    dict(B=1, H=21, W=28, C=96, heads=3, window=7, shift=5, mlp_ratio=4),     # fused: 12 windows, seams in both directions
    dict(B=2, H=16, W=24, C=96, heads=3, window=8, shift=4, mlp_ratio=0),     # fused: T = 64, two-deep row ring
    dict(B=40, H=14, W=14, C=96, heads=3, window=7, shift=3, mlp_ratio=0),    # fused: 80 pairs (one unit per CTA)
    dict(B=3, H=28, W=28, C=64, heads=2, window=7, shift=2, mlp_ratio=4),     # fused, two heads
])
def test_small_bf16_blocks(cfg):
    case(20, dtype="bf16", **cfg)


@pytest.mark.parametrize("offset,spread", [(40.0, 1.0), (-12.0, 0.25), (0.0, 30.0)])
def test_layernorm_statistics_on_rows_with_a_large_common_offset(offset, spread):
    """Rows whose mean dwarfs their spread (and rows with a huge spread): the fused kernels take both LayerNorm
    moments in one pass over data shifted by the row's first element, which must stay as accurate as two passes."""
    B, H, W, C, heads, ws = 2, 14, 14, 96, 3, 7
    inp = synth.swin_inputs(21, B, H, W, C, heads, ws, 4, "bf16")
    x = synth.to_f64(inp["x"]) * spread + offset
    inp["x"] = synth.f64_to_bf16_bits(x).reshape(x.shape)
    dev = {k: to_dev(v) for k, v in inp.items()}
    ref = oracle_block(inp, [0, 1], heads=heads, window=ws, shift=3, mlp_ratio=4)
    for mode in (sm.ELIMINATE, sm.ELIMINATE_UNFUSED, sm.EXPLICIT):
        y = run_block(inp, dev, B=B, H=H, W=W, C=C, heads=heads, window=ws, shift=3, mlp_ratio=4, dtype="bf16", mode=mode)
        assert_close_bf16(to_host_f64(y), ref, f"mode {mode}")


def test_config3_swin_t_stage1_full_size():
    """B=32, 56x56, C=96, 3 heads, window 7, shift 3, MLP x4 at full size; the oracle checks two images."""
    case(3, B=32, H=56, W=56, C=96, heads=3, window=7, shift=3, mlp_ratio=4, dtype="bf16", images=[0, 31])


def test_wide_block_on_cta_pairs_with_a_ragged_last_tile():
    """B=18, 14x14, C=512: 3528 rows = 27 full row tiles and 72 rows of a 28th, so the GEMMs run on CTA pairs (an even number
    of row tiles, more than a wave of 256-wide tiles) and the last pair tile ends inside its second CTA's rows: the output
    boxes of the lean epilogue are clipped by their tensor map, the per-thread stores of the others by the row bound."""
    case(4, B=18, H=14, W=14, C=512, heads=16, window=7, shift=3, mlp_ratio=4, dtype="bf16", images=[0, 17])


def test_config4_swin_b_stage3_block_pair():
    """B=64, 14x14, C=512, 16 heads: a regular block then a shifted block with independent weights."""
    B, H, W, C, heads, ws = 64, 14, 14, 512, 16, 7
    images = [0, 63]
    a = synth.swin_inputs(4, B, H, W, C, heads, ws, 4, "bf16", weight_set=0)
    b = synth.swin_inputs(4, B, H, W, C, heads, ws, 4, "bf16", weight_set=1)
    da, db = {k: to_dev(v) for k, v in a.items()}, {k: to_dev(v) for k, v in b.items()}
    outs = []
    for mode in (sm.ELIMINATE, sm.EXPLICIT):          # wide blocks: ELIMINATE runs kernel by kernel
        y1 = run_block(a, da, B=B, H=H, W=W, C=C, heads=heads, window=ws, shift=0, mlp_ratio=4, dtype="bf16", mode=mode)
        y2 = run_block(b, db, B=B, H=H, W=W, C=C, heads=heads, window=ws, shift=3, mlp_ratio=4, dtype="bf16", mode=mode,
                       x_dev=y1)
        outs.append((y1, y2))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    y1, y2 = outs[0]
    ref1 = oracle_block(a, images, heads=heads, window=ws, shift=0, mlp_ratio=4)
    assert_close_bf16(to_host_f64(y1)[images], ref1, "block A")
    # block B is checked on the GPU's own (bf16) block-A output, so that each block is compared
    # with the oracle on identical inputs
    y1_bits = y1.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    ref2 = oracle_block(b, images, heads=heads, window=ws, shift=3, mlp_ratio=4, x=y1_bits)
    assert_close_bf16(to_host_f64(y2)[images], ref2, "block B")


def test_swin_block_rejects_bad_arguments():
    inp = synth.swin_inputs(1, 1, 8, 8, 32, 2, 4, 0, "f32")
    dev = {k: to_dev(v) for k, v in inp.items()}
    base = dict(B=1, H=8, W=8, C=32, heads=2, window=4, shift=2, mlp_ratio=0, dtype="f32", mode=sm.ELIMINATE)
    for bad, code in [(dict(window=3), sm.ERR_SHAPE), (dict(shift=4), sm.ERR_SHAPE), (dict(heads=3), sm.ERR_SHAPE),
                      (dict(heads=4), sm.ERR_UNSUPPORTED), (dict(mode=9), sm.ERR_INVALID_ARG)]:
        with pytest.raises(sm.SmartmemError) as e:
            run_block(inp, dev, **{**base, **bad})
        assert e.value.code == code, bad


@pytest.mark.parametrize("cfg", [
    dict(B=2, H=14, W=14, C=96, heads=3, window=7, shift=3, mlp_ratio=4),      # fused halves
    dict(B=1, H=14, W=14, C=128, heads=4, window=7, shift=3, mlp_ratio=2),     # kernel by kernel
])
def test_block_halves_compose_to_the_block(cfg):
    """smartmem_swin_block_half: the attention half into a buffer, the MLP half from it = the block, bit for bit."""
    inp = synth.swin_inputs(22, cfg["B"], cfg["H"], cfg["W"], cfg["C"], cfg["heads"], cfg["window"], cfg["mlp_ratio"], "bf16")
    dev = {k: to_dev(v) for k, v in inp.items()}
    p = sm.SwinParams()
    p.dtype = sm.BF16
    for k, v in cfg.items():
        setattr(p, k, v)
    p.ln_eps = 1e-5
    for n in PARAM_NAMES:
        setattr(p, n, dev[n].data_ptr())
    for mode in (sm.ELIMINATE, sm.ELIMINATE_UNFUSED, sm.EXPLICIT):
        n = sm.smartmem_swin_block_workspace_bytes(p, mode)
        ws = torch.empty(n, dtype=torch.uint8, device="cuda")
        whole = torch.full_like(dev["x"], float("nan"))
        sm.smartmem_swin_block(p, dev["x"].data_ptr(), whole.data_ptr(), ws.data_ptr(), n, mode, stream())
        mid, out = torch.full_like(whole, float("nan")), torch.full_like(whole, float("nan"))
        sm.smartmem_swin_block_half(p, dev["x"].data_ptr(), mid.data_ptr(), ws.data_ptr(), n, mode, 0, stream())
        sm.smartmem_swin_block_half(p, mid.data_ptr(), out.data_ptr(), ws.data_ptr(), n, mode, 1, stream())
        check_status()
        assert torch.equal(out, whole), f"mode {mode}"
        assert not torch.equal(mid, whole)
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_swin_block_half(p, dev["x"].data_ptr(), out.data_ptr(), ws.data_ptr(), n, sm.ELIMINATE, 2, stream())
    assert e.value.code == sm.ERR_INVALID_ARG
