"""GPU parity of smartmem_attn_decode (one decode step against a key/value cache) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import llama as ollama
from paper_2404_13528_b200 import binding as sm
from paper_2404_13528_b200 import synth
from tests.gpu_util import assert_close_bf16, check_status, stream, to_dev, to_host_bits, to_host_f64

pytestmark = pytest.mark.gpu


def physical_cache(logical: torch.Tensor, s_max: int, mode: int) -> torch.Tensor:
    """logical [B,pos,H,D] bf16 -> the mode's cache buffer with room for s_max positions; unused rows are NaN."""
    B, pos, H, D = logical.shape
    if mode == sm.ELIMINATE:
        c = torch.full((B, s_max, H, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        c[:, :pos] = logical
    else:
        c = torch.full((B, H, s_max, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        c[:, :, :pos] = logical.permute(0, 2, 1, 3)
    return c


def logical_view(cache: torch.Tensor, mode: int) -> torch.Tensor:
    """cache buffer -> [B,S_max,H,D]."""
    return cache if mode == sm.ELIMINATE else cache.permute(0, 2, 1, 3)


def make_params(dev, B, s_max, hidden, heads, add_residual, rotary_dim=0):
    p = sm.AttnParams()
    p.rotary_dim = rotary_dim
    p.dtype, p.B, p.S, p.hidden, p.heads, p.head_dim, p.causal, p.add_residual = sm.BF16, B, s_max, hidden, heads, hidden // heads, 1, add_residual
    p.rms_eps, p.rope_theta = 1e-5, 10000.0
    p.rms_g, p.w_qkv, p.w_o = dev["rms_g"].data_ptr(), dev["w_qkv"].data_ptr(), dev["w_o"].data_ptr()
    return p


def run_decode(dev, kc, vc, *, B, pos, s_max, hidden, heads, add_residual, mode, rotary_dim=0):
    p = make_params(dev, B, s_max, hidden, heads, add_residual, rotary_dim)
    y = torch.full_like(dev["x"], float("nan"))
    n = sm.smartmem_attn_decode_workspace_bytes(p, mode)
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    sm.smartmem_attn_decode(p, pos, dev["x"].data_ptr(), kc.data_ptr(), vc.data_ptr(), y.data_ptr(), ws.data_ptr(), n, mode, stream())
    check_status()
    return y


def check_case(config_id, B, pos, s_max, hidden, heads, add_residual, sample=None, rotary_dim=0):
    D = hidden // heads
    inp = synth.decode_inputs(config_id, B, pos, hidden, heads)
    dev = {k: to_dev(v) for k, v in inp.items()}
    pf = {k: synth.to_f64(inp[k]) for k in ("rms_g", "w_qkv", "w_o")}
    rows = list(range(B)) if sample is None else sample
    y_ref, k_ref, v_ref = ollama.decode_step(synth.to_f64(inp["x"])[rows], synth.to_f64(inp["k_cache"])[rows],
                                             synth.to_f64(inp["v_cache"])[rows], pf, heads=heads, head_dim=D,
                                             add_residual=bool(add_residual), rotary_dim=rotary_dim or None)
    for mode in (sm.ELIMINATE, sm.EXPLICIT):
        kc = physical_cache(dev["k_cache"], s_max, mode)
        vc = physical_cache(dev["v_cache"], s_max, mode)
        y = run_decode(dev, kc, vc, B=B, pos=pos, s_max=s_max, hidden=hidden, heads=heads, add_residual=add_residual, mode=mode,
                       rotary_dim=rotary_dim)
        assert_close_bf16(to_host_f64(y)[rows], y_ref, f"y, mode {mode}")
        for name, cache, src, ref in (("k", kc, dev["k_cache"], k_ref), ("v", vc, dev["v_cache"], v_ref)):
            lv = logical_view(cache, mode)
            assert_close_bf16(to_host_f64(lv[:, pos])[rows], ref, f"appended {name}, mode {mode}")
            assert torch.equal(lv[:, :pos].contiguous().view(torch.int16), src.view(torch.int16)), f"{name} cache rows below pos changed"
            assert torch.isnan(lv[:, pos + 1:].float()).all(), f"{name} cache rows above pos were written"


@pytest.mark.parametrize("B,pos,s_max,hidden,heads,res", [
    (1, 0, 4, 256, 2, 0),            # empty cache: attends to the new token only
    (3, 5, 8, 256, 2, 1),            # fewer positions than one pass of the attention kernel covers
    (2, 200, 256, 512, 4, 0),        # several passes and a ragged tail (201 positions)
    (5, 63, 64, 256, 2, 1),          # the cache's last slot
    (130, 17, 32, 256, 2, 0),        # more sequences than one GEMM row tile
])
def test_small_decode_steps(B, pos, s_max, hidden, heads, res):
    check_case(40, B, pos, s_max, hidden, heads, res)


@pytest.mark.parametrize("rot", [32, 64])
def test_partial_rotary_decode_steps(rot):
    check_case(44, 3, 37, 64, 512, 4, 1, rotary_dim=rot)


def test_decode_step_llama_size_sampled_sequences():
    """hidden 4096, 32 heads x 128, 2047 cached positions, 8 sequences; the oracle checks three of them."""
    check_case(41, 8, 2047, 2048, 4096, 32, 0, sample=[0, 3, 7])


def test_decode_step_benchmark_launch_configuration():
    """The benchmark's launch: 64 sequences x 2047 cached positions, hidden 4096.  The cache of four seeded
    sequences is repeated 16 times on the device (every sequence still has its own new token), and the oracle
    checks sequences that cover all four cache copies and both ends of the batch."""
    B, B0, pos, s_max, hidden, heads = 64, 4, 2047, 2048, 4096, 32
    D = hidden // heads
    inp = synth.decode_inputs(43, B0, pos, hidden, heads)
    x = synth.normal(synth.SEED_BASE + 43, 6, (B, hidden), 1.0, 0.0, "bf16")
    dev = {k: to_dev(inp[k]) for k in ("rms_g", "w_qkv", "w_o")}
    dev["x"] = to_dev(x)
    kc0, vc0 = to_dev(inp["k_cache"]), to_dev(inp["v_cache"])
    rows = [0, 1, 22, 43, 63]
    pf = {k: synth.to_f64(inp[k]) for k in ("rms_g", "w_qkv", "w_o")}
    y_ref, k_ref, v_ref = ollama.decode_step(synth.to_f64(x)[rows], synth.to_f64(inp["k_cache"])[[r % B0 for r in rows]],
                                             synth.to_f64(inp["v_cache"])[[r % B0 for r in rows]], pf, heads=heads, head_dim=D)
    for mode in (sm.ELIMINATE, sm.EXPLICIT):
        kc = physical_cache(kc0.repeat(B // B0, 1, 1, 1), s_max, mode)
        vc = physical_cache(vc0.repeat(B // B0, 1, 1, 1), s_max, mode)
        y = run_decode(dev, kc, vc, B=B, pos=pos, s_max=s_max, hidden=hidden, heads=heads, add_residual=0, mode=mode)
        assert_close_bf16(to_host_f64(y)[rows], y_ref, f"y, mode {mode}")
        assert_close_bf16(to_host_f64(logical_view(kc, mode)[:, pos])[rows], k_ref, f"appended k, mode {mode}")
        assert_close_bf16(to_host_f64(logical_view(vc, mode)[:, pos])[rows], v_ref, f"appended v, mode {mode}")
        # sequences that share a cache copy and differ only in their new token must differ in y
        assert not torch.equal(y[0], y[4])
        del kc, vc
        torch.cuda.empty_cache()


def test_decode_rejects_bad_arguments():
    inp = synth.decode_inputs(42, 2, 3, 256, 2)
    dev = {k: to_dev(v) for k, v in inp.items()}
    kc = physical_cache(dev["k_cache"], 8, sm.ELIMINATE)
    vc = physical_cache(dev["v_cache"], 8, sm.ELIMINATE)
    with pytest.raises(sm.SmartmemError) as e:        # pos outside the cache
        run_decode(dev, kc, vc, B=2, pos=8, s_max=8, hidden=256, heads=2, add_residual=0, mode=sm.ELIMINATE)
    assert e.value.code == sm.ERR_SHAPE
    with pytest.raises(sm.SmartmemError) as e:        # head_dim 64
        run_decode(dev, kc, vc, B=2, pos=3, s_max=8, hidden=256, heads=4, add_residual=0, mode=sm.ELIMINATE)
    assert e.value.code == sm.ERR_UNSUPPORTED
    with pytest.raises(sm.SmartmemError) as e:        # no such mode for this entry point
        run_decode(dev, kc, vc, B=2, pos=3, s_max=8, hidden=256, heads=2, add_residual=0, mode=sm.ELIMINATE_NAIVE)
    assert e.value.code == sm.ERR_INVALID_ARG
