"""GPU parity of smartmem_run_chain: copy-only layout chains are bit-exact against the
oracle's materialised tensors; GEMM consumers are bit-identical between ELIMINATE and
EXPLICIT and within the bf16 tolerance of the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import chains
from oracle import swin as oswin
from paper_2404_13528_b200 import binding as sm
from paper_2404_13528_b200 import synth
from tests.gpu_util import assert_close_bf16, check_status, stream, to_dev, to_host_bits, to_host_f64
from tests.test_planner import _ops_from_chain

pytestmark = pytest.mark.gpu


def run_plan(ops, descs, mode, inputs, out_shape, dtype=torch.bfloat16):
    plan = sm.smartmem_plan(ops, descs, mode)
    try:
        wsb = sm.smartmem_plan_workspace_bytes(plan)
        ws = torch.empty(max(wsb, 16), dtype=torch.uint8, device="cuda")
        out = torch.full(out_shape, float("nan"), dtype=dtype, device="cuda")
        sm.smartmem_run_chain(plan, [t.data_ptr() for t in inputs], [out.data_ptr()], ws.data_ptr(), wsb, stream())
        check_status()
        return out
    finally:
        sm.smartmem_plan_destroy(plan)


def copy_chain_case(shape, chain, dtype="bf16"):
    x = synth.normal(77, 0, shape, dtype=dtype)
    ref = chains.apply_layout_chain(x, chain)           # moves the raw storage values: exact
    xd = to_dev(x)
    ops = _ops_from_chain(chain) + [sm.make_op(sm.OP_COPY)]
    desc = [sm.make_desc(shape, sm.BF16 if dtype == "bf16" else sm.F32)]
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    modes = [sm.ELIMINATE, sm.EXPLICIT, sm.ELIMINATE_NAIVE]
    if all(o["op"] != "slice" for o in chain):
        try:                                                # map placed on the consumer / producer side
            sm.smartmem_plan_destroy(sm.smartmem_plan(ops, desc, sm.ELIMINATE_SCATTER))
            modes += [sm.ELIMINATE_GATHER, sm.ELIMINATE_SCATTER]
        except sm.SmartmemError:
            pass                                            # chains whose inverse does not refine
    for mode in modes:
        out = run_plan(ops, desc, mode, [xd], ref.shape, tdt)
        assert np.array_equal(to_host_bits(out), ref), f"mode {mode}"


CH2A = lambda B, S, H, D: [{"op": "reshape", "shape": (B, S, H, D)}, {"op": "transpose", "perm": (0, 2, 1, 3)}]
CH2B = lambda B, C, H, W: [{"op": "transpose", "perm": (0, 2, 3, 1)}, {"op": "reshape", "shape": (B, H * W, C)}]


def swin_e1(s, ws):
    return [{"op": "roll", "shift": -s, "axis": 1}, {"op": "roll", "shift": -s, "axis": 2},
            {"op": "window_partition", "window": ws}]


@pytest.mark.parametrize("shape,chain", [
    ((2, 96, 4 * 64), CH2A(2, 96, 4, 64)),
    ((8, 1024, 16 * 64), CH2A(8, 1024, 16, 64)),                    # full size of the benchmark chain
    ((2, 64, 8, 24), CH2B(2, 64, 8, 24)),                           # ragged tiles -> gather path
    ((2, 128, 16, 16), CH2B(2, 128, 16, 16)),                       # tiled transpose path
    ((8, 256, 64, 64), CH2B(8, 256, 64, 64)),                       # full size
    ((1, 8, 8, 32), swin_e1(2, 4)),
    ((3, 14, 14, 96), swin_e1(3, 7)),
    ((2, 56, 56, 96), swin_e1(3, 7)),
    ((2 * 8 * 8, 49, 96), [{"op": "window_reverse", "window": 7, "B": 2, "H": 56, "W": 56},
                           {"op": "roll", "shift": 3, "axis": 1}, {"op": "roll", "shift": 3, "axis": 2}]),
    ((5, 5, 5), [{"op": "reshape", "shape": (5, 25)}, {"op": "transpose", "perm": (1, 0)}]),
    ((4, 6, 10), [{"op": "slice", "start": (1, 0, 2), "extent": (2, 6, 8)}, {"op": "transpose", "perm": (2, 0, 1)}]),
    ((2, 64, 12, 20), [{"op": "depth_to_space", "block": 2}]),                     # DtoS / StoD of Table 3
    ((2, 16, 24, 40), [{"op": "space_to_depth", "block": 2}]),
    ((3, 36, 5, 7), [{"op": "depth_to_space", "block": 3}, {"op": "transpose", "perm": (0, 2, 3, 1)}]),
    ((4, 128, 64, 64), [{"op": "depth_to_space", "block": 2}]),                    # a diffusion-decoder-sized upsample
    # split points that do not refine each other: only the sequential program can evaluate it
    ((4, 6), [{"op": "transpose", "perm": (1, 0)}, {"op": "reshape", "shape": (8, 3)}]),
    ((12, 10, 6), [{"op": "transpose", "perm": (2, 0, 1)}, {"op": "reshape", "shape": (8, 9, 10)}, {"op": "roll", "shift": 2, "axis": 1}]),
])
def test_copy_only_chains_bit_exact(shape, chain):
    copy_chain_case(shape, chain)


def test_copy_only_chain_fp32():
    copy_chain_case((1, 8, 8, 32), swin_e1(2, 4), dtype="f32")
    copy_chain_case((3, 7, 20), [{"op": "transpose", "perm": (1, 2, 0)}], dtype="f32")


@pytest.mark.parametrize("small", [True, False])
def test_chain_2a_qkt(small):
    inp = synth.chain_inputs(2, "2a", small=small)
    B, S, H, D = inp["dims"]
    xq, xk = to_dev(inp["xq"]), to_dev(inp["xk"])
    ops = _ops_from_chain(CH2A(B, S, H, D)) + [sm.make_op(sm.OP_BMM_NT, side_input=(1, 0))]
    descs = [sm.make_desc((B, S, H * D)), sm.make_desc((B, S, H * D))]
    outs = [run_plan(ops, descs, mode, [xq, xk], (B, H, S, S)) for mode in (sm.ELIMINATE, sm.EXPLICIT)]
    assert torch.equal(outs[0], outs[1])                 # same kernel, only the load path differs
    got = to_host_f64(outs[0])
    if small:
        ref = chains.chain_2a_scores(synth.to_f64(inp["xq"]), synth.to_f64(inp["xk"]), H)
        assert_close_bf16(got, ref, "2a scores")
    else:                                                # sampled (b, h) slices at full size
        q = synth.to_f64(inp["xq"]).reshape(B, S, H, D)
        k = synth.to_f64(inp["xk"]).reshape(B, S, H, D)
        for b, h in [(0, 0), (3, 7), (7, 15)]:
            assert_close_bf16(got[b, h], q[b, :, h] @ k[b, :, h].T, f"2a scores[{b},{h}]")


@pytest.mark.parametrize("small", [True, False])
def test_chain_2b_gemm(small):
    inp = synth.chain_inputs(2, "2b", small=small)
    B, C, Hh, Ww, N = inp["dims"]
    x, w = to_dev(inp["x"]), to_dev(inp["w"])
    ops = _ops_from_chain(CH2B(B, C, Hh, Ww)) + [sm.make_op(sm.OP_LINEAR, side_input=(1, 0))]
    descs = [sm.make_desc((B, C, Hh, Ww)), sm.make_desc((N, C))]
    outs = [run_plan(ops, descs, mode, [x, w], (B, Hh * Ww, N)) for mode in (sm.ELIMINATE, sm.EXPLICIT)]
    assert torch.equal(outs[0], outs[1])
    ref = chains.chain_2b_gemm(synth.to_f64(inp["x"]), synth.to_f64(inp["w"])).reshape(B, Hh * Ww, N)
    assert_close_bf16(to_host_f64(outs[0]), ref, "2b gemm")


def test_plain_linear_shapes():
    """Plain [M,K] x [N,K]^T with ragged M, several tile widths and a K tail."""
    for M, N, K in [(200, 96, 96), (128, 288, 96), (300, 384, 96), (130, 96, 384), (257, 512, 512), (64, 64, 64)]:
        a = synth.normal(5, M * 7 + N, (M, K), dtype="bf16")
        w = synth.normal(5, K * 3 + N + 1, (N, K), std=0.05, dtype="bf16")
        out = run_plan([sm.make_op(sm.OP_LINEAR, side_input=(1, 0))], [sm.make_desc((M, K)), sm.make_desc((N, K))],
                       sm.ELIMINATE, [to_dev(a), to_dev(w)], (M, N))
        assert_close_bf16(to_host_f64(out), synth.to_f64(a) @ synth.to_f64(w).T, f"linear {M}x{N}x{K}")


def test_linear_shapes_that_run_on_cta_pairs():
    """Enough 256-wide tiles for more than one wave, an even number of row tiles: two SMs share a 256 x 256 tile.  The
    short reduction takes the epilogue that releases its accumulator early, the long one the general epilogue; the ragged M
    leaves the last pair tile with out-of-range rows in its second half."""
    for M, N, K in [(2304, 2304, 576), (2264, 2304, 576), (2560, 2048, 1280)]:
        a = synth.normal(6, M + N, (M, K), dtype="bf16")
        w = synth.normal(6, K + N + 1, (N, K), std=K ** -0.5, dtype="bf16")
        out = run_plan([sm.make_op(sm.OP_LINEAR, side_input=(1, 0))], [sm.make_desc((M, K)), sm.make_desc((N, K))],
                       sm.ELIMINATE, [to_dev(a), to_dev(w)], (M, N))
        assert_close_bf16(to_host_f64(out), synth.to_f64(a) @ synth.to_f64(w).T, f"linear {M}x{N}x{K}")


def test_run_chain_rejects_bad_arguments():
    plan = sm.smartmem_plan([sm.make_op(sm.OP_TRANSPOSE, perm=(1, 0)), sm.make_op(sm.OP_COPY)],
                            [sm.make_desc((64, 64))], sm.EXPLICIT)
    x = torch.zeros(64 * 64 + 8, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_run_chain(plan, [x.data_ptr() + 2], [out.data_ptr()], 0, 0, stream())
    assert e.value.code == sm.ERR_ALIGNMENT
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_run_chain(plan, [x.data_ptr()], [out.data_ptr()], 0, 0, stream())
    assert e.value.code == sm.ERR_WORKSPACE
    sm.smartmem_plan_destroy(plan)


# ------------------------------------------------------------------ patch merging: gather -> LayerNorm -> linear
def patch_merging_case(B, H, W, C, dtype="bf16"):
    from tests.test_planner import _patch_merge_ops
    x = synth.normal(78, 0, (B, H, W, C), dtype=dtype)
    g = synth.normal(78, 1, (4 * C,), 0.02, 1.0, dtype)
    b = synth.normal(78, 2, (4 * C,), 0.02, 0.0, dtype)
    w = synth.normal(78, 3, (2 * C, 4 * C), 0.02, 0.0, dtype)
    ref = oswin.patch_merging(synth.to_f64(x), synth.to_f64(g), synth.to_f64(b), synth.to_f64(w))
    dt = sm.BF16 if dtype == "bf16" else sm.F32
    descs = [sm.make_desc((B, H, W, C), dt), sm.make_desc((4 * C,), dt), sm.make_desc((4 * C,), dt), sm.make_desc((2 * C, 4 * C), dt)]
    ins = [to_dev(t) for t in (x, g, b, w)]
    outs = {}
    for mode in (sm.ELIMINATE, sm.EXPLICIT):
        out = run_plan(_patch_merge_ops(B, H, W, C), descs, mode, ins, ref.shape)
        assert_close_bf16(to_host_f64(out), ref, f"mode {mode}")
        outs[mode] = out
    assert torch.equal(outs[sm.ELIMINATE].view(torch.int16), outs[sm.EXPLICIT].view(torch.int16))


@pytest.mark.parametrize("B,H,W,C", [(1, 4, 4, 8), (2, 14, 10, 32), (3, 28, 28, 96), (2, 6, 6, 12)])
def test_patch_merging_chain(B, H, W, C):
    """(2, 6, 6, 12): 12 channels are not a whole number of 16-byte vectors, so ELIMINATE materialises the gather as well."""
    patch_merging_case(B, H, W, C)


def test_patch_merging_swin_t_stage1_full_size():
    """[32,56,56,96] -> [32, 784, 192]: the merge between stages 1 and 2 of Swin-T at the benchmark's batch."""
    patch_merging_case(32, 56, 56, 96)


# ------------------------------------------------------------------ channels-first producer -> LayerNorm over C -> linear
def nchw_layernorm_linear_case(B, C, H, W, N, expect_copies_eliminate):
    """The implicit layout transformation of Fig. 1(b): a LayerNorm over the channel dimension of an NCHW tensor,
    followed by a linear layer.  ELIMINATE normalises straight out of the channels-first buffer."""
    from oracle import ops as oops
    x = synth.normal(79, 0, (B, C, H, W), dtype="bf16")
    g = synth.normal(79, 1, (C,), 0.02, 1.0, "bf16")
    b = synth.normal(79, 2, (C,), 0.02, 0.0, "bf16")
    w = synth.normal(79, 3, (N, C), 0.02, 0.0, "bf16")
    chain = [{"op": "transpose", "perm": (0, 2, 3, 1)}, {"op": "reshape", "shape": (B, H * W, C)}]
    xt = chains.apply_layout_chain(synth.to_f64(x), chain)
    ref = oops.linear(oops.layernorm(xt, synth.to_f64(g), synth.to_f64(b), 1e-5), synth.to_f64(w))
    ops = _ops_from_chain(chain) + [sm.make_op(sm.OP_LAYERNORM, side_input=(1, 2), eps=1e-5), sm.make_op(sm.OP_LINEAR, side_input=(3, 0))]
    descs = [sm.make_desc((B, C, H, W)), sm.make_desc((C,)), sm.make_desc((C,)), sm.make_desc((N, C))]
    plan = sm.smartmem_plan(ops, descs, sm.ELIMINATE)
    try:
        assert sm.smartmem_plan_num_steps(plan)[1] == expect_copies_eliminate
    finally:
        sm.smartmem_plan_destroy(plan)
    ins = [to_dev(t) for t in (x, g, b, w)]
    outs = {}
    for mode in (sm.ELIMINATE, sm.EXPLICIT):
        out = run_plan(ops, descs, mode, ins, ref.shape)
        assert_close_bf16(to_host_f64(out), ref, f"mode {mode}")
        outs[mode] = out
    # not bit-identical: the slab kernel sums a token's channels in another order than the row kernel that EXPLICIT
    # runs on the materialised tensor; the two agree to the last bf16 digit or two
    d = (outs[sm.ELIMINATE].float() - outs[sm.EXPLICIT].float()).abs().max().item()
    assert d <= 2e-2, d


@pytest.mark.parametrize("B,C,H,W,N,copies", [
    (2, 64, 8, 16, 64, 0),          # 128 tokens per image: two slabs each
    (1, 256, 16, 16, 128, 0),       # one image (the image atom vanishes)
    (3, 96, 8, 24, 32, 0),
    (2, 64, 6, 6, 64, 1),           # 36 tokens per image: not a multiple of the slab width, the gather is materialised
    (8, 256, 64, 64, 256, 0),       # the size of chain 2b
])
def test_nchw_layernorm_linear(B, C, H, W, N, copies):
    nchw_layernorm_linear_case(B, C, H, W, N, copies)
