"""GPU parity of a whole Swin-T stage assembled from the library's entry points -- block (shift 0), block (shift 3),
patch merging (gather -> LayerNorm -> linear chain) -- against the same composition of the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import swin as oswin
from paper_2404_13528_b200 import binding as sm
from paper_2404_13528_b200 import synth
from tests.gpu_util import assert_close_bf16, check_status, stream, to_dev, to_host_f64
from tests.test_gpu_swin import run_block
from tests.test_planner import _patch_merge_ops

pytestmark = pytest.mark.gpu


def stage_case(config_id, B, H, W, C, heads, window, images):
    blocks = [synth.swin_inputs(config_id, B, H, W, C, heads, window, 4, "bf16", weight_set=ws) for ws in (0, 1)]
    seed = synth.SEED_BASE + config_id
    pm = {"g": synth.normal(seed, 301, (4 * C,), 0.02, 1.0, "bf16"), "b": synth.normal(seed, 302, (4 * C,), 0.02, 0.0, "bf16"),
          "w": synth.normal(seed, 303, (2 * C, 4 * C), 0.02, 0.0, "bf16")}
    # oracle: the stage on the sampled images (images are independent through the whole stage)
    x = synth.to_f64(blocks[0]["x"])[images]
    for inp, shift in zip(blocks, (0, window // 2)):
        pf = {k: synth.to_f64(v) for k, v in inp.items() if k != "x"}
        x = oswin.swin_block(x, pf, heads=heads, window=window, shift=shift, mlp_ratio=4)
    ref = oswin.patch_merging(x, synth.to_f64(pm["g"]), synth.to_f64(pm["b"]), synth.to_f64(pm["w"]))
    descs = [sm.make_desc((B, H, W, C)), sm.make_desc((4 * C,)), sm.make_desc((4 * C,)), sm.make_desc((2 * C, 4 * C))]
    pmd = [to_dev(pm[k]) for k in ("g", "b", "w")]
    outs = {}
    for mode in (sm.ELIMINATE, sm.ELIMINATE_UNFUSED, sm.EXPLICIT):
        t = to_dev(blocks[0]["x"])
        for inp, shift in zip(blocks, (0, window // 2)):
            dev = {k: to_dev(v) for k, v in inp.items() if k != "x"}
            t = run_block(inp, dev, B=B, H=H, W=W, C=C, heads=heads, window=window, shift=shift, mlp_ratio=4, dtype="bf16",
                          mode=mode, x_dev=t)
        plan = sm.smartmem_plan(_patch_merge_ops(B, H, W, C), descs, sm.EXPLICIT if mode == sm.EXPLICIT else sm.ELIMINATE)
        try:
            wsb = sm.smartmem_plan_workspace_bytes(plan)
            ws = torch.empty(max(wsb, 16), dtype=torch.uint8, device="cuda")
            out = torch.full((B, (H // 2) * (W // 2), 2 * C), float("nan"), dtype=torch.bfloat16, device="cuda")
            sm.smartmem_run_chain(plan, [t.data_ptr()] + [p.data_ptr() for p in pmd], [out.data_ptr()], ws.data_ptr(), wsb, stream())
            check_status()
        finally:
            sm.smartmem_plan_destroy(plan)
        assert_close_bf16(to_host_f64(out)[images], ref, f"stage, mode {mode}")
        outs[mode] = out
    # kernel by kernel, the eliminated and the explicit chain are bit-identical (ELIMINATE fuses the attention halves)
    assert torch.equal(outs[sm.ELIMINATE_UNFUSED].view(torch.int16), outs[sm.EXPLICIT].view(torch.int16))


def test_small_stage():
    stage_case(50, 2, 14, 14, 64, 2, 7, [0, 1])


def test_swin_t_stage1_full_size_sampled_images():
    """[32,56,56,96] -> two blocks -> [32,784,192]; the oracle follows images 0 and 21."""
    stage_case(51, 32, 56, 56, 96, 3, 7, [0, 21])
