"""The allocation-free Swin block entry point (for callers that cannot allocate device memory:
a frozen memory pool, a plugin without the host's allocator, start-up code).

It must give exactly what smartmem_swin_block gives, on two calls in a row (the fixed scratch
array is shared and keeps the previous call's contents), and must refuse blocks that do not
fit the array.  This file sorts last on purpose: a run that stops at the first failure has
then already run every other test."""
import pytest
import torch

from paper_2404_13528_b200 import binding as sm
from paper_2404_13528_b200 import synth
from tests.gpu_util import check_status, stream, to_dev

pytestmark = pytest.mark.gpu


def _params(cfg, dev, dtype):
    p = sm.SwinParams()
    p.dtype = sm.BF16 if dtype == "bf16" else sm.F32
    for k, v in cfg.items():
        setattr(p, k, v)
    p.ln_eps = 1e-5
    for k, t in dev.items():
        if k != "x":
            setattr(p, k, t.data_ptr())
    return p


@pytest.mark.parametrize("dtype,cfg", [
    ("bf16", dict(B=4, H=14, W=14, C=96, heads=3, window=7, shift=3, mlp_ratio=4)),
    ("f32", dict(B=1, H=8, W=8, C=32, heads=2, window=4, shift=2, mlp_ratio=0)),
])
def test_noalloc_matches_workspace_entry_point_twice(dtype, cfg):
    outs = []
    for call in range(2):                      # second call: different input, scratch holds stale data
        inp = synth.swin_inputs(40 + call, cfg["B"], cfg["H"], cfg["W"], cfg["C"], cfg["heads"], cfg["window"],
                                cfg["mlp_ratio"], dtype)
        dev = {k: to_dev(v) for k, v in inp.items()}
        p = _params(cfg, dev, dtype)
        for mode in (sm.ELIMINATE, sm.ELIMINATE_UNFUSED, sm.EXPLICIT):
            n = sm.smartmem_swin_block_workspace_bytes(p, mode)
            assert n <= sm.smartmem_swin_block_static_scratch_bytes()
            ws = torch.empty(n, dtype=torch.uint8, device="cuda")
            ref = torch.full_like(dev["x"], float("nan"))
            sm.smartmem_swin_block(p, dev["x"].data_ptr(), ref.data_ptr(), ws.data_ptr(), n, mode, stream())
            got = torch.full_like(dev["x"], float("nan"))
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            sm.smartmem_swin_block_noalloc(p, dev["x"].data_ptr(), got.data_ptr(), mode, stream())
            check_status()
            if call == 1:                      # past the first call's one-time set-up: the device's free memory does not move
                assert torch.cuda.mem_get_info()[0] == free_before
            # same kernels on the same inputs: identical bits (well inside the bf16 / fp32 tolerances)
            assert torch.isfinite(got.float()).all()
            assert torch.equal(got, ref), f"call {call} mode {mode}"
            outs.append(got)
    assert not torch.equal(outs[0], outs[3])   # the two calls really had different inputs


def test_noalloc_rejects_blocks_beyond_the_fixed_array():
    cfg = dict(B=64, H=56, W=56, C=96, heads=3, window=7, shift=3, mlp_ratio=4)
    p = sm.SwinParams()
    p.dtype = sm.BF16
    for k, v in cfg.items():
        setattr(p, k, v)
    assert sm.smartmem_swin_block_workspace_bytes(p, sm.ELIMINATE) > sm.smartmem_swin_block_static_scratch_bytes()
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_swin_block_noalloc(p, x.data_ptr(), x.data_ptr(), sm.ELIMINATE, stream())
    assert e.value.code == sm.ERR_WORKSPACE
    assert "workspace too small" in str(e.value)
