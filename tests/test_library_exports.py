"""The C-ABI library loads without a GPU and exports every symbol include/smartmem.h declares."""
import ctypes
import os
import re

from paper_2404_13528_b200 import binding as sm

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "smartmem.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(smartmem_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = declared_symbols()
    assert len(names) >= 18
    L = ctypes.CDLL(sm.LIB_PATH)
    for n in names:
        assert hasattr(L, n), f"{n} declared in smartmem.h but not exported"
        assert n in sm.EXPORTED, f"{n} has no entry in the Python binding"
        assert hasattr(sm, n), f"binding lacks a function named {n}"


def test_host_only_calls_work_without_a_gpu():
    assert sm.smartmem_status_string(sm.OK) == "ok"
    assert sm.smartmem_launch_count() >= 0
    p = sm.SwinParams()
    p.dtype, p.B, p.H, p.W, p.C, p.heads, p.window, p.shift, p.mlp_ratio = sm.BF16, 2, 14, 14, 64, 2, 7, 3, 4
    e = sm.smartmem_swin_block_workspace_bytes(p, sm.ELIMINATE)
    x = sm.smartmem_swin_block_workspace_bytes(p, sm.EXPLICIT)
    u = sm.smartmem_swin_block_workspace_bytes(p, sm.ELIMINATE_UNFUSED)
    mc = 2 * 14 * 14 * 64 * 2
    # only what the chosen path writes is reserved.  ELIMINATE (attention half and MLP half each one kernel): the tensor between
    # the halves; kernel by kernel: qkv (3), attention output, the tensor between the halves; EXPLICIT adds the layout copies
    assert mc <= e < 2 * mc
    assert 5 * mc <= u < 6 * mc
    assert x >= u + 10 * mc
    p.C, p.heads = 512, 16                        # wide block: LayerNorm outputs and the hidden activation are materialised
    mcw = 2 * 14 * 14 * 512 * 2
    assert sm.smartmem_swin_block_workspace_bytes(p, sm.ELIMINATE) >= (1 + 3 + 1 + 1 + 1 + 4) * mcw
