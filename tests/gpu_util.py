"""Helpers for the GPU parity tests: numpy <-> device buffers and the tolerance rules."""
import numpy as np
import torch

from paper_2404_13528_b200 import binding as sm
from paper_2404_13528_b200 import synth


def to_dev(a: np.ndarray) -> torch.Tensor:
    """float32 array -> f32 tensor; uint16 array (bf16 bits) -> bf16 tensor."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16).copy()).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def to_host_bits(t: torch.Tensor) -> np.ndarray:
    """Device tensor -> numpy (bf16 comes back as uint16 bit patterns)."""
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def to_host_f64(t: torch.Tensor) -> np.ndarray:
    return synth.to_f64(to_host_bits(t))


def stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def assert_close_bf16(got: np.ndarray, ref: np.ndarray, what: str = "", max_strict_violations: int = 0,
                      allowed_rows=None):
    """bf16 rule, against the fp64 oracle: |got - ref| <= 2e-2 * max(1, |ref|) for every element.

    `max_strict_violations` is a named, counted exception for one known case (the first rows of a causal
    layer, whose softmax runs over one to three keys, so that the bf16 rounding of q and k is not averaged
    out): at most that many elements may exceed the per-element bound, each of them must lie in a row (index
    along the second-to-last axis) listed in `allowed_rows`, and each must still satisfy the bound scaled by
    the largest |ref| of its own output row."""
    err = np.abs(got - ref)
    bad = err > 2e-2 * np.maximum(1.0, np.abs(ref))
    n_bad = int(bad.sum())
    if n_bad == 0:
        return
    where = np.argwhere(bad)
    msg = (f"{what}: {n_bad} of {bad.size} elements beyond 2e-2 * max(1, |ref|); max err {err.max():.4g} at "
           f"{np.unravel_index(err.argmax(), err.shape)} (ref {ref.flat[err.argmax()]:.4g}); first at {where[:4].tolist()}")
    assert n_bad <= max_strict_violations, msg
    rows = set(int(w[-2]) for w in where)
    assert allowed_rows is not None and rows <= set(allowed_rows), msg + f"; rows {sorted(rows)} not in the allowed set"
    row_scale = np.maximum(1.0, np.abs(ref).max(axis=-1, keepdims=True))
    assert not (err > 2e-2 * row_scale).any(), msg + "; also beyond the row-scaled bound"


def assert_close_f32(got: np.ndarray, ref: np.ndarray, what: str = ""):
    """fp32 rule: max |got - ref| <= 1e-4."""
    err = np.abs(got - ref)
    assert err.max() <= 1e-4, f"{what}: max abs err {err.max():.3g}"


def check_status():
    st = sm.smartmem_last_device_status(stream())
    assert st == sm.OK, f"device status {st}: {sm.smartmem_status_string(st)}"
