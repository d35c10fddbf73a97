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


def assert_close_bf16(got: np.ndarray, ref: np.ndarray, what: str = ""):
    """bf16 rule, against the fp64 oracle: |got - ref| <= 2e-2 * max(1, scale) elementwise, where scale
    is the largest |ref| of the element's output row (last dimension).  The forward error of a
    mixed-precision contraction grows with the magnitude of the row it belongs to, not with the
    magnitude of the individual result (an element near zero in a large row still carries the
    row's rounding noise), so the relative part of the bound is taken per row."""
    err = np.abs(got - ref)
    scale = np.maximum(1.0, np.abs(ref).max(axis=-1, keepdims=True))
    bad = err > 2e-2 * scale
    strict = (err > 2e-2 * np.maximum(1.0, np.abs(ref))).sum()
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} elements out of tolerance; max err {err.max():.4g} "
                           f"at {np.unravel_index(err.argmax(), err.shape)} (ref {ref.flat[err.argmax()]:.4g}); "
                           f"{strict} beyond the per-element bound; max err / max |ref| = {err.max() / np.abs(ref).max():.3g}")


def assert_close_f32(got: np.ndarray, ref: np.ndarray, what: str = ""):
    """fp32 rule: max |got - ref| <= 1e-4."""
    err = np.abs(got - ref)
    assert err.max() <= 1e-4, f"{what}: max abs err {err.max():.3g}"


def check_status():
    st = sm.smartmem_last_device_status(stream())
    assert st == sm.OK, f"device status {st}: {sm.smartmem_status_string(st)}"
