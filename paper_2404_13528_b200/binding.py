"""ctypes binding of the C ABI in include/smartmem.h.

Argument marshalling only: every step of the hot path runs inside the CUDA library.  The
functions keep the C names.  Device buffers are passed as integers (``tensor.data_ptr()``),
streams as ``torch.cuda.current_stream().cuda_stream``.  If the shared library is missing
the import of any entry point raises -- there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsmartmem.so")

MAX_DIMS, MAX_ATOMS, MAX_ROLLS = 8, 16, 4
OK = 0
ERR_INVALID_ARG, ERR_SHAPE, ERR_UNSUPPORTED, ERR_WORKSPACE = -1, -2, -3, -4
ERR_ALIGNMENT, ERR_CUDA, ERR_TIMEOUT = -5, -6, -7
F32, BF16 = 0, 1
ELIMINATE, EXPLICIT, ELIMINATE_NAIVE, ELIMINATE_GATHER, ELIMINATE_SCATTER, ELIMINATE_UNFUSED = 0, 1, 2, 3, 4, 5
OP_RESHAPE, OP_TRANSPOSE, OP_ROLL, OP_SLICE, OP_WINDOW_PARTITION, OP_WINDOW_REVERSE = 0, 1, 2, 3, 4, 5
OP_DEPTH_TO_SPACE, OP_SPACE_TO_DEPTH = 6, 7
OP_COPY, OP_LINEAR, OP_BMM_NT, OP_LAYERNORM = 16, 17, 18, 19


class Op(C.Structure):
    _fields_ = [("kind", C.c_int32), ("ndim", C.c_int32), ("shape", C.c_int64 * MAX_DIMS),
                ("perm", C.c_int32 * MAX_DIMS), ("start", C.c_int64 * MAX_DIMS), ("shift", C.c_int64),
                ("axis", C.c_int32), ("window", C.c_int32), ("side_input", C.c_int32 * 2), ("eps", C.c_float),
                ("reserved", C.c_int32)]


class TensorDesc(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("ndim", C.c_int32), ("shape", C.c_int64 * MAX_DIMS),
                ("stride", C.c_int64 * MAX_DIMS)]


class IndexMap(C.Structure):
    _fields_ = [("n_atoms", C.c_int32), ("extent", C.c_int64 * MAX_ATOMS), ("src_stride", C.c_int64 * MAX_ATOMS),
                ("roll_of", C.c_int32 * MAX_ATOMS), ("roll_weight", C.c_int64 * MAX_ATOMS), ("n_rolls", C.c_int32),
                ("roll_shift", C.c_int64 * MAX_ROLLS), ("roll_mod", C.c_int64 * MAX_ROLLS),
                ("roll_stride", C.c_int64 * MAX_ROLLS), ("roll_n_parts", C.c_int32 * MAX_ROLLS),
                ("roll_part_extent", (C.c_int64 * MAX_ROLLS) * MAX_ROLLS),
                ("roll_part_stride", (C.c_int64 * MAX_ROLLS) * MAX_ROLLS), ("base", C.c_int64), ("n_elements", C.c_int64),
                ("vec_elems", C.c_int32), ("klass", C.c_int32)]


class SwinParams(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("dtype", "B", "H", "W", "C", "heads", "window", "shift", "mlp_ratio")] + \
               [("ln_eps", C.c_float)] + \
               [(n, C.c_void_p) for n in ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "rel_bias_table", "w_proj", "b_proj",
                                          "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2")]


class FanoutParams(C.Structure):
    _fields_ = [("B", C.c_int32), ("S", C.c_int32), ("K", C.c_int32), ("N", C.c_int32), ("Na", C.c_int32), ("Nb", C.c_int32),
                ("k_contig", C.c_int32), ("w_p", C.c_void_p), ("w_a", C.c_void_p), ("w_b", C.c_void_p)]


class AttnParams(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("dtype", "B", "S", "hidden", "heads", "head_dim", "causal", "add_residual")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)] + \
               [(n, C.c_void_p) for n in ("rms_g", "w_qkv", "w_o")] + \
               [("rotary_dim", C.c_int32), ("reserved", C.c_int32)]


EXPORTED = [
    "smartmem_op_quadrant", "smartmem_pair_decision", "smartmem_select_layouts", "smartmem_plan", "smartmem_plan_destroy",
    "smartmem_plan_num_steps", "smartmem_plan_get_map", "smartmem_plan_output_desc",
    "smartmem_plan_workspace_bytes", "smartmem_map_eval", "smartmem_plan_eval_sequential", "smartmem_run_chain",
    "smartmem_swin_block_workspace_bytes", "smartmem_swin_block", "smartmem_swin_block_half", "smartmem_attn_layer_workspace_bytes",
    "smartmem_attn_layer", "smartmem_attn_decode_workspace_bytes", "smartmem_attn_decode", "smartmem_swin_block_timed", "smartmem_swin_block_static_scratch_bytes",
    "smartmem_swin_block_noalloc", "smartmem_profile_begin", "smartmem_profile_end", "smartmem_last_device_status", "smartmem_set_wait_limit_ns", "smartmem_selftest_bounded_wait", "smartmem_fanout_plan", "smartmem_fanout", "smartmem_launch_count", "smartmem_status_string",
]

_lib = None


def lib() -> C.CDLL:
    """Loads libsmartmem.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2404_13528_b200.build` "
                           "(the hot path has no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    P = C.POINTER
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    sig = {
        "smartmem_op_quadrant": (C.c_int, [i32, P(i32)]),
        "smartmem_pair_decision": (C.c_int, [i32, i32, P(i32), P(i32), P(i32)]),
        "smartmem_select_layouts": (C.c_int, [i32, i32, P(i32), P(i64), i32, i32, P(i32), P(i32), P(i32)]),
        "smartmem_plan": (C.c_int, [P(Op), i32, P(TensorDesc), i32, i32, P(vp)]),
        "smartmem_plan_destroy": (C.c_int, [vp]),
        "smartmem_plan_num_steps": (C.c_int, [vp, P(i32), P(i32)]),
        "smartmem_plan_get_map": (C.c_int, [vp, i32, i32, P(IndexMap)]),
        "smartmem_plan_output_desc": (C.c_int, [vp, P(TensorDesc)]),
        "smartmem_plan_workspace_bytes": (C.c_int, [vp, P(C.c_size_t)]),
        "smartmem_map_eval": (i64, [P(IndexMap), i64]),
        "smartmem_plan_eval_sequential": (i64, [vp, i32, i32, i64]),
        "smartmem_run_chain": (C.c_int, [vp, P(vp), P(vp), vp, C.c_size_t, vp]),
        "smartmem_swin_block_workspace_bytes": (C.c_int, [P(SwinParams), i32, P(C.c_size_t)]),
        "smartmem_swin_block": (C.c_int, [P(SwinParams), vp, vp, vp, C.c_size_t, i32, vp]),
        "smartmem_swin_block_half": (C.c_int, [P(SwinParams), vp, vp, vp, C.c_size_t, i32, i32, vp]),
        "smartmem_swin_block_timed": (C.c_int, [P(SwinParams), vp, vp, vp, C.c_size_t, i32, vp, P(C.c_float), C.c_char_p,
                                      i32, i32, P(i32)]),
        "smartmem_swin_block_static_scratch_bytes": (C.c_int, [P(C.c_size_t)]),
        "smartmem_swin_block_noalloc": (C.c_int, [P(SwinParams), vp, vp, i32, vp]),
        "smartmem_attn_layer_workspace_bytes": (C.c_int, [P(AttnParams), i32, P(C.c_size_t)]),
        "smartmem_attn_layer": (C.c_int, [P(AttnParams), vp, vp, vp, C.c_size_t, i32, vp]),
        "smartmem_attn_decode_workspace_bytes": (C.c_int, [P(AttnParams), i32, P(C.c_size_t)]),
        "smartmem_attn_decode": (C.c_int, [P(AttnParams), i32, vp, vp, vp, vp, vp, C.c_size_t, i32, vp]),
        "smartmem_profile_begin": (C.c_int, []),
        "smartmem_profile_end": (C.c_int, [vp, P(C.c_float), C.c_char_p, i32, i32, P(i32)]),
        "smartmem_last_device_status": (C.c_int, [vp, P(i32)]),
        "smartmem_set_wait_limit_ns": (C.c_int, [C.c_uint64]),
        "smartmem_selftest_bounded_wait": (C.c_int, [vp]),
        "smartmem_fanout_plan": (C.c_int, [P(FanoutParams), i32, P(i32), P(i32), P(C.c_int64), P(C.c_int64), P(C.c_size_t)]),
        "smartmem_fanout": (C.c_int, [P(FanoutParams), vp, vp, vp, vp, C.c_size_t, i32, vp]),
        "smartmem_launch_count": (i64, []),
        "smartmem_status_string": (C.c_char_p, [i32]),
    }
    for name, (res, args) in sig.items():
        f = getattr(L, name)
        f.restype, f.argtypes = res, args
    _lib = L
    return L


class SmartmemError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {smartmem_status_string(code)} ({code})")


def _check(rc: int, where: str):
    if rc != OK:
        raise SmartmemError(rc, where)


# ---------------------------------------------------------------------------------------------
# helpers to build the C structures
# ---------------------------------------------------------------------------------------------
def make_op(kind: int, *, shape=(), perm=(), start=(), shift=0, axis=0, window=0, side_input=(0, 0), eps=0.0) -> Op:
    o = Op()
    o.kind = kind
    o.ndim = max(len(shape), len(perm), len(start))
    for i, v in enumerate(shape):
        o.shape[i] = int(v)
    for i, v in enumerate(perm):
        o.perm[i] = int(v)
    for i, v in enumerate(start):
        o.start[i] = int(v)
    o.shift, o.axis, o.window = int(shift), int(axis), int(window)
    o.side_input[0], o.side_input[1] = int(side_input[0]), int(side_input[1])
    o.eps = float(eps)
    return o


def make_desc(shape, dtype: int = BF16, stride=None) -> TensorDesc:
    d = TensorDesc()
    d.dtype, d.ndim = dtype, len(shape)
    for i, v in enumerate(shape):
        d.shape[i] = int(v)
    if stride is not None:
        for i, v in enumerate(stride):
            d.stride[i] = int(v)
    return d


# ---------------------------------------------------------------------------------------------
# entry points (same names as the C ABI)
# ---------------------------------------------------------------------------------------------
def smartmem_status_string(code: int) -> str:
    return lib().smartmem_status_string(code).decode()


def smartmem_op_quadrant(kind: int) -> int:
    q = C.c_int32()
    _check(lib().smartmem_op_quadrant(kind, C.byref(q)), "smartmem_op_quadrant")
    return q.value


def smartmem_select_layouts(ndim: int, reduction_dims, weights=None, k: int = 1, max_layouts: int = MAX_DIMS):
    """Returns (layouts, layout_of_consumer): layouts[l] = producer dimensions from outermost to contiguous."""
    n = len(reduction_dims)
    rd = (C.c_int32 * n)(*[int(v) for v in reduction_dims])
    w = None if weights is None else (C.c_int64 * n)(*[int(v) for v in weights])
    nl = C.c_int32()
    perm = (C.c_int32 * (max_layouts * MAX_DIMS))()
    loc = (C.c_int32 * n)()
    _check(lib().smartmem_select_layouts(ndim, n, rd, w, k, max_layouts, C.byref(nl), perm, loc), "smartmem_select_layouts")
    return [[perm[l * MAX_DIMS + p] for p in range(ndim)] for l in range(nl.value)], list(loc)


def smartmem_pair_decision(first: int, second: int):
    a, r, s = C.c_int32(), C.c_int32(), C.c_int32()
    _check(lib().smartmem_pair_decision(first, second, C.byref(a), C.byref(r), C.byref(s)), "smartmem_pair_decision")
    return a.value, r.value, s.value


def smartmem_plan(ops, inputs, mode: int) -> int:
    """ops: list of Op; inputs: list of TensorDesc.  Returns an opaque plan handle."""
    arr_o = (Op * len(ops))(*ops)
    arr_i = (TensorDesc * len(inputs))(*inputs)
    h = C.c_void_p()
    _check(lib().smartmem_plan(arr_o, len(ops), arr_i, len(inputs), mode, C.byref(h)), "smartmem_plan")
    return h.value


def smartmem_plan_destroy(plan: int):
    _check(lib().smartmem_plan_destroy(plan), "smartmem_plan_destroy")


def smartmem_plan_num_steps(plan: int):
    a, b = C.c_int32(), C.c_int32()
    _check(lib().smartmem_plan_num_steps(plan, C.byref(a), C.byref(b)), "smartmem_plan_num_steps")
    return a.value, b.value


def smartmem_plan_get_map(plan: int, step: int, operand: int = 0) -> IndexMap:
    m = IndexMap()
    _check(lib().smartmem_plan_get_map(plan, step, operand, C.byref(m)), "smartmem_plan_get_map")
    return m


def smartmem_plan_output_desc(plan: int) -> TensorDesc:
    d = TensorDesc()
    _check(lib().smartmem_plan_output_desc(plan, C.byref(d)), "smartmem_plan_output_desc")
    return d


def smartmem_plan_workspace_bytes(plan: int) -> int:
    n = C.c_size_t()
    _check(lib().smartmem_plan_workspace_bytes(plan, C.byref(n)), "smartmem_plan_workspace_bytes")
    return n.value


def smartmem_map_eval(m: IndexMap, i: int) -> int:
    return lib().smartmem_map_eval(C.byref(m), i)


def smartmem_plan_eval_sequential(plan: int, step: int, operand: int, i: int) -> int:
    return lib().smartmem_plan_eval_sequential(plan, step, operand, i)


def smartmem_run_chain(plan: int, inputs, outputs, workspace: int, workspace_bytes: int, stream: int):
    """inputs / outputs: lists of device pointers (ints)."""
    ai = (C.c_void_p * len(inputs))(*inputs)
    ao = (C.c_void_p * len(outputs))(*outputs)
    _check(lib().smartmem_run_chain(plan, ai, ao, workspace, workspace_bytes, stream), "smartmem_run_chain")


def smartmem_swin_block_workspace_bytes(p: SwinParams, mode: int) -> int:
    n = C.c_size_t()
    _check(lib().smartmem_swin_block_workspace_bytes(C.byref(p), mode, C.byref(n)), "smartmem_swin_block_workspace_bytes")
    return n.value


def smartmem_swin_block(p: SwinParams, x: int, y: int, workspace: int, workspace_bytes: int, mode: int, stream: int):
    _check(lib().smartmem_swin_block(C.byref(p), x, y, workspace, workspace_bytes, mode, stream), "smartmem_swin_block")


def smartmem_swin_block_half(p: SwinParams, x: int, y: int, workspace: int, workspace_bytes: int, mode: int, half: int, stream: int):
    _check(lib().smartmem_swin_block_half(C.byref(p), x, y, workspace, workspace_bytes, mode, half, stream), "smartmem_swin_block_half")


def smartmem_swin_block_timed(p: SwinParams, x: int, y: int, workspace: int, workspace_bytes: int, mode: int, stream: int):
    """Runs the block with an event before every kernel; returns [(label, milliseconds), ...]."""
    maxk, stride = 32, 48
    ms = (C.c_float * maxk)()
    names = C.create_string_buffer(maxk * stride)
    n = C.c_int32()
    _check(lib().smartmem_swin_block_timed(C.byref(p), x, y, workspace, workspace_bytes, mode, stream, ms, names, stride,
                                           maxk, C.byref(n)), "smartmem_swin_block_timed")
    raw = names.raw
    return [(raw[i * stride:(i + 1) * stride].split(b"\0", 1)[0].decode(), float(ms[i])) for i in range(n.value)]


def smartmem_swin_block_static_scratch_bytes() -> int:
    n = C.c_size_t()
    _check(lib().smartmem_swin_block_static_scratch_bytes(C.byref(n)), "smartmem_swin_block_static_scratch_bytes")
    return n.value


def smartmem_swin_block_noalloc(p: SwinParams, x: int, y: int, mode: int, stream: int):
    """The Swin block for callers that cannot allocate device memory: no workspace argument, the
    intermediates live in a fixed 32 MiB array inside the library.  Calls share that array, so
    calls that overlap on the GPU race; blocks that need more are rejected (ERR_WORKSPACE)."""
    _check(lib().smartmem_swin_block_noalloc(C.byref(p), x, y, mode, stream), "smartmem_swin_block_noalloc")


def smartmem_attn_layer_workspace_bytes(p: AttnParams, mode: int) -> int:
    n = C.c_size_t()
    _check(lib().smartmem_attn_layer_workspace_bytes(C.byref(p), mode, C.byref(n)), "smartmem_attn_layer_workspace_bytes")
    return n.value


def smartmem_attn_layer(p: AttnParams, x: int, y: int, workspace: int, workspace_bytes: int, mode: int, stream: int):
    _check(lib().smartmem_attn_layer(C.byref(p), x, y, workspace, workspace_bytes, mode, stream), "smartmem_attn_layer")


def smartmem_attn_decode_workspace_bytes(p: AttnParams, mode: int) -> int:
    n = C.c_size_t()
    _check(lib().smartmem_attn_decode_workspace_bytes(C.byref(p), mode, C.byref(n)), "smartmem_attn_decode_workspace_bytes")
    return n.value


def smartmem_attn_decode(p: AttnParams, pos: int, x: int, k_cache: int, v_cache: int, y: int, workspace: int,
                         workspace_bytes: int, mode: int, stream: int):
    _check(lib().smartmem_attn_decode(C.byref(p), pos, x, k_cache, v_cache, y, workspace, workspace_bytes, mode, stream),
           "smartmem_attn_decode")


def smartmem_profile_begin():
    _check(lib().smartmem_profile_begin(), "smartmem_profile_begin")


def smartmem_profile_end(stream: int):
    """Returns [(label, milliseconds), ...] for every kernel launched since smartmem_profile_begin()."""
    maxk, stride = 256, 32
    ms = (C.c_float * maxk)()
    names = C.create_string_buffer(maxk * stride)
    n = C.c_int32()
    _check(lib().smartmem_profile_end(stream, ms, names, stride, maxk, C.byref(n)), "smartmem_profile_end")
    raw = names.raw
    return [(raw[i * stride:(i + 1) * stride].split(b"\0", 1)[0].decode(), float(ms[i])) for i in range(n.value)]


def smartmem_last_device_status(stream: int) -> int:
    s = C.c_int32()
    _check(lib().smartmem_last_device_status(stream, C.byref(s)), "smartmem_last_device_status")
    return s.value


def smartmem_set_wait_limit_ns(limit_ns: int) -> None:
    _check(lib().smartmem_set_wait_limit_ns(int(limit_ns)), "smartmem_set_wait_limit_ns")


def smartmem_selftest_bounded_wait(stream: int) -> None:
    _check(lib().smartmem_selftest_bounded_wait(stream), "smartmem_selftest_bounded_wait")


def smartmem_fanout_plan(p: FanoutParams, mode: int) -> dict:
    n, lb, pb, cb, ws = C.c_int32(), C.c_int32(), C.c_int64(), C.c_int64(), C.c_size_t()
    _check(lib().smartmem_fanout_plan(C.byref(p), mode, C.byref(n), C.byref(lb), C.byref(pb), C.byref(cb), C.byref(ws)),
           "smartmem_fanout_plan")
    return {"copies_written": n.value, "layout_of_consumer_b": lb.value, "producer_bytes_written": pb.value,
            "copy_kernel_bytes": cb.value, "workspace_bytes": ws.value}


def smartmem_fanout(p: FanoutParams, x: int, ya: int, yb: int, workspace: int, workspace_bytes: int, mode: int, stream: int):
    _check(lib().smartmem_fanout(C.byref(p), x, ya, yb, workspace, workspace_bytes, mode, stream), "smartmem_fanout")


def smartmem_launch_count() -> int:
    return lib().smartmem_launch_count()
