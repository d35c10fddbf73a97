"""Host planner: classification tables, composed index maps against the oracle's
materialised operators (brute force over every consumer index), EXPLICIT expansion,
error handling.  CPU only (no CUDA call is made)."""
import itertools

import numpy as np
import pytest

from oracle import chains
from paper_2404_13528_b200 import binding as sm


def _ops_from_chain(chain):
    out = []
    for o in chain:
        k = o["op"]
        if k == "reshape":
            out.append(sm.make_op(sm.OP_RESHAPE, shape=o["shape"]))
        elif k == "transpose":
            out.append(sm.make_op(sm.OP_TRANSPOSE, perm=o["perm"]))
        elif k == "roll":
            out.append(sm.make_op(sm.OP_ROLL, shift=o["shift"], axis=o["axis"]))
        elif k == "slice":
            out.append(sm.make_op(sm.OP_SLICE, start=o["start"], shape=o["extent"]))
        elif k == "window_partition":
            out.append(sm.make_op(sm.OP_WINDOW_PARTITION, window=o["window"]))
        elif k == "window_reverse":
            out.append(sm.make_op(sm.OP_WINDOW_REVERSE, window=o["window"], shape=(o["B"], o["H"], o["W"])))
        elif k == "depth_to_space":
            out.append(sm.make_op(sm.OP_DEPTH_TO_SPACE, window=o["block"]))
        elif k == "space_to_depth":
            out.append(sm.make_op(sm.OP_SPACE_TO_DEPTH, window=o["block"]))
    return out


def _plan_copy(shape, chain, mode=sm.ELIMINATE, dtype=sm.BF16):
    ops = _ops_from_chain(chain) + [sm.make_op(sm.OP_COPY)]
    return sm.smartmem_plan(ops, [sm.make_desc(shape, dtype)], mode)


def _check_map_against_oracle(shape, chain, expect_klass=None):
    ref = chains.source_offsets(shape, chain).reshape(-1)
    plan = _plan_copy(shape, chain)
    try:
        assert sm.smartmem_plan_num_steps(plan) == (1, 0)
        m = sm.smartmem_plan_get_map(plan, 0)
        assert m.n_elements == ref.size
        seq = [sm.smartmem_plan_eval_sequential(plan, 0, 0, i) for i in range(ref.size)]
        assert seq == ref.tolist()
        if m.klass != 3:
            got = [sm.smartmem_map_eval(m, i) for i in range(ref.size)]
            assert got == ref.tolist()
            v = m.vec_elems          # a vector is contiguous in the source and never straddles a wrap
            if v > 1:
                r = ref.reshape(-1, v)
                assert (np.diff(r, axis=1) == 1).all() and (r[:, 0] % v == 0).all()
        if expect_klass is not None:
            assert m.klass == expect_klass
        d = sm.smartmem_plan_output_desc(plan)
        assert tuple(d.shape[: d.ndim]) == chains.source_offsets(shape, chain).shape
        return m
    finally:
        sm.smartmem_plan_destroy(plan)


# ------------------------------------------------------------------ Tables 3, 5, 6
def test_table3_quadrants():
    ILD_VAR, ILI_VAR, ILD_FIX, ILI_FIX = 0, 1, 2, 3
    assert sm.smartmem_op_quadrant(sm.OP_LINEAR) == ILD_VAR      # MatMul
    assert sm.smartmem_op_quadrant(sm.OP_BMM_NT) == ILD_VAR
    assert sm.smartmem_op_quadrant(sm.OP_COPY) == ILI_VAR        # Unary
    assert sm.smartmem_op_quadrant(sm.OP_RESHAPE) == ILD_FIX
    assert sm.smartmem_op_quadrant(sm.OP_TRANSPOSE) == ILD_FIX
    assert sm.smartmem_op_quadrant(sm.OP_SLICE) == ILI_FIX
    assert sm.smartmem_op_quadrant(sm.OP_ROLL) == ILI_FIX        # Gather class
    assert sm.smartmem_op_quadrant(sm.OP_DEPTH_TO_SPACE) == ILD_FIX    # DtoS
    assert sm.smartmem_op_quadrant(sm.OP_SPACE_TO_DEPTH) == ILD_FIX    # StoD
    assert sm.smartmem_op_quadrant(sm.OP_LAYERNORM) == ILD_VAR


def test_tables_5_and_6_all_cells():
    KEEP, FUSE, E1, E2, BOTH = 0, 1, 2, 3, 4
    NONE, S_BOTH, S_FUSED, S_1ST, S_2ND = 0, 1, 2, 3, 4
    # rows = first operator, columns = second; quadrant order ILD&Var, ILI&Var, ILD&Fixed, ILI&Fixed
    action = [[KEEP, FUSE, E2, E2], [FUSE, FUSE, E2, E2], [E1, E1, BOTH, BOTH], [E1, E1, BOTH, BOTH]]
    result = [[0, 0, 0, 0], [0, 1, 1, 1], [0, 1, -1, -1], [0, 1, -1, -1]]
    search = [[S_BOTH, S_FUSED, S_1ST, S_1ST], [S_FUSED, NONE, NONE, NONE], [S_2ND, NONE, NONE, NONE],
              [S_2ND, NONE, NONE, NONE]]
    for a, b in itertools.product(range(4), range(4)):
        assert sm.smartmem_pair_decision(a, b) == (action[a][b], result[a][b], search[a][b]), (a, b)
    with pytest.raises(sm.SmartmemError):
        sm.smartmem_pair_decision(4, 0)


# ------------------------------------------------------------------ composed maps
def test_paper_example_map():
    # Section 2.2: 5x5x5 -> Reshape 5x25 -> Transpose 25x5; consumer (5b+c, a) <- (a,b,c)
    m = _check_map_against_oracle((5, 5, 5), [{"op": "reshape", "shape": (5, 25)}, {"op": "transpose", "perm": (1, 0)}], 1)
    assert m.n_atoms == 2 and list(m.extent[:2]) == [25, 5] and list(m.src_stride[:2]) == [1, 25]


def test_reshape_only_chain_vanishes():
    m = _check_map_against_oracle((4, 6, 8), [{"op": "reshape", "shape": (24, 8)}, {"op": "reshape", "shape": (2, 12, 8)}], 0)
    assert m.n_atoms == 1 and m.vec_elems == 8


def test_chain_2a_and_2b_maps():
    B, S, H, D = 2, 16, 4, 8
    m = _check_map_against_oracle((B, S, H * D), [{"op": "reshape", "shape": (B, S, H, D)},
                                                  {"op": "transpose", "perm": (0, 2, 1, 3)}], 1)
    assert list(m.extent[:4]) == [B, H, S, D] and list(m.src_stride[:4]) == [S * H * D, D, H * D, 1]
    assert m.vec_elems == 8
    B, Cc, Hh, Ww = 2, 8, 4, 4
    m = _check_map_against_oracle((B, Cc, Hh, Ww), [{"op": "transpose", "perm": (0, 2, 3, 1)},
                                                    {"op": "reshape", "shape": (B * Hh * Ww, Cc)}], 1)
    assert list(m.extent[:3]) == [B, Hh * Ww, Cc] and list(m.src_stride[:3]) == [Cc * Hh * Ww, 1, Hh * Ww]
    assert m.vec_elems == 1


@pytest.mark.parametrize("B,H,W,C,ws,s", [(1, 8, 8, 8, 4, 2), (2, 14, 14, 8, 7, 3), (1, 21, 14, 16, 7, 3), (2, 8, 8, 8, 4, 0)])
def test_swin_shift_partition_map(B, H, W, C, ws, s):
    chain = [{"op": "roll", "shift": -s, "axis": 1}, {"op": "roll", "shift": -s, "axis": 2},
             {"op": "window_partition", "window": ws}]
    m = _check_map_against_oracle((B, H, W, C), chain, 2 if s else 1)
    assert m.vec_elems == 8 and m.n_rolls == (2 if s else 0)
    # the store-side map of the second half of the block: window reverse then reverse shift
    nW = B * (H // ws) * (W // ws)
    chain = [{"op": "window_reverse", "window": ws, "B": B, "H": H, "W": W},
             {"op": "roll", "shift": s, "axis": 1}, {"op": "roll", "shift": s, "axis": 2}]
    # (gather form: H and W are not affine coordinates of the windowed buffer; the rolled coordinate
    # is decomposed again over the window factors after the wrap)
    m2 = _check_map_against_oracle((nW, ws * ws, C), chain, 2 if s else 1)
    if s:
        assert m2.n_rolls == 2 and list(m2.roll_n_parts[:2]) == [2, 2] and m2.vec_elems == 8


def test_head_split_slice_map():
    nW, T, heads, d = 3, 4, 2, 8
    Cc = heads * d
    for which in range(3):
        chain = [{"op": "reshape", "shape": (nW, T, 3, heads, d)}, {"op": "transpose", "perm": (2, 0, 3, 1, 4)},
                 {"op": "slice", "start": (which, 0, 0, 0, 0), "extent": (1, nW, heads, T, d)}]
        m = _check_map_against_oracle((nW, T, 3 * Cc), chain, 1)
        assert m.base == which * Cc and m.vec_elems == 8


def test_rolls_compose_and_slice_of_rolled_dim():
    _check_map_against_oracle((6, 8), [{"op": "roll", "shift": 2, "axis": 0}, {"op": "roll", "shift": 3, "axis": 0}], 2)
    _check_map_against_oracle((6, 8), [{"op": "roll", "shift": 2, "axis": 0}, {"op": "roll", "shift": 4, "axis": 0}], 0)
    _check_map_against_oracle((6, 8), [{"op": "roll", "shift": -1, "axis": 0},
                                       {"op": "slice", "start": (2, 0), "extent": (3, 8)}], 2)
    _check_map_against_oracle((6, 8), [{"op": "roll", "shift": 1, "axis": 1}], 2)


def test_non_refinable_chain_falls_back_to_sequential():
    # [4,6] -> transpose -> [6,4] -> reshape [8,3]: split points do not refine
    m = _check_map_against_oracle((4, 6), [{"op": "transpose", "perm": (1, 0)}, {"op": "reshape", "shape": (8, 3)}], 3)
    assert sm.smartmem_map_eval(m, 0) == -1


def test_strided_input():
    ops = [sm.make_op(sm.OP_TRANSPOSE, perm=(1, 0)), sm.make_op(sm.OP_COPY)]
    plan = sm.smartmem_plan(ops, [sm.make_desc((4, 6), sm.F32, stride=(10, 1))], sm.ELIMINATE)
    m = sm.smartmem_plan_get_map(plan, 0)
    for j, i in itertools.product(range(6), range(4)):
        assert sm.smartmem_map_eval(m, j * 4 + i) == i * 10 + j
        assert sm.smartmem_plan_eval_sequential(plan, 0, 0, j * 4 + i) == i * 10 + j
    sm.smartmem_plan_destroy(plan)


def test_random_chains_bruteforce():
    rng = np.random.default_rng(2024)
    n_canonical = 0
    for trial in range(150):
        nd = int(rng.integers(2, 5))
        shape = tuple(int(rng.choice([2, 3, 4, 6, 8])) for _ in range(nd))
        cur = shape
        chain = []
        for _ in range(int(rng.integers(1, 5))):
            kind = rng.choice(["reshape", "transpose", "roll", "slice"])
            if kind == "reshape":
                n = int(np.prod(cur))
                dims = []
                rem = n
                while rem > 1 and len(dims) < 4:
                    divs = [d for d in range(2, rem + 1) if rem % d == 0]
                    d = int(rng.choice(divs))
                    dims.append(d)
                    rem //= d
                if rem > 1:
                    dims.append(rem)
                if not dims:
                    dims = [1]
                rng.shuffle(dims)
                chain.append({"op": "reshape", "shape": tuple(dims)})
                cur = tuple(dims)
            elif kind == "transpose":
                perm = tuple(int(p) for p in rng.permutation(len(cur)))
                chain.append({"op": "transpose", "perm": perm})
                cur = tuple(cur[p] for p in perm)
            elif kind == "roll":
                ax = int(rng.integers(0, len(cur)))
                chain.append({"op": "roll", "shift": int(rng.integers(-5, 6)), "axis": ax})
            else:
                start = tuple(int(rng.integers(0, n)) if rng.random() < 0.4 else 0 for n in cur)
                ext = tuple(int(rng.integers(1, n - s + 1)) if s or rng.random() < 0.3 else n for n, s in zip(cur, start))
                chain.append({"op": "slice", "start": start, "extent": ext})
                cur = ext
        m = _check_map_against_oracle(shape, chain)
        n_canonical += m.klass != 3
    assert n_canonical > 75        # the canonical form must cover most chains, not just trivial ones


# ------------------------------------------------------------------ EXPLICIT expansion
def test_explicit_mode_materialises_each_data_moving_op():
    B, H, W, Cc, ws, s = 1, 8, 8, 8, 4, 2
    chain = [{"op": "roll", "shift": -s, "axis": 1}, {"op": "roll", "shift": -s, "axis": 2},
             {"op": "reshape", "shape": (B, H, W, Cc)}, {"op": "window_partition", "window": ws}]
    plan = _plan_copy((B, H, W, Cc), chain, sm.EXPLICIT)
    steps, copies = sm.smartmem_plan_num_steps(plan)
    assert (steps, copies) == (4, 3)           # 2 rolls + 1 partition materialised, reshape is metadata, + the consumer
    cur = (B, H, W, Cc)
    singles = [chain[0:1], chain[1:2], chain[2:4]]
    for st, sub in enumerate(singles):
        ref = chains.source_offsets(cur, sub)
        m = sm.smartmem_plan_get_map(plan, st)
        assert [sm.smartmem_map_eval(m, i) for i in range(ref.size)] == ref.reshape(-1).tolist()
        cur = ref.shape
    assert sm.smartmem_plan_get_map(plan, 3).klass == 0          # the consumer reads a materialised buffer
    assert sm.smartmem_plan_workspace_bytes(plan) >= 3 * B * H * W * Cc * 2
    sm.smartmem_plan_destroy(plan)
    plan = _plan_copy((B, H, W, Cc), chain, sm.ELIMINATE)
    assert sm.smartmem_plan_num_steps(plan) == (1, 0) and sm.smartmem_plan_workspace_bytes(plan) == 0
    sm.smartmem_plan_destroy(plan)


def test_gemm_consumers_keep_reduction_atoms_separate():
    B, S, H, D = 2, 256, 4, 64
    ops = [sm.make_op(sm.OP_RESHAPE, shape=(B, S, H, D)), sm.make_op(sm.OP_TRANSPOSE, perm=(0, 2, 1, 3)),
           sm.make_op(sm.OP_BMM_NT, side_input=(1, 0))]
    descs = [sm.make_desc((B, S, H * D)), sm.make_desc((B, S, H * D))]
    plan = sm.smartmem_plan(ops, descs, sm.ELIMINATE)
    for operand in (0, 1):
        m = sm.smartmem_plan_get_map(plan, 0, operand)
        assert list(m.extent[:4]) == [B, H, S, D] and list(m.src_stride[:4]) == [S * H * D, D, H * D, 1]
    d = sm.smartmem_plan_output_desc(plan)
    assert tuple(d.shape[:4]) == (B, H, S, S)
    sm.smartmem_plan_destroy(plan)
    plan = sm.smartmem_plan(ops, descs, sm.EXPLICIT)
    assert sm.smartmem_plan_num_steps(plan) == (3, 2)            # one transpose copy per operand
    sm.smartmem_plan_destroy(plan)
    # identity chain into a linear layer: rows and reduction dim stay two atoms
    ops = [sm.make_op(sm.OP_LINEAR, side_input=(1, 0))]
    plan = sm.smartmem_plan(ops, [sm.make_desc((128, 64)), sm.make_desc((32, 64))], sm.ELIMINATE)
    m = sm.smartmem_plan_get_map(plan, 0)
    assert m.n_atoms == 2 and m.klass == 0
    sm.smartmem_plan_destroy(plan)


# ------------------------------------------------------------------ errors
def test_plan_errors():
    d = [sm.make_desc((4, 6))]
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_plan([sm.make_op(sm.OP_RESHAPE, shape=(5, 5)), sm.make_op(sm.OP_COPY)], d, sm.ELIMINATE)
    assert e.value.code == sm.ERR_SHAPE
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_plan([sm.make_op(sm.OP_TRANSPOSE, perm=(0, 0)), sm.make_op(sm.OP_COPY)], d, sm.ELIMINATE)
    assert e.value.code == sm.ERR_SHAPE
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_plan([sm.make_op(sm.OP_TRANSPOSE, perm=(1, 0))], d, sm.ELIMINATE)       # no consumer
    assert e.value.code == sm.ERR_INVALID_ARG
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_plan([sm.make_op(sm.OP_COPY)], d, 7)
    assert e.value.code == sm.ERR_INVALID_ARG
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_plan([sm.make_op(sm.OP_WINDOW_PARTITION, window=4), sm.make_op(sm.OP_COPY)],
                         [sm.make_desc((1, 6, 8, 4))], sm.ELIMINATE)
    assert e.value.code == sm.ERR_SHAPE
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_plan([sm.make_op(sm.OP_LINEAR, side_input=(1, 0))], [sm.make_desc((4, 6)), sm.make_desc((3, 5))], sm.ELIMINATE)
    assert e.value.code == sm.ERR_SHAPE
    assert sm.smartmem_status_string(sm.ERR_TIMEOUT) == "device-side wait timed out"


# ------------------------------------------------------------------ producer-side placement (Section 3.2.2)
@pytest.mark.parametrize("shape,chain", [
    ((2, 6, 4 * 3), [{"op": "reshape", "shape": (2, 6, 4, 3)}, {"op": "transpose", "perm": (0, 2, 1, 3)}]),
    ((2, 5, 3, 4), [{"op": "transpose", "perm": (0, 2, 3, 1)}, {"op": "reshape", "shape": (2, 12, 5)}]),
    ((2, 8, 8, 3), [{"op": "roll", "shift": -2, "axis": 1}, {"op": "roll", "shift": -2, "axis": 2},
                    {"op": "window_partition", "window": 4}]),
    ((2 * 2 * 2, 16, 3), [{"op": "window_reverse", "window": 4, "B": 2, "H": 8, "W": 8},
                          {"op": "roll", "shift": 2, "axis": 1}, {"op": "roll", "shift": 2, "axis": 2}]),
    ((5, 5, 5), [{"op": "reshape", "shape": (5, 25)}, {"op": "transpose", "perm": (1, 0)}]),
])
def test_scatter_placement_map_is_the_inverse_permutation(shape, chain):
    """ELIMINATE_SCATTER plans the inverted chain: its map sends input element i to the output position
    that, in the oracle's materialised result, holds input element i."""
    src = chains.source_offsets(shape, chain).reshape(-1)          # output position -> input element
    dest = np.empty_like(src)
    dest[src] = np.arange(src.size)                                # input element -> output position
    plan = _plan_copy(shape, chain, mode=sm.ELIMINATE_SCATTER)
    try:
        assert sm.smartmem_plan_num_steps(plan) == (1, 0)
        m = sm.smartmem_plan_get_map(plan, 0)
        assert m.klass != 3 and m.n_elements == src.size
        assert [sm.smartmem_map_eval(m, i) for i in range(src.size)] == dest.tolist()
        d = sm.smartmem_plan_output_desc(plan)
        assert tuple(d.shape[: d.ndim]) == chains.source_offsets(shape, chain).shape
    finally:
        sm.smartmem_plan_destroy(plan)
    g = _plan_copy(shape, chain, mode=sm.ELIMINATE_GATHER)         # consumer side: the usual map
    try:
        mg = sm.smartmem_plan_get_map(g, 0)
        assert [sm.smartmem_map_eval(mg, i) for i in range(src.size)] == src.tolist()
    finally:
        sm.smartmem_plan_destroy(g)


def test_placement_modes_reject_what_they_cannot_invert():
    sl = [{"op": "slice", "start": (1, 0), "extent": (2, 4)}]
    with pytest.raises(sm.SmartmemError):
        _plan_copy((4, 4), sl, mode=sm.ELIMINATE_SCATTER)           # a Slice drops elements
    ops = [sm.make_op(sm.OP_LINEAR, side_input=(1, 0))]
    with pytest.raises(sm.SmartmemError):
        sm.smartmem_plan(ops, [sm.make_desc((8, 8)), sm.make_desc((8, 8))], sm.ELIMINATE_SCATTER)   # copy-only chains


# ------------------------------------------------------------------ DtoS / StoD, LayerNorm consumer
@pytest.mark.parametrize("shape,chain", [
    ((2, 12, 3, 4), [{"op": "depth_to_space", "block": 2}]),
    ((2, 3, 4, 6), [{"op": "space_to_depth", "block": 2}]),
    ((1, 18, 2, 2), [{"op": "depth_to_space", "block": 3}]),
    ((2, 3, 4, 6), [{"op": "space_to_depth", "block": 2}, {"op": "depth_to_space", "block": 2}]),       # composes to the identity
    ((2, 8, 4, 4), [{"op": "depth_to_space", "block": 2}, {"op": "transpose", "perm": (0, 2, 3, 1)}]),  # NCHW -> NHWC after it
])
def test_depth_space_maps(shape, chain):
    m = _check_map_against_oracle(shape, chain)
    assert m.klass in (0, 1)
    if len(chain) == 2 and chain[0]["op"] == "space_to_depth" and chain[1]["op"] == "depth_to_space":
        assert m.klass == 0


def test_depth_space_shape_errors():
    for op, shape in ((sm.OP_DEPTH_TO_SPACE, (1, 6, 2, 2)), (sm.OP_SPACE_TO_DEPTH, (1, 2, 3, 4)), (sm.OP_SPACE_TO_DEPTH, (2, 4, 4))):
        with pytest.raises(sm.SmartmemError) as e:
            sm.smartmem_plan([sm.make_op(op, window=2), sm.make_op(sm.OP_COPY)], [sm.make_desc(shape)], sm.ELIMINATE)
        assert e.value.code == sm.ERR_SHAPE


def _patch_merge_ops(B, H, W, C):
    return [sm.make_op(sm.OP_RESHAPE, shape=(B, H // 2, 2, W // 2, 2, C)), sm.make_op(sm.OP_TRANSPOSE, perm=(0, 1, 3, 4, 2, 5)),
            sm.make_op(sm.OP_RESHAPE, shape=(B, (H // 2) * (W // 2), 4 * C)),
            sm.make_op(sm.OP_LAYERNORM, side_input=(1, 2), eps=1e-5), sm.make_op(sm.OP_LINEAR, side_input=(3, 0))]


def test_patch_merging_plan_folds_the_gather_into_the_layernorm():
    B, H, W, C = 2, 4, 6, 8
    descs = [sm.make_desc((B, H, W, C)), sm.make_desc((4 * C,)), sm.make_desc((4 * C,)), sm.make_desc((2 * C, 4 * C))]
    ref = chains.source_offsets((B, H, W, C), [{"op": "reshape", "shape": (B, H // 2, 2, W // 2, 2, C)},
                                               {"op": "transpose", "perm": (0, 1, 3, 4, 2, 5)},
                                               {"op": "reshape", "shape": (B, (H // 2) * (W // 2), 4 * C)}]).reshape(-1)
    plan = sm.smartmem_plan(_patch_merge_ops(B, H, W, C), descs, sm.ELIMINATE)
    try:
        assert sm.smartmem_plan_num_steps(plan) == (2, 0)                 # LayerNorm (gathering) + GEMM, no copy
        m = sm.smartmem_plan_get_map(plan, 0)
        assert m.vec_elems == 8 and m.klass == 1
        assert [sm.smartmem_map_eval(m, i) for i in range(ref.size)] == ref.tolist()
        d = sm.smartmem_plan_output_desc(plan)
        assert tuple(d.shape[: d.ndim]) == (B, (H // 2) * (W // 2), 2 * C)
    finally:
        sm.smartmem_plan_destroy(plan)
    plan = sm.smartmem_plan(_patch_merge_ops(B, H, W, C), descs, sm.EXPLICIT)
    try:
        assert sm.smartmem_plan_num_steps(plan) == (3, 1)                 # one materialised transpose
        assert sm.smartmem_plan_get_map(plan, 1).klass == 0
    finally:
        sm.smartmem_plan_destroy(plan)
    # channels that do not fill a 16-byte vector: ELIMINATE materialises the gather too
    descs6 = [sm.make_desc((B, H, W, 6)), sm.make_desc((24,)), sm.make_desc((24,)), sm.make_desc((12, 24))]
    plan = sm.smartmem_plan(_patch_merge_ops(B, H, W, 6), descs6, sm.ELIMINATE)
    try:
        assert sm.smartmem_plan_num_steps(plan) == (3, 1)
    finally:
        sm.smartmem_plan_destroy(plan)


def test_layernorm_consumer_argument_errors():
    B, H, W, C = 1, 2, 2, 8
    ops = _patch_merge_ops(B, H, W, C)
    good = [sm.make_desc((B, H, W, C)), sm.make_desc((4 * C,)), sm.make_desc((4 * C,)), sm.make_desc((2 * C, 4 * C))]
    bad_gamma = list(good)
    bad_gamma[1] = sm.make_desc((4 * C + 8,))
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_plan(ops, bad_gamma, sm.ELIMINATE)
    assert e.value.code == sm.ERR_SHAPE
    ops0 = list(ops)
    ops0[3] = sm.make_op(sm.OP_LAYERNORM, side_input=(1, 2), eps=0.0)
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_plan(ops0, good, sm.ELIMINATE)
    assert e.value.code == sm.ERR_INVALID_ARG
    ops1 = list(ops)
    ops1[3] = sm.make_op(sm.OP_LAYERNORM, side_input=(1, 9), eps=1e-5)
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_plan(ops1, good, sm.ELIMINATE)
    assert e.value.code == sm.ERR_INVALID_ARG


def test_layernorm_over_the_strided_dimension_of_a_channels_first_producer_is_folded():
    """NCHW -> (NHWC view) -> LayerNorm over C: tokens are contiguous in the producer, channels strided.  The planner keeps
    the map on the LayerNorm's load side when the tokens of an image are a multiple of 64, else materialises."""
    def steps(B, C, H, W):
        ops = [sm.make_op(sm.OP_TRANSPOSE, perm=(0, 2, 3, 1)), sm.make_op(sm.OP_RESHAPE, shape=(B, H * W, C)),
               sm.make_op(sm.OP_LAYERNORM, side_input=(1, 2), eps=1e-5), sm.make_op(sm.OP_COPY)]
        plan = sm.smartmem_plan(ops, [sm.make_desc((B, C, H, W)), sm.make_desc((C,)), sm.make_desc((C,))], sm.ELIMINATE)
        try:
            return sm.smartmem_plan_num_steps(plan)
        finally:
            sm.smartmem_plan_destroy(plan)
    assert steps(2, 64, 8, 16)[1] == 0
    assert steps(1, 32, 8, 8)[1] == 0
    assert steps(2, 64, 6, 6)[1] == 1          # 36 tokens per image
    assert steps(2, 63, 8, 8)[1] == 1          # odd channel count
