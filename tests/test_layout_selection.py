"""Reduction-dimension layout selection (host planner): the paper's worked example, invariants and a brute-force
optimality check, for the oracle's step-by-step form and for the library's smartmem_select_layouts."""
import itertools
import os

import numpy as np
import pytest

from oracle import layout_select
from paper_2404_13528_b200 import binding as sm

GOLD = os.path.join(os.path.dirname(__file__), "golden", "layout_selection_example.txt")


def _gold():
    d = {}
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        d[k] = [int(x) for x in v]
    return d


def both(ndim, rds, w=None, k=1):
    a = layout_select.select_layouts(ndim, rds, w, k)
    b = sm.smartmem_select_layouts(ndim, rds, w, k)
    assert a == (b[0], b[1]), (a, b)
    return a


def test_paper_example_one_layout_serves_both_reduction_dimensions():
    g = _gold()
    layouts, where = both(g["ndim"][0], g["consumers"], None, g["k"][0])
    assert len(layouts) == g["n_layouts"][0]
    assert sorted(layouts[0][-g["k"][0]:]) == g["served_dims_layout0"]
    assert layouts[0][-1] == 2                      # D3 has two consumers: it is the contiguous one
    assert where == [0, 0, 0]
    # linear memory (k = 1): the same consumers need two copies, D3 first
    layouts, where = both(3, g["consumers"], None, 1)
    assert layouts == [[0, 1, 2], [1, 2, 0]] and where == [1, 0, 0]


def check_invariants(ndim, rds, w, k):
    layouts, where = both(ndim, rds, w, k)
    ww = [1] * len(rds) if w is None else w
    demanded = sorted({r for r in rds if r >= 0})
    assert len(layouts) == max(1, -(-len(demanded) // k))
    for L in layouts:
        assert sorted(L) == list(range(ndim))                                   # a permutation
    for c, r in enumerate(rds):
        if r < 0:
            assert where[c] == 0
        else:
            assert r in layouts[where[c]][-k:]                                  # served among the k contiguous-most dims
    # no k-subset of dimensions covers more consumer weight than layout 0 does (brute force)
    cover = lambda dims: sum(x for r, x in zip(rds, ww) if r in dims)
    best = max(cover(set(s)) for s in itertools.combinations(range(ndim), min(k, ndim)))
    assert cover(set(layouts[0][-k:])) == best
    # dimensions that layout 0 does not serve keep their natural order
    outer = layouts[0][: ndim - min(k, len(demanded))]
    assert outer == sorted(outer)


def test_invariants_and_bruteforce_optimality():
    rng = np.random.default_rng(5)
    for _ in range(300):
        ndim = int(rng.integers(1, 7))
        n = int(rng.integers(1, 7))
        rds = [int(rng.integers(-1, ndim)) for _ in range(n)]
        w = None if rng.random() < 0.3 else [int(rng.integers(1, 9)) for _ in range(n)]
        k = int(rng.integers(1, ndim + 1))
        check_invariants(ndim, rds, w, k)


def test_special_cases():
    assert both(4, [-1, -1]) == ([[0, 1, 2, 3]], [0, 0])                        # no requirement: natural layout
    assert both(2, [1]) == ([[0, 1]], [0])                                      # MatMul A[i,k]: k already contiguous
    assert both(2, [0]) == ([[1, 0]], [0])                                      # reduction over rows: transposed store
    assert both(3, [0, 1, 1, 2, 2, 2], None, 1) == ([[0, 1, 2], [0, 2, 1], [1, 2, 0]], [2, 1, 1, 0, 0, 0])
    assert both(3, [0, 2], [5, 1], 1) == ([[1, 2, 0], [0, 1, 2]], [0, 1])      # weight beats count


def test_argument_errors():
    for args in ((0, [0]), (3, [3]), (3, [0], [0]), (3, [-2])):
        with pytest.raises(sm.SmartmemError) as e:
            sm.smartmem_select_layouts(*args)
        assert e.value.code == sm.ERR_INVALID_ARG
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_select_layouts(3, [0], None, 4)
    assert e.value.code == sm.ERR_INVALID_ARG
    with pytest.raises(sm.SmartmemError) as e:
        sm.smartmem_select_layouts(3, [0, 1, 2], None, 1, max_layouts=2)
    assert e.value.code == sm.ERR_UNSUPPORTED
