"""CPU oracle: TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 restatement of what the hot path computes.  Every layout operator
(Reshape, Transpose, cyclic shift, window partition/reverse, head split/merge) is
MATERIALISED into a fresh buffer, exactly as the unoptimised operator graph would do it
(the method eliminates these operators without changing the result, Section 3.2.1), and
every compute operator is its textbook definition.  Nothing here is blocked, fused or
reordered, and nothing is shared with the CUDA path.

Only the tests, the smoke check and the benchmark's cpu_baseline / reference arm may
import this package; the product path never does.

Pins (see tests/test_oracle_*.py): the paper's 5x5x5 -> 5x25 -> 25x5 example
(Section 2.2), brute-force Python loops on tiny inputs, closed forms and invariants.
Parity unpinned: the paper prints no numeric output of any whole chain, so full-size
block outputs are pinned only transitively, through the per-operator pins and the
closed-form block cases (uniform attention, zero weights, unshifted == shifted at s=0).
"""
