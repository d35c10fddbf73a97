"""A producer with two consumers of different reduction dimensions (Section 3.2.2, "Global"): what the planner
decides on the host, and -- on the GPU -- that every variant matches the oracle."""
import numpy as np
import pytest

from oracle import chains, layout_select
from paper_2404_13528_b200 import binding as sm
from paper_2404_13528_b200 import synth


def params(B, S, K, N, Na, Nb, k):
    p = sm.FanoutParams()
    p.B, p.S, p.K, p.N, p.Na, p.Nb, p.k_contig = B, S, K, N, Na, Nb, k
    return p


def test_planner_keeps_one_copy_when_two_dimensions_can_be_walked():
    p = params(4, 256, 128, 384, 256, 128, 2)
    d = sm.smartmem_fanout_plan(p, sm.ELIMINATE)
    pbytes = 4 * 256 * 384 * 2
    assert d["copies_written"] == 1 and d["layout_of_consumer_b"] == 0
    assert d["producer_bytes_written"] == pbytes and d["copy_kernel_bytes"] == 0
    assert d["workspace_bytes"] >= pbytes
    # the oracle's selection agrees: one layout, N innermost, S next
    lay, of = layout_select.select_layouts(3, [2, 1], None, 2)
    assert [list(l) for l in lay] == [[0, 1, 2]] and list(of) == [0, 0]


def test_planner_writes_a_redundant_copy_when_only_one_dimension_can():
    p = params(4, 256, 128, 384, 256, 128, 1)
    d = sm.smartmem_fanout_plan(p, sm.ELIMINATE)
    pbytes = 4 * 256 * 384 * 2
    assert d["copies_written"] == 2 and d["layout_of_consumer_b"] == 1
    assert d["producer_bytes_written"] == 2 * pbytes and d["copy_kernel_bytes"] == 0
    assert d["workspace_bytes"] >= 2 * pbytes
    lay, of = layout_select.select_layouts(3, [2, 1], None, 1)
    assert [list(l) for l in lay] == [[0, 1, 2], [0, 2, 1]] and list(of) == [0, 1]


def test_explicit_writes_the_default_layout_and_copies():
    p = params(4, 256, 128, 384, 256, 128, 1)
    d = sm.smartmem_fanout_plan(p, sm.EXPLICIT)
    pbytes = 4 * 256 * 384 * 2
    assert d["copies_written"] == 2 and d["layout_of_consumer_b"] == 1
    assert d["producer_bytes_written"] == pbytes and d["copy_kernel_bytes"] == 2 * pbytes


def test_planner_rejects_bad_requests():
    for bad in (params(0, 256, 128, 384, 256, 128, 1), params(4, 250, 128, 384, 256, 128, 1), params(4, 256, 128, 384, 256, 128, 3)):
        with pytest.raises(sm.SmartmemError):
            sm.smartmem_fanout_plan(bad, sm.ELIMINATE)
    with pytest.raises(sm.SmartmemError):
        sm.smartmem_fanout_plan(params(4, 256, 128, 384, 256, 128, 1), sm.ELIMINATE_NAIVE)


def fan_inputs(B, S, K, N, Na, Nb):
    x = synth.normal(91, 0, (B * S, K), dtype="bf16")
    w_p = synth.normal(91, 1, (N, K), std=K ** -0.5, dtype="bf16")
    w_a = synth.normal(91, 2, (Na, N), std=N ** -0.5, dtype="bf16")
    w_b = synth.normal(91, 3, (Nb, S), std=S ** -0.5, dtype="bf16")
    return x, w_p, w_a, w_b


@pytest.mark.gpu
@pytest.mark.parametrize("shape", [(2, 128, 64, 128, 64, 64),        # one tile each
                                   (3, 200, 96, 264, 136, 72),       # ragged tiles in every dimension
                                   (4, 512, 256, 384, 256, 128)])    # several tiles per GEMM
def test_fanout_matches_the_oracle_in_every_variant(shape):
    import torch
    from tests.gpu_util import assert_close_bf16, check_status, stream, to_dev, to_host_bits, to_host_f64

    B, S, K, N, Na, Nb = shape
    x, w_p, w_a, w_b = fan_inputs(*shape)
    ya_ref, yb_ref = chains.fanout(synth.to_f64(x), synth.to_f64(w_p), synth.to_f64(w_a), synth.to_f64(w_b), B, S)
    d = [to_dev(a) for a in (x, w_p, w_a, w_b)]
    got = {}
    for name, mode, k in (("one copy", sm.ELIMINATE, 2), ("two copies", sm.ELIMINATE, 1), ("explicit", sm.EXPLICIT, 1)):
        p = params(B, S, K, N, Na, Nb, k)
        p.w_p, p.w_a, p.w_b = d[1].data_ptr(), d[2].data_ptr(), d[3].data_ptr()
        info = sm.smartmem_fanout_plan(p, mode)
        ws = torch.empty(info["workspace_bytes"], dtype=torch.uint8, device="cuda")
        ya = torch.full((B * S, Na), float("nan"), dtype=torch.bfloat16, device="cuda")
        yb = torch.full((B, N, Nb), float("nan"), dtype=torch.bfloat16, device="cuda")
        sm.smartmem_fanout(p, d[0].data_ptr(), ya.data_ptr(), yb.data_ptr(), ws.data_ptr(), info["workspace_bytes"], mode, stream())
        check_status()
        assert_close_bf16(to_host_f64(ya), ya_ref, f"{name}: YA")
        assert_close_bf16(to_host_f64(yb), yb_ref, f"{name}: YB")
        got[name] = (to_host_bits(ya), to_host_bits(yb))
        if name == "two copies":                         # the producer's second copy is the transpose of its first, bit for bit
            pbytes = B * S * N * 2
            P = ws[:pbytes].view(torch.bfloat16).view(B, S, N)
            off = (pbytes + 255) // 256 * 256
            Pt = ws[off:off + pbytes].view(torch.bfloat16).view(B, N, S)
            assert torch.equal(Pt, P.transpose(1, 2).contiguous())
    # the layout of P never changes a value of P: consumer A is bit-identical across the variants, and consumer B between the
    # two variants that read the [B, N, S] copy
    assert np.array_equal(got["one copy"][0], got["two copies"][0]) and np.array_equal(got["one copy"][0], got["explicit"][0])
    assert np.array_equal(got["two copies"][1], got["explicit"][1])
