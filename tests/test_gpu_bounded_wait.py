"""A bounded device-side wait that runs out: the kernel returns, the host reads SMARTMEM_ERR_TIMEOUT, and
the context stays usable.  The wait is the kernels' own (`mbar_wait`), on a barrier nothing arrives at."""
import time

import pytest

pytestmark = pytest.mark.gpu


def test_wait_runs_out_and_the_context_survives():
    import torch
    from paper_2404_13528_b200 import binding as sm

    st = torch.cuda.current_stream().cuda_stream
    assert sm.smartmem_last_device_status(st) == sm.OK
    sm.smartmem_set_wait_limit_ns(50_000_000)            # 50 ms
    try:
        t0 = time.perf_counter()
        sm.smartmem_selftest_bounded_wait(st)
        status = sm.smartmem_last_device_status(st)      # synchronises the stream
        dt = time.perf_counter() - t0
        assert status == sm.ERR_TIMEOUT
        assert 0.04 < dt < 0.9, dt                       # it waited for the limit, and not for the default second
        assert sm.smartmem_last_device_status(st) == sm.OK   # reading the status cleared it
    finally:
        sm.smartmem_set_wait_limit_ns(1_000_000_000)
    # the context is intact: an ordinary call runs and matches
    from tests.test_gpu_chains import CH2A, copy_chain_case
    copy_chain_case((2, 96, 4 * 64), CH2A(2, 96, 4, 64))
    assert sm.smartmem_last_device_status(st) == sm.OK


def test_wait_limit_rejects_nonsense():
    from paper_2404_13528_b200 import binding as sm

    for bad in (0, 61_000_000_000):
        with pytest.raises(sm.SmartmemError):
            sm.smartmem_set_wait_limit_ns(bad)
