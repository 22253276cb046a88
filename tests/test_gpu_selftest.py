"""The time-out path of the kernels' bounded waits, exercised without hanging or faulting anything,
and the dense INT8 MMA loop the benchmark uses as its tensor-pipe denominator."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2608_21952_b200 import inputs
from paper_2608_21952_b200.inputs import CONFIGS

pytestmark = pytest.mark.gpu


def test_a_bounded_wait_that_runs_out_sets_the_status_word_and_leaves_the_context_usable():
    """One thread waits, through the library's own wait loop with a cap of 48 polls, on a barrier nothing
    arrives on: the status word reads SSDI8_ERR_DEVICE_TIMEOUT, the kernel returns normally, and an
    ordinary forward pass on the same device afterwards equals the one before bit for bit."""
    import torch
    import gpu_harness as gh
    from paper_2608_21952_b200 import binding as bd
    cfg = CONFIGS["cfg0"]
    t = inputs.make_prefill(cfg)
    q = orc.prepare_quantized(cfg, t)
    y0, fin0, _ = gh.gpu_fwd(cfg, q, taps=())
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    bd.ssdi8_selftest_bounded_wait(status)
    torch.cuda.synchronize()
    assert int(status.item()) == bd.ERR_DEVICE_TIMEOUT == -7
    y1, fin1, _ = gh.gpu_fwd(cfg, q, taps=())          # asserts its own status word is 0
    assert np.array_equal(y0, y1) and np.array_equal(fin0, fin1)
    with pytest.raises(bd.SSDi8Error) as e:
        bd.ssdi8_selftest_bounded_wait(None)
    assert e.value.code == bd.ERR_NULL


def test_int8_mma_peak_runs_and_reports_its_operation_count():
    import torch
    from paper_2608_21952_b200 import binding as bd
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    bd.ssdi8_int8_mma_peak(1024, status)
    e0.record()
    ops = bd.ssdi8_int8_mma_peak(8192, status)
    e1.record()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert ops == 2.0 * 128 * 256 * 32 * 8192 * sms
    tops = ops / (e0.elapsed_time(e1) * 1e-3) / 1e12
    print(f"int8 dense MMA: {tops:.0f} TOPS")
    assert 500 < tops < 9000       # a sanity window around the 4.5 POPS nominal figure
    with pytest.raises(bd.SSDi8Error) as e:
        bd.ssdi8_int8_mma_peak(5, status)
    assert e.value.code == bd.ERR_SHAPE
