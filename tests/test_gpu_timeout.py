"""The give-up path of the bounded device waits, run once on purpose.  Every wait inside the
tensor-core kernels is bounded: when it runs out it latches TORQ_ERR_TIMEOUT with the id of the wait
site, raises the CTA's abort flag, the other roles leave their loops, the kernel drains and returns.
A healthy run never gets there, so torq_selftest_wait_timeout makes a wait run out harmlessly (a
barrier nothing arrives on, a limit of a millisecond): nothing faults, traps or hangs."""
import pytest
import torch

from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu

TORQ_ERR_TIMEOUT, SITE_SELFTEST = 6, 7


def test_a_wait_that_runs_out_latches_the_error_word_and_the_library_stays_usable():
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    res = torq.torq_selftest_wait_timeout(1_000_000)            # 1 ms
    torch.cuda.synchronize()
    gave_up, left_by_flag, waited_ns = (int(v) for v in res.cpu())
    assert gave_up == 1 and left_by_flag == 1
    assert 500_000 <= waited_ns <= 500_000_000                    # about the limit, far below the 2 s of its own
    err = torq.torq_last_device_error()
    assert err & 0xFF == TORQ_ERR_TIMEOUT and (err >> 8) & 0xFF == SITE_SELFTEST
    assert torq.torq_last_device_error() == 0                     # reading clears it
    # the next ordinary call runs and reports nothing
    z = torch.randn((64, 256), device="cuda")
    codes, scales = torq.torq_quantize_mxfp4(z)
    X = torch.randn((256, 256), device="cuda").to(torch.bfloat16)
    R = torch.eye(256, device="cuda").to(torch.bfloat16)
    c2, s2 = torq.torq_rotate_quantize(X, R, None)
    c3, s3 = torq.torq_rotate_quantize(X, None, None)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    assert torch.equal(c2, c3) and torch.equal(s2, s3)            # identity rotation = quantize-only


def test_argument_errors_launch_nothing():
    before = torq.torq_launch_count()
    L = torq.lib()
    out = torch.zeros(4, dtype=torch.int64, device="cuda")
    import ctypes
    assert L.torq_selftest_wait_timeout(10, ctypes.c_void_p(out.data_ptr()), None) == 2
    assert L.torq_selftest_wait_timeout(1_000_000, None, None) == 1
    assert torq.torq_launch_count() == before
