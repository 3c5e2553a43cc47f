"""A bounded device-side wait that runs out.  Every tensor-core kernel of the library waits on mbarriers through
one bounded wait; here that wait is made to expire in the only safe way: a one-CTA self-test kernel waits (for a
millisecond) on a barrier nobody arrives on, must report Q8_ERR_TIMEOUT through the status word and return, and
the context must be as usable afterwards as before.  No GEMM is broken for this and nothing waits without a limit."""
import time

import numpy as np
import pytest
import torch

from paper_1910_06188_b200 import binding as q8
from paper_1910_06188_b200 import synth
from tests.gpu_util import check_linear

pytestmark = pytest.mark.gpu


def test_bounded_wait_expires_flags_timeout_and_returns():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    report = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    t0 = time.perf_counter()
    q8.q8_selftest_wait_timeout(1_000_000, status, report)          # 1 ms
    code, bits = q8.q8_poll_status(status)                           # synchronises: the kernel has exited
    dt = time.perf_counter() - t0
    assert code == q8.Q8_ERR_TIMEOUT and bits == 1 << q8.Q8_ERR_TIMEOUT
    assert q8.status_string(code) == "bounded device wait expired"
    assert report.tolist() == [1, 1]        # the wait returned "failed" and the CTA-wide abort flag was raised
    assert dt < 5.0                          # it gave up after its limit, not after seconds
    assert q8.q8_poll_status(status) == (q8.Q8_OK, 0)               # polling cleared the word
    # a longer limit is honoured too (20 ms), measured on the device
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    q8.q8_selftest_wait_timeout(20_000_000, status)
    e1.record()
    assert q8.q8_poll_status(status)[0] == q8.Q8_ERR_TIMEOUT
    assert 19.0 <= e0.elapsed_time(e1) < 500.0


def test_library_is_fully_usable_after_a_timeout():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    q8.q8_selftest_wait_timeout(1_000_000, status)
    assert q8.q8_poll_status(status)[0] == q8.Q8_ERR_TIMEOUT
    X = synth.activation(300, 272, seed=4100)
    W = synth.weight(200, 272, seed=4101)
    b = synth.bias(200, seed=4102)
    info = check_linear(X, W, b, act=1)                              # bit-exact against the oracle, status word clean
    assert info["gemm_kernel"] == 1


def test_selftest_argument_checks():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for bad in (0, 999, 100_000_001):
        with pytest.raises(q8.Q8Error) as e:
            q8.q8_selftest_wait_timeout(bad, status)
        assert e.value.status == q8.Q8_ERR_ARG
    with pytest.raises(q8.Q8Error) as e:
        q8.q8_selftest_wait_timeout(1_000_000, None)
    assert e.value.status == q8.Q8_ERR_NULL
    assert status.item() == 0
