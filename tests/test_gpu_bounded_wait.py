"""Failure detection without a GPU fault: a wait that nothing satisfies must expire after its (short) limit, the kernel
must end normally with TIMEOUT recorded in the device status word, and the library must keep working afterwards."""
import pytest
import torch

import paper_2608_03537_b200 as cf
import workloads as wl
from tests import parity as P

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_the_context_stays_usable(cuda_device):
    assert cf.last_device_status() == cf.OK
    expired = cf.selftest_bounded_wait(timeout_ms=20)
    assert expired == 64                                   # one thread timed out, the rest saw the abort flag
    assert cf.last_device_status() == cf.ERR_TIMEOUT       # reported ...
    assert cf.last_device_status() == cf.OK                # ... and cleared by the read
    # the context is intact: a real kernel still runs and matches the oracle
    w = wl.config(0)
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label="after timeout self-test")
    assert cf.last_device_status() == cf.OK


def test_selftest_rejects_long_limits(cuda_device):
    with pytest.raises(cf.ComfuseError) as e:
        cf.selftest_bounded_wait(timeout_ms=5000)
    assert e.value.status == cf.ERR_INVALID_ARG
