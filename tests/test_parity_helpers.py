"""The parity helpers themselves (no GPU): the canary pads around outputs catch a write on either side."""
import pytest
import torch

from tests import parity as P


def test_canary_pads_catch_writes_outside_the_tensor():
    t = P.guarded((3, 40), torch.bfloat16, float("nan"), "cpu")
    ws = P.guarded((100,), torch.uint8, 0xEE, "cpu")
    t._guard_ws = ws
    assert t.shape == (3, 40) and t.is_contiguous() and t.data_ptr() % 16 == 0
    P.check_canaries({"Y": t}, "untouched")
    t.fill_(1.0)                                   # writing the tensor itself is fine
    ws.fill_(7)
    P.check_canaries({"Y": t}, "inside")
    flat, n = t._guard
    flat[P.GUARD_BYTES + n + 3] = 0                # one byte behind the tensor
    with pytest.raises(AssertionError, match="behind output Y"):
        P.check_canaries({"Y": t}, "behind")
    flat[P.GUARD_BYTES + n + 3] = P.CANARY
    flat[P.GUARD_BYTES - 1] = 0                    # one byte in front of it
    with pytest.raises(AssertionError, match="in front of output Y"):
        P.check_canaries({"Y": t}, "front")
    flat[P.GUARD_BYTES - 1] = P.CANARY
    wflat, wn = ws._guard
    wflat[P.GUARD_BYTES + wn] = 1                  # first byte behind the workspace
    with pytest.raises(AssertionError, match="workspace"):
        P.check_canaries({"Y": t}, "workspace")
