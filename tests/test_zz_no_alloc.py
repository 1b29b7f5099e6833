"""The workspace-free entry point (comfuse_gemm_epilogue_static_scratch).

It serves callers that cannot allocate the workspace of the unfused path themselves -- for example code inside a
stream capture, or a plug-in that has no access to its host framework's allocator -- by keeping the intermediate
GEMM result in a fixed array inside the library.  The test calls it through the C ABI twice in a row, with different
problems so that the second call sees the first call's leftovers in the shared array, and checks each output against
the ordinary entry point (caller-provided workspace) within the tolerances used by the other parity tests.  This file
is collected last, so a run that stops at the first failure has already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2608_03537_b200 as cf
import workloads as wl
from tests import parity as P


def test_static_scratch_rejects_problems_beyond_its_limit():
    """Host-only: a problem whose intermediate does not fit the fixed array is refused before any CUDA call."""
    d = cf.GemmDesc()
    d.batch, d.M, d.N, d.K = 1, 8192, 4096, 64            # 64 MiB intermediate > 16 MiB
    d.lda, d.ldb, d.ldr, d.ldy = 64, 4096, 4096, 4096
    d.kind, d.mask, d.alpha, d.eps, d.fused, d.reserved = cf.EPI_BIAS_RES_LAYERNORM, cf.MASK_NONE, 1.0, 1e-5, 0, 0
    assert d.batch * d.M * d.N * 2 > cf.STATIC_SCRATCH_BYTES
    fake = ctypes.c_void_p(256)   # never dereferenced: the size check comes first
    st = cf.lib().comfuse_gemm_epilogue_static_scratch(ctypes.byref(d), fake, fake, fake, None, None)
    assert st == cf.ERR_WORKSPACE
    assert cf.lib().comfuse_gemm_epilogue_static_scratch(None, fake, fake, fake, None, None) == cf.ERR_INVALID_ARG


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_point_twice_in_a_row(cuda_device):
    cases = [wl.post_norm(300, 768, 200, seed=41, affine=True),   # first call
             wl.config(0),                                          # second call: smaller problem, stale bytes behind it
             wl.complex_subgraph(140, 768, 64, seed=42)]            # third: another op list over the same array
    for w in cases:
        T = P.dev_tensors(w)
        d = w.dims
        ref = P.run_gpu(w, T, fused=False)                          # existing entry point, caller workspace
        Y = torch.full((d["M"], d["N"]), float("nan"), dtype=torch.bfloat16, device=cuda_device)
        if w.kind == wl.KIND_BIAS_RES_LAYERNORM:
            cf.gemm_epilogue_static_scratch(T["A"], T["B"], Y, cf.EPI_BIAS_RES_LAYERNORM, bias=T["bias"],
                                            residual=T["residual"], gamma=T.get("gamma"), beta=T.get("beta"),
                                            alpha=w.scalars["alpha"], eps=w.scalars["eps"])
            got = {"Y": Y}
        else:
            rm = torch.full((d["M"],), float("nan"), dtype=torch.float32, device=cuda_device)
            am = torch.full((d["M"],), -1, dtype=torch.int32, device=cuda_device)
            cf.gemm_epilogue_static_scratch(T["A"], T["B"], Y, cf.EPI_BIAS_GELU_RES_RMSNORM_MAX, bias=T["bias"],
                                            residual=T["residual"], gamma=T["gamma"], alpha=w.scalars["alpha"],
                                            eps=w.scalars["eps"], row_max=rm, row_argmax=am)
            got = {"Y": Y, "row_max": rm, "row_argmax": am}
        assert cf.last_device_status() == cf.OK
        diff = (got["Y"].float() - ref["Y"].float()).abs()
        assert torch.isfinite(got["Y"].float()).all()
        assert diff.max().item() <= P.TOL_NORM_MAX and diff.mean().item() <= P.TOL_NORM_MEAN, w.name
        if "row_max" in got:
            assert (got["row_max"] - ref["row_max"]).abs().max().item() <= 3e-2
            assert torch.equal(got["row_argmax"], ref["row_argmax"])
        # and against the oracle, like every other parity test
        P.check_outputs(w, got, P.run_oracle(w), label=f"static scratch {w.name}", rowmax_tol=3e-2)
