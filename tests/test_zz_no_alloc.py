"""The workspace-free entry point (comfuse_gemm_epilogue_static_scratch).

It serves callers that cannot allocate the workspace of the unfused path themselves -- for example a loop in which
cudaMalloc is not allowed, or a plug-in that has no access to its host framework's allocator -- by keeping the
intermediate GEMM result in a fixed array inside the library.  The tests call it through the C ABI several times in a
row, with different problems so that each call sees the previous call's leftovers in the shared array, check each output
against the ordinary entry point (caller-provided workspace) within the tolerances used by the other parity tests, and
check that the amount of free device memory does not move across the calls.  This file is collected last, so a run that
stops at the first failure has already run every other test.
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


def _call_static(w, T, outs):
    """One call of the workspace-free entry point on workload `w` into the pre-allocated outputs `outs`."""
    flags = (cf.FLAG_POST_RELU if w.scalars.get("relu") else 0) | (0 if w.scalars.get("activation", True) else cf.FLAG_NO_ACTIVATION)
    if w.kind == wl.KIND_BIAS_RES_LAYERNORM:
        cf.gemm_epilogue_static_scratch(T["A"], T["B"], outs["Y"], cf.EPI_BIAS_RES_LAYERNORM, bias=T["bias"],
                                        residual=T["residual"], gamma=T.get("gamma"), beta=T.get("beta"),
                                        alpha=w.scalars["alpha"], eps=w.scalars["eps"], flags=flags)
    elif w.kind == wl.KIND_BIAS_GELU_RES_RMSNORM_MAX:
        cf.gemm_epilogue_static_scratch(T["A"], T["B"], outs["Y"], cf.EPI_BIAS_GELU_RES_RMSNORM_MAX, bias=T.get("bias"),
                                        residual=T.get("residual"), gamma=T["gamma"], alpha=w.scalars["alpha"],
                                        eps=w.scalars["eps"], row_max=outs["row_max"], row_argmax=outs["row_argmax"], flags=flags)
    else:
        cf.gemm_epilogue_static_scratch(T["A"], T["B"], outs["Y"], cf.EPI_SCALE_MASK_SOFTMAX, alpha=w.scalars["alpha"],
                                        mask=cf.MASK_CAUSAL if w.scalars.get("causal") else cf.MASK_NONE,
                                        softcap=w.scalars.get("softcap", 0.0))


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_point_several_times_in_a_row(cuda_device):
    cases = [wl.post_norm(300, 768, 200, seed=41, affine=True),           # first call
             wl.config(0),                                                  # second call: smaller problem, stale bytes behind it
             wl.complex_subgraph(140, 768, 64, seed=42),                    # another op list over the same array
             wl.post_norm(200, 1024, 72, seed=43, affine=True, relu=True),  # descriptor flag: ReLU behind the LayerNorm
             wl.complex_subgraph(100, 512, 96, seed=44, activation=False, residual=False),  # descriptor flag: no activation
             wl.scaled_masked_softmax(3, 512, 512, 64, seed=45, causal=True, softcap=4.0)]  # batched causal softmax, soft-capped
    # every tensor of every case exists before the first call, so that the free-memory readings below see only what the
    # library does
    prepared = []
    for w in cases:
        T = P.dev_tensors(w)
        d = w.dims
        ref = P.run_gpu(w, T, fused=False)                                  # existing entry point, caller workspace
        shape = (d["batch"], d["M"], d["N"]) if "batch" in d else (d["M"], d["N"])
        outs = {"Y": torch.full(shape, float("nan"), dtype=torch.bfloat16, device=cuda_device)}
        if w.kind == wl.KIND_BIAS_GELU_RES_RMSNORM_MAX:
            outs["row_max"] = torch.full((d["M"],), float("nan"), dtype=torch.float32, device=cuda_device)
            outs["row_argmax"] = torch.full((d["M"],), -1, dtype=torch.int32, device=cuda_device)
        prepared.append((w, T, ref, outs))
    torch.cuda.synchronize()
    free_before = None
    for k, (w, T, ref, outs) in enumerate(prepared):
        _call_static(w, T, outs)
        torch.cuda.synchronize()
        assert cf.last_device_status() == cf.OK
        free_now = torch.cuda.mem_get_info()[0]
        if k >= 1:   # the first call may load kernels; from the second call on, nothing may be allocated or freed
            assert free_now == free_before, f"free device memory moved by {free_before - free_now} bytes across call {k}"
        free_before = free_now
    for w, T, ref, outs in prepared:
        got = outs
        assert torch.isfinite(got["Y"].float()).all()
        diff = (got["Y"].float() - ref["Y"].float()).abs()
        if w.kind == wl.KIND_SCALE_MASK_SOFTMAX:
            assert diff.max().item() <= P.TOL_SOFTMAX_MAX, w.name
        else:
            assert diff.max().item() <= P.TOL_NORM_MAX and diff.mean().item() <= P.TOL_NORM_MEAN, w.name
        if "row_max" in got:
            assert (got["row_max"] - ref["row_max"]).abs().max().item() <= 3e-2
            assert torch.equal(got["row_argmax"], ref["row_argmax"])
        # and against the oracle, like every other parity test
        P.check_outputs(w, got, P.run_oracle(w), label=f"static scratch {w.name}", rowmax_tol=3e-2, softmax_tol=P.TOL_SOFTMAX_UNFUSED)


@pytest.mark.gpu
def test_static_scratch_rejects_an_oversized_problem_with_real_tensors(cuda_device):
    """The limit once more with device tensors behind the pointers: refused with a clear status, the output untouched, and
    the next call of ordinary size still right."""
    M, N, K = 4352, 2048, 64                                # 17 MiB intermediate > 16 MiB
    assert M * N * 2 > cf.STATIC_SCRATCH_BYTES
    A = torch.randn(M, K, device=cuda_device).bfloat16()
    B = torch.randn(K, N, device=cuda_device).bfloat16()
    Y = torch.full((M, N), 7.0, dtype=torch.bfloat16, device=cuda_device)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    with pytest.raises(cf.ComfuseError) as e:
        cf.gemm_epilogue_static_scratch(A, B, Y, cf.EPI_BIAS_RES_LAYERNORM)
    assert e.value.status == cf.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert (Y == 7.0).all().item()
    assert cf.last_device_status() == cf.OK
    w = wl.config(0)
    T = P.dev_tensors(w)
    Y2 = torch.full((w.dims["M"], w.dims["N"]), float("nan"), dtype=torch.bfloat16, device=cuda_device)
    cf.gemm_epilogue_static_scratch(T["A"], T["B"], Y2, cf.EPI_BIAS_RES_LAYERNORM, bias=T["bias"], residual=T["residual"],
                                    alpha=w.scalars["alpha"], eps=w.scalars["eps"])
    P.check_outputs(w, {"Y": Y2}, P.run_oracle(w), label="static scratch after a refusal")
