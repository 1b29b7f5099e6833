"""GPU: the host-buffer forms of the entry points (per-step tensors in pinned host memory, staged through a caller-provided
device buffer) give bit for bit what the device-pointer forms give, and reject a staging buffer that is too small."""
import numpy as np
import pytest
import torch

import workloads as wl
from tests import parity as P

pytestmark = pytest.mark.gpu


def _pinned(t):
    return t.cpu().pin_memory()


def test_layernorm_host_buffers_match_device_buffers(cuda_device):
    import paper_2608_03537_b200 as cf
    w = wl.post_norm(300, 768, 200, seed=17, affine=True)
    T = P.dev_tensors(w)
    dev = T["A"].device
    ref = P.run_gpu(w, T, fused=True)["Y"]
    hA, hR = _pinned(T["A"]), _pinned(T["residual"])
    hY = torch.empty(300, 768, dtype=torch.bfloat16).pin_memory()
    mask = cf.HOST_A | cf.HOST_RESIDUAL | cf.HOST_Y
    desc = cf.make_gemm_desc(hA, T["B"], hY, cf.EPI_BIAS_RES_LAYERNORM, residual=hR, fused=True)
    staging = torch.empty(cf.host_staging_size(desc, mask), dtype=torch.uint8, device=dev)
    for _ in range(2):
        hY.fill_(7.0)
        cf.gemm_epilogue_host(hA, T["B"], hY, cf.EPI_BIAS_RES_LAYERNORM, staging=staging, host_mask=mask, bias=T["bias"],
                              residual=hR, gamma=T["gamma"], beta=T["beta"], alpha=w.scalars["alpha"], eps=w.scalars["eps"])
        torch.cuda.synchronize()
        assert torch.equal(hY.view(torch.int16), ref.cpu().view(torch.int16))
    # against the oracle as well
    err = np.abs(wl.bf16_to_f64(hY.view(torch.int16).numpy().view(np.uint16)) - P.run_oracle(w)["Y"])
    assert err.max() <= P.TOL_NORM_MAX and err.mean() <= P.TOL_NORM_MEAN


def test_softmax_host_buffers_batched(cuda_device):
    import paper_2608_03537_b200 as cf
    w = wl.scaled_masked_softmax(3, 256, 256, 64, seed=5, causal=True)
    T = P.dev_tensors(w)
    dev = T["A"].device
    ref = P.run_gpu(w, T, fused=True)["Y"]
    hA, hB = _pinned(T["A"]), _pinned(T["B"])
    hY = torch.empty(3, 256, 256, dtype=torch.bfloat16).pin_memory()
    mask = cf.HOST_A | cf.HOST_B | cf.HOST_Y
    desc = cf.make_gemm_desc(hA, hB, hY, cf.EPI_SCALE_MASK_SOFTMAX, mask=cf.MASK_CAUSAL, fused=True)
    staging = torch.empty(cf.host_staging_size(desc, mask), dtype=torch.uint8, device=dev)
    cf.gemm_epilogue_host(hA, hB, hY, cf.EPI_SCALE_MASK_SOFTMAX, staging=staging, host_mask=mask, alpha=w.scalars["alpha"],
                          mask=cf.MASK_CAUSAL)
    torch.cuda.synchronize()
    assert torch.equal(hY.view(torch.int16), ref.cpu().view(torch.int16))


def test_softmax_host_buffers_with_keys_stored_one_per_row(cuda_device):
    """COMFUSE_FLAG_B_ROW_MAJOR_NK through the host-buffer form: the operand [batch, N, K] is staged with its own extent and
    read in place; same bits as the device-pointer call with the transposed operand."""
    import paper_2608_03537_b200 as cf
    w = wl.scaled_masked_softmax(3, 256, 512, 72, seed=6, causal=False)
    T = P.dev_tensors(w)
    dev = T["A"].device
    ref = P.run_gpu(w, T, fused=True)["Y"]
    hA, hB = _pinned(T["A"]), _pinned(T["B"].transpose(1, 2).contiguous())
    hY = torch.empty(3, 256, 512, dtype=torch.bfloat16).pin_memory()
    mask = cf.HOST_A | cf.HOST_B | cf.HOST_Y
    desc = cf.make_gemm_desc(hA, hB, hY, cf.EPI_SCALE_MASK_SOFTMAX, fused=True, flags=cf.FLAG_B_ROW_MAJOR_NK)
    staging = torch.empty(cf.host_staging_size(desc, mask), dtype=torch.uint8, device=dev)
    cf.gemm_epilogue_host(hA, hB, hY, cf.EPI_SCALE_MASK_SOFTMAX, staging=staging, host_mask=mask, alpha=w.scalars["alpha"],
                          flags=cf.FLAG_B_ROW_MAJOR_NK)
    torch.cuda.synchronize()
    assert torch.equal(hY.view(torch.int16), ref.cpu().view(torch.int16))


def test_b2b_host_buffers_match_device_buffers(cuda_device):
    import paper_2608_03537_b200 as cf
    w = wl.b2b_mlp(M=600, K=128, N1=512, N2=128, seed=8, affine=True)
    T = P.dev_tensors(w)
    dev = T["X"].device
    ref = P.run_gpu(w, T, fused=True)["Y"]
    hX = _pinned(T["X"])
    hO = torch.empty(600, 128, dtype=torch.bfloat16).pin_memory()
    desc = cf.make_b2b_desc(600, 128, 512, 128, w.scalars["eps"], True)
    staging = torch.empty(cf.b2b_host_staging_size(desc), dtype=torch.uint8, device=dev)
    cf.b2b_gemm_host(hX, T["W1"], T["b1"], T["W2"], T["b2"], hO, staging=staging, gamma=T.get("gamma"), beta=T.get("beta"),
                     eps=w.scalars["eps"])
    torch.cuda.synchronize()
    assert torch.equal(hO.view(torch.int16), ref.cpu().view(torch.int16))


def test_host_form_rejects_small_staging(cuda_device):
    import paper_2608_03537_b200 as cf
    w = wl.post_norm(256, 256, 64, seed=2, affine=False)
    T = P.dev_tensors(w)
    hA = _pinned(T["A"])
    hY = torch.empty(256, 256, dtype=torch.bfloat16).pin_memory()
    staging = torch.empty(1024, dtype=torch.uint8, device=T["B"].device)
    with pytest.raises(cf.ComfuseError) as ei:
        cf.gemm_epilogue_host(hA, T["B"], hY, cf.EPI_BIAS_RES_LAYERNORM, staging=staging, host_mask=cf.HOST_A | cf.HOST_Y,
                              bias=T["bias"], residual=T["residual"])
    assert ei.value.status == cf.ERR_WORKSPACE


@pytest.mark.parametrize("case", ["layernorm_fused", "layernorm_unfused", "rmsnorm_max", "layernorm_wide_rows"])
def test_pipelined_host_form_over_row_chunks_matches_device_form(case, cuda_device):
    """Enough rows for the host form to run as a pipeline of row ranges (copy-in, compute and copy-out streams): results,
    row outputs included, are bit for bit those of the device-pointer call; repeated calls on one stream reuse the staging
    buffer safely; an event recorded after the call on the caller's stream covers the whole call."""
    import paper_2608_03537_b200 as cf
    if case == "rmsnorm_max":
        w = wl.complex_subgraph(2100, 1024, 2048, seed=23)     # 8.6 MB of A + 4.3 MB of residual: three row ranges
        kind = cf.EPI_BIAS_GELU_RES_RMSNORM_MAX
    elif case == "layernorm_wide_rows":
        w = wl.post_norm(1100, 8192, 72, seed=24, affine=True)   # 18 MB of residual: four row ranges
        kind = cf.EPI_BIAS_RES_LAYERNORM
    else:
        w = wl.post_norm(4200, 768, 1024, seed=22, affine=True)  # 8.6 MB of A + 6.5 MB of residual: three row ranges
        kind = cf.EPI_BIAS_RES_LAYERNORM
    fused = case != "layernorm_unfused"
    M, N = w.dims["M"], w.dims["N"]
    T = P.dev_tensors(w)
    dev = T["A"].device
    ref = P.run_gpu(w, T, fused=fused)
    hA, hR = _pinned(T["A"]), _pinned(T["residual"])
    hY = torch.empty(M, N, dtype=torch.bfloat16).pin_memory()
    mask = cf.HOST_A | cf.HOST_RESIDUAL | cf.HOST_Y
    desc = cf.make_gemm_desc(hA, T["B"], hY, kind, residual=hR, fused=fused)
    staging = torch.empty(cf.host_staging_size(desc, mask), dtype=torch.uint8, device=dev)
    ws = torch.empty(max(16, cf.workspace_size(desc)), dtype=torch.uint8, device=dev)
    kw = dict(staging=staging, host_mask=mask, bias=T["bias"], residual=hR, gamma=T["gamma"], alpha=w.scalars["alpha"],
              eps=w.scalars["eps"], fused=fused, workspace=ws)
    if kind == cf.EPI_BIAS_RES_LAYERNORM:
        kw["beta"] = T["beta"]
    else:
        kw["row_max"] = torch.zeros(M, dtype=torch.float32, device=dev)
        kw["row_argmax"] = torch.zeros(M, dtype=torch.int32, device=dev)
    done = torch.cuda.Event()
    for it in range(3):
        hY.fill_(7.0)
        cf.gemm_epilogue_host(hA, T["B"], hY, kind, **kw)
        # an event recorded behind the call on the caller's stream covers the helper streams' copies as well
        done.record()
        done.synchronize()
        assert torch.equal(hY.view(torch.int16), ref["Y"].cpu().view(torch.int16)), (case, it)
    if "row_max" in kw:
        assert torch.equal(kw["row_max"], ref["row_max"]) and torch.equal(kw["row_argmax"], ref["row_argmax"])


def test_pipelined_b2b_host_forms_match_device_forms(cuda_device):
    """Large enough for the B2B host forms to run as pipelines (row ranges for the MLP kind, batch ranges for the attention
    kind): bit for bit the device-pointer results, and within tolerance of the oracle on sampled rows."""
    import paper_2608_03537_b200 as cf
    # MLP kind: 40000 rows, X = 10 MB -> two row ranges
    w = wl.b2b_mlp(M=40000, K=128, N1=512, N2=128, seed=31, affine=True)
    T = P.dev_tensors(w)
    dev = T["X"].device
    ref = P.run_gpu(w, T, fused=True)["Y"]
    hX = _pinned(T["X"])
    hO = torch.empty(40000, 128, dtype=torch.bfloat16).pin_memory()
    desc = cf.make_b2b_desc(40000, 128, 512, 128, w.scalars["eps"], True)
    staging = torch.empty(cf.b2b_host_staging_size(desc), dtype=torch.uint8, device=dev)
    for _ in range(2):
        hO.fill_(3.0)
        cf.b2b_gemm_host(hX, T["W1"], T["b1"], T["W2"], T["b2"], hO, staging=staging, gamma=T.get("gamma"), beta=T.get("beta"),
                         eps=w.scalars["eps"])
        torch.cuda.synchronize()
        assert torch.equal(hO.view(torch.int16), ref.cpu().view(torch.int16))
    rows = wl.sample_rows(40000, 64)
    P.check_outputs(w, {"Y": ref}, P.run_oracle(w, rows=rows), rows=rows, label="b2b host pipelined")
    # attention kind: 20 batches, Q = 10.5 MB -> batch ranges
    w = wl.target_attention(20, 2048, 256, 128, seed=32)
    T = P.dev_tensors(w)
    ref = P.run_gpu(w, T, fused=True)["Y"]
    hQ, hK, hV = _pinned(T["X"]), _pinned(T["W1"]), _pinned(T["W2"])
    hO = torch.empty(20, 2048, 128, dtype=torch.bfloat16).pin_memory()
    desc = cf.make_b2b_desc(2048, 128, 256, 128, 0.0, True, cf.B2B_SOFTMAX_ATTENTION, 20, w.scalars["alpha"])
    staging = torch.empty(cf.b2b_host_staging_size(desc), dtype=torch.uint8, device=dev)
    for _ in range(2):
        hO.fill_(3.0)
        cf.b2b_attention_host(hQ, hK, hV, hO, staging=staging, alpha=w.scalars["alpha"])
        torch.cuda.synchronize()
        assert torch.equal(hO.view(torch.int16), ref.cpu().view(torch.int16))


def test_b2b_host_forms_with_partial_last_chunks(cuda_device):
    """The host-buffer forms with a hidden width / source length that ends in a partial chunk (zero-filled loads on the
    device side), large enough to run as pipelines: bit for bit the device-pointer results, oracle parity on sampled rows."""
    import paper_2608_03537_b200 as cf
    w = wl.b2b_mlp(M=40000, K=128, N1=200, N2=128, seed=41, affine=True)
    T = P.dev_tensors(w)
    dev = T["X"].device
    ref = P.run_gpu(w, T, fused=True)["Y"]
    hX = _pinned(T["X"])
    hO = torch.empty(40000, 128, dtype=torch.bfloat16).pin_memory()
    desc = cf.make_b2b_desc(40000, 128, 200, 128, w.scalars["eps"], True)
    staging = torch.empty(cf.b2b_host_staging_size(desc), dtype=torch.uint8, device=dev)
    hO.fill_(3.0)
    cf.b2b_gemm_host(hX, T["W1"], T["b1"], T["W2"], T["b2"], hO, staging=staging, gamma=T.get("gamma"), beta=T.get("beta"),
                     eps=w.scalars["eps"])
    torch.cuda.synchronize()
    assert torch.equal(hO.view(torch.int16), ref.cpu().view(torch.int16))
    rows = wl.sample_rows(40000, 64)
    P.check_outputs(w, {"Y": ref}, P.run_oracle(w, rows=rows), rows=rows, label="b2b host, N1 = 200")
    for keys_row_major in (False, True):
        w = wl.target_attention(20, 2048, 200, 128, seed=42)
        T = P.dev_tensors(w)
        Kd = T["W1"].transpose(1, 2).contiguous() if keys_row_major else T["W1"]
        ref = torch.empty(20, 2048, 128, dtype=torch.bfloat16, device=dev)
        cf.b2b_attention(T["X"], Kd, T["W2"], ref, alpha=w.scalars["alpha"], keys_row_major=keys_row_major)
        hQ, hK, hV = _pinned(T["X"]), _pinned(Kd), _pinned(T["W2"])
        hO = torch.empty(20, 2048, 128, dtype=torch.bfloat16).pin_memory()
        desc = cf.make_b2b_desc(2048, 128, 200, 128, 0.0, True, cf.B2B_SOFTMAX_ATTENTION, 20, w.scalars["alpha"],
                                cf.B2B_FLAG_KEYS_ROW_MAJOR if keys_row_major else 0)
        staging = torch.empty(cf.b2b_host_staging_size(desc), dtype=torch.uint8, device=dev)
        hO.fill_(3.0)
        cf.b2b_attention_host(hQ, hK, hV, hO, staging=staging, alpha=w.scalars["alpha"], keys_row_major=keys_row_major)
        torch.cuda.synchronize()
        assert torch.equal(hO.view(torch.int16), ref.cpu().view(torch.int16))
        rows = wl.sample_rows(2048, 32)
        want = P.run_oracle(w, rows=rows)
        P.check_outputs(w, {"Y": ref}, want, rows=rows, label=f"attention host, 200 source positions, keys_row_major={keys_row_major}")
