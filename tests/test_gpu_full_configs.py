"""GPU parity at the full sizes of the named configurations, in the launch configuration the benchmark times.
Every output element is compared with the fp64 oracle (the softmax configuration one batch at a time, to bound the
oracle's memory); properties that need no oracle are checked over the whole output as well."""
import numpy as np
import pytest
import torch

import workloads as wl
from tests import parity as P

pytestmark = pytest.mark.gpu


def _finite_everywhere(Y):
    assert torch.isfinite(Y.float()).all().item(), "some output elements were never written (NaN poison left)"


def _unfused_bound(w, got, ref, label):
    """The in-library unfused baseline rounds the GEMM result to bf16 before the subgraph, i.e. twice in all: an occasional
    output of magnitude 4 .. 8 lands just above 3e-2.  It is held to 4e-2, with the number of elements above 3e-2 printed
    and bounded."""
    over = int((np.abs(P.to_f64(got["Y"]) - ref["Y"]) > P.TOL_NORM_MAX).sum())
    print(f"{label}: {over} of {ref['Y'].size} elements above 3e-2")
    assert over <= ref["Y"].size // 100_000
    return 4e-2


@pytest.mark.parametrize("fused", [True, False])
def test_config_bert_ffn_out_post_norm(fused, cuda_device):
    w = wl.config(1)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    _finite_everywhere(got["Y"])
    ref = P.run_oracle(w)
    res = P.check_outputs(w, got, ref, label=f"c2 fused={fused}",
                          norm_tol=P.TOL_NORM_MAX if fused else _unfused_bound(w, got, ref, "c2 unfused"))
    # property over every row: undoing the affine step leaves mean ~0 and variance ~1
    g = torch.from_numpy(wl.bf16_bits_to_f32(w.tensors["gamma"])).to(got["Y"].device)
    b = torch.from_numpy(wl.bf16_bits_to_f32(w.tensors["beta"])).to(got["Y"].device)
    Yn = (got["Y"].float() - b) / g
    assert Yn.mean(-1).abs().max().item() < 2e-2
    assert (Yn.var(-1, unbiased=False) - 1).abs().max().item() < 3e-2
    print("c2", fused, res)


@pytest.mark.parametrize("fused", [True, False])
def test_config_complex_subgraph(fused, cuda_device):
    w = wl.config(2)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    _finite_everywhere(got["Y"])
    ref = P.run_oracle(w)
    res = P.check_outputs(w, got, ref, label=f"c3 fused={fused}", rowmax_tol=5e-3 if fused else 3e-2,
                          norm_tol=P.TOL_NORM_MAX if fused else _unfused_bound(w, got, ref, "c3 unfused"))
    # property over every row: the stored row attains its maximum at the reported column, and bf16(row_max) is it
    Y = got["Y"].float()
    ymax = Y.max(-1).values
    picked = Y.gather(-1, got["row_argmax"].long()[:, None])[:, 0]
    assert torch.equal(picked, ymax)
    assert torch.equal(got["row_max"].to(torch.bfloat16).float(), ymax)
    print("c3", fused, res)


@pytest.mark.parametrize("fused", [True, False])
def test_config_scaled_causal_softmax(fused, cuda_device):
    w = wl.config(3)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    _finite_everywhere(got["Y"])
    res = {"max_abs": 0.0, "mean_abs": 0.0}
    for b in range(w.dims["batch"]):   # every batch, one at a time (the oracle's fp64 scores of one batch are 34 MB)
        r = P.check_outputs(w, got, P.run_oracle(w, batches=[b]), batches=[b], label=f"c4 fused={fused} batch {b}",
                            softmax_tol=P.TOL_SOFTMAX_MAX if fused else P.TOL_SOFTMAX_UNFUSED)
        res = {"max_abs": max(res["max_abs"], r["max_abs"]), "mean_abs": res["mean_abs"] + r["mean_abs"] / w.dims["batch"]}
    # properties over every row of every batch: strictly upper triangle exactly zero, rows sum to ~1, P[.,0,0] = 1
    Y = got["Y"]
    M = w.dims["M"]
    upper = torch.triu(torch.ones(M, M, dtype=torch.bool, device=Y.device), diagonal=1)
    assert (Y[:, upper] == 0).all().item()
    assert (Y.float().sum(-1) - 1).abs().max().item() < 2e-2
    assert (Y[:, 0, 0] == 1).all().item()
    print("c4", fused, res)


def test_config_tiny_post_norm_full(cuda_device):
    w = wl.config(0)
    for fused in (True, False):
        got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
        print("c1", fused, P.check_outputs(w, got, P.run_oracle(w), label=f"c1 fused={fused}"))


@pytest.mark.parametrize("cfg", [1, 3, 4])
def test_cuda_graph_replay_matches_direct_launches(cfg, cuda_device):
    """The benchmark replays its steps from a CUDA graph (one launch per buffer set, launched with programmatic stream
    serialization so consecutive launches overlap at their edges).  The replayed launches must write, bit for bit, what a
    direct launch writes; the direct launch is what the tests above compare with the oracle."""
    import paper_2608_03537_b200 as cf
    w = wl.config(cfg)
    T = P.dev_tensors(w)
    ref = P.run_gpu(w, T, fused=True)["Y"]
    outs = [torch.full_like(ref, float("nan")) for _ in range(3)]

    def launch(Y):
        if w.kind == wl.KIND_B2B_MLP_LAYERNORM:
            cf.b2b_gemm(T["X"], T["W1"], T["b1"], T["W2"], T["b2"], Y, gamma=T.get("gamma"), beta=T.get("beta"), eps=w.scalars["eps"])
        elif w.kind == wl.KIND_BIAS_RES_LAYERNORM:
            cf.gemm_epilogue(T["A"], T["B"], Y, cf.EPI_BIAS_RES_LAYERNORM, bias=T["bias"], residual=T["residual"], gamma=T["gamma"],
                             beta=T["beta"], alpha=w.scalars["alpha"], eps=w.scalars["eps"])
        else:
            cf.gemm_epilogue(T["A"], T["B"], Y, cf.EPI_SCALE_MASK_SOFTMAX, alpha=w.scalars["alpha"], mask=cf.MASK_CAUSAL)

    launch(outs[0])                      # first use outside the capture (configures the kernel)
    torch.cuda.synchronize()
    outs[0].fill_(float("nan"))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for Y in outs:
            launch(Y)
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    for Y in outs:
        assert torch.equal(Y.view(torch.int16), ref.view(torch.int16))
    assert cf.last_device_status() == cf.OK
