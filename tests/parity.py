"""Shared helpers for the GPU parity tests: move a seeded workload to the device, run it through the C ABI
binding, evaluate the fp64 oracle on the same bytes (all rows, or a sample of rows), and compare.

Tolerances (stated by the benchmark definition, checked here literally):
  normalised bf16 outputs (LayerNorm / RMSNorm):  max-abs <= 3e-2, mean-abs <= 3e-3
  softmax probabilities:                           max-abs <= 2e-3
The bf16 output rounding alone accounts for up to 1.56e-2 of the first (|y| in [4, 8)) and 1.95e-3 of the last
(p in [0.5, 1)), so both need round-to-nearest-even at the store.
"""
from __future__ import annotations

import numpy as np
import torch

import paper_2608_03537_b200 as cf
import workloads as wl
from oracle import comfuse_oracle as orc

TOL_NORM_MAX = 3e-2
TOL_NORM_MEAN = 3e-3
TOL_SOFTMAX_MAX = 2e-3
TOL_SOFTMAX_UNFUSED = 1e-2   # in-library unfused baseline only: it exponentiates bf16-rounded scores


def to_dev(bits: np.ndarray, device="cuda:0") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


def dev_tensors(w: wl.Workload, device="cuda:0") -> dict:
    return {k: to_dev(v, device) for k, v in w.tensors.items()}


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def f64(w: wl.Workload, name: str, rows=None):
    t = w.tensors.get(name)
    if t is None:
        return None
    if rows is not None:
        t = t[..., rows, :]
    return wl.bf16_to_f64(t)


# --------------------------------------------------------------------------------------------- GPU side
# Canary pads: every output (and the workspace) of prepare_gpu / run_gpu sits inside a larger allocation whose margins hold a
# fixed bit pattern; check_outputs (or check_canaries) verifies that no launch wrote outside the tensor it was given.
GUARD_BYTES = 4096
CANARY = 0x5A


def guarded(shape, dtype, fill, device):
    """A contiguous tensor of `shape` with GUARD_BYTES of canary before and after it in the same allocation."""
    n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
    pad = (-n) % 256
    flat = torch.full((GUARD_BYTES + n + pad + GUARD_BYTES,), CANARY, dtype=torch.uint8, device=device)
    t = flat[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(*shape)
    t.fill_(fill)
    t._guard = (flat, n)
    return t


def check_canaries(tensors, label=""):
    """Every guarded tensor among `tensors`: the bytes around it still hold the canary."""
    for name, t in (tensors.items() if isinstance(tensors, dict) else enumerate(tensors)):
        for what, u in ((f"output {name}", t), (f"the workspace of {name}", getattr(t, "_guard_ws", None))):
            g = getattr(u, "_guard", None) if u is not None else None
            if g is None:
                continue
            flat, n = g
            lead = flat[:GUARD_BYTES]
            tail = flat[GUARD_BYTES + n:]
            assert bool((lead == CANARY).all().item()), f"{label}: bytes in front of {what} were overwritten"
            assert bool((tail == CANARY).all().item()), f"{label}: bytes behind {what} were overwritten"


def _guarded_workspace(nbytes, device):
    ws = guarded((max(int(nbytes), 16),), torch.uint8, 0xEE, device)
    return ws

def prepare_gpu(w: wl.Workload, T: dict, fused: bool = True, poison: bool = True):
    """Allocate the outputs and the workspace of one workload once.  Returns (outputs on device, launch): launch()
    enqueues one call of the library on the current stream and nothing else, so that calls can be queued back to back."""
    dev = T[next(iter(T))].device
    d = w.dims
    fill = float("nan") if poison else 0.0
    if w.kind == wl.KIND_B2B_SOFTMAX_ATTENTION:
        O = guarded((d["batch"], d["M"], d["N2"]), torch.bfloat16, fill, dev)
        desc = cf.make_b2b_desc(d["M"], d["K"], d["N1"], d["N2"], 0.0, fused, cf.B2B_SOFTMAX_ATTENTION, d["batch"], w.scalars["alpha"])
        ws = _guarded_workspace(cf.b2b_workspace_size(desc), dev)
        O._guard_ws = ws
        return {"Y": O}, lambda: cf.b2b_attention(T["X"], T["W1"], T["W2"], O, alpha=w.scalars["alpha"], fused=fused, workspace=ws)
    if w.kind == wl.KIND_B2B_MLP_RELU:
        O = guarded((d["M"], d["N2"]), torch.bfloat16, fill, dev)
        desc = cf.make_b2b_desc(d["M"], d["K"], d["N1"], d["N2"], 0.0, fused, cf.B2B_MLP_RELU)
        ws = _guarded_workspace(cf.b2b_workspace_size(desc), dev)
        O._guard_ws = ws
        return {"Y": O}, lambda: cf.b2b_mlp_relu(T["X"], T["W1"], T.get("b1"), T["W2"], T.get("b2"), O, fused=fused, workspace=ws)
    if w.kind == wl.KIND_B2B_MLP_LAYERNORM:
        O = guarded((d["M"], d["N2"]), torch.bfloat16, fill, dev)
        desc = cf.make_b2b_desc(d["M"], d["K"], d["N1"], d["N2"], w.scalars["eps"], fused)
        ws = _guarded_workspace(cf.b2b_workspace_size(desc), dev)
        O._guard_ws = ws
        return {"Y": O}, lambda: cf.b2b_gemm(T["X"], T["W1"], T["b1"], T["W2"], T["b2"], O, gamma=T.get("gamma"), beta=T.get("beta"),
                                             eps=w.scalars["eps"], fused=fused, workspace=ws)
    shape = (d["batch"], d["M"], d["N"]) if "batch" in d else (d["M"], d["N"])
    Y = guarded(shape, torch.bfloat16, fill, dev)
    out = {"Y": Y}
    kw = {}
    if w.kind == wl.KIND_BIAS_RES_LAYERNORM:
        kind = cf.EPI_BIAS_RES_LAYERNORM
        kw = dict(bias=T.get("bias"), residual=T.get("residual"), gamma=T.get("gamma"), beta=T.get("beta"),
                  alpha=w.scalars["alpha"], eps=w.scalars["eps"])
    elif w.kind == wl.KIND_BIAS_GELU_RES_RMSNORM_MAX:
        kind = cf.EPI_BIAS_GELU_RES_RMSNORM_MAX
        out["row_max"] = guarded(shape[:-1], torch.float32, fill, dev)
        out["row_argmax"] = guarded(shape[:-1], torch.int32, -1, dev)
        kw = dict(bias=T.get("bias"), residual=T.get("residual"), gamma=T.get("gamma"), alpha=w.scalars["alpha"],
                  eps=w.scalars["eps"], row_max=out["row_max"], row_argmax=out["row_argmax"])
    else:
        kind = cf.EPI_SCALE_MASK_SOFTMAX
        kw = dict(alpha=w.scalars["alpha"], mask=cf.MASK_CAUSAL if w.scalars.get("causal") else cf.MASK_NONE)
        if "mask" in T:
            kw.update(mask=cf.MASK_ADDITIVE, mask_tensor=T["mask"])
    flags = (cf.FLAG_POST_RELU if w.scalars.get("relu") else 0) | (0 if w.scalars.get("activation", True) else cf.FLAG_NO_ACTIVATION)
    kw.update(flags=flags, softcap=w.scalars.get("softcap", 0.0))
    desc = cf.make_gemm_desc(T["A"], T["B"], Y, kind, residual=kw.get("residual"), alpha=kw.get("alpha", 1.0),
                             eps=kw.get("eps", 1e-5), mask=kw.get("mask", cf.MASK_NONE), fused=fused, flags=flags,
                             softcap=kw["softcap"])
    ws = _guarded_workspace(cf.workspace_size(desc), dev)
    Y._guard_ws = ws
    return out, lambda: cf.gemm_epilogue(T["A"], T["B"], Y, kind, fused=fused, workspace=ws, **kw)


def run_gpu(w: wl.Workload, T: dict, fused: bool = True, poison: bool = True):
    """Run one workload through the library.  Returns dict of output tensors (on device)."""
    out, launch = prepare_gpu(w, T, fused, poison)
    launch()
    return out


# --------------------------------------------------------------------------------------------- oracle side
def run_oracle(w: wl.Workload, rows=None, batches=None):
    """fp64 oracle on all rows, or on `rows` (indices into M); for batched workloads on `batches`."""
    d = w.dims
    if w.kind == wl.KIND_B2B_SOFTMAX_ATTENTION:
        bsel = list(range(d["batch"])) if batches is None else list(batches)
        Q = w.tensors["X"][bsel]
        if rows is not None:
            Q = Q[:, rows, :]
        return {"Y": orc.b2b_softmax_attention(wl.bf16_to_f64(Q), wl.bf16_to_f64(w.tensors["W1"][bsel]),
                                               wl.bf16_to_f64(w.tensors["W2"][bsel]), w.scalars["alpha"])}
    if w.kind == wl.KIND_B2B_MLP_RELU:
        return {"Y": orc.b2b_mlp_relu(f64(w, "X", rows), f64(w, "W1"), f64(w, "b1"), f64(w, "W2"), f64(w, "b2"))}
    if w.kind == wl.KIND_B2B_MLP_LAYERNORM:
        Y = orc.b2b_mlp_layernorm(f64(w, "X", rows), f64(w, "W1"), f64(w, "b1"), f64(w, "W2"), f64(w, "b2"),
                                  f64(w, "gamma"), f64(w, "beta"), w.scalars["eps"])
        return {"Y": Y}
    if w.kind == wl.KIND_BIAS_RES_LAYERNORM:
        Y = orc.bias_res_layernorm(f64(w, "A", rows), f64(w, "B"), f64(w, "bias"), f64(w, "residual", rows),
                                   f64(w, "gamma"), f64(w, "beta"), w.scalars["alpha"], w.scalars["eps"],
                                   relu=w.scalars.get("relu", False))
        return {"Y": Y}
    if w.kind == wl.KIND_BIAS_GELU_RES_RMSNORM_MAX:
        Y, mx, am = orc.bias_gelu_res_rmsnorm_max(f64(w, "A", rows), f64(w, "B"), f64(w, "bias"), f64(w, "residual", rows),
                                                  f64(w, "gamma"), w.scalars["alpha"], w.scalars["eps"],
                                                  activation=w.scalars.get("activation", True))
        return {"Y": Y, "row_max": mx, "row_argmax": am}
    # softmax
    bsel = list(range(d["batch"])) if batches is None else list(batches)
    A = w.tensors["A"][bsel]
    B = w.tensors["B"][bsel]
    if rows is not None:
        A = A[:, rows, :]
    mask = None
    if w.scalars.get("causal"):
        mask = orc.causal_mask(d["M"], d["N"], rows=rows)
    if "mask" in w.tensors:
        m = wl.bf16_to_f64(w.tensors["mask"])
        mask = m if rows is None else m[rows]
    P = orc.scale_mask_softmax(wl.bf16_to_f64(A), wl.bf16_to_f64(B), w.scalars["alpha"], mask, softcap=w.scalars.get("softcap", 0.0))
    return {"Y": P}


# --------------------------------------------------------------------------------------------- comparison
def check_outputs(w: wl.Workload, got: dict, ref: dict, rows=None, batches=None, label="", rowmax_tol=5e-3, softmax_tol=TOL_SOFTMAX_MAX,
                  norm_tol=TOL_NORM_MAX):
    """Element-by-element comparison against the oracle with the stated tolerances; returns the error figures.
    `rowmax_tol`: absolute tolerance of the fp32 row maximum (and the slack within which a reported arg max column
    must reach the oracle's maximum).  The fused path keeps fp32 up to that point (5e-3 covers tanh.approx); the
    unfused path has rounded the GEMM result to bf16 first, so it gets the normalised-tensor tolerance 3e-2.
    `softmax_tol`: 2e-3 for the fused kernel; the unfused path exponentiates bf16-rounded scores (relative error
    2^-9 on |score| up to ~4 after scaling), which alone moves a probability near 0.5 by up to ~4e-3, so the tests
    give it 1e-2 and say so.  `norm_tol`: max-abs bound of normalised outputs (3e-2 unless a caller says otherwise)."""
    check_canaries(got, label)
    Y = got["Y"]
    if batches is not None:
        Y = Y[list(batches)]
    if rows is not None:
        Y = Y[..., torch.as_tensor(rows, device=Y.device), :]
    Yg = to_f64(Y)
    assert Yg.shape == ref["Y"].shape, (Yg.shape, ref["Y"].shape)
    assert np.isfinite(Yg).all(), f"{label}: non-finite output (unwritten or NaN)"
    err = np.abs(Yg - ref["Y"])
    res = {"max_abs": float(err.max()), "mean_abs": float(err.mean())}
    if w.kind == wl.KIND_SCALE_MASK_SOFTMAX:
        assert res["max_abs"] <= softmax_tol, f"{label}: softmax max-abs {res['max_abs']:.3e}"
        dead = ref["Y"] == 0.0
        assert (Yg[dead] == 0.0).all(), f"{label}: masked entries must be exactly zero"
    else:
        assert res["max_abs"] <= norm_tol, f"{label}: max-abs {res['max_abs']:.3e}"
        assert res["mean_abs"] <= TOL_NORM_MEAN, f"{label}: mean-abs {res['mean_abs']:.3e}"
    if w.kind == wl.KIND_BIAS_GELU_RES_RMSNORM_MAX:
        rm, am = got["row_max"], got["row_argmax"]
        if rows is not None:
            idx = torch.as_tensor(rows, device=rm.device)
            rm, am = rm[idx], am[idx]
        rm = rm.cpu().numpy().astype(np.float64)
        am = am.cpu().numpy().astype(np.int64)
        assert np.abs(rm - ref["row_max"]).max() <= rowmax_tol, f"{label}: row max off by {np.abs(rm - ref['row_max']).max():.3e}"
        # several columns can be within fp32 / tanh-approximation noise of the maximum: the index is valid if the
        # oracle's value at the reported column is within `rowmax_tol` of the oracle's maximum
        n = ref["Y"].shape[-1]
        assert ((am >= 0) & (am < n)).all()
        at = np.take_along_axis(ref["Y"], am[:, None], axis=-1)[:, 0]
        slack = rowmax_tol
        assert (at >= ref["row_max"] - slack).all(), f"{label}: argmax points at a non-maximal column"
        res["argmax_mismatch"] = int((am != ref["row_argmax"]).sum())
        # invariants that need no oracle: rounding is monotone, so the stored bf16 row attains its maximum at the
        # reported column and that maximum is the rounded row max
        Yfull = got["Y"] if rows is None else got["Y"][torch.as_tensor(rows, device=got["Y"].device)]
        Ymax = Yfull.float().max(dim=-1).values.cpu().numpy()
        picked = np.take_along_axis(to_f64(Yfull), am[:, None], axis=-1)[:, 0]
        assert (picked == Ymax).all(), f"{label}: Y[argmax] is not the stored row maximum"
        rm_b = torch.from_numpy(rm.astype(np.float32)).to(torch.bfloat16).float().numpy()
        assert (rm_b == Ymax).all(), f"{label}: bf16(row_max) differs from the stored row maximum"
    return res
