"""Seeded synthetic inputs for the ComFuse joint compute-memory fusion path.

This module only *generates data*: tensor shapes, value distributions and the
bf16 storage format.  It contains none of the method's arithmetic (no GEMM, no
normalisation, no softmax) and is the one module that both the CPU oracle's
tests and the CUDA path's tests / benchmark import, so that both sides see the
same bytes.

Every tensor is produced as fp32 from a numpy ``Generator`` (PCG64) seeded with
``[seed, tensor_index]``, rounded to bfloat16 with round-to-nearest-even, and
returned as the raw ``uint16`` bit pattern.  ``bf16_to_f64`` widens those bits
exactly, which is what the oracle consumes; the GPU side reinterprets the same
bits as ``torch.bfloat16``.

The five named workloads follow the paper's two experiment families: a MatMul
followed by a reduction-bearing epilogue (post-norm / softmax patterns,
Sec. 6.1) and a back-to-back GEMM MLP (Sec. 6.2, Table II).  The paper uses
synthetic microbenchmarks without public datasets; so do these.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

# ----------------------------------------------------------------------------
# bf16 storage helpers (format conversion only)
# ----------------------------------------------------------------------------


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (round-to-nearest-even); returns uint16 bits."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    # NaN stays NaN (quiet); everything else: add 0x7FFF + lsb, truncate.
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    nan = np.isnan(x)
    out = rounded.astype(np.uint16)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bits to fp32."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_to_f64(b: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bits to fp64 (what the oracle consumes)."""
    return bf16_bits_to_f32(b).astype(np.float64)


# ----------------------------------------------------------------------------
# random tensors
# ----------------------------------------------------------------------------


def _rng(seed: int, index: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([int(seed), int(index)]))


def normal_bf16(seed: int, index: int, shape, mean: float = 0.0, std: float = 1.0) -> np.ndarray:
    g = _rng(seed, index)
    x = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    if mean != 0.0:
        x += np.float32(mean)
    return f32_to_bf16_bits(x)


def uniform_bf16(seed: int, index: int, shape, lo: float, hi: float) -> np.ndarray:
    g = _rng(seed, index)
    x = g.random(size=shape, dtype=np.float32)
    x = x * np.float32(hi - lo) + np.float32(lo)
    return f32_to_bf16_bits(x)


# ----------------------------------------------------------------------------
# workload descriptions
# ----------------------------------------------------------------------------

KIND_BIAS_RES_LAYERNORM = "bias_res_layernorm"
KIND_BIAS_GELU_RES_RMSNORM_MAX = "bias_gelu_res_rmsnorm_max"
KIND_SCALE_MASK_SOFTMAX = "scale_mask_softmax"
KIND_B2B_MLP_LAYERNORM = "b2b_mlp_layernorm"
KIND_B2B_SOFTMAX_ATTENTION = "b2b_softmax_attention"
KIND_B2B_MLP_RELU = "b2b_mlp_relu"
KIND_GEMM_PROGRAM = "gemm_program"   # epilogue given as a node list (Workload.program)


@dataclass
class Workload:
    """One problem instance: a kind, its sizes, scalars and bf16 tensors (uint16 bits)."""

    name: str
    kind: str
    dims: dict
    scalars: dict
    tensors: dict = field(default_factory=dict)
    program: object = None  # SpecProgram for KIND_GEMM_PROGRAM; its parameter slot k is tensors[f"p{k}"]

    def gemm_flops(self) -> float:
        d = self.dims
        if self.kind in (KIND_B2B_MLP_LAYERNORM, KIND_B2B_SOFTMAX_ATTENTION, KIND_B2B_MLP_RELU):
            return d.get("batch", 1) * (2.0 * d["M"] * d["K"] * d["N1"] + 2.0 * d["M"] * d["N1"] * d["N2"])
        return 2.0 * d.get("batch", 1) * d["M"] * d["N"] * d["K"]

    def min_hbm_bytes(self) -> float:
        """Every operand read once and every output written once, nothing else."""
        d = self.dims
        if self.kind == KIND_B2B_SOFTMAX_ATTENTION:
            return 2.0 * d["batch"] * (d["M"] * d["K"] + d["K"] * d["N1"] + d["N1"] * d["N2"] + d["M"] * d["N2"])
        if self.kind == KIND_B2B_MLP_RELU:
            M, K, N1, N2 = d["M"], d["K"], d["N1"], d["N2"]
            return 2.0 * (M * K + K * N1 + N1 * N2 + N1 + N2 + M * N2)
        if self.kind == KIND_B2B_MLP_LAYERNORM:
            M, K, N1, N2 = d["M"], d["K"], d["N1"], d["N2"]
            return 2.0 * (M * K + K * N1 + N1 * N2 + N1 + N2 + M * N2) + (
                4.0 * N2 if "gamma" in self.tensors else 0.0
            )
        b, M, N, K = d.get("batch", 1), d["M"], d["N"], d["K"]
        total = 2.0 * b * (M * K + K * N + M * N)
        if self.kind == KIND_GEMM_PROGRAM:
            total += sum(2.0 * v.size for k, v in self.tensors.items() if k.startswith("p"))
            total += 4.0 * M * len(self.program.row_outputs)
        if self.kind == KIND_BIAS_RES_LAYERNORM:
            total += 2.0 * (M * N + N)  # residual, bias
            total += 2.0 * 2 * N if "gamma" in self.tensors else 0.0
        elif self.kind == KIND_BIAS_GELU_RES_RMSNORM_MAX:
            total += 2.0 * (M * N + 2 * N) + 8.0 * M  # residual, bias, g, rowmax+argmax
        return total


def _gemm_epilogue_ln(name, seed, M, N, K, affine, relu=False):
    t = {
        "A": normal_bf16(seed, 0, (M, K)),
        "B": normal_bf16(seed, 1, (K, N), std=1.0 / math.sqrt(K)),
        "bias": uniform_bf16(seed, 2, (N,), -0.1, 0.1),
        "residual": normal_bf16(seed, 3, (M, N)),
    }
    if affine:
        t["gamma"] = normal_bf16(seed, 4, (N,), mean=1.0, std=0.02)
        t["beta"] = normal_bf16(seed, 5, (N,), mean=0.0, std=0.02)
    return Workload(name, KIND_BIAS_RES_LAYERNORM, {"M": M, "N": N, "K": K},
                    {"alpha": 1.0, "eps": 1e-5, "relu": bool(relu)}, t)


def post_norm(M=256, N=256, K=256, seed=0, affine=False, name=None, relu=False) -> Workload:
    """Y = LayerNorm(X.W + b + R) (then ReLU if ``relu``).  X,R ~ N(0,1); W ~ N(0, var 1/K); b ~ U(-0.1, 0.1)."""
    return _gemm_epilogue_ln(name or f"post_norm_{M}x{N}x{K}", seed, M, N, K, affine, relu)


def complex_subgraph(M=8192, N=4096, K=4096, seed=2, name=None, activation=True, residual=True) -> Workload:
    """Z = X.W + b; H = GELU_tanh(Z) + R; Y = RMSNorm(H).g; row max / argmax of Y.  Without the activation and the
    residual this is the plain bias + RMSNorm pattern."""
    t = {
        "A": normal_bf16(seed, 0, (M, K)),
        "B": normal_bf16(seed, 1, (K, N), std=1.0 / math.sqrt(K)),
        "bias": uniform_bf16(seed, 2, (N,), -0.1, 0.1),
        "residual": normal_bf16(seed, 3, (M, N)),
        "gamma": normal_bf16(seed, 4, (N,), mean=1.0, std=0.02),
    }
    if not residual:
        del t["residual"]
    return Workload(name or f"complex_subgraph_{M}x{N}x{K}", KIND_BIAS_GELU_RES_RMSNORM_MAX,
                    {"M": M, "N": N, "K": K}, {"alpha": 1.0, "eps": 1e-5, "activation": bool(activation)}, t)


def scaled_masked_softmax(batch=64, M=2048, N=2048, K=64, seed=3, causal=True, name=None, softcap=0.0) -> Workload:
    """P = softmax(alpha * A.B + mask) per batch; alpha = 1/sqrt(K); causal 0 / -inf mask; ``softcap`` > 0 passes the
    scaled scores through softcap * tanh(. / softcap) first."""
    t = {
        "A": normal_bf16(seed, 0, (batch, M, K)),
        "B": normal_bf16(seed, 1, (batch, K, N)),
    }
    return Workload(name or f"softmax_{batch}x{M}x{N}x{K}", KIND_SCALE_MASK_SOFTMAX,
                    {"batch": batch, "M": M, "N": N, "K": K},
                    {"alpha": 1.0 / math.sqrt(K), "causal": bool(causal), "softcap": float(softcap)}, t)


def b2b_mlp(M=32768, K=128, N1=512, N2=128, seed=4, affine=False, name=None) -> Workload:
    """O = LayerNorm(GELU_tanh(X.W1 + b1).W2 + b2 + X); needs N2 == K for the residual."""
    assert N2 == K
    t = {
        "X": normal_bf16(seed, 0, (M, K)),
        "W1": normal_bf16(seed, 1, (K, N1), std=1.0 / math.sqrt(K)),
        "b1": uniform_bf16(seed, 2, (N1,), -0.1, 0.1),
        "W2": normal_bf16(seed, 3, (N1, N2), std=1.0 / math.sqrt(N1)),
        "b2": uniform_bf16(seed, 4, (N2,), -0.1, 0.1),
    }
    if affine:
        t["gamma"] = normal_bf16(seed, 5, (N2,), mean=1.0, std=0.02)
        t["beta"] = normal_bf16(seed, 6, (N2,), mean=0.0, std=0.02)
    return Workload(name or f"b2b_mlp_{M}x{K}x{N1}x{N2}", KIND_B2B_MLP_LAYERNORM,
                    {"M": M, "K": K, "N1": N1, "N2": N2}, {"eps": 1e-5}, t)


def dlrm_bottom_mlp(M=32768, K=1024, N1=512, N2=128, seed=8, name=None) -> Workload:
    """O = ReLU(ReLU(X.W1 + b1).W2 + b2): the two-layer bottom MLP with the paper's DLRM feature dimensions
    1024 -> 512 -> 128.  X ~ N(0, 1), weights ~ N(0, 1 / fan-in), biases ~ U(-0.1, 0.1)."""
    t = {
        "X": normal_bf16(seed, 0, (M, K)),
        "W1": normal_bf16(seed, 1, (K, N1), std=1.0 / math.sqrt(K)),
        "b1": uniform_bf16(seed, 2, (N1,), -0.1, 0.1),
        "W2": normal_bf16(seed, 3, (N1, N2), std=1.0 / math.sqrt(N1)),
        "b2": uniform_bf16(seed, 4, (N2,), -0.1, 0.1),
    }
    return Workload(name or f"dlrm_bottom_mlp_{M}x{K}x{N1}x{N2}", KIND_B2B_MLP_RELU,
                    {"M": M, "K": K, "N1": N1, "N2": N2}, {}, t)


# The five named configurations (index = position in the benchmark's config list).
def target_attention(batch=32, M=4096, S=256, d=128, seed=5, name=None) -> Workload:
    """O = softmax(Q.Kt / sqrt(d)).V per batch: M target positions attend to S source positions (the paper's
    Target-Attention shape is M = 4096, S = 256).  Q, Kt, V ~ N(0, 1)."""
    t = {
        "X": normal_bf16(seed, 0, (batch, M, d)),
        "W1": normal_bf16(seed, 1, (batch, d, S)),
        "W2": normal_bf16(seed, 2, (batch, S, d)),
    }
    return Workload(name or f"target_attention_{batch}x{M}x{S}x{d}", KIND_B2B_SOFTMAX_ATTENTION,
                    {"batch": batch, "M": M, "K": d, "N1": S, "N2": d}, {"alpha": 1.0 / math.sqrt(d)}, t)


def config(index: int) -> Workload:
    if index == 0:   # post-norm tiny, gamma = 1, beta = 0, seed 0
        return post_norm(256, 256, 256, seed=0, affine=False, name="c1_post_norm_tiny")
    if index == 1:   # BERT-base-shaped post-norm FFN output (batch 16 x seq 512)
        return post_norm(8192, 768, 3072, seed=1, affine=True, name="c2_bert_ffn_out_post_norm")
    if index == 2:   # complex subgraph over wide rows
        return complex_subgraph(8192, 4096, 4096, seed=2, name="c3_complex_subgraph")
    if index == 3:   # GEMM + scaled causal row softmax
        return scaled_masked_softmax(64, 2048, 2048, 64, seed=3, name="c4_scaled_causal_softmax")
    if index == 4:   # back-to-back GEMM MLP with post-norm
        return b2b_mlp(32768, 128, 512, 128, seed=4, name="c5_b2b_mlp")
    if index == 5:   # beyond the five named configurations: B2B with a reduction as F (attention form)
        return target_attention(32, 4096, 256, 128, seed=5, name="a1_target_attention")
    if index == 7:   # beyond the five: the Self-Attention 512 x 512 shape of Sec. 6.2 (two sub-tiles of 256 source positions)
        return target_attention(256, 512, 512, 128, seed=7, name="a2_self_attention_512")
    if index == 8:   # beyond the five: the DLRM bottom-MLP shape of Sec. 6.2 (K streamed through the first GEMM)
        return dlrm_bottom_mlp(32768, 1024, 512, 128, seed=8, name="d1_dlrm_bottom_mlp")
    if index == 6:   # beyond the five: an epilogue given as data that no compiled kind covers
        return program_range_normalise(8192, 1024, 1024, seed=6, name="p1_program_range_normalise")
    raise IndexError(index)


def sample_rows(M: int, count: int, seed: int = 12345) -> np.ndarray:
    """A sorted sample of row indices that always includes the first and last rows
    and both sides of every 128-row boundary near the ends."""
    g = _rng(seed, M)
    fixed = {0, 1, 127, 128, M - 129 if M > 129 else 0, M - 128 if M > 128 else 0, M - 2 if M > 1 else 0, M - 1}
    fixed = {r for r in fixed if 0 <= r < M}
    extra = max(0, count - len(fixed))
    pool = g.choice(M, size=min(M, extra), replace=False)
    rows = sorted(fixed.union(int(r) for r in pool))
    return np.asarray(rows[:max(count, len(fixed))], dtype=np.int64)


# ----------------------------------------------------------------------------
# epilogue programs as data (node lists; no arithmetic here, only the lists)
# ----------------------------------------------------------------------------
# A node is (op, in0, in1, param, imm): op is a name of the Fusion-Spec vocabulary (Sec. 5.2: accumulator entry,
# broadcasts, element-wise computations, reductions), in0/in1 index earlier nodes, param indexes the call's parameter
# table, imm is the value of a "const" node.


class _Prog:
    def __init__(self):
        self.nodes = []

    def add(self, op, a=-1, b=-1, param=-1, imm=0.0):
        self.nodes.append((op, int(a), int(b), int(param), float(imm)))
        return len(self.nodes) - 1


@dataclass
class SpecProgram:
    """An epilogue program: ordered nodes, the terminal node stored as Y, per-row outputs, and what each parameter slot
    holds ("rowvec" [N] / "tensor" [M, N])."""
    nodes: list
    terminal: int
    row_outputs: tuple = ()
    param_kinds: tuple = ()


def spec_layernorm(eps=1e-5, bias=True, residual=True, affine=True, relu=False) -> SpecProgram:
    """MatMul-BiasAdd(-Residual)-LayerNorm(-ReLU) spelled with primitive nodes: two mean reductions (Sec. 3.2, Fig. 3;
    the MBLR pattern of Sec. 6.1 with relu=True).  Parameter slots in order: bias, residual, gamma, beta (those present)."""
    g = _Prog()
    kinds = []
    x = g.add("acc")
    if bias:
        kinds.append("rowvec")
        x = g.add("add", x, g.add("rowvec", param=len(kinds) - 1))
    if residual:
        kinds.append("tensor")
        x = g.add("add", x, g.add("tensor", param=len(kinds) - 1))
    mean = g.add("mean", x)
    d = g.add("sub", x, mean)
    var = g.add("mean", g.add("square", d))
    rstd = g.add("rsqrt", g.add("add", var, g.add("const", imm=eps)))
    y = g.add("mul", d, rstd)
    if affine:
        kinds.append("rowvec")
        y = g.add("mul", y, g.add("rowvec", param=len(kinds) - 1))
        kinds.append("rowvec")
        y = g.add("add", y, g.add("rowvec", param=len(kinds) - 1))
    if relu:
        y = g.add("relu", y)
    return SpecProgram(g.nodes, y, (), tuple(kinds))


def spec_rmsnorm_max(eps=1e-5, activation=True, residual=True) -> SpecProgram:
    """MatMul-BiasAdd(-GELU)(-Residual)-RMSNorm, then the chained row max / arg max (Sec. 3.2 chaining; the MBR pattern
    of Sec. 6.1 with activation=False, residual=False).  Parameter slots: bias, [residual], gain."""
    g = _Prog()
    kinds = ["rowvec"]
    x = g.add("add", g.add("acc"), g.add("rowvec", param=0))
    if activation:
        x = g.add("gelu_tanh", x)
    if residual:
        kinds.append("tensor")
        x = g.add("add", x, g.add("tensor", param=len(kinds) - 1))
    ms = g.add("mean", g.add("square", x))
    rstd = g.add("rsqrt", g.add("add", ms, g.add("const", imm=eps)))
    kinds.append("rowvec")
    y = g.add("mul", g.add("mul", x, rstd), g.add("rowvec", param=len(kinds) - 1))
    mx = g.add("rmax", y)
    am = g.add("argmax", y)
    return SpecProgram(g.nodes, y, (mx, am), tuple(kinds))


def spec_softmax(alpha=1.0, causal=False, softcap=0.0) -> SpecProgram:
    """MatMul-Scale(-TanhSoftcap)(-Mask)-Softmax spelled with primitive nodes (the MSTS pattern of Sec. 6.1): a max and a
    sum reduction."""
    g = _Prog()
    t = g.add("mul", g.add("acc"), g.add("const", imm=alpha))
    if softcap > 0.0:
        t = g.add("mul", g.add("tanh", g.add("mul", t, g.add("const", imm=1.0 / softcap))), g.add("const", imm=softcap))
    if causal:
        t = g.add("add", t, g.add("causal_mask"))
    e = g.add("exp", g.add("sub", t, g.add("rmax", t)))
    y = g.add("div", e, g.add("sum", e))
    return SpecProgram(g.nodes, y, (), ())


def spec_gated_minmax() -> SpecProgram:
    """A program outside the compiled patterns: a gate x * sigmoid(x) spelled with two uses of x (a DAG, not a chain),
    rescaled to the row's range with a min and a max reduction, plus the row product of the gate's sigmoid as a
    per-row output (exercises the min / max / prod reduction operators of Sec. 5).  Parameter slot 0: bias."""
    g = _Prog()
    x = g.add("add", g.add("acc"), g.add("rowvec", param=0))
    sg = g.add("sigmoid", x)
    s = g.add("mul", x, sg)
    lo = g.add("rmin", s)
    hi = g.add("rmax", s)
    rng = g.add("add", g.add("sub", hi, lo), g.add("const", imm=1e-3))
    y = g.add("div", g.add("sub", s, lo), rng)
    pr = g.add("prod", g.add("add", g.add("mul", sg, g.add("const", imm=0.01)), g.add("const", imm=0.995)))
    return SpecProgram(g.nodes, y, (lo, hi, pr), ("rowvec",))


def spec_range_normalise() -> SpecProgram:
    """A chain program outside the compiled patterns that keeps ONE tensor resident: x = acc + bias, rescaled to the row's
    range with a min and a max reduction (same stage boundary), then chained reductions on the result (sum, arg max) and a
    product reduction of a function of x (the sum / prod / max / min operators of Sec. 5).  Parameter slot 0: bias."""
    g = _Prog()
    x = g.add("add", g.add("acc"), g.add("rowvec", param=0))
    lo = g.add("rmin", x)
    hi = g.add("rmax", x)
    rng = g.add("add", g.add("sub", hi, lo), g.add("const", imm=1e-3))
    y = g.add("div", g.add("sub", x, lo), rng)
    pr = g.add("prod", g.add("add", g.add("mul", g.add("sigmoid", x), g.add("const", imm=0.01)), g.add("const", imm=0.995)))
    sm = g.add("sum", y)
    am = g.add("argmax", y)
    return SpecProgram(g.nodes, y, (lo, hi, pr, sm, am), ("rowvec",))


def program_range_normalise(M=8192, N=1024, K=1024, seed=6, name=None) -> Workload:
    """GEMM followed by the range-normalising chain program (spec_range_normalise): inputs as for the post-norm pattern."""
    t = {
        "A": normal_bf16(seed, 0, (M, K)),
        "B": normal_bf16(seed, 1, (K, N), std=1.0 / math.sqrt(K)),
        "p0": uniform_bf16(seed, 2, (N,), -0.1, 0.1),
    }
    return Workload(name or f"program_range_normalise_{M}x{N}x{K}", KIND_GEMM_PROGRAM, {"M": M, "N": N, "K": K}, {}, t,
                    program=spec_range_normalise())
