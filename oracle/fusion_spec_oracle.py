"""fp64 CPU oracle for epilogues given as DATA: an ordered node list evaluated behind a MatMul.

TEST INFRASTRUCTURE ONLY.  Imported by the test-suite, the smoke check and the benchmark's CPU legs, by nothing on
the product path; shares no code with the CUDA library and never imports it.

What it defines (Sec. 5.2): the memory-intensive subgraph is a topologically ordered sequence of nodes of four
categories -- accumulator entry, broadcast (scalar constant, row vector, full tensor), element-wise computation
(unary / binary) and reduction over the last dimension -- with data-dependency edges, one terminal node whose value
is the output tensor, and a table of runtime parameters.  A reduction's per-row result can feed later element-wise
nodes (Sec. 5.3: the statistics and the passed-through original tensor enter the nested sub-program), which is how
LayerNorm, RMSNorm and Softmax are spelled with primitive nodes.  The value of a program is the plain evaluation of
its nodes in list order on the fp64 MatMul result: no stages, no tiling, no intermediate rounding.

A node is a tuple ``(op, in0, in1, param, imm)``; ``in0``/``in1`` index earlier nodes (-1 = unused), ``param``
indexes the parameter table (-1 = unused), ``imm`` is the constant of a ``const`` node.

Readings where the paper gives no formula: ``mean`` divides by N; ``argmax`` is the lowest column attaining the row
maximum; ``causal_mask`` is the additive mask 0 for column <= row and -inf above the diagonal; ``topk`` (the
parameterised Top-K mode of the StreamReduction node, Sec. 5) yields the K largest values of each row in falling order, equal values
in rising column order, with their columns.

Pins (tests/test_oracle_spec_pins.py, no GPU): a pure-Python loop evaluator on tiny inputs, fp64 library routines
(layer_norm, softmax, rms_norm, gelu) for the programs that spell them, closed forms (LayerNorm of a ramp, uniform
causal rows), hand-computed min / prod / argmax / top-k rows.
"""
from __future__ import annotations

import math

import numpy as np

_SQRT_2_OVER_PI = math.sqrt(2.0 / math.pi)

ENTRY_OPS = ("acc",)
BROADCAST_OPS = ("const", "rowvec", "tensor", "causal_mask")
UNARY_OPS = ("neg", "abs", "square", "sqrt", "rsqrt", "recip", "exp", "log", "tanh", "relu", "gelu_tanh", "sigmoid")
BINARY_OPS = ("add", "sub", "mul", "div", "max", "min")
REDUCE_OPS = ("sum", "mean", "rmax", "rmin", "prod", "argmax")
TOPK_OPS = ("topk_values", "topk_indices")  # K is the node's ``param``; the value is [M, K] and can only be a row output


def _unary(op: str, a: np.ndarray) -> np.ndarray:
    with np.errstate(all="ignore"):
        if op == "neg":
            return -a
        if op == "abs":
            return np.abs(a)
        if op == "square":
            return a * a
        if op == "sqrt":
            return np.sqrt(a)
        if op == "rsqrt":
            return 1.0 / np.sqrt(a)
        if op == "recip":
            return 1.0 / a
        if op == "exp":
            return np.exp(a)
        if op == "log":
            return np.log(a)
        if op == "tanh":
            return np.tanh(a)
        if op == "relu":
            return np.maximum(a, 0.0)
        if op == "gelu_tanh":
            return 0.5 * a * (1.0 + np.tanh(_SQRT_2_OVER_PI * (a + 0.044715 * a * a * a)))
        if op == "sigmoid":
            return 1.0 / (1.0 + np.exp(-a))
    raise ValueError(f"unknown unary op {op!r}")


def _binary(op: str, a: np.ndarray, b: np.ndarray) -> np.ndarray:
    with np.errstate(all="ignore"):
        if op == "add":
            return a + b
        if op == "sub":
            return a - b
        if op == "mul":
            return a * b
        if op == "div":
            return a / b
        if op == "max":
            return np.maximum(a, b)
        if op == "min":
            return np.minimum(a, b)
    raise ValueError(f"unknown binary op {op!r}")


def _reduce(op: str, a: np.ndarray, N: int) -> np.ndarray:
    """Row-wise reduction of an [M, N] value to [M, 1]."""
    if op == "sum":
        return a.sum(axis=1, keepdims=True)
    if op == "mean":
        return a.sum(axis=1, keepdims=True) / N
    if op == "rmax":
        return a.max(axis=1, keepdims=True)
    if op == "rmin":
        return a.min(axis=1, keepdims=True)
    if op == "prod":
        return a.prod(axis=1, keepdims=True)
    if op == "argmax":
        return a.argmax(axis=1).astype(np.float64)[:, None]  # numpy returns the first (lowest) maximiser
    raise ValueError(f"unknown reduction {op!r}")


def eval_nodes(nodes, Z: np.ndarray, params=(), row0: int = 0):
    """All node values of the program on the MatMul result ``Z`` [M, N] (fp64), in list order (Sec. 5.2).

    ``row0`` is the global index of Z's first row (only the causal mask looks at it).  Returns the list of values:
    [M, N] arrays for tensor-valued nodes, [M, 1] for per-row values, 0-d for constants.
    """
    Z = np.asarray(Z, dtype=np.float64)
    M, N = Z.shape
    vals = []
    for k, (op, in0, in1, param, imm) in enumerate(nodes):
        for e in (in0, in1):
            if not (e == -1 or 0 <= e < k):
                raise ValueError(f"node {k}: edge {e} does not point at an earlier node")
        if op == "acc":
            v = Z
        elif op == "const":
            v = np.float64(imm)
        elif op == "rowvec":
            v = np.asarray(params[param], dtype=np.float64).reshape(1, N)
        elif op == "tensor":
            v = np.asarray(params[param], dtype=np.float64).reshape(M, N)
        elif op == "causal_mask":
            rows = np.arange(row0, row0 + M)[:, None]
            v = np.where(np.arange(N)[None, :] <= rows, 0.0, -np.inf)
        elif op in UNARY_OPS:
            v = _unary(op, np.asarray(vals[in0]))
        elif op in BINARY_OPS:
            v = _binary(op, np.asarray(vals[in0]), np.asarray(vals[in1]))
        elif op in REDUCE_OPS:
            a = np.asarray(vals[in0])
            if a.ndim < 2:
                a = np.broadcast_to(a, (M, N))
            elif a.shape[1] != N:
                a = np.broadcast_to(a, (a.shape[0], N))
            if a.shape[0] != M:
                a = np.broadcast_to(a, (M, N))
            v = _reduce(op, a, N)
        elif op in TOPK_OPS:
            a = np.broadcast_to(np.asarray(vals[in0]), (M, N))
            tv, ti = topk_rows(a, param)
            v = tv if op == "topk_values" else ti.astype(np.float64)
        else:
            raise ValueError(f"node {k}: unknown op {op!r}")
        vals.append(v)
    return vals


def gemm_spec(A, B, nodes, terminal: int, params=(), row_outputs=()):
    """Y = value of node ``terminal`` of the program evaluated on Z = A B, as [M, N]; plus the per-row values of the
    nodes listed in ``row_outputs`` (each [M]; [M, K] for a Top-K node)  (Sec. 5.2: terminal node, parameter table; Sec. 3: Y = epilogue(A B))."""
    Z = np.matmul(np.asarray(A, dtype=np.float64), np.asarray(B, dtype=np.float64))
    M, N = Z.shape
    vals = eval_nodes(nodes, Z, params)
    Y = np.broadcast_to(np.asarray(vals[terminal], dtype=np.float64), (M, N)).copy()
    rows = []
    for r in row_outputs:
        if nodes[r][0] in TOPK_OPS:
            rows.append(np.asarray(vals[r], dtype=np.float64).copy())  # [M, K]
        else:
            rows.append(np.broadcast_to(np.asarray(vals[r], dtype=np.float64), (M, 1))[:, 0].copy())
    return Y, rows


def topk_rows(Y: np.ndarray, k: int):
    """The K largest values of every row in falling order and their columns; equal values in rising column order
    (the StreamReduction node's hyper-parameter K, Sec. 5)."""
    Y = np.asarray(Y, dtype=np.float64)
    order = np.argsort(-Y, axis=1, kind="stable")[:, :k]
    return np.take_along_axis(Y, order, axis=1), order
