"""Pins for the node-list oracle (epilogue programs as data, Sec. 5.2 / 5.3): CPU only.  The evaluator is compared with
things other than itself -- fp64 library routines for the programs that spell LayerNorm / RMSNorm / Softmax / GELU,
closed forms, hand-computed rows, and a scalar-loop evaluator written separately on tiny inputs."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import workloads as wl
from oracle import fusion_spec_oracle as spo


def _rng(seed):
    return np.random.default_rng(seed)


def _inputs(seed, M, K, N):
    g = _rng(seed)
    return g.standard_normal((M, K)), g.standard_normal((K, N)) / math.sqrt(K)


# ----------------------------------------------------------------------------- library routines (special cases)
@pytest.mark.parametrize("relu", [False, True])
def test_layernorm_program_equals_library_layer_norm(relu):
    M, K, N = 7, 12, 40
    A, B = _inputs(1, M, K, N)
    g = _rng(2)
    bias, R, gamma, beta = g.standard_normal(N), g.standard_normal((M, N)), g.standard_normal(N), g.standard_normal(N)
    prog = wl.spec_layernorm(eps=1e-5, relu=relu)
    Y, rows = spo.gemm_spec(A, B, prog.nodes, prog.terminal, (bias, R, gamma, beta))
    H = torch.from_numpy(A @ B + bias + R)
    ref = F.layer_norm(H, (N,), torch.from_numpy(gamma), torch.from_numpy(beta), 1e-5)
    if relu:
        ref = torch.relu(ref)
    np.testing.assert_allclose(Y, ref.numpy(), rtol=0, atol=1e-12)
    assert rows == []


def test_rmsnorm_max_program_equals_library_rms_norm_and_gelu():
    M, K, N = 6, 9, 33
    A, B = _inputs(3, M, K, N)
    g = _rng(4)
    bias, R, gain = g.standard_normal(N), g.standard_normal((M, N)), g.standard_normal(N)
    prog = wl.spec_rmsnorm_max(eps=1e-5)
    Y, (mx, am) = spo.gemm_spec(A, B, prog.nodes, prog.terminal, (bias, R, gain), prog.row_outputs)
    H = F.gelu(torch.from_numpy(A @ B + bias), approximate="tanh") + torch.from_numpy(R)
    ref = F.rms_norm(H, (N,), torch.from_numpy(gain), 1e-5)
    np.testing.assert_allclose(Y, ref.numpy(), rtol=0, atol=1e-12)
    v, i = ref.max(dim=1)
    np.testing.assert_allclose(mx, v.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_array_equal(am.astype(np.int64), i.numpy())


@pytest.mark.parametrize("causal,softcap", [(False, 0.0), (True, 0.0), (False, 3.0), (True, 1.5)])
def test_softmax_program_equals_library_softmax(causal, softcap):
    M, K, N = 11, 8, 11
    A, B = _inputs(5, M, K, N)
    prog = wl.spec_softmax(alpha=0.37, causal=causal, softcap=softcap)
    Y, _ = spo.gemm_spec(A, B, prog.nodes, prog.terminal)
    T = torch.from_numpy(A @ B) * 0.37
    if softcap > 0:
        T = torch.tanh(T / softcap) * softcap
    if causal:
        T = T.masked_fill(torch.ones(M, N, dtype=torch.bool).triu(1), float("-inf"))
    np.testing.assert_allclose(Y, torch.softmax(T, dim=1).numpy(), rtol=0, atol=1e-13)
    if causal:
        assert np.all(Y[np.triu_indices(M, 1, N)] == 0.0)


# ----------------------------------------------------------------------------- closed forms
@pytest.mark.parametrize("N", [4, 16, 768])
def test_layernorm_program_on_a_ramp_closed_form(N):
    # A = I makes Z = B; every row of B is the ramp 1..N: mean (N+1)/2, variance (N^2-1)/12
    B = np.tile(np.arange(1, N + 1, dtype=np.float64), (3, 1))
    prog = wl.spec_layernorm(eps=0.0, bias=False, residual=False, affine=False)
    Y, _ = spo.gemm_spec(np.eye(3), B, prog.nodes, prog.terminal)
    expect = (np.arange(1, N + 1) - (N + 1) / 2) / math.sqrt((N * N - 1) / 12)
    np.testing.assert_allclose(Y, np.tile(expect, (3, 1)), rtol=0, atol=1e-12)


def test_causal_softmax_program_of_zero_scores_is_uniform():
    M = 9
    prog = wl.spec_softmax(alpha=0.125, causal=True)
    Y, _ = spo.gemm_spec(np.zeros((M, 4)), np.ones((4, M)), prog.nodes, prog.terminal)
    for i in range(M):
        np.testing.assert_allclose(Y[i, : i + 1], 1.0 / (i + 1), rtol=0, atol=1e-15)
        assert np.all(Y[i, i + 1:] == 0.0)
    assert Y[0, 0] == 1.0


# ----------------------------------------------------------------------------- hand-computed rows
def test_reduction_operators_on_hand_computed_rows():
    Z = np.array([[3.0, 1.0, 4.0, 1.0, 5.0], [2.0, 7.0, 7.0, 1.0, -1.0]])
    nodes = [("acc", -1, -1, -1, 0.0), ("sum", 0, -1, -1, 0.0), ("mean", 0, -1, -1, 0.0), ("rmax", 0, -1, -1, 0.0),
             ("rmin", 0, -1, -1, 0.0), ("prod", 0, -1, -1, 0.0), ("argmax", 0, -1, -1, 0.0)]
    vals = spo.eval_nodes(nodes, Z)
    expect = {1: [14.0, 16.0], 2: [2.8, 3.2], 3: [5.0, 7.0], 4: [1.0, -1.0], 5: [60.0, -98.0], 6: [4.0, 1.0]}
    for k, e in expect.items():
        np.testing.assert_allclose(vals[k][:, 0], e, rtol=0, atol=1e-15)


def test_topk_rows_hand_computed_with_ties():
    v, c = spo.topk_rows(np.array([[2.0, 7.0, 7.0, 1.0], [0.5, -1.0, 0.5, 0.5]]), 3)
    np.testing.assert_array_equal(v, [[7.0, 7.0, 2.0], [0.5, 0.5, 0.5]])
    np.testing.assert_array_equal(c, [[1, 2, 0], [0, 2, 3]])


def test_topk_nodes_hand_computed_through_the_program_evaluator():
    # top-2 of relu(z): rows [0 5 0 5 1] -> (5, 5) at columns (1, 3); [2 0 0 0 3] -> (3, 2) at (4, 0)
    Z = np.array([[-1.0, 5.0, -3.0, 5.0, 1.0], [2.0, -7.0, -7.0, -1.0, 3.0]])
    nodes = [("acc", -1, -1, -1, 0.0), ("relu", 0, -1, -1, 0.0), ("topk_values", 1, -1, 2, 0.0), ("topk_indices", 1, -1, 2, 0.0)]
    Y, (tv, ti) = spo.gemm_spec(np.eye(2), Z, nodes, 1, (), (2, 3))
    np.testing.assert_array_equal(Y, np.maximum(Z, 0.0))
    np.testing.assert_array_equal(tv, [[5.0, 5.0], [3.0, 2.0]])
    np.testing.assert_array_equal(ti, [[1, 3], [4, 0]])


def test_topk_agrees_with_the_library_sort_on_distinct_values():
    g = _rng(21)
    Yv = g.permutation(200).astype(np.float64).reshape(4, 50)  # all distinct: no tie rule involved
    v, c = spo.topk_rows(Yv, 7)
    tv, tc = torch.topk(torch.from_numpy(Yv), 7, dim=1)
    np.testing.assert_array_equal(v, tv.numpy())
    np.testing.assert_array_equal(c, tc.numpy())


def test_row_scalar_and_constant_operands_broadcast():
    # y = (z - min z) / 2 + 1, per-row value fed back into an element-wise node, constants on either side
    Z = np.array([[1.0, 5.0, 3.0], [-2.0, -6.0, 0.0]])
    nodes = [("acc", -1, -1, -1, 0.0), ("rmin", 0, -1, -1, 0.0), ("sub", 0, 1, -1, 0.0), ("const", -1, -1, -1, 2.0),
             ("div", 2, 3, -1, 0.0), ("const", -1, -1, -1, 1.0), ("add", 5, 4, -1, 0.0)]
    vals = spo.eval_nodes(nodes, Z)
    np.testing.assert_array_equal(vals[6], [[1.0, 3.0, 2.0], [3.0, 1.0, 4.0]])


# ----------------------------------------------------------------------------- scalar-loop evaluator on tiny inputs
def _loop_eval(nodes, Z, params):
    """Element by element, with Python floats and the math module only."""
    M, N = len(Z), len(Z[0])
    un = {"neg": lambda a: -a, "abs": abs, "square": lambda a: a * a, "sqrt": math.sqrt, "rsqrt": lambda a: a ** -0.5,
          "recip": lambda a: 1 / a, "exp": math.exp, "log": math.log, "tanh": math.tanh, "relu": lambda a: a if a > 0 else 0.0,
          "gelu_tanh": lambda a: 0.5 * a * (1 + math.tanh(math.sqrt(2 / math.pi) * (a + 0.044715 * a ** 3))),
          "sigmoid": lambda a: 1 / (1 + math.exp(-a))}
    bi = {"add": lambda a, b: a + b, "sub": lambda a, b: a - b, "mul": lambda a, b: a * b, "div": lambda a, b: a / b,
          "max": max, "min": min}
    out = []
    for i in range(M):
        vals = []  # per node: list of N floats
        for (op, a, b, prm, imm) in nodes:
            if op == "acc":
                v = list(Z[i])
            elif op == "const":
                v = [imm] * N
            elif op == "rowvec":
                v = list(params[prm])
            elif op == "tensor":
                v = list(params[prm][i])
            elif op == "causal_mask":
                v = [0.0 if j <= i else -math.inf for j in range(N)]
            elif op in un:
                v = [un[op](x) for x in vals[a]]
            elif op in bi:
                v = [bi[op](x, y) for x, y in zip(vals[a], vals[b])]
            else:
                r = vals[a]
                if op == "sum":
                    s = math.fsum(r)
                elif op == "mean":
                    s = math.fsum(r) / N
                elif op == "rmax":
                    s = max(r)
                elif op == "rmin":
                    s = min(r)
                elif op == "prod":
                    s = 1.0
                    for x in r:
                        s *= x
                elif op == "argmax":
                    s = float(min(j for j in range(N) if r[j] == max(r)))
                else:
                    raise AssertionError(op)
                v = [s] * N
            vals.append(v)
        out.append(vals)
    return out


@pytest.mark.parametrize("name", ["layernorm", "rmsnorm_max", "softmax", "gated"])
def test_programs_against_scalar_loops(name):
    M, K, N = 4, 3, 6
    A, B = _inputs(11, M, K, N)
    g = _rng(12)
    prog = {"layernorm": wl.spec_layernorm(relu=True), "rmsnorm_max": wl.spec_rmsnorm_max(),
            "softmax": wl.spec_softmax(alpha=0.5, causal=False, softcap=2.0), "gated": wl.spec_gated_minmax()}[name]
    params = [g.standard_normal(N) if k == "rowvec" else g.standard_normal((M, N)) for k in prog.param_kinds]
    Y, rows = spo.gemm_spec(A, B, prog.nodes, prog.terminal, params, prog.row_outputs)
    Z = [[math.fsum(A[i, k] * B[k, j] for k in range(K)) for j in range(N)] for i in range(M)]
    loop = _loop_eval(prog.nodes, Z, params)
    for i in range(M):
        np.testing.assert_allclose(Y[i], loop[i][prog.terminal], rtol=1e-12, atol=1e-13)
        for r, node in zip(rows, prog.row_outputs):
            np.testing.assert_allclose(r[i], loop[i][node][0], rtol=1e-12, atol=1e-13)


def test_forward_edges_are_rejected():
    with pytest.raises(ValueError):
        spo.eval_nodes([("acc", -1, -1, -1, 0.0), ("add", 0, 2, -1, 0.0), ("const", -1, -1, -1, 1.0)], np.zeros((2, 2)))


# ----------------------------------------------------------------------------- the two oracles agree where they overlap
def test_programs_agree_with_the_op_list_oracle():
    """The primitive spellings evaluated by the node-list oracle equal the op-list oracle's closed definitions (both are
    pinned separately above and in test_oracle_pins.py; this ties the two together)."""
    from oracle import comfuse_oracle as orc
    M, K, N = 9, 16, 48
    A, B = _inputs(31, M, K, N)
    g = _rng(32)
    bias, R, gamma, beta = g.standard_normal(N), g.standard_normal((M, N)), g.standard_normal(N), g.standard_normal(N)
    p = wl.spec_layernorm(eps=1e-5, relu=True)
    Y, _ = spo.gemm_spec(A, B, p.nodes, p.terminal, (bias, R, gamma, beta))
    np.testing.assert_allclose(Y, orc.bias_res_layernorm(A, B, bias, R, gamma, beta, 1.0, 1e-5, relu=True), rtol=0, atol=1e-12)
    p = wl.spec_rmsnorm_max(eps=1e-5)
    Y, (mx, am) = spo.gemm_spec(A, B, p.nodes, p.terminal, (bias, R, gamma), p.row_outputs)
    Y2, mx2, am2 = orc.bias_gelu_res_rmsnorm_max(A, B, bias, R, gamma, 1.0, 1e-5)
    np.testing.assert_allclose(Y, Y2, rtol=0, atol=1e-12)
    np.testing.assert_allclose(mx, mx2, rtol=0, atol=1e-12)
    np.testing.assert_array_equal(am.astype(np.int64), am2)
    p = wl.spec_rmsnorm_max(eps=1e-5, activation=False, residual=False)
    Y, _ = spo.gemm_spec(A, B, p.nodes, p.terminal, (bias, gamma), p.row_outputs)
    np.testing.assert_allclose(Y, orc.bias_gelu_res_rmsnorm_max(A, B, bias, None, gamma, 1.0, 1e-5, activation=False)[0], rtol=0, atol=1e-12)
    As, Bs = _inputs(33, 12, 8, 12)
    p = wl.spec_softmax(alpha=0.3, causal=True, softcap=2.5)
    Y, _ = spo.gemm_spec(As, Bs, p.nodes, p.terminal)
    np.testing.assert_allclose(Y, orc.scale_mask_softmax(As, Bs, 0.3, orc.causal_mask(12, 12), softcap=2.5), rtol=0, atol=1e-13)
