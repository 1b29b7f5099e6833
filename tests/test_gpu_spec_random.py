"""Randomised differential test of the three pathways for epilogue programs: seeded random node lists (element-wise nodes,
broadcasts, reductions whose per-row values feed later nodes, row outputs) are evaluated by the fp64 node-list oracle and
by the library with `fused` = 1 (best path), 2 (on-chip interpreter where the program lowers to it) and 0 (row program).
Exercises typing, constant folding, liveness / buffer assignment and chain extraction on shapes nobody wrote by hand."""
import numpy as np
import pytest
import torch

import paper_2608_03537_b200 as cf
import workloads as wl
from oracle import fusion_spec_oracle as spo
from tests.parity import to_dev, to_f64

pytestmark = pytest.mark.gpu


def _N(default):
    """Seeds per test; COMFUSE_FUZZ_SEEDS scales the sweep for a longer soak."""
    import os
    return range(int(os.environ.get("COMFUSE_FUZZ_SEEDS", default)))

UNARY = ["neg", "abs", "square", "tanh", "relu", "sigmoid", "gelu_tanh", "exp"]
BINARY = ["add", "sub", "mul", "max", "min", "div"]
REDUCE = ["sum", "mean", "rmax", "rmin"]


def _reference_on_rounded_z(A, B, nodes, terminal, params, row_outputs):
    """The oracle evaluated behind the GEMM result rounded to bf16 (fp32 accumulate, round to nearest even): what the
    row-program pathway is defined to compute."""
    f = wl.bf16_to_f64
    Z = (f(A) @ f(B)).astype(np.float32)
    Zb = wl.bf16_to_f64(wl.f32_to_bf16_bits(Z))
    vals = spo.eval_nodes(nodes, Zb, [f(p) for p in params])
    M, N = Zb.shape
    Y = np.broadcast_to(np.asarray(vals[terminal], dtype=np.float64), (M, N)).copy()
    rows = [np.broadcast_to(np.asarray(vals[r], dtype=np.float64), (M, 1))[:, 0].copy() for r in row_outputs]
    return Y, rows


def _random_program(seed):
    g = np.random.default_rng(seed)
    nodes = [("acc", -1, -1, -1, 0.0), ("rowvec", -1, -1, 0, 0.0), ("const", -1, -1, -1, float(np.round(g.uniform(0.3, 1.5), 3)))]
    kinds = ["t", "t", "c"]  # tensor / row / const typed
    if g.random() < 0.5:
        nodes.append(("tensor", -1, -1, 1, 0.0))
        kinds.append("t")
    n_extra = int(g.integers(4, 14))
    for _ in range(n_extra):
        r = g.random()
        tensors = [i for i, k in enumerate(kinds) if k == "t"]
        anyv = list(range(len(nodes)))
        if r < 0.35:
            op = UNARY[int(g.integers(len(UNARY)))]
            a = int(g.choice(anyv))
            if op == "exp":   # keep the exponent bounded
                nodes.append(("tanh", a, -1, -1, 0.0)); kinds.append(kinds[a]); a = len(nodes) - 1
            nodes.append((op, a, -1, -1, 0.0)); kinds.append(kinds[a])
        elif r < 0.8:
            op = BINARY[int(g.integers(len(BINARY)))]
            a, b = int(g.choice(anyv)), int(g.choice(anyv))
            if op == "div":   # denominator bounded away from zero: 1.5 + tanh(.)
                nodes.append(("tanh", b, -1, -1, 0.0)); kinds.append(kinds[b])
                nodes.append(("const", -1, -1, -1, 1.5)); kinds.append("c")
                nodes.append(("add", len(nodes) - 2, len(nodes) - 1, -1, 0.0))
                kinds.append("t" if kinds[b] == "t" else ("r" if kinds[b] == "r" else "c"))
                b = len(nodes) - 1
            ka, kb = kinds[a], kinds[b]
            nodes.append((op, a, b, -1, 0.0))
            kinds.append("t" if "t" in (ka, kb) else ("r" if "r" in (ka, kb) else "c"))
        else:
            op = REDUCE[int(g.integers(len(REDUCE)))]
            a = int(g.choice(tensors))
            nodes.append((op, a, -1, -1, 0.0)); kinds.append("r")
    tensors = [i for i, k in enumerate(kinds) if k == "t" and nodes[i][0] not in ("rowvec", "tensor", "acc")]
    terminal = int(tensors[-1]) if tensors else 0
    rows = [i for i, k in enumerate(kinds) if k == "r"]
    row_outputs = tuple(int(x) for x in rows[-2:])
    n_params = 2 if any(n[0] == "tensor" for n in nodes) else 1
    return nodes, terminal, row_outputs, n_params


@pytest.mark.parametrize("seed", _N(64))
def test_random_program_matches_the_oracle_on_every_pathway(seed):
    M, N, K = 130, 256, 64
    nodes, terminal, row_outputs, n_params = _random_program(1000 + seed)
    A = wl.normal_bf16(seed, 0, (M, K))
    B = wl.normal_bf16(seed, 1, (K, N), std=K ** -0.5)
    params = [wl.normal_bf16(seed, 2, (N,), std=0.5), wl.normal_bf16(seed, 3, (M, N))][:n_params]
    f = wl.bf16_to_f64
    vals = spo.eval_nodes(nodes, f(A) @ f(B), [f(p) for p in params])
    big = max(float(np.max(np.abs(np.asarray(v)))) if np.all(np.isfinite(np.asarray(v))) else np.inf for v in vals)
    if not np.isfinite(big) or big > 1e3:
        pytest.skip("program leaves the bounded range")
    ref_exact = spo.gemm_spec(f(A), f(B), nodes, terminal, [f(p) for p in params], row_outputs)
    ref_rounded = _reference_on_rounded_z(A, B, nodes, terminal, params, row_outputs)
    spec = cf.make_spec(nodes, terminal, n_params, row_outputs)
    shape = cf.make_gemm_shape(1, M, N, K)
    plan = cf.spec_plan(spec, shape)
    dev = "cuda:0"
    dA, dB, dP = to_dev(A), to_dev(B), [to_dev(p) for p in params]
    seen = set()
    for fused in (1, 2, 0):
        path = plan.path if fused == 1 else (plan.program_path if fused == 2 else cf.SPEC_PATH_ROW_PROGRAM)
        # the row-program pathway is defined on the bf16-rounded GEMM result: random programs can be arbitrarily sensitive
        # to that rounding (tanh of a row sum near zero), so it is compared with the oracle evaluated on the rounded Z
        Yref, Rref = ref_rounded if path == cf.SPEC_PATH_ROW_PROGRAM else ref_exact
        scale = max(1.0, float(np.abs(Yref).max()))
        Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev)
        ro = [torch.full((M,), float("nan"), dtype=torch.float32, device=dev) for _ in row_outputs]
        ws = torch.empty(max(16, cf.gemm_spec_workspace_size(spec, shape, fused)), dtype=torch.uint8, device=dev)
        cf.gemm_spec(dA, dB, Y, spec, params=dP, row_out=ro, fused=fused, workspace=ws)
        torch.cuda.synchronize()
        assert cf.last_device_status() == cf.OK
        err = np.abs(to_f64(Y) - Yref)
        assert np.isfinite(err).all() and err.max() <= 3e-2 * scale, (seed, fused, plan.path, plan.program_path, err.max(), scale)
        for got, ref in zip(ro, Rref):
            rs = max(1.0, float(np.abs(ref).max()))
            assert np.abs(got.cpu().numpy().astype(np.float64) - ref).max() <= 3e-2 * rs, (seed, fused, "row output")
        seen.add(path)
    assert cf.SPEC_PATH_ROW_PROGRAM in seen


def _random_chain_program(seed):
    """A random program of the shape the on-chip interpreter takes: ONE resident tensor x, chains on it."""
    g = np.random.default_rng(seed)
    nodes = []

    def add(op, a=-1, b=-1, param=-1, imm=0.0):
        nodes.append((op, int(a), int(b), int(param), float(imm)))
        return len(nodes) - 1

    n_params = 1
    acc = add("acc")
    vec = [add("rowvec", param=0)]
    if g.random() < 0.5:
        vec.append(add("rowvec", param=1)); n_params = 2
    tensor = None
    if g.random() < 0.5:
        tensor = add("tensor", param=n_params); n_params += 1
    scalars = []

    def operand(allow_tensor):
        pool = [("const", None)] + [("vec", v) for v in vec] + [("row", s) for s in scalars]
        if allow_tensor and tensor is not None:
            pool.append(("tensor", tensor))
        kind, ix = pool[int(g.integers(len(pool)))]
        return add("const", imm=float(np.round(g.uniform(0.4, 1.6), 3))) if kind == "const" else ix

    def chain(v, n_ops, allow_tensor):
        for _ in range(n_ops):
            if g.random() < 0.4:
                op = ["tanh", "relu", "abs", "sigmoid", "neg", "square", "gelu_tanh"][int(g.integers(7))]
                if op == "square":
                    v = add("tanh", v)
                v = add(op, v)
            else:
                op = ["add", "sub", "mul", "max", "min", "div"][int(g.integers(6))]
                o = operand(allow_tensor)
                if op == "div":   # a row-uniform denominator bounded away from zero (constant, or 1.5 + tanh(statistic))
                    o = add("add", add("tanh", scalars[int(g.integers(len(scalars)))]), add("const", imm=1.5)) if scalars and g.random() < 0.5 \
                        else add("const", imm=float(np.round(g.uniform(0.5, 2.0), 3)))
                if op == "mul":
                    v = add("tanh", v)
                v = add(op, v, o) if g.random() < 0.7 or op == "div" else add(op, o, v)
        return v

    x = chain(acc, int(g.integers(0, 4)), True)
    n_stages = int(g.integers(0, 3))
    for _ in range(n_stages):
        new = []
        for _ in range(int(g.integers(1, 3))):
            u = chain(x, int(g.integers(0, 3)), False)
            r = add(["sum", "mean", "rmax", "rmin"][int(g.integers(4))], u)
            if g.random() < 0.5:   # per-row arithmetic on the statistic
                r = add("rsqrt", add("add", add("abs", r), add("const", imm=1.0)))
            new.append(r)
        scalars.extend(new)
    y = chain(x, int(g.integers(1, 5)), False)
    if nodes[y][0] in ("acc", "rowvec", "tensor"):
        y = add("relu", y)
    outs = list(scalars[-2:])
    if g.random() < 0.6:
        outs.append(add(["rmax", "sum", "argmax"][int(g.integers(3))], y))
    return nodes, y, tuple(outs), n_params


@pytest.mark.parametrize("seed", _N(160))
def test_random_chain_program_on_the_on_chip_interpreter(seed):
    M, N, K = (300, 1024, 72) if seed % 2 else (130, 256, 64)
    nodes, terminal, row_outputs, n_params = _random_chain_program(5000 + seed)
    A = wl.normal_bf16(seed, 0, (M, K))
    B = wl.normal_bf16(seed, 1, (K, N), std=K ** -0.5)
    params = []
    for q in range(n_params):
        is_tensor = any(n[0] == "tensor" and n[3] == q for n in nodes)
        params.append(wl.normal_bf16(seed, 2 + q, (M, N) if is_tensor else (N,), std=0.5))
    f = wl.bf16_to_f64
    vals = spo.eval_nodes(nodes, f(A) @ f(B), [f(p) for p in params])
    big = max(float(np.max(np.abs(np.asarray(v)))) if np.all(np.isfinite(np.asarray(v))) else np.inf for v in vals)
    if not np.isfinite(big) or big > 1e3 * N:
        pytest.skip("program leaves the bounded range")
    ref_exact = spo.gemm_spec(f(A), f(B), nodes, terminal, [f(p) for p in params], row_outputs)
    ref_rounded = _reference_on_rounded_z(A, B, nodes, terminal, params, row_outputs)
    spec = cf.make_spec(nodes, terminal, n_params, row_outputs)
    shape = cf.make_gemm_shape(1, M, N, K)
    plan = cf.spec_plan(spec, shape)
    if plan.program_path != cf.SPEC_PATH_FUSED_PROGRAM:
        pytest.skip("beyond the interpreter's limits")
    dev = "cuda:0"
    dA, dB, dP = to_dev(A), to_dev(B), [to_dev(p) for p in params]
    for fused in (2, 0):
        Yref, Rref = ref_exact if fused == 2 else ref_rounded
        scale = max(1.0, float(np.abs(Yref).max()))
        Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev)
        ro = [torch.full((M,), -1, dtype=torch.int32 if nodes[r][0] == "argmax" else torch.float32, device=dev) for r in row_outputs]
        ws = torch.empty(max(16, cf.gemm_spec_workspace_size(spec, shape, fused)), dtype=torch.uint8, device=dev)
        before = cf.launch_count()
        cf.gemm_spec(dA, dB, Y, spec, params=dP, row_out=ro, fused=fused, workspace=ws)
        torch.cuda.synchronize()
        assert cf.last_device_status() == cf.OK
        assert cf.launch_count() - before == (1 if fused == 2 else 2)
        err = np.abs(to_f64(Y) - Yref)
        assert np.isfinite(err).all() and err.max() <= 3e-2 * scale, (seed, fused, err.max(), scale)
        for r, got, ref in zip(row_outputs, ro, Rref):
            if nodes[r][0] == "argmax":
                idx = got.cpu().numpy().astype(np.int64)
                assert np.all((idx >= 0) & (idx < N))
                chosen = Yref[np.arange(M), idx]
                assert np.all(chosen >= Yref.max(axis=1) - 3e-2 * scale)
            else:
                rs = max(1.0, float(np.abs(ref).max()))
                assert np.abs(got.cpu().numpy().astype(np.float64) - ref).max() <= 3e-2 * rs, (seed, fused, "row output", nodes[r])
