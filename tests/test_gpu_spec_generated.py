"""The kernel generated for a program (`fused` = 3, Sec. 5: the fused epilogue as generated code).

The program's structure is compiled into the fused kernel at run time; the interpreter (`fused` = 2) runs the same lowering
as data.  Compiled without floating-point contraction the generated kernel must reproduce the interpreter bit for bit --
output and every row output -- on hand-written programs, Top-K programs and a seeded random sweep; compiled the default
way it is compared with the fp64 oracle at the interpreter's tolerances.
"""
import numpy as np
import pytest
import torch

import paper_2608_03537_b200 as cf
import workloads as wl
from oracle import fusion_spec_oracle as spo
from tests.parity import to_dev, to_f64
from tests.test_gpu_spec import CASES, _check_rows, _inputs, _oracle, _run, _run_topk, _topk_prog
from tests.test_gpu_spec_random import _random_chain_program

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _compiler_present():
    st, why = cf.program_compiler_status()
    if st != cf.OK:
        pytest.skip(f"no run-time compiler on this machine: {why}")


@pytest.fixture
def no_contraction(monkeypatch):
    monkeypatch.setenv("COMFUSE_GENERATED_FMAD", "0")


def _bits(t):
    return t.view(torch.int16) if t.dtype == torch.bfloat16 else t.view(torch.int32)


def _same(a, b):
    return torch.equal(_bits(a), _bits(b))


@pytest.mark.parametrize("name", sorted(CASES))
def test_generated_kernel_equals_the_interpreter_bit_for_bit(name, no_contraction):
    prog, batch, M, N, K, kind, tmax, tmean = CASES[name]
    A, B, params = _inputs(61, batch, M, N, K, prog.param_kinds)
    Yi, roi, plan, _ = _run(prog, A, B, params, 2, batch, M, N)
    assert plan.program_path == cf.SPEC_PATH_FUSED_PROGRAM
    Yg, rog, _, launches = _run(prog, A, B, params, cf.GENERATED, batch, M, N)
    assert launches == 1
    assert _same(Yi, Yg)
    for a, b in zip(roi, rog):
        assert _same(a, b)


@pytest.mark.parametrize("name", sorted(CASES))
def test_generated_kernel_matches_the_oracle(name):
    prog, batch, M, N, K, kind, tmax, tmean = CASES[name]
    A, B, params = _inputs(62, batch, M, N, K, prog.param_kinds)
    Y, ro, plan, launches = _run(prog, A, B, params, cf.GENERATED, batch, M, N)
    assert launches == 1
    Yref, Rref = _oracle(prog, A, B, params, batch)
    err = np.abs(to_f64(Y) - Yref)
    assert np.isfinite(err).all() and err.max() <= tmax and err.mean() <= tmean, (err.max(), err.mean())
    _check_rows(prog, ro, Rref, Yref)


# one, two, four, eight and sixteen CTAs per row block; the last two shapes give every cluster several tiles
@pytest.mark.parametrize("M,N,K", [(129, 256, 64), (300, 512, 72), (260, 768, 264), (300, 1024, 136), (200, 2048, 64), (520, 4096, 72),
                                   (4000, 4096, 64), (9000, 256, 64)])
def test_generated_range_normalise_over_every_instantiation(M, N, K, no_contraction):
    prog = wl.spec_range_normalise()
    A, B, params = _inputs(63, 1, M, N, K, prog.param_kinds)
    Yi, roi, plan, _ = _run(prog, A, B, params, 2, 1, M, N)
    Yg, rog, _, launches = _run(prog, A, B, params, cf.GENERATED, 1, M, N)
    assert launches == 1 and _same(Yi, Yg)
    for a, b in zip(roi, rog):
        assert _same(a, b)
    Yref, Rref = _oracle(prog, A, B, params, 1)
    err = np.abs(to_f64(Yg) - Yref)
    assert np.isfinite(err).all() and err.max() <= 4e-3 and err.mean() <= 1e-3


@pytest.mark.parametrize("M,N,K", [(300, 256, 72), (260, 1024, 136), (4000, 2048, 64)])
def test_generated_gated_program_equals_the_interpreter(M, N, K, no_contraction):
    prog = wl.spec_gated_minmax()       # the resident tensor is an operand of its own chain: x * sigmoid(x)
    A, B, params = _inputs(67, 1, M, N, K, prog.param_kinds)
    Yi, roi, _, _ = _run(prog, A, B, params, 2, 1, M, N)
    Yg, rog, _, launches = _run(prog, A, B, params, cf.GENERATED, 1, M, N)
    assert launches == 1 and _same(Yi, Yg) and all(_same(a, b) for a, b in zip(roi, rog))
    Yref, Rref = _oracle(prog, A, B, params, 1)
    err = np.abs(to_f64(Yg) - Yref)
    assert np.isfinite(err).all() and err.max() <= 4e-3


@pytest.mark.parametrize("M,N,K", [(300, 1280, 72), (520, 1536, 136), (260, 1792, 64), (300, 2560, 72), (1300, 3072, 64), (260, 3584, 200)])
def test_generated_kernels_at_row_lengths_the_library_has_no_instantiation_for(M, N, K):
    """Clusters of 10, 6, 14, 10, 12 and 14 CTAs: an instantiation of a generated kernel is a table entry.  The interpreter
    and the compiled kinds' on-chip forms do not exist at these row lengths."""
    prog = wl.spec_range_normalise()
    A, B, params = _inputs(69, 1, M, N, K, prog.param_kinds)
    Y, ro, plan, launches = _run(prog, A, B, params, 1, 1, M, N)
    assert launches == 1 and plan.path == cf.SPEC_PATH_FUSED_PROGRAM and plan.program_path == cf.SPEC_PATH_ROW_PROGRAM
    Yref, Rref = _oracle(prog, A, B, params, 1)
    err = np.abs(to_f64(Y) - Yref)
    assert np.isfinite(err).all() and err.max() <= 4e-3 and err.mean() <= 1e-3
    lo, hi, pr, sm, am = [t.cpu().numpy() for t in ro]
    np.testing.assert_allclose(lo, Rref[0], atol=1e-4, rtol=1e-5)
    np.testing.assert_allclose(hi, Rref[1], atol=1e-4, rtol=1e-5)
    np.testing.assert_allclose(pr, Rref[2], rtol=1e-4)
    np.testing.assert_allclose(sm, Rref[3], rtol=1e-4)
    assert np.mean(am == Rref[4].astype(np.int64)) > 0.995
    # a LayerNorm with an extra row output (not a compiled kind) with its residual through the operand ring
    ln = wl.spec_layernorm(relu=True)
    ln = wl.SpecProgram(ln.nodes, ln.terminal, (ln.nodes.index(("mean", 4, -1, -1, 0.0)),), ln.param_kinds)
    A, B, params = _inputs(70, 1, M, N, K, ln.param_kinds)
    Y, ro, plan, launches = _run(ln, A, B, params, cf.GENERATED, 1, M, N)
    Yref, Rref = _oracle(ln, A, B, params, 1)
    err = np.abs(to_f64(Y) - Yref)
    assert launches == 1 and np.isfinite(err).all() and err.max() <= 3e-2 and err.mean() <= 3e-3
    np.testing.assert_allclose(ro[0].cpu().numpy(), Rref[0], atol=2e-3)


def _dag_programs():
    N_ = ("acc", -1, -1, -1, 0.0)
    progs = {}
    # relu(x) * tanh(x) with x = acc + bias, minus its row maximum
    progs["two_factors"] = wl.SpecProgram(
        [N_, ("rowvec", -1, -1, 0, 0.0), ("add", 0, 1, -1, 0.0), ("relu", 2, -1, -1, 0.0), ("tanh", 2, -1, -1, 0.0), ("mul", 3, 4, -1, 0.0),
         ("rmax", 5, -1, -1, 0.0), ("sub", 5, 6, -1, 0.0)], 7, (6,), ("rowvec",))
    # three computed tensors alive at once: (sigmoid(x) - tanh(x)) / (1.5 + tanh(abs(x) * g)), normalised by its row mean square
    progs["three_live"] = wl.SpecProgram(
        [N_, ("sigmoid", 0, -1, -1, 0.0), ("tanh", 0, -1, -1, 0.0), ("sub", 1, 2, -1, 0.0), ("abs", 0, -1, -1, 0.0), ("rowvec", -1, -1, 0, 0.0),
         ("mul", 4, 5, -1, 0.0), ("tanh", 6, -1, -1, 0.0), ("const", -1, -1, -1, 1.5), ("add", 7, 8, -1, 0.0), ("div", 3, 9, -1, 0.0),
         ("square", 10, -1, -1, 0.0), ("mean", 11, -1, -1, 0.0), ("const", -1, -1, -1, 1e-3), ("add", 12, 13, -1, 0.0), ("rsqrt", 14, -1, -1, 0.0),
         ("mul", 10, 15, -1, 0.0)], 16, (12,), ("rowvec",))
    # the two factors are used again behind the reduction, with a residual tensor inside one of them
    progs["residual_gate"] = wl.SpecProgram(
        [N_, ("tensor", -1, -1, 0, 0.0), ("add", 0, 1, -1, 0.0), ("gelu_tanh", 2, -1, -1, 0.0), ("neg", 0, -1, -1, 0.0), ("sigmoid", 4, -1, -1, 0.0),
         ("mul", 3, 5, -1, 0.0), ("rmin", 6, -1, -1, 0.0), ("rmax", 6, -1, -1, 0.0), ("sub", 8, 7, -1, 0.0), ("const", -1, -1, -1, 1e-3),
         ("add", 9, 10, -1, 0.0), ("sub", 6, 7, -1, 0.0), ("div", 12, 11, -1, 0.0)], 13, (7, 8), ("tensor",))
    return progs


@pytest.mark.parametrize("M,N,K", [(300, 256, 72), (260, 1024, 136), (1100, 2048, 64)])
@pytest.mark.parametrize("name", ["two_factors", "three_live", "residual_gate"])
def test_programs_in_which_computed_tensors_meet_run_as_generated_code(name, M, N, K):
    """Two or three computed tensors alive at once: temporaries of the generated kernel (registers); the interpreter has
    none, so `fused` = 2 takes the row program, and both are compared with the node-list oracle."""
    prog = _dag_programs()[name]
    A, B, params = _inputs(68, 1, M, N, K, prog.param_kinds)
    Y, ro, plan, launches = _run(prog, A, B, params, cf.GENERATED, 1, M, N)
    assert launches == 1 and plan.path == cf.SPEC_PATH_FUSED_PROGRAM and plan.program_path == cf.SPEC_PATH_ROW_PROGRAM
    Yref, Rref = _oracle(prog, A, B, params, 1)
    err = np.abs(to_f64(Y) - Yref)
    scale = max(1.0, float(np.abs(Yref).max()))
    assert np.isfinite(err).all() and err.max() <= 8e-3 * scale and err.mean() <= 1e-3 * scale, (err.max(), err.mean(), scale)
    for got, ref in zip(ro, Rref):
        np.testing.assert_allclose(got.cpu().numpy(), ref, rtol=2e-3, atol=2e-3)
    Y1, ro1, _, launches1 = _run(prog, A, B, params, 1, 1, M, N)     # the best path is the same kernel
    assert launches1 == 1 and _same(Y, Y1)


def test_generated_kernel_with_the_operand_stored_n_by_k(no_contraction):
    prog = wl.spec_range_normalise()
    A, B, params = _inputs(64, 1, 300, 1024, 136, prog.param_kinds)
    Y0, ro0, _, _ = _run(prog, A, B, params, cf.GENERATED, 1, 300, 1024)
    Y1, ro1, _, _ = _run(prog, A, B, params, cf.GENERATED, 1, 300, 1024, b_nk=True)
    assert _same(Y0, Y1) and all(_same(a, b) for a, b in zip(ro0, ro1))


@pytest.mark.parametrize("M,N,K,k", [(70, 256, 16, 8), (300, 512, 16, 3), (200, 1024, 16, 8), (257, 4096, 16, 4)])
def test_generated_topk_exact_on_integer_data_with_ties(M, N, K, k):
    g = np.random.default_rng(70 + N)
    A = wl.f32_to_bf16_bits(g.integers(-1, 2, size=(M, K)).astype(np.float32))
    B = wl.f32_to_bf16_bits(g.integers(-2, 3, size=(K, N)).astype(np.float32))
    bias = wl.f32_to_bf16_bits(np.zeros(N, dtype=np.float32))
    Y, tv, ti, Yref, rv, ri = _run_topk(A, B, bias, k, fused=cf.GENERATED)
    np.testing.assert_array_equal(to_f64(Y), Yref)
    np.testing.assert_array_equal(tv.astype(np.float64), rv)
    np.testing.assert_array_equal(ti.astype(np.int64), ri.astype(np.int64))


@pytest.mark.parametrize("seed", range(0, 160, 5))
def test_random_chain_program_generated_equals_interpreted(seed, no_contraction):
    M, N, K = (300, 1024, 72) if seed % 2 else (130, 256, 64)
    nodes, terminal, row_outputs, n_params = _random_chain_program(5000 + seed)
    A = wl.normal_bf16(seed, 0, (M, K))
    B = wl.normal_bf16(seed, 1, (K, N), std=K ** -0.5)
    params = []
    for q in range(n_params):
        is_tensor = any(n[0] == "tensor" and n[3] == q for n in nodes)
        params.append(wl.normal_bf16(seed, 2 + q, (M, N) if is_tensor else (N,), std=0.5))
    spec = cf.make_spec(nodes, terminal, n_params, row_outputs)
    shape = cf.make_gemm_shape(1, M, N, K)
    if cf.spec_plan(spec, shape).program_path != cf.SPEC_PATH_FUSED_PROGRAM:
        pytest.skip("beyond the on-chip lowering's limits")
    dev = "cuda:0"
    dA, dB, dP = to_dev(A), to_dev(B), [to_dev(p) for p in params]
    out = {}
    for fused in (2, cf.GENERATED):
        Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev)
        ro = [torch.full((M,), -1, dtype=torch.int32 if nodes[r][0] == "argmax" else torch.float32, device=dev) for r in row_outputs]
        cf.gemm_spec(dA, dB, Y, spec, params=dP, row_out=ro, fused=fused)
        torch.cuda.synchronize()
        assert cf.last_device_status() == cf.OK
        out[fused] = (Y, ro)
    # NaN-free programs only compare equal bit for bit; a NaN the program itself produces has the same bits on both paths
    assert _same(out[2][0], out[cf.GENERATED][0]), seed
    for a, b in zip(out[2][1], out[cf.GENERATED][1]):
        assert _same(a, b), seed


def test_programs_that_differ_in_constants_share_a_kernel(tmp_path, monkeypatch):
    """Constants are run-time arguments of the generated kernel.  The generated translation unit is dumped only when a kernel
    is actually compiled, so the second program -- same structure, other constants -- must leave no dump behind."""
    def prog(c0, c1):
        nodes = [("acc", -1, -1, -1, 0.0), ("const", -1, -1, -1, c0), ("mul", 0, 1, -1, 0.0), ("tanh", 2, -1, -1, 0.0),
                 ("rmax", 3, -1, -1, 0.0), ("sub", 3, 4, -1, 0.0), ("const", -1, -1, -1, c1), ("mul", 5, 6, -1, 0.0), ("exp", 7, -1, -1, 0.0),
                 ("abs", 8, -1, -1, 0.0)]
        return wl.SpecProgram(nodes, 9, (4,), ())
    M, N, K = 260, 512, 72
    A, B, _ = _inputs(65, 1, M, N, K, ())
    first, second = tmp_path / "first.cu", tmp_path / "second.cu"
    monkeypatch.setenv("COMFUSE_GENERATED_DUMP", str(first))
    Y0, ro0, _, _ = _run(prog(0.7, 1.3), A, B, [], cf.GENERATED, 1, M, N)
    assert first.exists()
    monkeypatch.setenv("COMFUSE_GENERATED_DUMP", str(second))
    Y1, ro1, _, _ = _run(prog(0.9, 0.6), A, B, [], cf.GENERATED, 1, M, N)
    assert not second.exists()                                   # the second call found the first call's kernel
    for (c0, c1), Y, ro in (((0.7, 1.3), Y0, ro0), ((0.9, 0.6), Y1, ro1)):
        Yref, Rref = _oracle(prog(c0, c1), A, B, [], 1)
        assert np.abs(to_f64(Y) - Yref).max() <= 1e-2
        np.testing.assert_allclose(ro[0].cpu().numpy(), Rref[0], atol=2e-3)


def test_generated_kernel_is_refused_where_the_program_has_no_on_chip_lowering():
    N_ = ("acc", -1, -1, -1, 0.0)       # a full tensor used behind a reduction
    prog = wl.SpecProgram([N_, ("mean", 0, -1, -1, 0.0), ("sub", 0, 1, -1, 0.0), ("tensor", -1, -1, 0, 0.0), ("add", 2, 3, -1, 0.0)], 4, (),
                          ("tensor",))
    A, B, params = _inputs(66, 1, 130, 256, 64, prog.param_kinds)
    with pytest.raises(cf.ComfuseError) as e:
        _run(prog, A, B, params, cf.GENERATED, 1, 130, 256)
    assert e.value.status == cf.ERR_UNSUPPORTED


def test_p1_sized_program_generated_against_sampled_oracle_rows():
    w = wl.config(6)
    prog = w.program
    A, B, p0 = w.tensors["A"], w.tensors["B"], w.tensors["p0"]
    M, N = A.shape[0], B.shape[1]
    Y, ro, plan, launches = _run(prog, A, B, [p0], cf.GENERATED, 1, M, N)
    assert launches == 1
    rows = np.random.default_rng(5).choice(M, size=256, replace=False)
    f = wl.bf16_to_f64
    Yref, Rref = spo.gemm_spec(f(A[rows]), f(B), prog.nodes, prog.terminal, [f(p0)], prog.row_outputs)
    err = np.abs(to_f64(Y)[rows] - Yref)
    assert np.isfinite(err).all() and err.max() <= 4e-3
    for k in range(4):
        np.testing.assert_allclose(ro[k].cpu().numpy()[rows], Rref[k], rtol=2e-4, atol=1e-4)
