"""Parity of epilogue programs given as data (comfuse_gemm_spec) against the node-list oracle, element by element:
programs that lower to a fused kernel (and must then equal the enum entry point bit for bit), the same programs forced
onto the row-program pathway, and a program outside the compiled patterns."""
import numpy as np
import pytest
import torch

import paper_2608_03537_b200 as cf
import workloads as wl
from oracle import fusion_spec_oracle as spo
from tests.parity import TOL_NORM_MAX, TOL_NORM_MEAN, TOL_SOFTMAX_MAX, TOL_SOFTMAX_UNFUSED, to_dev, to_f64

pytestmark = pytest.mark.gpu


def _inputs(seed, batch, M, N, K, kinds):
    shp = (lambda *s: (batch, *s) if batch > 1 else s)
    A = wl.normal_bf16(seed, 0, shp(M, K))
    B = wl.normal_bf16(seed, 1, shp(K, N), std=K ** -0.5)
    params = []
    for i, kd in enumerate(kinds):
        if kd == "rowvec":
            params.append(wl.normal_bf16(seed, 10 + i, (N,), mean=1.0 if i >= 2 else 0.0, std=0.1))
        else:
            params.append(wl.normal_bf16(seed, 10 + i, shp(M, N)))
    return A, B, params


def _run(prog, A, B, params, fused, batch, M, N, b_nk=False):
    fused = int(fused)
    dev = "cuda:0"
    spec = cf.make_spec(prog.nodes, prog.terminal, len(prog.param_kinds), prog.row_outputs)
    dA, dB = to_dev(A), to_dev(B)
    if b_nk:
        dB = dB.transpose(-1, -2).contiguous()      # the operand as a layer stores it: [N, K]
    dP = [to_dev(p) for p in params]
    Y = torch.full((batch, M, N) if batch > 1 else (M, N), float("nan"), dtype=torch.bfloat16, device=dev)
    rows = batch * M
    ro = [torch.full((rows,), -7, dtype=torch.int32 if prog.nodes[r][0] == "argmax" else torch.float32, device=dev)
          for r in prog.row_outputs]
    shape = cf.make_gemm_shape(batch, M, N, A.shape[-1], flags=cf.FLAG_B_ROW_MAJOR_NK if b_nk else 0)
    plan = cf.spec_plan(spec, shape)
    ws = torch.empty(max(16, cf.gemm_spec_workspace_size(spec, shape, fused)), dtype=torch.uint8, device=dev)
    before = cf.launch_count()
    cf.gemm_spec(dA, dB, Y, spec, params=dP, row_out=ro, fused=fused, workspace=ws, b_nk=b_nk)
    torch.cuda.synchronize()
    assert cf.last_device_status() == cf.OK
    return Y, ro, plan, cf.launch_count() - before


def _oracle(prog, A, B, params, batch):
    f = wl.bf16_to_f64
    if batch == 1:
        return spo.gemm_spec(f(A), f(B), prog.nodes, prog.terminal, [f(p) for p in params], prog.row_outputs)
    Ys, Rs = [], []
    for b in range(batch):
        Y, R = spo.gemm_spec(f(A[b]), f(B[b]), prog.nodes, prog.terminal, [f(p) if p.ndim == 1 else f(p[b]) for p in params], prog.row_outputs)
        Ys.append(Y)
        Rs.append(R)
    return np.stack(Ys), [np.concatenate([r[k] for r in Rs]) for k in range(len(prog.row_outputs))]


CASES = {
    # name: (program, batch, M, N, K, fused kind it lowers to, max tolerance, mean tolerance)
    "layernorm_relu": (wl.spec_layernorm(relu=True), 1, 520, 768, 264, cf.EPI_BIAS_RES_LAYERNORM, TOL_NORM_MAX, TOL_NORM_MEAN),
    "layernorm_plain": (wl.spec_layernorm(bias=False, residual=False, affine=False), 1, 300, 256, 128, cf.EPI_BIAS_RES_LAYERNORM, TOL_NORM_MAX, TOL_NORM_MEAN),
    "rmsnorm_max": (wl.spec_rmsnorm_max(), 1, 392, 1024, 200, cf.EPI_BIAS_GELU_RES_RMSNORM_MAX, TOL_NORM_MAX, TOL_NORM_MEAN),
    "rmsnorm_mbr": (wl.spec_rmsnorm_max(activation=False, residual=False), 1, 260, 2048, 136, cf.EPI_BIAS_GELU_RES_RMSNORM_MAX, TOL_NORM_MAX, TOL_NORM_MEAN),
    "softmax_causal": (wl.spec_softmax(0.125, True, 0.0), 2, 512, 512, 64, cf.EPI_SCALE_MASK_SOFTMAX, TOL_SOFTMAX_MAX, 1e-4),
    "softmax_softcap": (wl.spec_softmax(0.2, False, 2.0), 1, 300, 1024, 72, cf.EPI_SCALE_MASK_SOFTMAX, TOL_SOFTMAX_MAX, 1e-4),
}


def _check_rows(prog, got, ref, Yref, tol=5e-3):
    for k, node in enumerate(prog.row_outputs):
        if prog.nodes[node][0] == "argmax":
            # near-ties: the chosen column must attain the oracle's maximum within the tolerance of the values
            idx = got[k].cpu().numpy().astype(np.int64)
            Y2 = Yref.reshape(-1, Yref.shape[-1])
            assert np.all((idx >= 0) & (idx < Y2.shape[1]))
            chosen = Y2[np.arange(Y2.shape[0]), idx]
            slack = 1e-3 if tol <= 5e-3 else tol  # the row-program pathway ranks values computed from the bf16-rounded GEMM result
            assert np.all(chosen >= Y2.max(axis=1) - slack * np.maximum(1.0, np.abs(Y2.max(axis=1))))
            assert np.mean(idx == ref[k].astype(np.int64)) > (0.99 if tol <= 5e-3 else 0.9)
        else:
            np.testing.assert_allclose(got[k].cpu().numpy().astype(np.float64), ref[k], rtol=tol, atol=tol)


@pytest.mark.parametrize("name", sorted(CASES))
def test_program_lowers_to_the_fused_kernel_and_matches_the_oracle(name):
    prog, batch, M, N, K, kind, tmax, tmean = CASES[name]
    A, B, params = _inputs(31, batch, M, N, K, prog.param_kinds)
    Y, ro, plan, launches = _run(prog, A, B, params, True, batch, M, N)
    assert plan.path == cf.SPEC_PATH_FUSED_KERNEL and plan.fused_kind == kind and plan.n_stages == 3
    assert launches == 1
    Yref, Rref = _oracle(prog, A, B, params, batch)
    err = np.abs(to_f64(Y) - Yref)
    assert np.isfinite(err).all() and err.max() <= tmax and err.mean() <= tmean, (err.max(), err.mean())
    _check_rows(prog, ro, Rref, Yref)


@pytest.mark.parametrize("fused", [1, 2, 0])
@pytest.mark.parametrize("name", ["layernorm_relu", "rmsnorm_max", "softmax_causal"])
def test_second_operand_stored_n_by_k_on_every_pathway(name, fused):
    """comfuse_gemm_shape_t.flags = COMFUSE_FLAG_B_ROW_MAJOR_NK: the compiled kind (1), the on-chip interpreter (2) and the
    GEMM + row-program pair (0) read B [N, K] in place and give the same bits as with B [K, N]."""
    prog, batch, M, N, K, kind, tmax, tmean = CASES[name]
    A, B, params = _inputs(37, batch, M, N, K, prog.param_kinds)
    Y0, ro0, plan0, _ = _run(prog, A, B, params, fused, batch, M, N)
    Y1, ro1, plan1, _ = _run(prog, A, B, params, fused, batch, M, N, b_nk=True)
    assert plan0.path == plan1.path
    assert torch.equal(Y0.view(torch.int16), Y1.view(torch.int16))
    for a, b in zip(ro0, ro1):
        assert torch.equal(a, b)


@pytest.mark.parametrize("name", sorted(CASES))
def test_same_program_on_the_row_program_pathway(name):
    prog, batch, M, N, K, kind, tmax, tmean = CASES[name]
    A, B, params = _inputs(32, batch, M, N, K, prog.param_kinds)
    Y, ro, plan, launches = _run(prog, A, B, params, False, batch, M, N)
    assert launches == 2  # GEMM, row program
    Yref, Rref = _oracle(prog, A, B, params, batch)
    err = np.abs(to_f64(Y) - Yref)
    # this pathway exponentiates / normalises the bf16-rounded GEMM result, like the in-library unfused baseline
    tmax = TOL_SOFTMAX_UNFUSED if kind == cf.EPI_SCALE_MASK_SOFTMAX else tmax
    assert np.isfinite(err).all() and err.max() <= tmax and err.mean() <= tmean, (err.max(), err.mean())
    _check_rows(prog, ro, Rref, Yref, tol=2e-2)


@pytest.mark.parametrize("name", sorted(CASES))
def test_same_program_on_the_on_chip_interpreter(name):
    prog, batch, M, N, K, kind, tmax, tmean = CASES[name]
    A, B, params = _inputs(35, batch, M, N, K, prog.param_kinds)
    Y, ro, plan, launches = _run(prog, A, B, params, 2, batch, M, N)
    assert plan.program_path == cf.SPEC_PATH_FUSED_PROGRAM and launches == 1
    Yref, Rref = _oracle(prog, A, B, params, batch)
    err = np.abs(to_f64(Y) - Yref)
    assert np.isfinite(err).all() and err.max() <= tmax and err.mean() <= tmean, (err.max(), err.mean())
    _check_rows(prog, ro, Rref, Yref)


# the last two shapes give every cluster several tiles (persistent walk, staging boxes reused, last tile staged in the ring)
@pytest.mark.parametrize("M,N,K", [(300, 1024, 136), (520, 4096, 72), (129, 256, 64), (260, 768, 264), (4000, 4096, 64), (9000, 256, 64)])
def test_chain_program_outside_the_compiled_patterns_runs_on_chip(M, N, K):
    prog = wl.spec_range_normalise()
    A, B, params = _inputs(36, 1, M, N, K, prog.param_kinds)
    Y, ro, plan, launches = _run(prog, A, B, params, True, 1, M, N)
    assert plan.path == cf.SPEC_PATH_FUSED_PROGRAM and plan.n_passes == 2 and launches == 1
    Yref, Rref = _oracle(prog, A, B, params, 1)
    err = np.abs(to_f64(Y) - Yref)
    assert np.isfinite(err).all() and err.max() <= 4e-3 and err.mean() <= 1e-3, (err.max(), err.mean())
    lo, hi, pr, sm, am = [t.cpu().numpy() for t in ro]
    np.testing.assert_allclose(lo, Rref[0], atol=1e-4, rtol=1e-5)
    np.testing.assert_allclose(hi, Rref[1], atol=1e-4, rtol=1e-5)
    np.testing.assert_allclose(pr, Rref[2], rtol=1e-4)
    np.testing.assert_allclose(sm, Rref[3], rtol=1e-4)
    # y's maximum is attained where x's is; the gap to the runner-up is far above fp32 rounding for Gaussian rows
    assert np.mean(am == Rref[4].astype(np.int64)) > 0.995
    chosen = Yref[np.arange(M), am.astype(np.int64)]
    assert np.all(chosen >= Yref.max(axis=1) - 1e-5)


def test_interpreter_with_residual_over_several_tiles_per_cluster():
    # LayerNorm-ReLU in primitives forced onto the interpreter: the residual rides the operand ring tile after tile
    prog = wl.spec_layernorm(relu=True)
    M, N, K = 5000, 2048, 72
    A, B, params = _inputs(38, 1, M, N, K, prog.param_kinds)
    Y, ro, plan, launches = _run(prog, A, B, params, 2, 1, M, N)
    assert plan.program_path == cf.SPEC_PATH_FUSED_PROGRAM and launches == 1
    Yref, _ = _oracle(prog, A, B, params, 1)
    err = np.abs(to_f64(Y) - Yref)
    assert np.isfinite(err).all() and err.max() <= TOL_NORM_MAX and err.mean() <= TOL_NORM_MEAN, (err.max(), err.mean())


def test_near_miss_of_a_compiled_kind_runs_on_chip():
    # residual inside the activation (the compiled RMSNorm kind has it outside), no row outputs
    N_ = ("acc", -1, -1, -1, 0.0)
    nodes = [N_, ("rowvec", -1, -1, 0, 0), ("add", 0, 1, -1, 0), ("tensor", -1, -1, 1, 0), ("add", 2, 3, -1, 0), ("gelu_tanh", 4, -1, -1, 0),
             ("square", 5, -1, -1, 0), ("mean", 6, -1, -1, 0), ("const", -1, -1, -1, 1e-5), ("add", 7, 8, -1, 0), ("rsqrt", 9, -1, -1, 0),
             ("mul", 5, 10, -1, 0)]
    prog = wl.SpecProgram(nodes, 11, (), ("rowvec", "tensor"))
    M, N, K = 392, 2048, 136
    A, B, params = _inputs(37, 1, M, N, K, prog.param_kinds)
    Y, ro, plan, launches = _run(prog, A, B, params, True, 1, M, N)
    assert plan.path == cf.SPEC_PATH_FUSED_PROGRAM and launches == 1
    Yref, _ = _oracle(prog, A, B, params, 1)
    err = np.abs(to_f64(Y) - Yref)
    assert np.isfinite(err).all() and err.max() <= TOL_NORM_MAX and err.mean() <= TOL_NORM_MEAN, (err.max(), err.mean())


def test_fused_lowering_equals_the_enum_entry_point_bit_for_bit():
    prog, batch, M, N, K, kind, _, _ = CASES["layernorm_relu"]
    A, B, params = _inputs(33, batch, M, N, K, prog.param_kinds)
    Y, _, _, _ = _run(prog, A, B, params, True, batch, M, N)
    dP = [to_dev(p) for p in params]
    Y2 = torch.empty_like(Y)
    cf.gemm_epilogue(to_dev(A), to_dev(B), Y2, cf.EPI_BIAS_RES_LAYERNORM, bias=dP[0], residual=dP[1], gamma=dP[2], beta=dP[3],
                     eps=1e-5, flags=cf.FLAG_POST_RELU)
    torch.cuda.synchronize()
    assert torch.equal(Y.view(torch.int16), Y2.view(torch.int16))


@pytest.mark.parametrize("M,N,K", [(260, 1000, 136), (64, 4096, 64), (130, 264, 72)])
def test_program_outside_the_compiled_patterns(M, N, K):
    prog = wl.spec_gated_minmax()
    A, B, params = _inputs(34, 1, M, N, K, prog.param_kinds)
    Y, ro, plan, launches = _run(prog, A, B, params, True, 1, M, N)
    # a gate x * sigmoid(x): on-chip where the row length has an instantiation (x stays resident, the gate is a chain with x
    # as its operand), else GEMM + row program
    on_chip = N == 4096
    assert plan.path == (cf.SPEC_PATH_FUSED_PROGRAM if on_chip else cf.SPEC_PATH_ROW_PROGRAM) and plan.n_stages == 2
    assert launches == (1 if on_chip else 2)
    Yref, Rref = _oracle(prog, A, B, params, 1)
    err = np.abs(to_f64(Y) - Yref)
    assert np.isfinite(err).all() and err.max() <= 1.5e-2 and err.mean() <= 2e-3, (err.max(), err.mean())
    np.testing.assert_allclose(ro[0].cpu().numpy(), Rref[0], atol=3e-2)   # row min of the gate
    np.testing.assert_allclose(ro[1].cpu().numpy(), Rref[1], atol=3e-2)   # row max
    np.testing.assert_allclose(ro[2].cpu().numpy(), Rref[2], rtol=2e-3)   # row product


@pytest.mark.parametrize("fused", [2, 0])
@pytest.mark.parametrize("M,N,K", [(300, 256, 72), (260, 1024, 136), (4000, 2048, 64)])
def test_gated_program_on_the_interpreter_and_on_the_row_program(M, N, K, fused):
    """x * sigmoid(x) spelled with two uses of x, rescaled to the row's range, plus the row product of a function of the
    sigmoid: the resident tensor is an operand of its own chain."""
    prog = wl.spec_gated_minmax()
    A, B, params = _inputs(37, 1, M, N, K, prog.param_kinds)
    Y, ro, plan, launches = _run(prog, A, B, params, fused, 1, M, N)
    assert plan.program_path == cf.SPEC_PATH_FUSED_PROGRAM and plan.n_passes == 2
    assert launches == (1 if fused else 2)
    Yref, Rref = _oracle(prog, A, B, params, 1)
    err = np.abs(to_f64(Y) - Yref)
    tol = 4e-3 if fused else 1.5e-2
    assert np.isfinite(err).all() and err.max() <= tol and err.mean() <= tol / 4, (err.max(), err.mean())
    np.testing.assert_allclose(ro[0].cpu().numpy(), Rref[0], atol=1e-4 if fused else 3e-2)   # row min of the gate
    np.testing.assert_allclose(ro[1].cpu().numpy(), Rref[1], atol=1e-4 if fused else 3e-2, rtol=1e-5)   # row max
    np.testing.assert_allclose(ro[2].cpu().numpy(), Rref[2], rtol=2e-4 if fused else 2e-3)   # row product


def test_row_program_rejects_rows_that_do_not_fit_shared_memory():
    prog = wl.spec_gated_minmax()
    spec = cf.make_spec(prog.nodes, prog.terminal, 1, prog.row_outputs)
    with pytest.raises(cf.ComfuseError) as e:
        cf.spec_plan(spec, cf.make_gemm_shape(1, 128, 65536, 64))
    assert e.value.status == cf.ERR_UNSUPPORTED


def _topk_prog(k):
    nodes = [("acc", -1, -1, -1, 0.0), ("rowvec", -1, -1, 0, 0.0), ("add", 0, 1, -1, 0.0), ("relu", 2, -1, -1, 0.0),
             ("topk_values", 3, -1, k, 0.0), ("topk_indices", 3, -1, k, 0.0)]
    return wl.SpecProgram(nodes, 3, (4, 5), ("rowvec",))


def _run_topk(A, B, bias, k, fused=1):
    prog = _topk_prog(k)
    M, N = A.shape[0], B.shape[1]
    spec = cf.make_spec(prog.nodes, prog.terminal, 1, prog.row_outputs)
    shape = cf.make_gemm_shape(1, M, N, A.shape[1])
    dev = "cuda:0"
    Y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
    tv = torch.full((M, k), float("nan"), dtype=torch.float32, device=dev)
    ti = torch.full((M, k), -1, dtype=torch.int32, device=dev)
    ws = torch.empty(max(16, cf.gemm_spec_workspace_size(spec, shape, fused)), dtype=torch.uint8, device=dev)
    cf.gemm_spec(to_dev(A), to_dev(B), Y, spec, params=[to_dev(bias)], row_out=[tv, ti], workspace=ws, fused=fused)
    torch.cuda.synchronize()
    assert cf.last_device_status() == cf.OK
    f = wl.bf16_to_f64
    Yref, (rv, ri) = spo.gemm_spec(f(A), f(B), prog.nodes, prog.terminal, [f(bias)], prog.row_outputs)
    return Y, tv.cpu().numpy(), ti.cpu().numpy(), Yref, rv, ri


def test_topk_row_outputs_exact_on_integer_data_with_ties():
    # small integers: the GEMM result is exact in bf16, so values AND columns must equal the oracle's, ties included
    g = np.random.default_rng(5)
    M, N, K = 70, 264, 16
    A = wl.f32_to_bf16_bits(g.integers(-1, 2, size=(M, K)).astype(np.float32))
    B = wl.f32_to_bf16_bits(g.integers(-2, 3, size=(K, N)).astype(np.float32))
    bias = wl.f32_to_bf16_bits(np.zeros(N, dtype=np.float32))
    Y, tv, ti, Yref, rv, ri = _run_topk(A, B, bias, 9)
    np.testing.assert_array_equal(to_f64(Y), Yref)
    np.testing.assert_array_equal(tv.astype(np.float64), rv)
    np.testing.assert_array_equal(ti.astype(np.int64), ri.astype(np.int64))
    assert (rv[:, :-1] == rv[:, 1:]).any()  # the data does contain ties


def test_topk_row_outputs_on_gaussian_data():
    M, N, K, k = 300, 1024, 136, 5
    A, B, (bias,) = _inputs(41, 1, M, N, K, ("rowvec",))
    Y, tv, ti, Yref, rv, ri = _run_topk(A, B, bias, k)
    assert np.abs(to_f64(Y) - Yref).max() <= 3e-2
    np.testing.assert_allclose(tv, rv, atol=3e-2)
    assert np.all(np.diff(tv, axis=1) <= 0)                       # falling order
    assert np.all((ti >= 0) & (ti < N)) and all(len(set(r)) == k for r in ti.tolist())
    np.testing.assert_allclose(np.take_along_axis(Yref, ti.astype(np.int64), axis=1), tv, atol=3e-2)  # the picked columns hold those values
    assert np.mean(ti == ri.astype(np.int64)) > 0.9


@pytest.mark.parametrize("M,N,K,k", [(70, 256, 16, 8), (300, 512, 16, 3), (200, 1024, 16, 8), (130, 2048, 16, 1), (257, 4096, 16, 4)])
def test_topk_on_chip_exact_on_integer_data_with_ties(M, N, K, k):
    """Top-K inside the fused kernel (K rounds of an arg max over the resident tensor, merged across the cluster): with
    small integers the GEMM result is exact, so values AND columns must equal the oracle's, ties included.  Row lengths with
    one, two, four, eight and sixteen CTAs per row block."""
    g = np.random.default_rng(50 + N)
    A = wl.f32_to_bf16_bits(g.integers(-1, 2, size=(M, K)).astype(np.float32))
    B = wl.f32_to_bf16_bits(g.integers(-2, 3, size=(K, N)).astype(np.float32))
    bias = wl.f32_to_bf16_bits(np.zeros(N, dtype=np.float32))
    prog = _topk_prog(k)
    plan = cf.spec_plan(cf.make_spec(prog.nodes, prog.terminal, 1, prog.row_outputs), cf.make_gemm_shape(1, M, N, K))
    assert plan.path == cf.SPEC_PATH_FUSED_PROGRAM     # no detour through a materialised GEMM result
    Y, tv, ti, Yref, rv, ri = _run_topk(A, B, bias, k, fused=2)
    np.testing.assert_array_equal(to_f64(Y), Yref)
    np.testing.assert_array_equal(tv.astype(np.float64), rv)
    np.testing.assert_array_equal(ti.astype(np.int64), ri.astype(np.int64))
    if k > 1:
        assert (rv[:, :-1] == rv[:, 1:]).any()  # the data does contain ties


def test_topk_on_chip_on_gaussian_data():
    M, N, K, k = 300, 1024, 136, 5
    A, B, (bias,) = _inputs(41, 1, M, N, K, ("rowvec",))
    Y, tv, ti, Yref, rv, ri = _run_topk(A, B, bias, k, fused=2)
    assert np.abs(to_f64(Y) - Yref).max() <= 3e-2
    np.testing.assert_allclose(tv, rv, atol=1e-3)                 # fp32 values, not values that went through bf16
    assert np.all(np.diff(tv, axis=1) <= 0)                       # falling order
    assert np.all((ti >= 0) & (ti < N)) and all(len(set(r)) == k for r in ti.tolist())
    np.testing.assert_allclose(np.take_along_axis(Yref, ti.astype(np.int64), axis=1), tv, atol=1e-3)
    assert np.mean(ti == ri.astype(np.int64)) > 0.99


def test_program_workload_at_bench_size_sampled_rows_and_graph_replay():
    """p1 at the size bench.py times, launched the way it launches it (captured once, replayed): sampled rows against the
    oracle, properties that hold for every row, and replay = direct launch bit for bit."""
    w = wl.config(6)
    prog, d = w.program, w.dims
    M, N, K = d["M"], d["N"], d["K"]
    dev = "cuda:0"
    spec = cf.make_spec(prog.nodes, prog.terminal, len(prog.param_kinds), prog.row_outputs)
    shape = cf.make_gemm_shape(1, M, N, K)
    assert cf.spec_plan(spec, shape).path == cf.SPEC_PATH_FUSED_PROGRAM
    A, B, p0 = to_dev(w.tensors["A"]), to_dev(w.tensors["B"]), to_dev(w.tensors["p0"])

    def outputs():
        Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev)
        ro = [torch.full((M,), -7, dtype=torch.int32 if prog.nodes[r][0] == "argmax" else torch.float32, device=dev) for r in prog.row_outputs]
        return Y, ro

    Y, ro = outputs()
    cf.gemm_spec(A, B, Y, spec, params=[p0], row_out=ro)
    torch.cuda.synchronize()
    Yg, rog = outputs()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        cf.gemm_spec(A, B, Yg, spec, params=[p0], row_out=rog)   # warm-up on the capture stream
        torch.cuda.synchronize()
        Yg.fill_(float("nan"))
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            cf.gemm_spec(A, B, Yg, spec, params=[p0], row_out=rog)
    g.replay()
    torch.cuda.synchronize()
    assert cf.last_device_status() == cf.OK
    assert torch.equal(Y.view(torch.int16), Yg.view(torch.int16))
    for a, b in zip(ro, rog):
        assert torch.equal(a, b)
    # sampled rows against the oracle
    rows = wl.sample_rows(M, 128)
    f = wl.bf16_to_f64
    Yref, Rref = spo.gemm_spec(f(w.tensors["A"][rows]), f(w.tensors["B"]), prog.nodes, prog.terminal, [f(w.tensors["p0"])], prog.row_outputs)
    err = np.abs(to_f64(Y[torch.from_numpy(rows).to(dev)]) - Yref)
    assert err.max() <= 4e-3 and err.mean() <= 1e-3, (err.max(), err.mean())
    got_rows = [t.cpu().numpy()[rows] for t in ro]
    np.testing.assert_allclose(got_rows[0], Rref[0], atol=1e-4, rtol=1e-5)
    np.testing.assert_allclose(got_rows[1], Rref[1], atol=1e-4, rtol=1e-5)
    np.testing.assert_allclose(got_rows[2], Rref[2], rtol=1e-4)
    np.testing.assert_allclose(got_rows[3], Rref[3], rtol=1e-4)
    # every row: y lies in [0, 1), is 0 at the row minimum, attains its maximum at the reported column
    Yf = Y.float()
    assert torch.isfinite(Yf).all().item() and Yf.min().item() == 0.0 and Yf.max().item() <= 1.0
    assert torch.equal(Yf.min(-1).values, torch.zeros(M, device=dev))
    picked = Yf.gather(-1, ro[4].long()[:, None])[:, 0]
    assert torch.equal(picked, Yf.max(-1).values)


@pytest.mark.parametrize("act", [None, "relu", "gelu_tanh", "tanh", "sigmoid"])
@pytest.mark.parametrize("M,N,K", [(300, 1000, 136), (520, 128, 1024), (64, 4096, 64)])
def test_reduction_free_program_runs_on_the_plain_tiling(act, M, N, K):
    """act(alpha * acc + bias) lowers to the GEMM kernel with the activation in its store epilogue: one launch, any N."""
    nodes = [("acc", -1, -1, -1, 0.0), ("const", -1, -1, -1, 0.75), ("mul", 0, 1, -1, 0.0), ("rowvec", -1, -1, 0, 0.0), ("add", 3, 2, -1, 0.0)]
    if act:
        nodes.append((act, 4, -1, -1, 0.0))
    prog = wl.SpecProgram(nodes, len(nodes) - 1, (), ("rowvec",))
    A, B, params = _inputs(51, 1, M, N, K, prog.param_kinds)
    Y, _, plan, launches = _run(prog, A, B, params, True, 1, M, N)
    assert plan.path == cf.SPEC_PATH_FUSED_KERNEL and plan.fused_kind == cf.EPI_BIAS_ACTIVATION and launches == 1
    assert plan.alpha == pytest.approx(0.75)
    Yref, _ = _oracle(prog, A, B, params, 1)
    err = np.abs(to_f64(Y) - Yref)
    scale = max(1.0, float(np.abs(Yref).max()))
    assert np.isfinite(err).all() and err.max() <= 2.0 ** -8 * scale, (err.max(), scale)   # bf16 output rounding + approximations


def test_two_layer_mlp_of_the_dlrm_shape_as_two_program_calls():
    """1024 -> 512 -> 128 with ReLU after each layer (the DLRM shape of Sec. 6.2, Table II, which has no fused B2B kernel
    here): two reduction-free program calls, the bf16 hidden layer goes through global memory."""
    M = 1000
    g = 61
    X = wl.normal_bf16(g, 0, (M, 1024))
    W1 = wl.normal_bf16(g, 1, (1024, 512), std=1024 ** -0.5)
    W2 = wl.normal_bf16(g, 2, (512, 128), std=512 ** -0.5)
    b1 = wl.uniform_bf16(g, 3, (512,), -0.1, 0.1)
    b2 = wl.uniform_bf16(g, 4, (128,), -0.1, 0.1)
    layer = wl.SpecProgram([("acc", -1, -1, -1, 0.0), ("rowvec", -1, -1, 0, 0.0), ("add", 0, 1, -1, 0.0), ("relu", 2, -1, -1, 0.0)], 3, (), ("rowvec",))
    H, _, plan1, l1 = _run(layer, X, W1, [b1], True, 1, M, 512)
    Hbits = H.view(torch.int16).cpu().numpy().view(np.uint16)
    O, _, plan2, l2 = _run(layer, Hbits, W2, [b2], True, 1, M, 128)
    assert plan1.fused_kind == plan2.fused_kind == cf.EPI_BIAS_ACTIVATION and l1 == l2 == 1
    f = wl.bf16_to_f64
    Href = np.maximum(f(X) @ f(W1) + f(b1), 0.0)
    Oref = np.maximum(Href @ f(W2) + f(b2), 0.0)
    assert np.abs(to_f64(H) - Href).max() <= 2.0 ** -8 * max(1.0, np.abs(Href).max())
    # the second layer sees the bf16-rounded hidden activations
    assert np.abs(to_f64(O) - Oref).max() <= 3e-2 and np.abs(to_f64(O) - Oref).mean() <= 3e-3
