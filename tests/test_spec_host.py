"""Host-side analysis of epilogue programs (no GPU): validation, typing, stage numbering at the reductions (Sec. 5.3),
canonicalisation onto the fused instantiations in any operand order (Sec. 5.4), liveness-based buffer assignment of
the row program."""
import pytest

import paper_2608_03537_b200 as cf
import workloads as wl

SHAPE = cf.make_gemm_shape(1, 512, 1024, 256)


def _plan(nodes, terminal, n_params=0, row_outputs=(), shape=SHAPE):
    return cf.spec_plan(cf.make_spec(nodes, terminal, n_params, row_outputs), shape)


def _status(nodes, terminal, n_params=0, row_outputs=(), shape=SHAPE):
    with pytest.raises(cf.ComfuseError) as e:
        _plan(nodes, terminal, n_params, row_outputs, shape)
    return e.value.status


N_ = ("acc", -1, -1, -1, 0.0)


def test_stage_numbering_follows_the_reductions():
    assert _plan([N_], 0).n_stages == 1
    assert _plan([N_, ("relu", 0, -1, -1, 0)], 1).n_stages == 1
    p = wl.spec_layernorm()
    assert _plan(p.nodes, p.terminal, 4).n_stages == 3          # x | x - mean | normalise
    p = wl.spec_softmax(0.5)
    assert _plan(p.nodes, p.terminal).n_stages == 3             # max | sum of exp | scale
    p = wl.spec_rmsnorm_max()
    pl = _plan(p.nodes, p.terminal, 3, p.row_outputs)
    assert pl.n_stages == 3 and pl.n_reductions == 3            # mean square | max and arg max of Y (same stage)
    p = wl.spec_gated_minmax()
    pl = _plan(p.nodes, p.terminal, 1, p.row_outputs)
    assert pl.n_stages == 2 and pl.n_reductions == 3            # three independent reductions share one boundary


def test_dead_nodes_are_not_counted():
    nodes = [N_, ("exp", 0, -1, -1, 0), ("sum", 1, -1, -1, 0), ("relu", 0, -1, -1, 0)]
    pl = _plan(nodes, 3)
    assert pl.n_live_nodes == 2 and pl.n_reductions == 0 and pl.n_stages == 1 and pl.n_instructions == 1


def test_constants_are_folded_on_the_host():
    # y = acc * (1 / sqrt(4))  ->  one instruction, no per-row arithmetic
    nodes = [N_, ("const", -1, -1, -1, 4.0), ("rsqrt", 1, -1, -1, 0), ("mul", 0, 2, -1, 0)]
    pl = _plan(nodes, 3)
    assert pl.n_instructions == 1 and pl.n_slots == 1


@pytest.mark.parametrize("prog,n_params,kind,flags", [
    (wl.spec_layernorm(), 4, cf.EPI_BIAS_RES_LAYERNORM, 0),
    (wl.spec_layernorm(relu=True, residual=False), 3, cf.EPI_BIAS_RES_LAYERNORM, cf.FLAG_POST_RELU),
    (wl.spec_layernorm(bias=False, residual=False, affine=False), 0, cf.EPI_BIAS_RES_LAYERNORM, 0),
    (wl.spec_rmsnorm_max(), 3, cf.EPI_BIAS_GELU_RES_RMSNORM_MAX, 0),
    (wl.spec_rmsnorm_max(activation=False, residual=False), 2, cf.EPI_BIAS_GELU_RES_RMSNORM_MAX, cf.FLAG_NO_ACTIVATION),
    (wl.spec_softmax(0.125), 0, cf.EPI_SCALE_MASK_SOFTMAX, 0),
])
def test_primitive_spellings_lower_to_the_fused_kernels(prog, n_params, kind, flags):
    pl = _plan(prog.nodes, prog.terminal, n_params, prog.row_outputs)
    assert pl.path == cf.SPEC_PATH_FUSED_KERNEL and pl.fused_kind == kind and pl.fused_flags == flags


def _swap_commutative(nodes):
    return [(op, b, a, p, i) if op in ("add", "mul") else (op, a, b, p, i) for (op, a, b, p, i) in nodes]


@pytest.mark.parametrize("prog,n_params", [(wl.spec_layernorm(relu=True), 4), (wl.spec_rmsnorm_max(), 3), (wl.spec_softmax(0.3, False, 5.0), 0)])
def test_operand_order_of_commutative_nodes_does_not_matter(prog, n_params):
    a = _plan(prog.nodes, prog.terminal, n_params, prog.row_outputs)
    b = _plan(_swap_commutative(prog.nodes), prog.terminal, n_params, prog.row_outputs)
    assert a.path == b.path == cf.SPEC_PATH_FUSED_KERNEL and a.fused_kind == b.fused_kind and a.fused_flags == b.fused_flags


def test_recovered_constants():
    p = wl.spec_softmax(alpha=0.125, causal=True, softcap=30.0)
    pl = _plan(p.nodes, p.terminal, shape=cf.make_gemm_shape(4, 1024, 1024, 64))
    assert pl.path == cf.SPEC_PATH_FUSED_KERNEL and pl.causal == 1
    assert pl.alpha == pytest.approx(0.125) and pl.softcap == pytest.approx(30.0)
    p = wl.spec_layernorm(eps=3e-4)
    assert _plan(p.nodes, p.terminal, 4).eps == pytest.approx(3e-4)


@pytest.mark.parametrize("generate", [False, True])
def test_near_misses_do_not_take_a_compiled_kind(generate, monkeypatch):
    """With COMFUSE_GENERATE=0 an on-chip program is interpreted, and the cost model sends exponential-heavy three-pass
    programs to the row program; run as generated code (the default where the run-time compiler is there) they stay on-chip."""
    if generate and cf.program_compiler_status()[0] != cf.OK:
        pytest.skip("no run-time compiler on this machine")
    monkeypatch.setenv("COMFUSE_GENERATE", "1" if generate else "0")
    PROG = cf.SPEC_PATH_FUSED_PROGRAM
    ROW = PROG if generate else cf.SPEC_PATH_ROW_PROGRAM
    # residual added INSIDE the activation: not the compiled RMSNorm entry, but still one resident tensor -> on-chip interpreter
    g = [N_, ("rowvec", -1, -1, 0, 0), ("add", 0, 1, -1, 0), ("tensor", -1, -1, 1, 0), ("add", 2, 3, -1, 0), ("gelu_tanh", 4, -1, -1, 0),
         ("square", 5, -1, -1, 0), ("mean", 6, -1, -1, 0), ("const", -1, -1, -1, 1e-5), ("add", 7, 8, -1, 0), ("rsqrt", 9, -1, -1, 0),
         ("mul", 5, 10, -1, 0)]
    assert _plan(g, 11, 2).path == PROG
    # soft-cap whose two constants are not reciprocal
    p = wl.spec_softmax(0.5, False, 2.0)
    nodes = [(op, a, b, q, 0.7 if (op == "const" and abs(i - 0.5) < 1e-9 and k > 1) else i) for k, (op, a, b, q, i) in enumerate(p.nodes)]
    pl = _plan(nodes, p.terminal)
    assert pl.path == ROW and pl.program_path == PROG   # exponential-heavy, three passes: the cost model prefers the row program
    # LayerNorm with an extra row output
    p = wl.spec_layernorm()
    assert _plan(p.nodes, p.terminal, 4, (p.nodes.index(("mean", 4, -1, -1, 0.0)),)).path == PROG
    # causal softmax on a non-square problem: no compiled softmax kind; both interpreters can run it, and the cost model
    # sends the exponential-heavy three-pass program to the row program
    p = wl.spec_softmax(0.5, True)
    pl = _plan(p.nodes, p.terminal, shape=cf.make_gemm_shape(1, 256, 512, 64))
    assert pl.path == ROW and pl.program_path == PROG
    # a row length without an on-chip instantiation: the compiled LayerNorm kind takes it as two kernels (256-column tiles,
    # a partial last one); a program outside the compiled kinds has no on-chip form there and goes to the row program
    p = wl.spec_layernorm()
    assert _plan(p.nodes, p.terminal, 4, shape=cf.make_gemm_shape(1, 256, 1000, 64)).path == cf.SPEC_PATH_FUSED_KERNEL
    p = wl.spec_range_normalise()
    assert _plan(p.nodes, p.terminal, 1, p.row_outputs, shape=cf.make_gemm_shape(1, 256, 1000, 64)).path == cf.SPEC_PATH_ROW_PROGRAM


def test_on_chip_lowering_needs_one_resident_tensor():
    PROG, ROW = cf.SPEC_PATH_FUSED_PROGRAM, cf.SPEC_PATH_ROW_PROGRAM
    # compiled kinds are also expressible on-chip (what `fused` = 2 runs), with one pass per stage that reads x
    for prog, n_params, passes in ((wl.spec_layernorm(relu=True), 4, 3), (wl.spec_rmsnorm_max(), 3, 2), (wl.spec_softmax(0.2, True, 3.0), 0, 3)):
        pl = _plan(prog.nodes, prog.terminal, n_params, prog.row_outputs, shape=cf.make_gemm_shape(1, 1024, 1024, 64))
        assert pl.path == cf.SPEC_PATH_FUSED_KERNEL and pl.program_path == PROG and pl.n_passes == passes
    # x * sigmoid(x): a computed tensor meets the resident tensor itself (a gate) -> x = acc + bias stays resident and the
    # gate is a chain with x as its operand, recomputed where a later stage reads it
    p = wl.spec_gated_minmax()
    pl = _plan(p.nodes, p.terminal, 1, p.row_outputs)
    assert pl.path == PROG and pl.program_path == PROG and pl.n_passes == 2
    # relu(x) * tanh(x): two COMPUTED tensors meet in one node -> the first waits in a temporary, which only a kernel
    # generated for the program has (registers); the interpreter sends it to the row program
    nodes = [N_, ("rowvec", -1, -1, 0, 0), ("add", 0, 1, -1, 0), ("relu", 2, -1, -1, 0), ("tanh", 2, -1, -1, 0), ("mul", 3, 4, -1, 0),
             ("rmax", 5, -1, -1, 0), ("sub", 5, 6, -1, 0)]
    pl = _plan(nodes, 7, 1)
    assert pl.program_path == ROW
    assert pl.path == (PROG if cf.program_compiler_status()[0] == cf.OK else ROW)
    # no reduction at all: act(acc + bias) is a compiled reduction-free kind (the plain GEMM's tiling, any N); on the
    # interpreter it is a single pass
    pl = _plan([N_, ("rowvec", -1, -1, 0, 0), ("add", 0, 1, -1, 0), ("relu", 2, -1, -1, 0)], 3, 1)
    assert pl.path == cf.SPEC_PATH_FUSED_KERNEL and pl.fused_kind == cf.EPI_BIAS_ACTIVATION and pl.program_path == PROG and pl.n_passes == 1
    pl = _plan([N_, ("rowvec", -1, -1, 0, 0), ("add", 0, 1, -1, 0), ("relu", 2, -1, -1, 0)], 3, 1, shape=cf.make_gemm_shape(1, 300, 1000, 72))
    assert pl.path == cf.SPEC_PATH_FUSED_KERNEL and pl.program_path == ROW          # any row length
    # two element-wise steps behind the bias: not that kind, still one resident tensor
    pl = _plan([N_, ("rowvec", -1, -1, 0, 0), ("add", 0, 1, -1, 0), ("relu", 2, -1, -1, 0), ("square", 3, -1, -1, 0)], 4, 1)
    assert pl.path == PROG and pl.n_passes == 1
    # a reduction of something below the tensor the later stages read (max of the raw accumulator, x = acc + bias used later):
    # the accumulator itself stays resident and acc + bias is recomputed from it
    nodes = [N_, ("rowvec", -1, -1, 0, 0), ("add", 0, 1, -1, 0), ("rmax", 0, -1, -1, 0), ("mean", 2, -1, -1, 0), ("sub", 2, 4, -1, 0),
             ("mul", 5, 3, -1, 0)]
    pl = _plan(nodes, 6, 1)
    assert pl.path == PROG and pl.n_passes == 2
    # four row vectors: more than the kernel stages in shared memory
    nodes = [N_] + [("rowvec", -1, -1, q, 0) for q in range(4)] + [("add", 0, 1, -1, 0), ("mul", 5, 2, -1, 0), ("add", 6, 3, -1, 0), ("mul", 7, 4, -1, 0)]
    assert _plan(nodes, 8, 4).path == ROW
    # a full tensor used after a reduction (the operand ring delivers it in pass 0 only)
    nodes = [N_, ("mean", 0, -1, -1, 0), ("sub", 0, 1, -1, 0), ("tensor", -1, -1, 0, 0), ("add", 2, 3, -1, 0)]
    assert _plan(nodes, 4, 1).path == ROW


def test_row_program_reuses_buffers_by_liveness():
    p = wl.spec_layernorm(relu=True)
    spec = cf.make_spec(p.nodes, p.terminal, 4)
    # forced row program: x, x - mean and its square are the only tensors alive together
    assert cf.gemm_spec_workspace_size(spec, SHAPE, fused=False) == 512 * 1024 * 2
    chain = [N_] + [("relu", k, -1, -1, 0) for k in range(20)]
    pl = _plan(chain, 20)
    assert pl.n_instructions == 20 and pl.n_slots == 1           # a chain runs in place
    p = wl.spec_gated_minmax()
    assert _plan(p.nodes, p.terminal, 1, p.row_outputs).n_slots == 2


def test_malformed_programs_are_rejected():
    INV = cf.ERR_INVALID_ARG
    assert _status([N_, ("add", 0, 2, -1, 0), ("const", -1, -1, -1, 1.0)], 1) == INV          # forward edge
    assert _status([N_, ("add", 0, -1, -1, 0)], 1) == INV                                      # missing operand
    assert _status([N_, (99, 0, -1, -1, 0)], 1) == INV                                         # outside the vocabulary
    assert _status([N_, ("relu", 0, 0, -1, 0)], 1) == INV                                      # unary with two inputs
    assert _status([N_, ("rowvec", -1, -1, 0, 0)], 1, n_params=0) == INV                       # parameter slot out of range
    assert _status([N_, ("rowvec", -1, -1, 0, 0), ("tensor", -1, -1, 0, 0), ("add", 1, 2, -1, 0)], 3, n_params=1) == INV  # one slot, two shapes
    assert _status([N_], 1) == INV                                                             # terminal out of range
    assert _status([N_, ("relu", 0, -1, -1, 0)], 1, row_outputs=(1,)) == INV                   # row output must be per-row
    assert _status([N_], 0, shape=cf.make_gemm_shape(1, 64, 100, 64)) == cf.ERR_ALIGNMENT      # N not a multiple of 8
    assert _status([("acc", 0, -1, -1, 0)], 0) == INV                                          # entry node with an input


def test_topk_nodes_are_row_outputs_only(monkeypatch):
    monkeypatch.setenv("COMFUSE_GENERATE", "0")   # the path expected below is the cost model's choice for interpreted programs
    INV = cf.ERR_INVALID_ARG
    tk = ("topk_values", 0, -1, 4, 0.0)
    assert _plan([N_, tk], 0, row_outputs=(1,)).path == cf.SPEC_PATH_ROW_PROGRAM
    assert _plan([N_, tk], 0, row_outputs=(1,)).n_stages == 2
    assert _status([N_, tk], 1) == INV                                           # cannot be the terminal
    assert _status([N_, tk, ("relu", 1, -1, -1, 0)], 2) == INV                   # cannot feed a node
    assert _status([N_, ("topk_values", 0, -1, 0, 0.0)], 0, row_outputs=(1,)) == INV    # K >= 1
    assert _status([N_, ("topk_indices", 0, -1, 65, 0.0)], 0, row_outputs=(1,)) == INV  # K <= 64
    assert _status([N_, ("topk_values", 0, -1, 40, 0.0)], 0, row_outputs=(1,), shape=cf.make_gemm_shape(1, 64, 32, 64)) == INV  # K <= N


def test_random_node_lists_never_crash_the_analysis():
    """Fuzz: arbitrary op codes, edges, parameter indices and terminals are either accepted or rejected with a status --
    and whatever is accepted can be planned on every pathway selector and sized."""
    import ctypes
    import numpy as np
    g = np.random.default_rng(123)
    codes = sorted(cf.OPS.values()) + [5, 15, 28, 31, 38, 47, 56, 99, -1]
    L = cf.lib()
    accepted = 0
    for _ in range(3000):
        n = int(g.integers(1, 20))
        nodes = [(0, -1, -1, -1, 0.0)]
        for k in range(1, n):
            op = int(g.choice(sorted(cf.OPS.values())))
            a = int(g.integers(0, k)) if op >= 16 else -1
            b = int(g.integers(0, k)) if 32 <= op <= 37 else -1
            prm = int(g.integers(0, 3)) if op in (2, 3) else (int(g.integers(1, 9)) if op in (54, 55) else -1)
            nodes.append((op, a, b, prm, float(g.normal())))
        if g.random() < 0.4:   # corrupt one field of one node
            k = int(g.integers(0, n))
            f = list(nodes[k])
            f[int(g.integers(0, 4))] = int(g.choice(codes)) if g.random() < 0.5 else int(g.integers(-3, n + 3))
            nodes[k] = tuple(f)
        n_params = int(g.integers(2, 5))
        terminal = int(g.integers(-1, n + 1)) if g.random() < 0.2 else int(g.integers(0, n))
        ro = tuple(int(x) for x in g.integers(0, n, size=int(g.integers(0, 3))))
        spec = cf.make_spec(nodes, terminal, n_params, ro)
        shape = cf.make_gemm_shape(1, int(g.integers(1, 600)), int(g.choice([64, 256, 768, 1000, 4096, 12])), int(g.integers(1, 40)) * 8)
        plan = cf.SpecPlan()
        st = L.comfuse_spec_plan(ctypes.byref(spec), ctypes.byref(shape), ctypes.byref(plan))
        assert st in (cf.OK, cf.ERR_INVALID_ARG, cf.ERR_UNSUPPORTED, cf.ERR_ALIGNMENT), st
        for fused in (0, 1, 2):
            nbytes = ctypes.c_size_t(0)
            st2 = L.comfuse_gemm_spec_workspace_size(ctypes.byref(spec), ctypes.byref(shape), fused, ctypes.byref(nbytes))
            assert st2 in (cf.OK, cf.ERR_INVALID_ARG, cf.ERR_UNSUPPORTED, cf.ERR_ALIGNMENT), st2
            if st in (cf.ERR_INVALID_ARG, cf.ERR_ALIGNMENT):
                assert st2 == st
        if st == cf.OK:
            accepted += 1
            assert plan.n_stages >= 1 and plan.n_live_nodes >= 1
            assert plan.path in (cf.SPEC_PATH_FUSED_KERNEL, cf.SPEC_PATH_ROW_PROGRAM, cf.SPEC_PATH_FUSED_PROGRAM)
    assert accepted > 20
