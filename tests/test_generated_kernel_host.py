"""The kernel generated for a program, as far as it goes without a GPU: the run-time compiler is found, a program's kernel
compiles for sm_100a (the device image is made on the host; only loading it needs a device), and the requests the pathway
refuses are refused by status code."""
import os
import subprocess
import sys

import pytest

import paper_2608_03537_b200 as cf
import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _spec(prog):
    return cf.make_spec(prog.nodes, prog.terminal, len(prog.param_kinds), prog.row_outputs)


@pytest.fixture
def compiler():
    st, why = cf.program_compiler_status()
    if st != cf.OK:
        pytest.skip(f"no run-time compiler on this machine: {why}")


def test_compiler_status_names_what_is_missing():
    st, why = cf.program_compiler_status()
    assert (st == cf.OK and why == "") or (st == cf.ERR_UNSUPPORTED and len(why) > 10)


@pytest.mark.parametrize("N", [256, 768, 4096])
def test_a_chain_program_compiles_for_every_kind_of_instantiation(compiler, N):
    prog = wl.spec_range_normalise()
    cf.gemm_spec_prepare(_spec(prog), cf.make_gemm_shape(1, 300, N, 64), cf.GENERATED)
    assert cf.gemm_spec_workspace_size(_spec(prog), cf.make_gemm_shape(1, 300, N, 64), cf.GENERATED) == 0


def test_topk_program_compiles(compiler):
    nodes = [("acc", -1, -1, -1, 0.0), ("relu", 0, -1, -1, 0.0), ("topk_values", 1, -1, 8, 0.0), ("topk_indices", 1, -1, 8, 0.0)]
    prog = wl.SpecProgram(nodes, 1, (2, 3), ())
    cf.gemm_spec_prepare(_spec(prog), cf.make_gemm_shape(1, 300, 1024, 64), cf.GENERATED)


def test_requests_the_pathway_refuses(compiler):
    N_ = ("acc", -1, -1, -1, 0.0)     # a full tensor used behind a reduction: no on-chip lowering
    dag = wl.SpecProgram([N_, ("mean", 0, -1, -1, 0.0), ("sub", 0, 1, -1, 0.0), ("tensor", -1, -1, 0, 0.0), ("add", 2, 3, -1, 0.0)], 4, (),
                         ("tensor",))
    with pytest.raises(cf.ComfuseError) as e:
        cf.gemm_spec_prepare(_spec(dag), cf.make_gemm_shape(1, 300, 1024, 64), cf.GENERATED)
    assert e.value.status == cf.ERR_UNSUPPORTED
    chain = wl.spec_range_normalise()
    with pytest.raises(cf.ComfuseError) as e:   # a row length without an instantiation
        cf.gemm_spec_prepare(_spec(chain), cf.make_gemm_shape(1, 300, 1000, 64), cf.GENERATED)
    assert e.value.status == cf.ERR_UNSUPPORTED
    with pytest.raises(cf.ComfuseError) as e:
        cf.gemm_spec_prepare(_spec(chain), cf.make_gemm_shape(1, 300, 1024, 64), 4)
    assert e.value.status == cf.ERR_INVALID_ARG
    with pytest.raises(cf.ComfuseError) as e:
        cf.gemm_spec_workspace_size(_spec(chain), cf.make_gemm_shape(1, 300, 1024, 64), 4)
    assert e.value.status == cf.ERR_INVALID_ARG
    # the other pathways have nothing to prepare
    for fused in (0, 1, 2):
        cf.gemm_spec_prepare(_spec(chain), cf.make_gemm_shape(1, 300, 1024, 64), fused)


def test_without_a_toolkit_the_pathway_says_so():
    """A child process that is pointed at an empty toolkit directory and cannot see the default one reports UNSUPPORTED with
    the reason; nothing falls back silently."""
    # the default location is compiled in; the child can only check the reason string when the toolkit is absent there
    if os.path.exists("/usr/local/cuda/lib64/libnvrtc.so.12"):
        pytest.skip("the default toolkit location exists on this machine: the library finds it whatever the environment says")
    r = subprocess.run([sys.executable, "-c", "import paper_2608_03537_b200 as cf; print(cf.program_compiler_status())"],
                       cwd=ROOT, capture_output=True, text=True, env=dict(os.environ, CUDA_HOME="/nonexistent"))
    assert r.returncode == 0 and "not found" in r.stdout


def test_two_computed_tensors_meet_in_generated_code_only(compiler, monkeypatch):
    """relu(x) * tanh(x): the first factor waits in a temporary while the second is computed -- registers of the generated
    kernel; the interpreter has none, so `fused` = 2 plans the row program and `fused` = 1 the on-chip form."""
    N_ = ("acc", -1, -1, -1, 0.0)
    nodes = [N_, ("rowvec", -1, -1, 0, 0.0), ("add", 0, 1, -1, 0.0), ("relu", 2, -1, -1, 0.0), ("tanh", 2, -1, -1, 0.0),
             ("mul", 3, 4, -1, 0.0), ("rmax", 5, -1, -1, 0.0), ("sub", 5, 6, -1, 0.0)]
    prog = wl.SpecProgram(nodes, 7, (6,), ("rowvec",))
    shape = cf.make_gemm_shape(1, 300, 1024, 64)
    plan = cf.spec_plan(_spec(prog), shape)
    assert plan.path == cf.SPEC_PATH_FUSED_PROGRAM and plan.program_path == cf.SPEC_PATH_ROW_PROGRAM
    cf.gemm_spec_prepare(_spec(prog), shape, cf.GENERATED)
    monkeypatch.setenv("COMFUSE_GENERATE", "0")
    assert cf.spec_plan(_spec(prog), shape).path == cf.SPEC_PATH_ROW_PROGRAM


def test_the_generated_translation_unit_can_be_dumped(compiler, tmp_path, monkeypatch):
    path = tmp_path / "generated.cu"
    monkeypatch.setenv("COMFUSE_GENERATED_DUMP", str(path))
    nodes = [("acc", -1, -1, -1, 0.0), ("const", -1, -1, -1, 0.37), ("mul", 0, 1, -1, 0.0), ("abs", 2, -1, -1, 0.0),
             ("rmax", 3, -1, -1, 0.0), ("sub", 3, 4, -1, 0.0)]
    prog = wl.SpecProgram(nodes, 5, (4,), ())
    cf.gemm_spec_prepare(_spec(prog), cf.make_gemm_shape(1, 300, 512, 64), cf.GENERATED)
    text = path.read_text()
    assert "kCompiledProgram" in text and "fused_pair_kernel<comfuse::EPI_PROGRAM, 256, 256, 1, 3, 1, 2>" in text
    assert "0.37" not in text            # constants stay run-time arguments: programs that differ only in them share the kernel


def test_device_images_can_be_kept_on_disk(compiler, tmp_path):
    """COMFUSE_KERNEL_CACHE=<directory>: a second process finds the image the first one compiled (the generated translation
    unit is dumped only when a kernel is actually compiled, so the second process leaves no dump behind)."""
    cache = tmp_path / "cache"
    cache.mkdir()
    code = (
        "import sys, paper_2608_03537_b200 as cf, workloads as wl\n"
        "p = wl.spec_range_normalise()\n"
        "spec = cf.make_spec(p.nodes, p.terminal, len(p.param_kinds), p.row_outputs)\n"
        "cf.gemm_spec_prepare(spec, cf.make_gemm_shape(1, 300, 2048, 64), cf.GENERATED)\n"
    )
    for dump in ("first.cu", "second.cu"):
        env = dict(os.environ, COMFUSE_KERNEL_CACHE=str(cache), COMFUSE_GENERATED_DUMP=str(tmp_path / dump),
                   PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
        r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
        assert r.returncode == 0, r.stderr[-2000:]
    files = [f for f in os.listdir(cache) if f.endswith(".cubin")]
    assert len(files) == 1 and os.path.getsize(cache / files[0]) > 10_000
    assert (tmp_path / "first.cu").exists() and not (tmp_path / "second.cu").exists()
    # a damaged file is ignored (and replaced by a fresh compilation), not trusted
    with open(cache / files[0], "r+b") as f:
        f.write(b"garbage")
    env = dict(os.environ, COMFUSE_KERNEL_CACHE=str(cache), COMFUSE_GENERATED_DUMP=str(tmp_path / "third.cu"),
               PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and (tmp_path / "third.cu").exists()
