"""The checked build of the library (-DCOMFUSE_CHECKED).

In that build every kernel evaluates a predicate in front of its global stores -- the coordinates of the output TMA stores,
the indices of the row-statistic and partial-statistic writes -- and a predicate that fails records a bit in the device
status word and skips the access (nothing traps).  The ordinary build compiles the predicates out.  Here a child process
loads the checked library in place of the ordinary one (COMFUSE_LIB), runs one case of every kernel family against the fp64
oracle, and requires the status word to stay clear; the predicate machinery itself is exercised by a self-test kernel whose
predicate is false by construction and whose access is therefore skipped.
"""
import os
import subprocess
import sys

import pytest

import paper_2608_03537_b200 as cf
from paper_2608_03537_b200 import build as cf_build

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CHECKED_LIB = os.path.join(os.path.dirname(cf_build.LIB_PATH), "libcomfuse_checked.so")

CHILD = r"""
import torch
import paper_2608_03537_b200 as cf
import workloads as wl
from tests import parity as P

assert cf.LIB_PATH.endswith("libcomfuse_checked.so"), cf.LIB_PATH
torch.cuda.set_device(0)
assert cf.selftest_bounds_predicate() is True
assert cf.last_device_status() == cf.ERR_BOUNDS       # recorded, and cleared by the read
assert cf.last_device_status() == cf.OK
cases = [
    wl.post_norm(300, 768, 200, seed=11, affine=True),
    wl.complex_subgraph(150, 4096, 128, seed=12),
    wl.scaled_masked_softmax(2, 2048, 2048, 64, seed=13),
    wl.scaled_masked_softmax(1, 1024, 1024, 320, seed=15),
    wl.b2b_mlp(512, 128, 512, 128, seed=14),
    wl.target_attention(2, 300, 256, 128, seed=16),
    wl.dlrm_bottom_mlp(600, 320, 512, 128, seed=18),
    wl.post_norm(130, 8192, 64, seed=17, affine=True, relu=True),
    wl.config(1),
]
for i, w in enumerate(cases):
    for fused in (True, False):
        got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
        assert cf.last_device_status() == cf.OK, (w.name, fused)
        if i + 1 < len(cases):   # the full-size case: status word only (its parity is covered by the ordinary build)
            P.check_outputs(w, got, P.run_oracle(w), label=f"{w.name} fused={fused}", rowmax_tol=5e-3 if fused else 3e-2,
                            softmax_tol=P.TOL_SOFTMAX_MAX if fused else P.TOL_SOFTMAX_UNFUSED,
                            norm_tol=P.TOL_NORM_MAX if fused else 4e-2)
# an epilogue program on the interpreter and as a generated kernel (compiled with the predicates as well)
import numpy as np
from oracle import fusion_spec_oracle as spo
prog = wl.spec_range_normalise()
M, N, K = 300, 1024, 72
A = wl.normal_bf16(21, 0, (M, K)); B = wl.normal_bf16(21, 1, (K, N), std=K ** -0.5); bias = wl.normal_bf16(21, 2, (N,), std=0.1)
f = wl.bf16_to_f64
Yref, Rref = spo.gemm_spec(f(A), f(B), prog.nodes, prog.terminal, [f(bias)], prog.row_outputs)
spec = cf.make_spec(prog.nodes, prog.terminal, 1, prog.row_outputs)
modes = [2] + ([cf.GENERATED] if cf.program_compiler_status()[0] == cf.OK else [])
for fused in modes:
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda:0")
    ro = [torch.zeros(M, dtype=torch.int32 if prog.nodes[r][0] == "argmax" else torch.float32, device="cuda:0") for r in prog.row_outputs]
    cf.gemm_spec(P.to_dev(A), P.to_dev(B), Y, spec, params=[P.to_dev(bias)], row_out=ro, fused=fused)
    torch.cuda.synchronize()
    assert cf.last_device_status() == cf.OK, ("program", fused)
    assert float(np.abs(P.to_f64(Y) - Yref).max()) <= 4e-3, ("program", fused)
print("checked build ok")
"""


def test_ordinary_build_has_no_predicates(cuda_device):
    if cf.LIB_PATH.endswith("libcomfuse_checked.so"):
        pytest.skip("the checked library is loaded in this process")
    assert cf.selftest_bounds_predicate() is False
    assert cf.last_device_status() == cf.OK


def test_checked_build_runs_every_kernel_family_with_a_clear_status_word(cuda_device):
    try:
        cf_build.build(checked=True)     # incremental: nothing happens when the library is up to date
    except Exception as e:               # no nvcc on this machine: a library that came with the tree will do
        if not os.path.exists(CHECKED_LIB):
            pytest.skip(f"checked library not built: {e}")
    env = dict(os.environ, COMFUSE_LIB=CHECKED_LIB, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    r = subprocess.run([sys.executable, "-c", CHILD], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "checked build ok" in r.stdout
