"""Cross-CTA aggregation modes of the row statistics (Sec. 3.1): leader-follower must give the same bits as all-to-all,
because both merge the CTAs' partials in rank order.  The mode is read once per process, so each mode runs in a child."""
import os
import subprocess
import sys

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys, numpy as np, torch
import workloads as wl
from tests.parity import dev_tensors, run_gpu
import paper_2608_03537_b200 as cf
out = {}
for name, w in (("ln", wl.post_norm(M=520, N=2048, K=264, seed=7, affine=True)),
                ("rms", wl.complex_subgraph(M=392, N=4096, K=136, seed=8)),
                ("sm", wl.scaled_masked_softmax(batch=2, M=512, N=512, K=320, seed=9))):
    got = run_gpu(w, dev_tensors(w))
    torch.cuda.synchronize()
    assert cf.last_device_status() == cf.OK
    for k, v in got.items():
        out[name + "_" + k] = v.view(torch.int16).cpu().numpy() if v.dtype == torch.bfloat16 else v.cpu().numpy()
np.savez(sys.argv[1], **out)
"""


def _run(mode, path):
    env = dict(os.environ, COMFUSE_REDUCE_MODE=mode, PYTHONPATH=ROOT)
    r = subprocess.run([sys.executable, "-c", CHILD, path], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    return np.load(path)


def test_leader_follower_aggregation_equals_all_to_all_bit_for_bit(tmp_path):
    a = _run("all2all", str(tmp_path / "a.npz"))
    b = _run("leader", str(tmp_path / "b.npz"))
    assert sorted(a.files) == sorted(b.files) and len(a.files) >= 5
    for k in a.files:
        x, y = a[k], b[k]
        if x.dtype.kind == "f":
            x, y = x.view(np.int32), y.view(np.int32)
        assert np.array_equal(x, y), k
