"""GPU parity of the two-layer ReLU MLP form of the back-to-back GEMM (the DLRM workload's shape class): the fused kernel
that streams K through the first GEMM and keeps the hidden layer on-chip, and the in-library unfused path (bf16 hidden layer
in the workspace), against the fp64 oracle."""
import os

import numpy as np
import pytest
import torch

import paper_2608_03537_b200 as cf
import workloads as wl
from tests import parity as P

pytestmark = pytest.mark.gpu

CASES = [
    # M, K, N1
    (256, 64, 256),      # one K block, one half: ML1 -> Epi1 -> ML2 -> Epi2 with nothing to overlap
    (256, 128, 512),     # two K blocks, two halves: the two slots change roles once
    (300, 1024, 512),    # the DLRM feature dimensions; ragged rows (a partial block and an empty one)
    (1000, 1000, 256),   # K not a multiple of 64: the last K block is zero-filled
    (77, 8, 256),        # the smallest K
    (2048, 192, 512),    # odd number of K blocks
    (40000, 128, 512),   # 157 tiles: up to three tiles per cluster, every slot reused in both roles
    (41000, 64, 256),    # single-half tiles alternate between the two slots
    (300, 200, 8),       # the narrowest hidden layer: all but 8 columns of the half are zero-filled
    (520, 1024, 200),    # a partial single half
    (1000, 136, 264),    # the second half holds 8 columns
    (300, 64, 384),      # one and a half halves
    (2048, 1024, 504),   # the last 8 columns missing
]


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("M,K,N1", CASES)
def test_b2b_mlp_relu(M, K, N1, fused, cuda_device):
    w = wl.dlrm_bottom_mlp(M, K, N1, 128, seed=M + K + N1)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    res = P.check_outputs(w, got, P.run_oracle(w), label=f"relu mlp M{M} K{K} N1{N1} fused={fused}")
    assert (got["Y"].float() >= 0).all().item()
    assert cf.last_device_status() == cf.OK
    print(M, K, N1, fused, res)


@pytest.mark.parametrize("fused", [True, False])
def test_dlrm_shape_full_size(fused, cuda_device):
    """32768 x (1024 -> 512 -> 128): every element against the oracle, every element finite and non-negative."""
    w = wl.config(8)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    Y = got["Y"].float()
    assert torch.isfinite(Y).all().item() and (Y >= 0).all().item()
    res = P.check_outputs(w, got, P.run_oracle(w), label=f"d1 fused={fused}")
    print("d1", fused, res)


def test_relu_mlp_without_biases_and_identity_second_layer(cuda_device):
    """b1 = b2 = NULL; W2 = the first 128 columns of I: O = ReLU(X W1)[:, :128] (ReLU of a non-negative value is itself)."""
    M, K, N1 = 512, 256, 256
    w = wl.dlrm_bottom_mlp(M, K, N1, 128, seed=11)
    T = P.dev_tensors(w)
    W2 = torch.zeros(N1, 128, dtype=torch.bfloat16, device=T["X"].device)
    W2[:128, :] = torch.eye(128, dtype=torch.bfloat16, device=W2.device)
    O = torch.full((M, 128), float("nan"), dtype=torch.bfloat16, device=W2.device)
    cf.b2b_mlp_relu(T["X"], T["W1"], None, W2, None, O, fused=True)
    ref = np.maximum(wl.bf16_to_f64(w.tensors["X"]) @ wl.bf16_to_f64(w.tensors["W1"]), 0.0)[:, :128]
    err = np.abs(P.to_f64(O) - ref)
    assert err.max() <= 3e-2 and err.mean() <= 3e-3
    # exact zeros where the hidden unit is clearly off
    assert (P.to_f64(O)[ref == 0.0] == 0.0).all()


def test_relu_mlp_bitwise_repeatable_and_equal_rows(cuda_device):
    """Run twice: same bits.  Rows are independent: the result of a row does not depend on which tile it sits in."""
    w = wl.dlrm_bottom_mlp(20000, 320, 512, 128, seed=5)
    T = P.dev_tensors(w)
    a = P.run_gpu(w, T, fused=True)["Y"]
    b = P.run_gpu(w, T, fused=True)["Y"]
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    X2 = T["X"][19000:19300].contiguous()       # the same rows as their own problem
    O2 = torch.empty(300, 128, dtype=torch.bfloat16, device=X2.device)
    cf.b2b_mlp_relu(X2, T["W1"], T["b1"], T["W2"], T["b2"], O2, fused=True)
    assert torch.equal(O2.view(torch.int16), a[19000:19300].view(torch.int16))


def test_relu_mlp_argument_checks(cuda_device):
    dev = "cuda:0"
    X = torch.zeros(256, 64, dtype=torch.bfloat16, device=dev)
    W1 = torch.zeros(64, 640, dtype=torch.bfloat16, device=dev)
    W2 = torch.zeros(640, 128, dtype=torch.bfloat16, device=dev)
    O = torch.zeros(256, 128, dtype=torch.bfloat16, device=dev)
    with pytest.raises(cf.ComfuseError) as e:     # N1 = 640: more than the two halves of 256 columns tensor memory holds
        cf.b2b_mlp_relu(X, W1, None, W2, None, O, fused=True)
    assert e.value.status == cf.ERR_UNSUPPORTED
    ws = torch.empty(256 * 640 * 2, dtype=torch.uint8, device=dev)
    cf.b2b_mlp_relu(X, W1, None, W2, None, O, fused=False, workspace=ws)   # ... but runs unfused
    assert cf.last_device_status() == cf.OK
    with pytest.raises(cf.ComfuseError) as e:     # unfused without its workspace
        cf.b2b_mlp_relu(X, W1, None, W2, None, O, fused=False)
    assert e.value.status == cf.ERR_WORKSPACE


def test_relu_mlp_random_shapes(cuda_device):
    """Seeded random shapes (M 1 .. 3000 and a few beyond one wave of clusters, K any multiple of 8 up to 1536, N1 any
    multiple of 8 up to 512), fused kernel against the oracle; the unfused path on every fourth shape.  COMFUSE_FUZZ_SEEDS lengthens the sweep."""
    rng = np.random.default_rng(20240)
    worst = 0.0
    for i in range(int(os.environ.get("COMFUSE_FUZZ_SEEDS", 60))):
        M = int(rng.integers(1, 3001)) if i % 10 else int(rng.integers(19000, 60000))
        K = 8 * int(rng.integers(1, 193))
        N1 = 256 * int(rng.integers(1, 3)) if i % 3 else 8 * int(rng.integers(1, 65))
        w = wl.dlrm_bottom_mlp(M, K, N1, 128, seed=1000 + i)
        T = P.dev_tensors(w)
        ref = P.run_oracle(w)
        res = P.check_outputs(w, P.run_gpu(w, T, fused=True), ref, label=f"random relu mlp #{i} M{M} K{K} N1{N1}")
        worst = max(worst, res["max_abs"])
        if i % 4 == 0:
            P.check_outputs(w, P.run_gpu(w, T, fused=False), ref, label=f"random relu mlp unfused #{i} M{M} K{K} N1{N1}")
    assert cf.last_device_status() == cf.OK
    print("worst max-abs", worst)


@pytest.mark.parametrize("M", [600, 9000])
def test_relu_mlp_host_buffers_match_device_buffers(M, cuda_device):
    """X and O in pinned host memory (M = 9000 x K = 1024 is 18 MB of activations: the call runs as a pipeline of row ranges):
    bit for bit the device-pointer call."""
    w = wl.dlrm_bottom_mlp(M, 1024, 512, 128, seed=31)
    T = P.dev_tensors(w)
    ref = P.run_gpu(w, T, fused=True)["Y"]
    hX = T["X"].cpu().pin_memory()
    hO = torch.empty(M, 128, dtype=torch.bfloat16).pin_memory()
    desc = cf.make_b2b_desc(M, 1024, 512, 128, 0.0, True, cf.B2B_MLP_RELU)
    staging = torch.empty(cf.b2b_host_staging_size(desc), dtype=torch.uint8, device=T["X"].device)
    for _ in range(2):
        cf.b2b_mlp_relu_host(hX, T["W1"], T["b1"], T["W2"], T["b2"], hO, staging=staging)
    torch.cuda.synchronize()
    assert torch.equal(hO.view(torch.int16), ref.cpu().view(torch.int16))
    assert cf.last_device_status() == cf.OK


def test_relu_mlp_back_to_back_dependent_launches(cuda_device):
    """The kernel is launched with programmatic stream serialization (its set-up may overlap the previous kernel's tail; it
    waits for that kernel before it touches global memory).  A chain in which every call consumes the previous call's
    output, enqueued without synchronisation, gives bit for bit what the chain gives with a synchronisation per call."""
    M, K, N1 = 3000, 128, 512
    w = wl.dlrm_bottom_mlp(M, K, N1, 128, seed=41)
    T = P.dev_tensors(w)
    dev = T["X"].device
    W2 = (T["W2"].float() * 4.0).to(torch.bfloat16)          # keeps the activations from dying out along the chain

    def chain(sync):
        x = T["X"].clone()                                    # [M, 128]; N2 == K so the output can feed the next call
        bufs = [torch.empty(M, 128, dtype=torch.bfloat16, device=dev) for _ in range(2)]
        for i in range(10):
            y = bufs[i & 1]
            cf.b2b_mlp_relu(x, T["W1"], T["b1"], W2, T["b2"], y, fused=True)
            if sync:
                torch.cuda.synchronize()
            x = y
        torch.cuda.synchronize()
        return x.clone()

    a = chain(sync=True)
    assert a.float().abs().max().item() > 0
    for _ in range(3):
        b = chain(sync=False)
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    assert cf.last_device_status() == cf.OK


_SCHEDULE_CHILD = r"""
import sys, numpy as np, torch
import workloads as wl
from tests import parity as P
import paper_2608_03537_b200 as cf
out = {}
for name, (M, K) in (("many_tiles", (40000, 128)), ("dlrm_dims", (300, 1024)), ("odd_blocks", (2048, 192))):
    w = wl.dlrm_bottom_mlp(M, K, 512, 128, seed=M + K)
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label=name)
    assert cf.last_device_status() == cf.OK
    out[name] = got["Y"].view(torch.int16).cpu().numpy()
np.savez(sys.argv[1], **out)
"""


def test_both_schedules_for_two_halves_agree_bit_for_bit(tmp_path, cuda_device):
    """N1 = 512 runs with both halves in lock-step by default; COMFUSE_B2B_STREAM_LOCK=0 (read once per process, hence the
    child processes) selects the alternating-slot schedule that N1 = 256 always uses.  Both accumulate every output element in
    the same order: same bits, and each is checked against the oracle in its child."""
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = {}
    for flag in ("1", "0"):
        path = str(tmp_path / f"s{flag}.npz")
        env = dict(os.environ, COMFUSE_B2B_STREAM_LOCK=flag, PYTHONPATH=root)
        r = subprocess.run([sys.executable, "-c", _SCHEDULE_CHILD, path], cwd=root, env=env, capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, r.stderr[-2000:]
        res[flag] = np.load(path)
    assert sorted(res["0"].files) == sorted(res["1"].files) and len(res["0"].files) == 3
    for k in res["0"].files:
        assert np.array_equal(res["0"][k], res["1"][k]), k


def test_relu_mlp_million_rows_sampled(cuda_device):
    """A million ragged rows (3907 tiles, 53 per CTA pair): sampled rows against the oracle, everything finite."""
    M, K, N1 = 1_000_003, 64, 512
    w = wl.dlrm_bottom_mlp(M, K, N1, 128, seed=77)
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    assert torch.isfinite(got["Y"].float()).all().item()
    rows = np.unique(np.concatenate([wl.sample_rows(M, 600), np.arange(M - 300, M)]))
    P.check_outputs(w, got, P.run_oracle(w, rows=rows), rows=rows, label="relu mlp 1e6 rows")
    assert cf.last_device_status() == cf.OK
