"""Input generators: storage-format conversion, determinism and the stated distributions."""
import numpy as np
import torch

import workloads as wl


def test_bf16_round_to_nearest_even_matches_torch():
    g = np.random.default_rng(0)
    x = (g.standard_normal(100000) * 10 ** g.uniform(-6, 6, 100000)).astype(np.float32)
    bits = wl.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, ref)
    # exact ties: 1 + 2^-8 is halfway between bf16(1.0) and the next value -> rounds to even (1.0)
    tie = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8], dtype=np.float32)
    np.testing.assert_array_equal(wl.f32_to_bf16_bits(tie), [0x3F80, 0x3F82])


def test_bf16_widening_is_exact():
    bits = np.arange(0, 0x7F80, 7, dtype=np.uint16)
    f = wl.bf16_bits_to_f32(bits)
    np.testing.assert_array_equal(wl.f32_to_bf16_bits(f), bits)
    np.testing.assert_array_equal(wl.bf16_to_f64(bits), f.astype(np.float64))


def test_generators_are_deterministic_and_independent():
    a = wl.post_norm(64, 48, 32, seed=5, affine=True)
    b = wl.post_norm(64, 48, 32, seed=5, affine=True)
    for k in a.tensors:
        np.testing.assert_array_equal(a.tensors[k], b.tensors[k])
    c = wl.post_norm(64, 48, 32, seed=6, affine=True)
    assert not np.array_equal(a.tensors["A"], c.tensors["A"])
    assert not np.array_equal(a.tensors["A"][:, :32], a.tensors["residual"][:, :32])


def test_distributions_of_config_one():
    w = wl.config(0)
    assert w.dims == {"M": 256, "N": 256, "K": 256} and "gamma" not in w.tensors
    A = wl.bf16_to_f64(w.tensors["A"])
    B = wl.bf16_to_f64(w.tensors["B"])
    bias = wl.bf16_to_f64(w.tensors["bias"])
    assert abs(A.mean()) < 0.02 and abs(A.std() - 1.0) < 0.02
    assert abs(B.mean()) < 0.002 and abs(B.var() - 1.0 / 256) < 2e-4      # N(0, var 1/K)
    assert bias.min() >= -0.1001 and bias.max() <= 0.1001
    Z = A @ B
    assert abs(Z.std() - 1.0) < 0.05                                       # unit-variance GEMM output


def test_affine_and_b2b_shapes():
    w = wl.post_norm(32, 64, 16, seed=1, affine=True)
    g = wl.bf16_to_f64(w.tensors["gamma"])
    assert abs(g.mean() - 1.0) < 0.02 and g.std() < 0.05
    m = wl.b2b_mlp(256, 128, 512, 128, seed=4)
    assert m.tensors["W1"].shape == (128, 512) and m.tensors["W2"].shape == (512, 128)
    assert m.gemm_flops() == 2 * 256 * 128 * 512 * 2
    d = wl.dlrm_bottom_mlp(256, 1024, 512, 128)
    assert d.tensors["X"].shape == (256, 1024) and d.tensors["W1"].shape == (1024, 512) and d.tensors["W2"].shape == (512, 128)
    assert d.gemm_flops() == 2 * 256 * (1024 * 512 + 512 * 128)
    assert d.min_hbm_bytes() == 2 * (256 * 1024 + 1024 * 512 + 512 * 128 + 512 + 128 + 256 * 128)
    s = wl.scaled_masked_softmax(2, 128, 128, 64, seed=3)
    assert s.scalars["alpha"] == 0.125 and s.tensors["B"].shape == (2, 64, 128)


def test_min_hbm_bytes_of_named_configs_without_materialising():
    # closed-form byte counts: every operand once, every output once
    M, N, K = 8192, 768, 3072
    expect = 2 * (M * K + K * N + M * N) + 2 * (M * N + N) + 4 * N
    w = wl.Workload("x", wl.KIND_BIAS_RES_LAYERNORM, {"M": M, "N": N, "K": K}, {}, {"gamma": None})
    assert w.min_hbm_bytes() == expect
    assert abs(expect / 1e6 - 80.2) < 0.1


def test_sample_rows_covers_edges():
    r = wl.sample_rows(8192, 64)
    assert r[0] == 0 and r[-1] == 8191 and 127 in r and 128 in r and len(set(r.tolist())) == len(r)
    assert np.all(r[:-1] < r[1:])
