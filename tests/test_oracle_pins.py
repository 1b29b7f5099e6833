"""Pins for the fp64 oracle: everything here runs on the CPU and compares the oracle with something
other than itself -- hand-computed numbers, closed forms, invariants, pure-Python brute force written
from the definitions with scalar loops, and library routines used only as special-case cross-checks."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import comfuse_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


# ----------------------------------------------------------------------------- GEMM
def _read_gemm_cases():
    cases, cur = [], {}
    with open(os.path.join(GOLDEN, "gemm_small_integer.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            tag, r, c, *vals = line.split()
            cur[tag] = np.array([float(v) for v in vals]).reshape(int(r), int(c))
            if tag == "Z":
                cases.append(cur)
                cur = {}
    return cases


def test_gemm_hand_computed_integers():
    cases = _read_gemm_cases()
    assert len(cases) == 3
    for c in cases:
        np.testing.assert_array_equal(orc.gemm(c["A"], c["B"]), c["Z"])


def test_gemm_brute_force_loops():
    g = _rng(1)
    A = g.integers(-4, 5, size=(5, 7)).astype(np.float64)
    B = g.integers(-4, 5, size=(7, 6)).astype(np.float64)
    Z = np.zeros((5, 6))
    for i in range(5):
        for j in range(6):
            s = 0.0
            for k in range(7):
                s += A[i, k] * B[k, j]
            Z[i, j] = s
    np.testing.assert_array_equal(orc.gemm(A, B), Z)


def test_gemm_identity_and_associativity():
    g = _rng(2)
    B = g.standard_normal((9, 11))
    np.testing.assert_array_equal(orc.gemm(np.eye(9), B), B)
    X, W1, W2 = g.standard_normal((6, 8)), g.standard_normal((8, 10)), g.standard_normal((10, 4))
    np.testing.assert_allclose(orc.gemm(orc.gemm(X, W1), W2), orc.gemm(X, orc.gemm(W1, W2)), rtol=0, atol=1e-12)


def test_gemm_batched_matches_per_batch():
    g = _rng(3)
    A, B = g.standard_normal((3, 4, 5)), g.standard_normal((3, 5, 6))
    Z = orc.gemm(A, B)
    for b in range(3):
        np.testing.assert_allclose(Z[b], orc.gemm(A[b], B[b]), rtol=0, atol=1e-14)


# ----------------------------------------------------------------------------- GELU
def test_gelu_tabulated_values():
    with open(os.path.join(GOLDEN, "gelu_tanh_values.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    assert len(rows) == 8
    for x, gx, tol in rows:
        assert abs(float(orc.gelu_tanh(np.array(float(x)))) - float(gx)) <= float(tol), x


def test_gelu_identities_and_limits():
    x = np.linspace(-8, 8, 4001)
    G = orc.gelu_tanh(x)
    np.testing.assert_allclose(G - orc.gelu_tanh(-x), x, rtol=0, atol=1e-14)   # G(x) - G(-x) = x
    assert orc.gelu_tanh(np.array(0.0)) == 0.0
    big = np.array([6.0, 8.0, 20.0])
    np.testing.assert_allclose(orc.gelu_tanh(big), big, rtol=0, atol=1e-9)
    small = orc.gelu_tanh(-big)
    assert np.all(small <= 0) and np.all(small > -1e-9)
    # the function has one minimum near x = -0.75 with value about -0.17
    i = int(np.argmin(G))
    assert -0.80 < x[i] < -0.70 and -0.171 < G[i] < -0.169


def test_gelu_library_special_case():
    x = torch.linspace(-6, 6, 1001, dtype=torch.float64)
    ref = torch.nn.functional.gelu(x, approximate="tanh").numpy()
    np.testing.assert_allclose(orc.gelu_tanh(x.numpy()), ref, rtol=0, atol=1e-14)


# ----------------------------------------------------------------------------- LayerNorm
def test_layernorm_ramp_closed_form():
    with open(os.path.join(GOLDEN, "layernorm_ramp.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for n, mean, var in rows:
        n, mean, var = int(n), float(mean), float(var)
        eps = 1e-5
        x = np.arange(1, n + 1, dtype=np.float64)[None, :]
        expect = (x - mean) / math.sqrt(var + eps)
        np.testing.assert_allclose(orc.layernorm_rows(x, eps=eps), expect, rtol=0, atol=1e-12)


def test_layernorm_invariants():
    g = _rng(4)
    H = g.standard_normal((17, 96)) * 3.0 + 5.0
    eps = 1e-5
    Y = orc.layernorm_rows(H, eps=eps)
    var = H.var(axis=-1)   # numpy's biased variance, an independent computation
    np.testing.assert_allclose(Y.mean(axis=-1), 0.0, atol=1e-12)
    np.testing.assert_allclose(Y.var(axis=-1), var / (var + eps), rtol=1e-12)
    # shift / positive-scale invariance as eps -> 0
    Y0 = orc.layernorm_rows(H, eps=0.0)
    np.testing.assert_allclose(orc.layernorm_rows(2.5 * H - 7.0, eps=0.0), Y0, rtol=0, atol=1e-11)
    # affine is a row-vector broadcast applied after normalisation
    gamma, beta = g.standard_normal(96), g.standard_normal(96)
    np.testing.assert_allclose(orc.layernorm_rows(H, gamma, beta, eps), Y * gamma[None, :] + beta[None, :], atol=1e-13)


def test_layernorm_brute_force_and_library():
    g = _rng(5)
    H = g.standard_normal((4, 9))
    gamma, beta = g.standard_normal(9), g.standard_normal(9)
    eps = 1e-3
    out = np.zeros_like(H)
    for i in range(4):
        mu = sum(H[i, j] for j in range(9)) / 9
        var = sum((H[i, j] - mu) ** 2 for j in range(9)) / 9
        for j in range(9):
            out[i, j] = (H[i, j] - mu) / math.sqrt(var + eps) * gamma[j] + beta[j]
    np.testing.assert_allclose(orc.layernorm_rows(H, gamma, beta, eps), out, rtol=0, atol=1e-13)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(H), (9,), torch.from_numpy(gamma), torch.from_numpy(beta), eps)
    np.testing.assert_allclose(orc.layernorm_rows(H, gamma, beta, eps), ref.numpy(), rtol=0, atol=1e-12)


# ----------------------------------------------------------------------------- RMSNorm
def test_rmsnorm_constant_row_and_identity():
    eps = 1e-5
    for c in (0.5, -3.0, 7.0):
        Y = orc.rmsnorm_rows(np.full((2, 33), c), eps=eps)
        np.testing.assert_allclose(Y, c / math.sqrt(c * c + eps), rtol=1e-14)
    g = _rng(6)
    H = g.standard_normal((11, 40)) * 2
    gain = g.standard_normal(40) + 3.0
    Y = orc.rmsnorm_rows(H, gain, eps)
    ms = np.mean(H * H, axis=-1)
    np.testing.assert_allclose(((Y / gain) ** 2).sum(-1), 40 * ms / (ms + eps), rtol=1e-12)
    # no mean subtraction: adding a constant changes the result
    assert np.abs(orc.rmsnorm_rows(H + 1.0, gain, eps) - Y).max() > 1e-2


def test_rmsnorm_library_special_case():
    g = _rng(7)
    H, gain = g.standard_normal((5, 24)), g.standard_normal(24)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(H), (24,), torch.from_numpy(gain), 1e-4).numpy()
    np.testing.assert_allclose(orc.rmsnorm_rows(H, gain, 1e-4), ref, rtol=0, atol=1e-12)


# ----------------------------------------------------------------------------- softmax
def test_softmax_rows_sum_to_one_shift_invariance():
    g = _rng(8)
    T = g.standard_normal((13, 50)) * 4
    P = orc.softmax_rows(T)
    np.testing.assert_allclose(P.sum(-1), 1.0, rtol=0, atol=1e-12)
    np.testing.assert_allclose(orc.softmax_rows(T + 123.0), P, rtol=0, atol=1e-13)
    assert np.all(P > 0)
    ref = torch.softmax(torch.from_numpy(T), dim=-1).numpy()
    np.testing.assert_allclose(P, ref, rtol=0, atol=1e-14)


def test_softmax_causal_zero_scores_is_uniform():
    n = 12
    A = np.zeros((n, 4))
    B = np.zeros((4, n))
    P = orc.scale_mask_softmax(A, B, alpha=0.125, mask=orc.causal_mask(n, n))
    assert P[0, 0] == 1.0
    for i in range(n):
        np.testing.assert_allclose(P[i, : i + 1], 1.0 / (i + 1), rtol=1e-15)
        assert np.all(P[i, i + 1:] == 0.0)        # masked entries are exactly zero


def test_softmax_fully_masked_row_is_zero():
    T = np.array([[0.0, 1.0, 2.0], [-np.inf, -np.inf, -np.inf], [-np.inf, 0.0, -np.inf]])
    P = orc.softmax_rows(T)
    assert np.all(P[1] == 0.0)
    np.testing.assert_array_equal(P[2], [0.0, 1.0, 0.0])
    np.testing.assert_allclose(P[0].sum(), 1.0, atol=1e-15)


def test_softmax_brute_force_with_scale_and_mask():
    g = _rng(9)
    A, B = g.standard_normal((6, 5)), g.standard_normal((5, 6))
    alpha = 0.37
    P = orc.scale_mask_softmax(A, B, alpha=alpha, mask=orc.causal_mask(6, 6))
    for i in range(6):
        t = []
        for j in range(6):
            s = sum(A[i, k] * B[k, j] for k in range(5)) * alpha
            t.append(s if j <= i else -math.inf)
        m = max(t)
        e = [math.exp(v - m) if v != -math.inf else 0.0 for v in t]
        z = sum(e)
        np.testing.assert_allclose(P[i], [v / z for v in e], rtol=0, atol=1e-14)


def test_causal_mask_row_subset():
    full = orc.causal_mask(9, 9)
    rows = np.array([0, 4, 8])
    np.testing.assert_array_equal(orc.causal_mask(9, 9, rows=rows), full[rows])


# ----------------------------------------------------------------------------- max / argmax
def test_row_max_argmax_spike_and_ties():
    g = _rng(10)
    Y = g.standard_normal((7, 64))
    cols = [0, 63, 17, 17, 5, 40, 1]
    for i, c in enumerate(cols):
        Y[i, c] = 100.0 + i
    mx, am = orc.row_max_argmax(Y)
    np.testing.assert_array_equal(am, cols)
    np.testing.assert_array_equal(mx, 100.0 + np.arange(7))
    T = np.array([[1.0, 3.0, 3.0, 2.0], [5.0, 5.0, 5.0, 5.0]])
    _, am = orc.row_max_argmax(T)
    np.testing.assert_array_equal(am, [1, 0])   # lowest index on ties


# ----------------------------------------------------------------------------- whole op lists vs scalar brute force
def _gelu_scalar(x):
    return 0.5 * x * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (x + 0.044715 * x ** 3)))


def test_bias_res_layernorm_brute_force():
    g = _rng(11)
    M, N, K = 4, 6, 5
    A, B = g.standard_normal((M, K)), g.standard_normal((K, N))
    bias, R = g.standard_normal(N), g.standard_normal((M, N))
    gamma, beta = g.standard_normal(N), g.standard_normal(N)
    alpha, eps = 0.7, 1e-5
    out = np.zeros((M, N))
    for i in range(M):
        h = [alpha * sum(A[i, k] * B[k, j] for k in range(K)) + bias[j] + R[i, j] for j in range(N)]
        mu = sum(h) / N
        var = sum((v - mu) ** 2 for v in h) / N
        for j in range(N):
            out[i, j] = (h[j] - mu) / math.sqrt(var + eps) * gamma[j] + beta[j]
    np.testing.assert_allclose(orc.bias_res_layernorm(A, B, bias, R, gamma, beta, alpha, eps), out, rtol=0, atol=1e-12)


def test_bias_gelu_res_rmsnorm_max_brute_force():
    g = _rng(12)
    M, N, K = 3, 7, 4
    A, B = g.standard_normal((M, K)), g.standard_normal((K, N))
    bias, R, gain = g.standard_normal(N), g.standard_normal((M, N)), g.standard_normal(N) + 2
    eps = 1e-5
    Y, mx, am = orc.bias_gelu_res_rmsnorm_max(A, B, bias, R, gain, 1.0, eps)
    for i in range(M):
        h = [_gelu_scalar(sum(A[i, k] * B[k, j] for k in range(K)) + bias[j]) + R[i, j] for j in range(N)]
        ms = sum(v * v for v in h) / N
        y = [h[j] / math.sqrt(ms + eps) * gain[j] for j in range(N)]
        np.testing.assert_allclose(Y[i], y, rtol=0, atol=1e-13)
        assert mx[i] == pytest.approx(max(y), abs=1e-13)
        assert am[i] == y.index(max(y))


def test_b2b_equals_two_step_and_brute_force():
    g = _rng(13)
    M, K, N1 = 5, 4, 9
    X, W1, W2 = g.standard_normal((M, K)), g.standard_normal((K, N1)), g.standard_normal((N1, K))
    b1, b2 = g.standard_normal(N1), g.standard_normal(K)
    gamma, beta = g.standard_normal(K), g.standard_normal(K)
    eps = 1e-5
    O = orc.b2b_mlp_layernorm(X, W1, b1, W2, b2, gamma, beta, eps)
    S = orc.b2b_intermediate(X, W1, b1)
    np.testing.assert_allclose(orc.b2b_from_intermediate(S, X, W2, b2, gamma, beta, eps), O, rtol=0, atol=1e-13)
    for i in range(M):
        s = [_gelu_scalar(sum(X[i, k] * W1[k, n] for k in range(K)) + b1[n]) for n in range(N1)]
        o = [sum(s[n] * W2[n, j] for n in range(N1)) + b2[j] + X[i, j] for j in range(K)]
        mu = sum(o) / K
        var = sum((v - mu) ** 2 for v in o) / K
        expect = [(o[j] - mu) / math.sqrt(var + eps) * gamma[j] + beta[j] for j in range(K)]
        np.testing.assert_allclose(O[i], expect, rtol=0, atol=1e-12)


def test_b2b_identity_second_weight_reduces_to_post_norm():
    g = _rng(14)
    M, K = 6, 8
    X, W1, b1 = g.standard_normal((M, K)), g.standard_normal((K, K)), g.standard_normal(K)
    O = orc.b2b_mlp_layernorm(X, W1, b1, np.eye(K), np.zeros(K), eps=1e-5)
    expect = orc.layernorm_rows(orc.gelu_tanh(X @ W1 + b1) + X, eps=1e-5)
    np.testing.assert_allclose(O, expect, rtol=0, atol=1e-13)


# ----------------------------------------------------------------------------- partial-statistic merges
@pytest.mark.parametrize("splits", [[5, 95], [32, 32, 36], [1, 1, 98], [25, 25, 25, 25], [64, 36]])
def test_welford_merge_any_split(splits):
    g = _rng(15)
    x = g.standard_normal((9, 100)) * 3 + 10
    acc, o = None, 0
    for s in splits:
        part = orc.welford_partial(x[:, o:o + s])
        acc = part if acc is None else orc.welford_merge(acc, part)
        o += s
    n, mean, m2 = acc
    assert n == 100
    np.testing.assert_allclose(mean, x.mean(-1), rtol=0, atol=1e-12)
    np.testing.assert_allclose(m2 / n, x.var(-1), rtol=1e-12)


@pytest.mark.parametrize("splits", [[5, 95], [32, 32, 36], [50, 50], [99, 1]])
def test_softmax_merge_any_split(splits):
    g = _rng(16)
    x = g.standard_normal((9, 100)) * 5
    x[3, 60:] = -np.inf           # a fully masked partial in some splits
    x[4, :50] = -np.inf
    acc, o = None, 0
    for s in splits:
        part = orc.softmax_partial(x[:, o:o + s])
        acc = part if acc is None else orc.softmax_merge(acc, part)
        o += s
    m, l = acc
    np.testing.assert_allclose(m, x.max(-1), rtol=0, atol=0)
    P = orc.softmax_rows(x)
    with np.errstate(invalid="ignore"):
        np.testing.assert_allclose(np.where(np.isneginf(x), 0.0, np.exp(x - m[:, None])) / l[:, None], P, rtol=0, atol=1e-13)


# ----------------------------------------------------------------------------- the Sec. 6.1 pattern variants
def test_layernorm_relu_variant_brute_force_and_sign():
    """MatMul-BiasAdd-LayerNorm-ReLU: scalar-loop brute force; every output is >= 0 and equals the plain result where
    that is positive (so the ReLU sits after the affine step, not before the normalisation)."""
    r = _rng(40)
    A, B = r.standard_normal((5, 7)), r.standard_normal((7, 6))
    bias, gamma, beta = r.standard_normal(6), r.standard_normal(6), r.standard_normal(6)
    eps = 1e-5
    want = np.zeros((5, 6))
    for i in range(5):
        h = [sum(A[i, k] * B[k, j] for k in range(7)) + bias[j] for j in range(6)]
        mu = sum(h) / 6
        var = sum((x - mu) ** 2 for x in h) / 6
        for j in range(6):
            y = (h[j] - mu) / math.sqrt(var + eps) * gamma[j] + beta[j]
            want[i, j] = y if y > 0 else 0.0
    got = orc.bias_res_layernorm(A, B, bias, None, gamma, beta, 1.0, eps, relu=True)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    plain = orc.bias_res_layernorm(A, B, bias, None, gamma, beta, 1.0, eps)
    assert (got >= 0).all() and (got[plain > 0] == plain[plain > 0]).all() and (got[plain <= 0] == 0).all()
    assert (plain < 0).any()          # the case actually exercises the clamp


def test_rmsnorm_without_activation_is_bias_rmsnorm():
    """MatMul-BiasAdd-RMSNorm: with the activation off and no residual the op list is RMSNorm(A.B + bias) * g:
    brute force, and the identity sum_j (Y_j / g_j)^2 = N * ms / (ms + eps)."""
    r = _rng(41)
    A, B, bias, g = r.standard_normal((4, 9)), r.standard_normal((9, 8)), r.standard_normal(8), r.uniform(0.5, 1.5, 8)
    eps = 1e-3
    Y, mx, am = orc.bias_gelu_res_rmsnorm_max(A, B, bias, None, g, 1.0, eps, activation=False)
    for i in range(4):
        z = [sum(A[i, k] * B[k, j] for k in range(9)) + bias[j] for j in range(8)]
        ms = sum(x * x for x in z) / 8
        row = [z[j] / math.sqrt(ms + eps) * g[j] for j in range(8)]
        np.testing.assert_allclose(Y[i], row, rtol=0, atol=1e-12)
        assert abs(sum((row[j] / g[j]) ** 2 for j in range(8)) - 8 * ms / (ms + eps)) < 1e-12
        assert mx[i] == max(row) and am[i] == row.index(max(row))
    with_act = orc.bias_gelu_res_rmsnorm_max(A, B, bias, None, g, 1.0, eps)[0]
    assert np.abs(with_act - Y).max() > 1e-2      # the switch does something


def test_softcap_softmax_bounds_limit_and_library():
    """MatMul-Scale-TanhSoftcap-Softmax.  (1) brute force with math.tanh / math.exp; (2) the capped scores lie in
    (-c, c), so no two probabilities of a row differ by more than a factor e^(2c); (3) c -> infinity recovers the
    plain softmax; (4) library cross-check in fp64; (5) the mask applies after the cap: masked entries are exactly 0."""
    r = _rng(42)
    A, B = 3.0 * r.standard_normal((6, 5)), 3.0 * r.standard_normal((5, 7))
    alpha, c = 0.7, 2.0
    P = orc.scale_mask_softmax(A, B, alpha, None, softcap=c)
    for i in range(6):
        t = [c * math.tanh(alpha * sum(A[i, k] * B[k, j] for k in range(5)) / c) for j in range(7)]
        m = max(t)
        e = [math.exp(x - m) for x in t]
        np.testing.assert_allclose(P[i], [x / sum(e) for x in e], rtol=0, atol=1e-14)
    assert (P.max(-1) / P.min(-1) < math.exp(2 * c)).all()
    plain = orc.scale_mask_softmax(A, B, alpha, None)
    assert (plain.max(-1) / plain.min(-1)).max() > math.exp(2 * c)        # uncapped rows exceed the bound: the cap matters
    np.testing.assert_allclose(orc.scale_mask_softmax(A, B, alpha, None, softcap=1e9), plain, rtol=0, atol=1e-12)
    Z = torch.from_numpy(A) @ torch.from_numpy(B) * alpha
    lib = torch.softmax(c * torch.tanh(Z / c), dim=-1).numpy()
    np.testing.assert_allclose(P, lib, rtol=0, atol=1e-14)
    Pm = orc.scale_mask_softmax(A[:, :5], B[:, :6], alpha, orc.causal_mask(6, 6), softcap=c)
    assert (Pm[np.triu_indices(6, 1)] == 0).all() and np.allclose(Pm.sum(-1), 1.0, atol=1e-12) and Pm[0, 0] == 1.0


# ----------------------------------------------------------------------------- B2B with a reduction as F (attention form)
def test_b2b_softmax_attention_brute_force_and_properties():
    """Scalar-loop brute force; zero queries attend uniformly (every output row is the mean of the value rows); every output
    lies inside the per-column range of V (rows of softmax are convex weights); a key that dominates one query's scores
    makes that query's output its value row; batched call equals per-batch calls; library cross-check in fp64."""
    r = _rng(50)
    Q, Kt, V = r.standard_normal((5, 4)), r.standard_normal((4, 6)), r.standard_normal((6, 3))
    alpha = 0.5
    O = orc.b2b_softmax_attention(Q, Kt, V, alpha)
    for i in range(5):
        s = [alpha * sum(Q[i, k] * Kt[k, j] for k in range(4)) for j in range(6)]
        m = max(s)
        e = [math.exp(x - m) for x in s]
        pr = [x / sum(e) for x in e]
        for c in range(3):
            assert abs(O[i, c] - sum(pr[j] * V[j, c] for j in range(6))) < 1e-13
    np.testing.assert_allclose(orc.b2b_softmax_attention(np.zeros((2, 4)), Kt, V, alpha), np.tile(V.mean(0), (2, 1)), atol=1e-14)
    assert (O >= V.min(0) - 1e-12).all() and (O <= V.max(0) + 1e-12).all()
    Kd = Kt.copy()
    Kd[:, 2] = 50.0 * Q[1] / np.dot(Q[1], Q[1])          # query 1 . key 2 = 50 / alpha-scaled: dominates that row
    Od = orc.b2b_softmax_attention(Q, Kd, V, 1.0)
    np.testing.assert_allclose(Od[1], V[2], atol=1e-9)
    Qb, Kb, Vb = r.standard_normal((3, 5, 4)), r.standard_normal((3, 4, 6)), r.standard_normal((3, 6, 3))
    Ob = orc.b2b_softmax_attention(Qb, Kb, Vb, alpha)
    for b in range(3):
        np.testing.assert_allclose(Ob[b], orc.b2b_softmax_attention(Qb[b], Kb[b], Vb[b], alpha), atol=1e-14)
    lib = torch.softmax(torch.from_numpy(Q) @ torch.from_numpy(Kt) * alpha, dim=-1) @ torch.from_numpy(V)
    np.testing.assert_allclose(O, lib.numpy(), atol=1e-13)


def test_b2b_mlp_relu_brute_force_and_properties():
    """The ReLU two-layer MLP (Sec. 4, Eq. 2 with F = ReLU(. + b1) and a ReLU tail; the DLRM workload of Sec. 6.2).
    Scalar-loop brute force; a hand-computed 2 x 2 case with one clipped unit per layer; outputs are non-negative; without
    biases the map is positively homogeneous (f(aX) = a f(X) for a > 0); a large positive b1 keeps every hidden unit active,
    which reduces the hidden layer to an affine map; W2 = I, b2 = 0 leaves ReLU(X W1 + b1); library cross-check in fp64."""
    r = _rng(60)
    X, W1, b1 = r.standard_normal((5, 7)), r.standard_normal((7, 6)), r.standard_normal(6)
    W2, b2 = r.standard_normal((6, 3)), r.standard_normal(3)
    O = orc.b2b_mlp_relu(X, W1, b1, W2, b2)
    for i in range(5):
        s = [max(sum(X[i, k] * W1[k, j] for k in range(7)) + b1[j], 0.0) for j in range(6)]
        for c in range(3):
            assert abs(O[i, c] - max(sum(s[j] * W2[j, c] for j in range(6)) + b2[c], 0.0)) < 1e-13
    # hand-computed: X = [[1, -2]], W1 = [[1, 2], [3, 1]] -> P = [-5, 0]; + b1 = [6, -1] -> [1, -1] -> S = [1, 0];
    # W2 = [[2, -3], [5, 7]] -> [2, -3]; + b2 = [0.5, 1] -> [2.5, -2] -> O = [2.5, 0]
    Oh = orc.b2b_mlp_relu([[1.0, -2.0]], [[1.0, 2.0], [3.0, 1.0]], [6.0, -1.0], [[2.0, -3.0], [5.0, 7.0]], [0.5, 1.0])
    np.testing.assert_array_equal(Oh, [[2.5, 0.0]])
    assert (O >= 0.0).all() and (O == 0.0).any() and (O > 0.0).any()
    z6, z3 = np.zeros(6), np.zeros(3)
    np.testing.assert_allclose(orc.b2b_mlp_relu(3.5 * X, W1, z6, W2, z3), 3.5 * orc.b2b_mlp_relu(X, W1, z6, W2, z3), atol=1e-12)
    big = np.full(6, 100.0)
    np.testing.assert_allclose(orc.b2b_mlp_relu(X, W1, big, W2, b2), np.maximum((X @ W1 + big) @ W2 + b2, 0.0), atol=1e-11)
    np.testing.assert_allclose(orc.b2b_mlp_relu(X, W1, b1, np.eye(6), z6), np.maximum(X @ W1 + b1, 0.0), atol=1e-14)
    lin = torch.nn.functional.linear
    tX, tW1, tW2 = torch.from_numpy(X), torch.from_numpy(W1), torch.from_numpy(W2)
    lib = torch.relu(lin(torch.relu(lin(tX, tW1.T, torch.from_numpy(b1))), tW2.T, torch.from_numpy(b2)))
    np.testing.assert_allclose(O, lib.numpy(), atol=1e-13)
