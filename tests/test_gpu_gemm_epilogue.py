"""GPU parity: the fused kernels and the in-library unfused path against the fp64 oracle, element by element, on
seeded inputs small enough for the oracle to finish in seconds yet spanning several tiles, clusters of 1, 2, 4 and 8
CTAs, ragged row-block tails and K tails."""
import numpy as np
import pytest
import torch

import paper_2608_03537_b200 as cf
import workloads as wl
from tests import parity as P

pytestmark = pytest.mark.gpu

LN_SHAPES = [
    (256, 256, 256),    # the tiny post-norm configuration: 2 row blocks, 1 CTA per block
    (300, 768, 200),    # 2-CTA cluster, ragged M (300 = 2*128 + 44), K tail (200 = 3*64 + 8)
    (130, 512, 72),     # single CTA, 512 TMEM columns
    (257, 1024, 128),   # 2-CTA cluster of 512 columns
    (200, 2048, 96),    # 4-CTA cluster
    (200, 4096, 128),   # 8-CTA cluster, TMEM completely full
    (1, 256, 8),        # degenerate: one row, one 16-byte K line
]


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("M,N,K", LN_SHAPES)
def test_layernorm_epilogue(M, N, K, fused, cuda_device):
    w = wl.post_norm(M, N, K, seed=M + N + K, affine=(N != 256))
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    P.check_outputs(w, got, P.run_oracle(w), label=f"LN {M}x{N}x{K} fused={fused}")


def test_layernorm_without_bias_or_residual(cuda_device):
    w = wl.post_norm(200, 768, 128, seed=9, affine=True)
    del w.tensors["bias"], w.tensors["residual"]
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label="LN no bias/residual")


def test_layernorm_alpha_and_padded_leading_dims(cuda_device):
    """alpha != 1 and leading dimensions larger than the row length (strided views)."""
    import paper_2608_03537_b200 as cf
    from oracle import comfuse_oracle as orc
    w = wl.post_norm(260, 768, 136, seed=21, affine=True)
    T = P.dev_tensors(w)
    dev = T["A"].device
    Abig = torch.zeros(260, 136 + 24, dtype=torch.bfloat16, device=dev); Abig[:, :136] = T["A"]
    Bbig = torch.zeros(136, 768 + 8, dtype=torch.bfloat16, device=dev); Bbig[:, :768] = T["B"]
    Rbig = torch.zeros(260, 768 + 16, dtype=torch.bfloat16, device=dev); Rbig[:, :768] = T["residual"]
    Ybig = torch.full((260, 768 + 32), 7.0, dtype=torch.bfloat16, device=dev)
    A, B, R, Y = Abig[:, :136], Bbig[:, :768], Rbig[:, :768], Ybig[:, :768]
    cf.gemm_epilogue(A, B, Y, cf.EPI_BIAS_RES_LAYERNORM, bias=T["bias"], residual=R, gamma=T["gamma"], beta=T["beta"],
                     alpha=0.5, eps=1e-3, fused=True)
    ref = orc.bias_res_layernorm(P.f64(w, "A"), P.f64(w, "B"), P.f64(w, "bias"), P.f64(w, "residual"), P.f64(w, "gamma"),
                                 P.f64(w, "beta"), 0.5, 1e-3)
    err = np.abs(P.to_f64(Y) - ref)
    assert err.max() <= P.TOL_NORM_MAX and err.mean() <= P.TOL_NORM_MEAN
    assert (Ybig[:, 768:] == 7.0).all()      # the pad columns of the output were not touched


RMS_SHAPES = [(300, 256, 200), (140, 768, 64), (200, 1024, 128), (150, 4096, 128)]


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("M,N,K", RMS_SHAPES)
def test_gelu_rmsnorm_max_epilogue(M, N, K, fused, cuda_device):
    w = wl.complex_subgraph(M, N, K, seed=M + N)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    P.check_outputs(w, got, P.run_oracle(w), label=f"RMS {M}x{N}x{K} fused={fused}",
                    rowmax_tol=5e-3 if fused else 3e-2)


WIDE_SHAPES = [(300, 8192, 72), (129, 12288, 64)]   # rows wider than the largest cluster (16 CTAs x 256 columns)


@pytest.mark.parametrize("M,N,K", WIDE_SHAPES)
def test_layernorm_wide_rows_two_kernel_path(M, N, K, cuda_device):
    """fused = 1 with N > 4096 and a short contraction: per-4096-column-block stage 1 with partial statistics, then the
    normalising kernel.  The row leaves the chip once as fp16 before it is normalised, so the fused tolerance holds."""
    import paper_2608_03537_b200 as cf
    w = wl.post_norm(M, N, K, seed=N + K, affine=True)
    T = P.dev_tensors(w)
    desc = cf.make_gemm_desc(T["A"], T["B"], torch.empty(M, N, dtype=torch.bfloat16, device=T["A"].device),
                             cf.EPI_BIAS_RES_LAYERNORM, residual=T["residual"], fused=True)
    assert cf.workspace_size(desc) == M * (N // 4096) * 8      # one (mean, M2) pair per row and block
    got = P.run_gpu(w, T, fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label=f"LN wide {M}x{N}x{K}")


@pytest.mark.parametrize("M,N,K", WIDE_SHAPES)
def test_gelu_rmsnorm_max_wide_rows_two_kernel_path(M, N, K, cuda_device):
    w = wl.complex_subgraph(M, N, K, seed=M + N)
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label=f"RMS wide {M}x{N}x{K}", rowmax_tol=3e-2)


@pytest.mark.parametrize("M,N,K", [(300, 8192, 1024), (260, 6144, 1088), (129, 5120, 1024)])
def test_wide_rows_behind_a_long_contraction_run_in_256_column_tiles(M, N, K, cuda_device):
    """N > 4096 with K >= 1024: the first kernel works in 256-column tiles on every SM instead of 4096-column blocks on clusters
    of sixteen (one partial per row and tile), which also covers row lengths that are multiples of 256 but not of 4096."""
    import paper_2608_03537_b200 as cf
    w = wl.post_norm(M, N, K, seed=N + K, affine=True)
    T = P.dev_tensors(w)
    desc = cf.make_gemm_desc(T["A"], T["B"], torch.empty(M, N, dtype=torch.bfloat16, device=T["A"].device),
                             cf.EPI_BIAS_RES_LAYERNORM, residual=T["residual"], fused=True)
    assert cf.workspace_size(desc) == M * (N // 256) * 8
    got = P.run_gpu(w, T, fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label=f"LN wide 256-tiles {M}x{N}x{K}")
    w = wl.complex_subgraph(M, N, K, seed=M + N)
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label=f"RMS wide 256-tiles {M}x{N}x{K}", rowmax_tol=3e-2)


@pytest.mark.parametrize("M,N,K", [(300, 1536, 200), (129, 1280, 520), (1100, 1280, 2056), (260, 1792, 136), (4100, 1536, 72), (520, 1792, 1032)])
def test_on_chip_forms_on_clusters_of_six_ten_and_fourteen_ctas(M, N, K, cuda_device):
    """1536, 1280 and 1792 columns: three, five and seven column ranges per row block.  Which of these shapes run on chip and
    which as two kernels follows the measured rule of the library; here whatever it picks is checked against the oracle, and
    the on-chip form where the rule says so needs no workspace."""
    import paper_2608_03537_b200 as cf
    w = wl.post_norm(M, N, K, seed=N + K, affine=True, relu=(N == 1792))
    T = P.dev_tensors(w)
    desc = cf.make_gemm_desc(T["A"], T["B"], torch.empty(M, N, dtype=torch.bfloat16, device=T["A"].device),
                             cf.EPI_BIAS_RES_LAYERNORM, residual=T["residual"], fused=True)
    on_chip = N == 1280 or (N == 1536 and K <= 1024) or (N == 1792 and K <= 2048)
    assert cf.workspace_size(desc) == (0 if on_chip else M * (N // 256) * 8)
    got = P.run_gpu(w, T, fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label=f"LN {M}x{N}x{K}")
    w = wl.complex_subgraph(M, N, K, seed=M + N)
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label=f"RMS {M}x{N}x{K}", rowmax_tol=3e-2)


@pytest.mark.parametrize("M,N,K", [(300, 1536, 2048), (520, 3072, 64), (260, 5120, 136), (4100, 2560, 72)])
def test_row_lengths_without_a_single_kernel_form_run_in_256_column_tiles(M, N, K, cuda_device):
    """Multiples of 256 that no on-chip instantiation covers (1280, 1536, 2560, 3072, 5120, ...), at any K: the two-kernel form."""
    import paper_2608_03537_b200 as cf
    w = wl.post_norm(M, N, K, seed=N + K, affine=True, relu=(N == 3072))
    T = P.dev_tensors(w)
    desc = cf.make_gemm_desc(T["A"], T["B"], torch.empty(M, N, dtype=torch.bfloat16, device=T["A"].device),
                             cf.EPI_BIAS_RES_LAYERNORM, residual=T["residual"], fused=True)
    assert cf.workspace_size(desc) == M * (N // 256) * 8
    got = P.run_gpu(w, T, fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label=f"LN 256-tiles {M}x{N}x{K}")
    w = wl.complex_subgraph(M, N, K, seed=M + N)
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label=f"RMS 256-tiles {M}x{N}x{K}", rowmax_tol=3e-2)


@pytest.mark.parametrize("M,N,K", [(300, 1000, 200), (520, 1600, 64), (129, 200, 520), (260, 5000, 136), (1100, 384, 72), (70, 128, 64),
                                   (200, 8200, 1024), (130, 40, 32), (544, 3272, 216), (300, 3496, 256), (260, 4000, 72)])
def test_row_lengths_that_are_not_a_multiple_of_256_end_in_a_partial_tile(M, N, K, cuda_device):
    """Any row length (a multiple of 8).  A row a little shorter than an on-chip form runs on it with the surplus columns
    masked (exact zeros; the statistic is taken over N).  Otherwise the last 256-column tile of the two-kernel form is a partial
    one -- operands outside the matrix read as zeros, the stores are clipped, the second kernel corrects that tile's statistic."""
    import paper_2608_03537_b200 as cf
    w = wl.post_norm(M, N, K, seed=N + K, affine=True)
    T = P.dev_tensors(w)
    desc = cf.make_gemm_desc(T["A"], T["B"], torch.empty(M, N, dtype=torch.bfloat16, device=T["A"].device),
                             cf.EPI_BIAS_RES_LAYERNORM, residual=T["residual"], fused=True)
    # a little shorter than 1024 / 2048 / 256 / 4096: that form, surplus columns masked (3272 and 3496 leave the last of the
    # sixteen CTAs' column ranges without a single valid column: its accumulator must still be computed, as zeros)
    on_chip = N in (1000, 1600, 200, 3272, 3496, 4000)
    assert cf.workspace_size(desc) == (0 if on_chip else M * ((N + 255) // 256) * 8)
    got = P.run_gpu(w, T, fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label=f"LN partial tile {M}x{N}x{K}")
    w = wl.complex_subgraph(M, N, K, seed=M + N)
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label=f"RMS partial tile {M}x{N}x{K}", rowmax_tol=3e-2)


def test_wide_rows_need_their_workspace(cuda_device):
    import paper_2608_03537_b200 as cf
    w = wl.post_norm(128, 8192, 64, seed=3, affine=False)
    T = P.dev_tensors(w)
    Y = torch.empty(128, 8192, dtype=torch.bfloat16, device=T["A"].device)
    with pytest.raises(cf.ComfuseError) as ei:
        cf.gemm_epilogue(T["A"], T["B"], Y, cf.EPI_BIAS_RES_LAYERNORM, bias=T["bias"], residual=T["residual"], fused=True)
    assert ei.value.status == cf.ERR_WORKSPACE


def test_argmax_planted_spike(cuda_device):
    """A residual spike pins the arg max of chosen rows, in every CTA of the cluster and at the chunk borders."""
    M, N, K = 128, 768, 64
    w = wl.complex_subgraph(M, N, K, seed=5)
    R = wl.bf16_bits_to_f32(w.tensors["residual"]).copy()
    cols = {0: 0, 1: 767, 2: 383, 3: 384, 64: 500, 127: 31}
    for r, c in cols.items():
        R[r, c] = 8.0
    w.tensors["residual"] = wl.f32_to_bf16_bits(R)
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    ref = P.run_oracle(w)
    P.check_outputs(w, got, ref, label="argmax spike")
    am = got["row_argmax"].cpu().numpy()
    for r, c in cols.items():
        assert am[r] == c == ref["row_argmax"][r]


@pytest.mark.parametrize("fused", [True, False])
def test_argmax_exact_tie_reports_lowest_column(fused, cuda_device):
    """With A = 0 and bias = 0 the pre-norm value is the residual itself (GELU(0) = 0) and gain 1 keeps equal
    entries equal, so equal spikes are exact ties: the lower column must win across threads, halves and CTAs."""
    M, N, K = 128, 768, 64
    w = wl.complex_subgraph(M, N, K, seed=8)
    w.tensors["A"][:] = 0
    w.tensors["bias"][:] = 0
    w.tensors["gamma"] = wl.f32_to_bf16_bits(np.ones(N, dtype=np.float32))
    R = wl.bf16_bits_to_f32(w.tensors["residual"]).copy()
    ties = {0: (5, 6), 1: (10, 50), 2: (31, 32), 3: (100, 500), 4: (383, 384), 5: (700, 767), 77: (0, 767)}
    for r, (c1, c2) in ties.items():
        R[r, c1] = 8.0
        R[r, c2] = 8.0
    w.tensors["residual"] = wl.f32_to_bf16_bits(R)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    ref = P.run_oracle(w)
    P.check_outputs(w, got, ref, label="argmax tie", rowmax_tol=5e-3 if fused else 3e-2)
    am = got["row_argmax"].cpu().numpy()
    for r, (c1, _) in ties.items():
        assert am[r] == c1 == ref["row_argmax"][r]


SOFTMAX_CASES = [
    # batch, M, N, K, causal
    (2, 256, 256, 64, True),
    (3, 512, 512, 64, True),
    (2, 1024, 1024, 32, True),
    (2, 2048, 2048, 64, True),     # the attention-score configuration (short K: row kernel, chunks computed twice)
    (1, 300, 512, 64, False),      # no mask, ragged M
    (2, 200, 2048, 40, False),
    (1, 4096, 4096, 16, True),
    (1, 1000, 1000, 64, True),     # row kernel: N not a multiple of the 64-column box, diagonal inside a chunk
    (2, 136, 1096, 128, False),    # row kernel: two K blocks, ragged last chunk
    (1, 384, 8192, 256, False),    # row kernel: N beyond what one cluster can hold, four K blocks, odd row-block count
    (37, 256, 256, 8, True),       # row kernel: more tiles than one round, minimal K
    # K > 256: the cluster kernel (row block resident on-chip, statistics exchanged through distributed shared memory)
    (2, 256, 256, 320, True),
    (3, 512, 512, 320, True),
    (2, 1024, 1024, 264, True),
    (2, 2048, 2048, 320, True),
    (1, 300, 512, 320, False),
    (2, 200, 2048, 272, False),
    (1, 4096, 4096, 264, True),
    # row lengths on clusters of 10, 6, 14, 10, 12 and 14 CTAs (instead of the row kernel's two MainLoop passes)
    (1, 300, 768, 320, False),
    (2, 768, 768, 520, True),
    (1, 300, 1280, 320, False),
    (1, 1536, 1536, 264, True),
    (2, 200, 1792, 520, False),
    (1, 520, 2560, 776, False),
    (1, 3072, 3072, 264, True),
    (1, 260, 3584, 1032, False),
    # row lengths between two instantiations run on the next wider one, the columns from N on masked
    (1, 300, 1000, 320, False),
    (2, 1000, 1000, 264, True),
    (1, 200, 72, 520, False),
    (1, 260, 2056, 776, False),
    (1, 3000, 3000, 328, True),
    (3, 130, 4088, 1032, False),
    # K >= 768: the cluster kernel's long-contraction form (three stages, sub-tiles in lock step, eight epilogue warps)
    (1, 300, 1024, 776, False),
    (2, 1024, 1024, 768, True),
    (1, 2048, 2048, 1032, True),
    (1, 260, 4096, 800, False),
]


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("batch,M,N,K,causal", SOFTMAX_CASES)
def test_scaled_masked_softmax_epilogue(batch, M, N, K, causal, fused, cuda_device):
    w = wl.scaled_masked_softmax(batch, M, N, K, seed=N + K, causal=causal)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    ref = P.run_oracle(w)
    res = P.check_outputs(w, got, ref, label=f"softmax b{batch} {M}x{N}x{K} causal={causal} fused={fused}",
                          softmax_tol=P.TOL_SOFTMAX_MAX if fused else P.TOL_SOFTMAX_UNFUSED)
    rowsum = got["Y"].float().sum(-1)
    assert (rowsum - 1).abs().max().item() < 2e-2       # bf16-rounded probabilities still sum to ~1


def test_softmax_large_scores_do_not_overflow(cuda_device):
    """Scores of magnitude ~1e2 (alpha = 4): exp(x - max) must stay finite, rows must sum to one."""
    w = wl.scaled_masked_softmax(1, 256, 256, 64, seed=77, causal=True)
    w.scalars["alpha"] = 4.0
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label="softmax large scores")


@pytest.mark.parametrize("batch,M,N,K,causal", [(1, 300, 8192, 320, False), (2, 200, 1000, 512, False), (1, 1536, 1536, 320, True),
                                               (1, 257, 12288, 264, False)])
def test_softmax_long_k_rows_without_a_cluster_instantiation(batch, M, N, K, causal, cuda_device):
    """Long K with a row wider than the largest cluster holds (or of a length without a cluster instantiation): fused through
    the statistics pass + second MainLoop pass of the row kernel, at the fused tolerance."""
    w = wl.scaled_masked_softmax(batch, M, N, K, seed=5 + N, causal=causal)
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label=f"softmax long K N={N}")
    assert (got["Y"].float().sum(-1) - 1).abs().max().item() < 2e-2
    assert cf.last_device_status() == cf.OK


def _additive_mask(M, N, seed, dead_rows=(5,)):
    """A mask tensor with moderate finite entries, 30 % of -inf, and whole rows of -inf."""
    g = np.random.default_rng(seed)
    mask = (g.standard_normal((M, N)) * 0.5).astype(np.float32)
    mask[g.random((M, N)) < 0.3] = -np.inf
    for r in dead_rows:
        if r < M:
            mask[r, :] = -np.inf
    return wl.f32_to_bf16_bits(mask)


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("batch,M,N,K,softcap", [
    (2, 96, 256, 64, 0.0),       # short K: the row kernel; fewer rows than a tile
    (3, 300, 1000, 72, 0.0),     # ragged M and N, several chunks per row
    (1, 512, 2048, 128, 3.0),    # soft-cap in front of the mask
    (2, 200, 1024, 320, 0.0),    # long K: the cluster kernel (4 CTA pairs per row block)
    (1, 256, 512, 512, 2.5),     # cluster kernel, soft-capped
    (1, 300, 1024, 840, 2.0),    # cluster kernel behind a long contraction, soft-capped
    (2, 260, 2048, 768, 0.0),
    (1, 300, 1536, 320, 0.0),    # cluster of 6 CTAs
    (2, 200, 768, 264, 3.0),     # sub-tiles of 256 and 128 columns in lock step
    (1, 300, 1000, 328, 0.0),    # the 1024-column form with 24 columns masked, the mask tensor's rows 1000 long
    (2, 200, 1160, 64, 2.5),     # a small problem behind a short contraction: the cluster kernel, 1280-column form
    (1, 260, 3072, 520, 2.0),    # cluster of 12 CTAs, soft-capped
])
def test_softmax_additive_mask_with_fully_masked_rows(batch, M, N, K, softcap, fused, cuda_device):
    """The additive-mask variant: the mask tensor is one more operand of the epilogue; -inf entries give exact zeros, a
    fully masked row gives a row of zeros (the plain definition would give NaN)."""
    w = wl.scaled_masked_softmax(batch, M, N, K, seed=31 + K, causal=False, softcap=softcap)
    dead = (5, M - 1, 130)
    w.tensors["mask"] = _additive_mask(M, N, seed=K, dead_rows=dead)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    ref = P.run_oracle(w)
    P.check_outputs(w, got, ref, label=f"softmax additive mask fused={fused}", softmax_tol=P.TOL_SOFTMAX_MAX if fused else P.TOL_SOFTMAX_UNFUSED)
    for r in dead:
        if r < M:
            assert (got["Y"][:, r, :] == 0).all()
    rows_alive = [r for r in range(M) if r not in dead]
    assert (got["Y"][:, rows_alive, :].float().sum(-1) - 1).abs().max().item() < 2e-2


def test_fused_and_unfused_runs_are_bitwise_repeatable(cuda_device):
    """Merge order across the cluster is fixed (rank order), so two runs give identical bits."""
    for w in (wl.post_norm(300, 768, 200, seed=3, affine=True), wl.complex_subgraph(150, 4096, 128, seed=4),
              wl.scaled_masked_softmax(2, 2048, 2048, 64, seed=6)):
        T = P.dev_tensors(w)
        a = P.run_gpu(w, T, fused=True)
        b = P.run_gpu(w, T, fused=True)
        for k in a:
            assert torch.equal(a[k].view(torch.int16) if a[k].dtype == torch.bfloat16 else a[k],
                               b[k].view(torch.int16) if b[k].dtype == torch.bfloat16 else b[k]), (w.name, k)


def test_no_timeout_recorded(cuda_device):
    import paper_2608_03537_b200 as cf
    assert cf.last_device_status() == cf.OK


def test_back_to_back_dependent_launches_see_each_others_results(cuda_device):
    """Kernels are launched with programmatic stream serialization: the set-up of a kernel overlaps the tail of the previous
    one, and it waits for that kernel before it touches global memory.  A chain in which every call consumes the previous
    call's output, enqueued without any synchronisation, must give bit-for-bit what the same chain gives with a
    synchronisation after every call."""
    import paper_2608_03537_b200 as cf
    M, N, K = 512, 256, 256
    w = wl.post_norm(M, N, K, seed=11, affine=True)
    T = P.dev_tensors(w)
    dev = T["A"].device

    def chain(sync):
        x = T["A"].clone()                       # [M, 256]; N == K so the output can feed the next call
        bufs = [torch.empty(M, N, dtype=torch.bfloat16, device=dev) for _ in range(2)]
        for i in range(12):
            y = bufs[i & 1]                      # ping-pong: a call overwrites what the call before the previous one wrote
            cf.gemm_epilogue(x, T["B"], y, cf.EPI_BIAS_RES_LAYERNORM, bias=T["bias"], residual=T["residual"],
                             gamma=T["gamma"], beta=T["beta"], fused=True)
            if sync:
                torch.cuda.synchronize()
            x = y
        torch.cuda.synchronize()
        return x.clone()

    a = chain(sync=True)
    for _ in range(3):
        b = chain(sync=False)
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    assert cf.last_device_status() == cf.OK


# --------------------------------------------------------------------------------------------- the Sec. 6.1 patterns
@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("M,N,K", [(300, 768, 200), (200, 4096, 128), (300, 8192, 72)])
def test_matmul_bias_layernorm_relu_pattern(M, N, K, fused, cuda_device):
    w = wl.post_norm(M, N, K, seed=M + N + K + 1, affine=True, relu=True)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    P.check_outputs(w, got, P.run_oracle(w), label=f"LN+ReLU {M}x{N}x{K} fused={fused}")
    Y = got["Y"].float()
    assert (Y >= 0).all().item() and (Y == 0).float().mean().item() > 0.3     # about half the values are clamped


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("M,N,K", [(140, 768, 64), (150, 4096, 128), (129, 8192, 64)])
def test_matmul_bias_rmsnorm_pattern(M, N, K, fused, cuda_device):
    """RMSNorm(A.B + bias) * g: no activation, no residual (the row max / argmax outputs are still produced)."""
    w = wl.complex_subgraph(M, N, K, seed=M + N + 2, activation=False, residual=False)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    P.check_outputs(w, got, P.run_oracle(w), label=f"bias+RMS {M}x{N}x{K} fused={fused}",
                    rowmax_tol=5e-3 if (fused and N <= 4096) else 3e-2)


SOFTCAP_CASES = [
    # batch, M, N, K, causal, softcap
    (2, 512, 512, 64, True, 5.0),      # row kernel (short K), strong cap
    (1, 300, 1000, 64, False, 30.0),   # row kernel, ragged N, mild cap
    (2, 256, 2048, 320, False, 5.0),   # cluster kernel (K > 256)
    (1, 1024, 1024, 264, True, 2.0),   # cluster kernel, causal
]


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("batch,M,N,K,causal,cap", SOFTCAP_CASES)
def test_matmul_scale_tanh_softcap_softmax_pattern(batch, M, N, K, causal, cap, fused, cuda_device):
    w = wl.scaled_masked_softmax(batch, M, N, K, seed=N + K + 7, causal=causal, softcap=cap)
    # make the cap bite: scores of standard deviation ~4 instead of ~1
    w.scalars["alpha"] *= 4.0
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    P.check_outputs(w, got, P.run_oracle(w), label=f"softcap {cap} b{batch} {M}x{N}x{K} causal={causal} fused={fused}",
                    softmax_tol=P.TOL_SOFTMAX_MAX if fused else P.TOL_SOFTMAX_UNFUSED)


@pytest.mark.parametrize("fused", [True, False])
def test_layernorm_with_a_large_common_offset(fused, cuda_device):
    """Rows whose mean is ~60 times their standard deviation: the statistics must not cancel (chunk-centred partial sums
    merged with the pairwise update, not sum and sum of squares)."""
    w = wl.post_norm(300, 1024, 136, seed=91, affine=True)
    w.tensors["bias"] = wl.f32_to_bf16_bits(np.full(1024, 64.0, dtype=np.float32))
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    P.check_outputs(w, got, P.run_oracle(w), label=f"large offset fused={fused}")


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("batch,M,N,K,causal", [
    (2, 256, 256, 64, True),       # one chunk
    (3, 300, 1000, 72, False),     # ragged M, N and K
    (2, 2048, 2048, 64, True),     # the attention-score shape of the fifth... fourth configuration, two batches
    (1, 200, 1024, 320, False),    # long K: the row kernel's second MainLoop pass
    (1, 129, 8192, 128, False),    # rows wider than a cluster
])
def test_softmax_second_operand_stored_n_by_k(batch, M, N, K, causal, fused, cuda_device):
    """COMFUSE_FLAG_B_ROW_MAJOR_NK: the second operand as [batch, N, K] (attention keys, one per row).  Every GEMM kernel
    reads it in place as a K-major operand and gives the same bits as the call with the operand transposed."""
    w = wl.scaled_masked_softmax(batch, M, N, K, seed=N + K, causal=causal)
    T = P.dev_tensors(w)
    Bnk = T["B"].transpose(1, 2).contiguous()                        # [batch, N, K]
    Y = torch.full((batch, M, N), float("nan"), dtype=torch.bfloat16, device=cuda_device)
    mask = cf.MASK_CAUSAL if causal else cf.MASK_NONE
    desc = cf.make_gemm_desc(T["A"], Bnk, Y, cf.EPI_SCALE_MASK_SOFTMAX, alpha=w.scalars["alpha"], mask=mask, fused=fused,
                             flags=cf.FLAG_B_ROW_MAJOR_NK)
    need = cf.workspace_size(desc)
    assert need == (0 if fused else batch * M * N * 2)
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device=cuda_device)
    cf.gemm_epilogue(T["A"], Bnk, Y, cf.EPI_SCALE_MASK_SOFTMAX, alpha=w.scalars["alpha"], mask=mask, fused=fused, workspace=ws,
                     flags=cf.FLAG_B_ROW_MAJOR_NK)
    torch.cuda.synchronize()
    assert cf.last_device_status() == cf.OK
    P.check_outputs(w, {"Y": Y}, P.run_oracle(w), label=f"softmax B[N,K] {batch}x{M}x{N}x{K} fused={fused}",
                    softmax_tol=P.TOL_SOFTMAX_MAX if fused else P.TOL_SOFTMAX_UNFUSED)
    ref = P.run_gpu(w, T, fused=fused)["Y"]      # same kernels, same arithmetic as with B [K, N]
    assert torch.equal(Y.view(torch.int16), ref.view(torch.int16))


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("kind", ["ln_small", "ln_lockstep", "rms_cluster16", "rms_two_kernels"])
def test_second_operand_n_by_k_normalising_kinds(kind, fused, cuda_device):
    """A linear layer's weight as it is stored, [out, in] = [N, K]: the LayerNorm and RMSNorm kinds on every tiling of the
    fused kernel (one sub-tile, lock-step sub-tiles, clusters of sixteen, the two-kernel form) and on the unfused path give the
    same bits as with the transposed operand, and match the oracle."""
    w = {"ln_small": lambda: wl.post_norm(300, 256, 200, seed=71, affine=True),
         "ln_lockstep": lambda: wl.post_norm(300, 768, 200, seed=72, affine=True),
         "rms_cluster16": lambda: wl.complex_subgraph(150, 4096, 128, seed=73),
         "rms_two_kernels": lambda: wl.complex_subgraph(520, 2048, 1024, seed=74)}[kind]()
    T = P.dev_tensors(w)
    ref, _ = P.prepare_gpu(w, T, fused=fused)
    T2 = dict(T)
    T2["B"] = T["B"].t().contiguous()
    d = w.dims
    Y = torch.full((d["M"], d["N"]), float("nan"), dtype=torch.bfloat16, device=cuda_device)
    if w.kind == wl.KIND_BIAS_RES_LAYERNORM:
        epi = cf.EPI_BIAS_RES_LAYERNORM
        kw = dict(bias=T.get("bias"), residual=T.get("residual"), gamma=T.get("gamma"), beta=T.get("beta"), alpha=w.scalars["alpha"], eps=w.scalars["eps"])
        outs = {"Y": Y}
    else:
        epi = cf.EPI_BIAS_GELU_RES_RMSNORM_MAX
        outs = {"Y": Y, "row_max": torch.empty(d["M"], dtype=torch.float32, device=cuda_device),
                "row_argmax": torch.empty(d["M"], dtype=torch.int32, device=cuda_device)}
        kw = dict(bias=T.get("bias"), residual=T.get("residual"), gamma=T.get("gamma"), alpha=w.scalars["alpha"], eps=w.scalars["eps"],
                  row_max=outs["row_max"], row_argmax=outs["row_argmax"])
    desc = cf.make_gemm_desc(T["A"], T2["B"], Y, epi, residual=T.get("residual"), fused=fused, flags=cf.FLAG_B_ROW_MAJOR_NK)
    ws = torch.empty(max(cf.workspace_size(desc), 16), dtype=torch.uint8, device=cuda_device)
    cf.gemm_epilogue(T["A"], T2["B"], Y, epi, fused=fused, workspace=ws, flags=cf.FLAG_B_ROW_MAJOR_NK, **kw)
    torch.cuda.synchronize()
    assert cf.last_device_status() == cf.OK
    P.check_outputs(w, outs, P.run_oracle(w), label=f"{kind} B[N,K] fused={fused}", rowmax_tol=3e-2, norm_tol=P.TOL_NORM_MAX if fused else 4e-2)
    base = P.run_gpu(w, T, fused=fused)
    for k in outs:
        a, b = outs[k], base[k]
        assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a, b.view(torch.int16) if b.dtype == torch.bfloat16 else b), k


def test_second_operand_n_by_k_through_the_workspace_free_entry_point(cuda_device):
    """The workspace-free (unfused, fixed scratch) entry point passes the operand-layout flag through."""
    w = wl.post_norm(300, 768, 200, seed=91, affine=True)
    T = P.dev_tensors(w)
    Bnk = T["B"].t().contiguous()
    Y = torch.full((300, 768), float("nan"), dtype=torch.bfloat16, device=cuda_device)
    cf.gemm_epilogue_static_scratch(T["A"], Bnk, Y, cf.EPI_BIAS_RES_LAYERNORM, bias=T["bias"], residual=T["residual"],
                                    gamma=T["gamma"], beta=T["beta"], alpha=w.scalars["alpha"], eps=w.scalars["eps"],
                                    flags=cf.FLAG_B_ROW_MAJOR_NK)
    torch.cuda.synchronize()
    assert cf.last_device_status() == cf.OK
    ref = P.run_gpu(w, T, fused=False)["Y"]
    assert torch.equal(Y.view(torch.int16), ref.view(torch.int16))
    P.check_outputs(w, {"Y": Y}, P.run_oracle(w), label="static scratch B[N,K]", norm_tol=4e-2)
