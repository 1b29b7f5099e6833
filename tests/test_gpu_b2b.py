"""GPU parity of the back-to-back GEMM: fused kernel (P and S never leave the chip) and the in-library unfused path
(three bf16 intermediates) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import paper_2608_03537_b200 as cf
import workloads as wl
from tests import parity as P

pytestmark = pytest.mark.gpu

CASES = [
    # M, N1, affine
    (256, 512, False),     # one row-block pair, all four N1 chunks
    (300, 512, True),      # ragged: second pair has one partial block and one empty block
    (1000, 256, True),     # two chunks
    (130, 128, False),     # a single chunk: ML1 -> Epi1 -> ML2 with no overlap partner
    (2048, 384, True),     # three chunks, several tiles per cluster on small grids
    (300, 640, True),      # five chunks: an odd count beyond four
    (520, 2048, False),    # sixteen chunks per tile
    (260, 4096, True),     # the widest hidden layer the bias buffer holds
    (300, 8, True),        # the narrowest: 8 of the chunk's 128 columns, the rest zero-filled
    (520, 200, False),     # a whole chunk and a partial one
    (260, 1000, True),     # seven chunks and 104 columns
    (300, 4088, False),    # the last 8 columns missing
]


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("M,N1,affine", CASES)
def test_b2b_mlp_layernorm(M, N1, affine, fused, cuda_device):
    w = wl.b2b_mlp(M, 128, N1, 128, seed=M + N1, affine=affine)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    P.check_outputs(w, got, P.run_oracle(w), label=f"b2b M{M} N1{N1} fused={fused}")
    assert cf.last_device_status() == cf.OK


@pytest.mark.parametrize("fused", [True, False])
def test_config_b2b_mlp_full_size(fused, cuda_device):
    """c5 at full size: every element against the oracle; over every row, the un-normalised statistics property."""
    w = wl.config(4)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    assert torch.isfinite(got["Y"].float()).all().item()
    res = P.check_outputs(w, got, P.run_oracle(w), label=f"c5 fused={fused}")
    Y = got["Y"].float()          # gamma = 1, beta = 0: every row has mean ~0 and variance ~1
    assert Y.mean(-1).abs().max().item() < 2e-2
    assert (Y.var(-1, unbiased=False) - 1).abs().max().item() < 3e-2
    print("c5", fused, res)


def test_b2b_identity_second_weight(cuda_device):
    """W2 = I, b2 = 0: the fused chain must reduce to LayerNorm(GELU(X W1 + b1) + X) (needs N1 = N2 = 128)."""
    w = wl.b2b_mlp(384, 128, 128, 128, seed=7)
    w.tensors["W2"] = wl.f32_to_bf16_bits(np.eye(128, dtype=np.float32))
    w.tensors["b2"][:] = 0
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label="b2b identity W2")


def test_b2b_bitwise_repeatable(cuda_device):
    w = wl.b2b_mlp(2048, 128, 512, 128, seed=3)
    T = P.dev_tensors(w)
    a = P.run_gpu(w, T, fused=True)["Y"]
    b = P.run_gpu(w, T, fused=True)["Y"]
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_b2b_unsupported_shapes_are_refused_for_the_fused_path(cuda_device):
    d = cf.make_b2b_desc(256, 128, 4224, 128, fused=True)      # N1 > 4096
    with pytest.raises(cf.ComfuseError) as e:
        cf.b2b_workspace_size(d)
    assert e.value.status == cf.ERR_UNSUPPORTED
    assert cf.b2b_workspace_size(cf.make_b2b_desc(256, 128, 4224, 128, fused=False)) == 256 * 4224 * 2 + 256 * 128 * 2


# --------------------------------------------------------------------------------------------- attention form (F = softmax)
@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("batch,M", [(2, 256), (3, 600), (37, 128), (1, 1)])
def test_b2b_softmax_attention(batch, M, fused, cuda_device):
    """O = softmax(Q.Kt / sqrt(d)).V with 256 source positions and head size 128: several tiles, ragged M, more tiles than
    one round of CTA pairs, the one-row edge."""
    w = wl.target_attention(batch, M, 256, 128, seed=batch + M)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    P.check_outputs(w, got, P.run_oracle(w), label=f"attention b{batch} M{M} fused={fused}")


def test_b2b_softmax_attention_sharp_and_flat_rows(cuda_device):
    """Large scores (one key dominates: the output is that value row; no overflow) and zero queries (uniform weights: the
    output is the mean of the value rows)."""
    w = wl.target_attention(2, 256, 256, 128, seed=9)
    w.scalars["alpha"] = 4.0                       # scores of standard deviation ~45
    w.tensors["X"][1, 128:] = 0                    # zero queries in the second half of batch 1 (bf16 bits 0 = 0.0)
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    ref = P.run_oracle(w)
    P.check_outputs(w, got, ref, label="attention sharp/flat")
    V1 = wl.bf16_to_f64(w.tensors["W2"][1])
    assert np.abs(P.to_f64(got["Y"][1, 128:]) - V1.mean(0)).max() < 2e-3


def test_b2b_attention_full_size(cuda_device):
    w = wl.config(5)                               # 32 x (4096 x 128 -> 256 -> 128)
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    assert torch.isfinite(got["Y"].float()).all().item()
    for b in range(w.dims["batch"]):               # every element, one batch at a time
        P.check_outputs(w, got, P.run_oracle(w, batches=[b]), batches=[b], label=f"a1 target attention batch {b}")


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("batch,M", [(4, 512), (3, 600), (40, 256), (100, 512), (1, 1)])
def test_b2b_softmax_attention_512_source_positions(batch, M, fused, cuda_device):
    """The Self-Attention 512 x 512 shape of Sec. 6.2 (Table II) and neighbours: a score row of 512 runs as two sub-tiles of
    256 with their own maxima, combined at the normalisation; ragged M, up to three row tiles (six sub-tiles) per CTA pair, the
    one-row edge."""
    w = wl.target_attention(batch, M, 512, 128, seed=batch + M + 1)
    got = P.run_gpu(w, P.dev_tensors(w), fused=fused)
    P.check_outputs(w, got, P.run_oracle(w), label=f"attention S=512 b{batch} M{M} fused={fused}")


def test_b2b_softmax_attention_512_sharp_rows_in_either_half(cuda_device):
    """Large scores: the dominant key lies in the first half for some rows and in the second half for others, so the two
    sub-tiles' maxima differ by tens of units either way; no overflow, the output is the dominant value row."""
    w = wl.target_attention(2, 256, 512, 128, seed=77)
    w.scalars["alpha"] = 4.0
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    P.check_outputs(w, got, P.run_oracle(w), label="attention S=512 sharp")


@pytest.mark.parametrize("keys_row_major", [False, True])
@pytest.mark.parametrize("batch,M,S", [(2, 300, 8), (3, 260, 64), (2, 600, 200), (5, 256, 248), (2, 300, 264), (3, 520, 384), (40, 256, 504)])
def test_b2b_softmax_attention_any_source_length_up_to_512(batch, M, S, keys_row_major, cuda_device):
    """Source lengths that are not 256 or 512: the fused kernel masks the positions from S on (their keys and values read as
    zeros, their scores count as -inf), in the 256-position form up to 256 and in the two-sub-tile form beyond."""
    import paper_2608_03537_b200 as cf
    w = wl.target_attention(batch, M, S, 128, seed=5 * batch + M + S)
    T = P.dev_tensors(w)
    O = torch.full((batch, M, 128), float("nan"), dtype=torch.bfloat16, device=cuda_device)
    keys = T["W1"].transpose(1, 2).contiguous() if keys_row_major else T["W1"]
    desc = cf.make_b2b_desc(M, 128, S, 128, 0.0, True, cf.B2B_SOFTMAX_ATTENTION, batch, w.scalars["alpha"],
                            cf.B2B_FLAG_KEYS_ROW_MAJOR if keys_row_major else 0)
    assert cf.b2b_workspace_size(desc) == 0
    before = cf.launch_count()
    cf.b2b_attention(T["X"], keys, T["W2"], O, alpha=w.scalars["alpha"], fused=True, keys_row_major=keys_row_major)
    torch.cuda.synchronize()
    assert cf.last_device_status() == cf.OK and cf.launch_count() - before == 1
    P.check_outputs(w, {"Y": O}, P.run_oracle(w), label=f"attention b{batch} M{M} S{S} keys_row_major={keys_row_major}")


@pytest.mark.parametrize("batch,M,S,d", [(4, 512, 1024, 128), (2, 300, 1000, 64)])
def test_b2b_softmax_attention_other_shapes_unfused_path(batch, M, S, d, cuda_device):
    """Shapes without a fused instantiation: the fused call says UNSUPPORTED, the in-library unfused path (batched GEMM, row
    softmax, batched GEMM) matches the oracle."""
    import paper_2608_03537_b200 as cf
    w = wl.target_attention(batch, M, S, d, seed=S + d)
    with pytest.raises(cf.ComfuseError) as e:
        P.run_gpu(w, P.dev_tensors(w), fused=True)
    assert e.value.status == cf.ERR_UNSUPPORTED
    got = P.run_gpu(w, P.dev_tensors(w), fused=False)
    P.check_outputs(w, got, P.run_oracle(w), label=f"attention {batch}x{M}x{S}x{d} unfused")


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("batch,M,S", [(2, 256, 256), (3, 600, 256), (3, 600, 512), (40, 256, 512), (1, 1, 256)])
def test_b2b_softmax_attention_row_major_keys(batch, M, S, fused, cuda_device):
    """COMFUSE_B2B_FLAG_KEYS_ROW_MAJOR: the keys as [batch, S, d], one key per row; the fused kernel and the unfused path's
    GEMM read them in place as a K-major operand.  Same oracle, same tolerance, and the same bits as the call with the keys
    already transposed."""
    w = wl.target_attention(batch, M, S, 128, seed=3 * batch + M + S)
    T = P.dev_tensors(w)
    keys = T["W1"].transpose(1, 2).contiguous()                     # [batch, S, d]
    O = torch.full((batch, M, 128), float("nan"), dtype=torch.bfloat16, device=cuda_device)
    desc = cf.make_b2b_desc(M, 128, S, 128, 0.0, fused, cf.B2B_SOFTMAX_ATTENTION, batch, w.scalars["alpha"], cf.B2B_FLAG_KEYS_ROW_MAJOR)
    need = cf.b2b_workspace_size(desc)
    assert need == (0 if fused else batch * M * S * 2)
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device=cuda_device)
    cf.b2b_attention(T["X"], keys, T["W2"], O, alpha=w.scalars["alpha"], fused=fused, workspace=ws, keys_row_major=True)
    torch.cuda.synchronize()
    assert cf.last_device_status() == cf.OK
    P.check_outputs(w, {"Y": O}, P.run_oracle(w), label=f"attention row-major keys b{batch} M{M} S{S} fused={fused}")
    ref = P.run_gpu(w, T, fused=fused)["Y"]
    assert torch.equal(O.view(torch.int16), ref.view(torch.int16))
