"""Launches queued back to back.

The other parity tests run one launch at a time, with a synchronisation behind each.  A stream of launches differs in three
ways: the next launch's set-up overlaps the previous launch's tail (programmatic dependent launch), the inputs sit in L2 so
every load is fast except the very first ones, which all CTAs issue at once, and the shared memory and tensor memory a CTA
finds still hold the previous launch's last tile, so a consumer that looked at a buffer too early would read plausible
numbers instead of garbage.  Here every workload's fused kernel runs 40 times behind a busy-wait kernel with nothing in
between; the output of the last launch must equal the output of one isolated launch bit for bit (the kernels are
deterministic), and the isolated launch is compared with the fp64 oracle -- element by element in the full-size tests, on
the rows of each CTA pair's first tile here for the shape no other test runs at full size.
"""
import numpy as np
import pytest
import torch

import paper_2608_03537_b200 as cf
import workloads as wl
from tests import parity as P

pytestmark = pytest.mark.gpu

LAUNCHES = 40


def _same_bits(a, b):
    if a.dtype == torch.bfloat16:
        return torch.equal(a.view(torch.int16), b.view(torch.int16))
    if a.dtype == torch.float32:
        return torch.equal(a.view(torch.int32), b.view(torch.int32))
    return torch.equal(a, b)


@pytest.mark.parametrize("index", [1, 2, 3, 4, 5, 7, 8], ids=["c2", "c3", "c4", "c5", "a1", "a2", "d1"])
def test_forty_launches_back_to_back_equal_one_isolated_launch(index, cuda_device):
    w = wl.config(index)
    T = P.dev_tensors(w)
    first, launch = P.prepare_gpu(w, T, fused=True)
    launch()
    torch.cuda.synchronize()
    assert cf.last_device_status() == cf.OK
    first = {k: v.clone() for k, v in first.items()}
    for rounds in range(3):
        out, launch = P.prepare_gpu(w, T, fused=True)
        torch.cuda.synchronize()
        torch.cuda._sleep(2_000_000)          # the host queues the launches while this runs
        for _ in range(LAUNCHES):
            launch()
        torch.cuda.synchronize()
        assert cf.last_device_status() == cf.OK
        for k in first:
            assert _same_bits(out[k], first[k]), f"{w.name}: output {k} of launch {LAUNCHES} of round {rounds} differs from an isolated launch"


SMALL = {
    "post_norm_ragged": lambda: wl.post_norm(300, 768, 200, seed=3, affine=True),
    "post_norm_short_k": lambda: wl.post_norm(600, 256, 64, seed=4, affine=False),
    "complex_subgraph_cluster16": lambda: wl.complex_subgraph(150, 4096, 128, seed=5),
    "complex_subgraph_two_kernels": lambda: wl.complex_subgraph(520, 2048, 1024, seed=6),
    "softmax_rows_causal": lambda: wl.scaled_masked_softmax(2, 2048, 2048, 64, seed=7, causal=True),
    "softmax_cluster_long_k": lambda: wl.scaled_masked_softmax(2, 200, 1024, 320, seed=8, causal=False),
    "b2b_mlp_ragged": lambda: wl.b2b_mlp(300, 128, 512, 128, seed=9, affine=True),
    "b2b_mlp_one_chunk": lambda: wl.b2b_mlp(130, 128, 128, 128, seed=10),
    "attention_256": lambda: wl.target_attention(3, 600, 256, 128, seed=11),
    "attention_512": lambda: wl.target_attention(3, 600, 512, 128, seed=12),
    "attention_one_row": lambda: wl.target_attention(1, 1, 256, 128, seed=13),
    "dlrm_small": lambda: wl.dlrm_bottom_mlp(700, 200, 512, 128, seed=14),
}


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("name", sorted(SMALL))
def test_small_and_ragged_shapes_back_to_back(name, fused, cuda_device):
    """The same check on shapes with few tiles, ragged edges and one-chunk pipelines, where a launch is little more than
    its first tile, on the fused kernels and on the in-library unfused path (plain GEMM + row kernels); the isolated launch
    is compared with the oracle as well."""
    w = SMALL[name]()
    T = P.dev_tensors(w)
    first, launch = P.prepare_gpu(w, T, fused=fused)
    launch()
    torch.cuda.synchronize()
    assert cf.last_device_status() == cf.OK
    P.check_outputs(w, first, P.run_oracle(w), label=f"{name} fused={fused} isolated",
                    softmax_tol=P.TOL_SOFTMAX_MAX if fused else P.TOL_SOFTMAX_UNFUSED, rowmax_tol=3e-2, norm_tol=P.TOL_NORM_MAX if fused else 4e-2)
    out, launch = P.prepare_gpu(w, T, fused=fused)
    torch.cuda.synchronize()
    torch.cuda._sleep(1_000_000)
    for _ in range(LAUNCHES):
        launch()
    torch.cuda.synchronize()
    assert cf.last_device_status() == cf.OK
    for k in first:
        assert _same_bits(out[k], first[k]), f"{name} fused={fused}: output {k} of launch {LAUNCHES} differs from an isolated launch"


def test_self_attention_512_full_size_first_and_last_tiles_against_the_oracle(cuda_device):
    """a2 at full size (256 x (512 x 128 -> 512 -> 128), seven row tiles = fourteen sub-tiles per CTA pair): the batches
    that hold every CTA pair's first tile, and the last ones, element by element."""
    w = wl.config(7)
    got = P.run_gpu(w, P.dev_tensors(w), fused=True)
    assert torch.isfinite(got["Y"].float()).all().item()
    nb = w.dims["batch"]
    for b in list(range(0, 40)) + list(range(nb - 8, nb)):
        P.check_outputs(w, got, P.run_oracle(w, batches=[b]), batches=[b], label=f"a2 self-attention batch {b}")
