"""Host-side checks that need no GPU: the shared library loads, exports every function that include/comfuse.h
declares, and rejects bad arguments before it touches CUDA."""
import ctypes
import os
import re

import paper_2608_03537_b200 as cf

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE = ctypes.c_void_p(4096)       # 16-byte aligned, never dereferenced: validation comes first
ODD = ctypes.c_void_p(4096 + 2)    # misaligned


def _desc(**kw):
    d = cf.GemmDesc()
    d.batch, d.M, d.N, d.K = 1, 256, 768, 512
    d.lda, d.ldb, d.ldr, d.ldy = 512, 768, 768, 768
    d.batch_stride_a = d.batch_stride_b = d.batch_stride_r = d.batch_stride_y = 0
    d.kind, d.mask, d.alpha, d.eps, d.fused, d.reserved = cf.EPI_BIAS_RES_LAYERNORM, cf.MASK_NONE, 1.0, 1e-5, 1, 0
    for k, v in kw.items():
        setattr(d, k, v)
    return d


def _ws(d):
    n = ctypes.c_size_t(12345)
    return cf.lib().comfuse_workspace_size(ctypes.byref(d), ctypes.byref(n)), n.value


def test_library_exports_every_declared_function():
    header = open(os.path.join(ROOT, "include", "comfuse.h")).read()
    declared = set(re.findall(r"\b(comfuse_[a-z0-9_]+)\s*\(", header))
    assert declared == set(cf.EXPORTED_SYMBOLS), declared ^ set(cf.EXPORTED_SYMBOLS)
    L = cf.lib()
    for name in declared:
        assert getattr(L, name) is not None


def test_status_strings_and_launch_counter():
    L = cf.lib()
    texts = [L.comfuse_status_string(i).decode() for i in range(9)]
    assert texts[0] == "ok" and len(set(texts)) == 9
    assert "unknown" in L.comfuse_status_string(99).decode()
    assert cf.launch_count() >= 0


def test_workspace_size_rules():
    assert _ws(_desc()) == (cf.OK, 0)                                      # fused: no workspace
    assert _ws(_desc(fused=0)) == (cf.OK, 256 * 768 * 2)                   # unfused: dense bf16 Z
    assert _ws(_desc(fused=0, batch=3, batch_stride_a=256 * 512, batch_stride_b=512 * 768, batch_stride_y=256 * 768,
                     batch_stride_r=256 * 768)) == (cf.OK, 3 * 256 * 768 * 2)
    assert _ws(_desc(N=776, ldb=776, ldr=776, ldy=776)) == (cf.OK, 0)                  # N = 776 runs on the 1024-column form, 248 columns masked
    assert _ws(_desc(N=520, ldb=520, ldr=520, ldy=520)) == (cf.OK, 256 * 3 * 8)        # too short for the 768-column form: two kernels,
                                                                                      # 256-column tiles, the last one partial
    assert _ws(_desc(N=70000, ldb=70000, ldr=70000, ldy=70000))[0] == cf.ERR_UNSUPPORTED   # beyond 65536 columns
    assert _ws(_desc(N=776, ldb=776, ldr=776, ldy=776, fused=0))[0] == cf.OK          # ... but the unfused path takes it
    assert _ws(_desc(N=770, ldb=776, ldr=776, ldy=776))[0] == cf.ERR_ALIGNMENT        # N must be a multiple of 8
    assert _ws(_desc(lda=516))[0] == cf.ERR_ALIGNMENT                                  # leading dims too
    assert _ws(_desc(lda=256))[0] == cf.ERR_INVALID_ARG                                # lda < K
    assert _ws(_desc(M=0))[0] == cf.ERR_INVALID_ARG
    assert _ws(_desc(kind=7))[0] == cf.ERR_INVALID_ARG
    assert _ws(_desc(reserved=1))[0] == cf.ERR_INVALID_ARG
    assert _ws(_desc(mask=cf.MASK_CAUSAL))[0] == cf.ERR_INVALID_ARG                    # masks belong to the softmax kind
    sm = dict(kind=cf.EPI_SCALE_MASK_SOFTMAX, N=2048, ldb=2048, ldr=2048, ldy=2048)
    assert _ws(_desc(**sm, mask=cf.MASK_CAUSAL))[0] == cf.ERR_UNSUPPORTED              # causal needs M == N
    assert _ws(_desc(**sm, M=2048, mask=cf.MASK_CAUSAL))[0] == cf.OK
    assert _ws(_desc(**sm, mask=cf.MASK_ADDITIVE)) == (cf.OK, 0)                       # additive mask: fused and unfused
    assert _ws(_desc(**sm, mask=cf.MASK_ADDITIVE, fused=0))[0] == cf.OK
    long_k = dict(sm, K=512, lda=512, N=8192, ldb=8192, ldr=8192, ldy=8192)
    assert _ws(_desc(**long_k)) == (cf.OK, 0)                                          # softmax rows of any length run fused
    assert cf.lib().comfuse_workspace_size(None, None) == cf.ERR_INVALID_ARG


def test_wide_row_and_host_staging_sizes():
    wide = dict(N=8192, ldb=8192, ldr=8192, ldy=8192)
    assert _ws(_desc(**wide)) == (cf.OK, 256 * 2 * 8)                      # fused wide rows: (mean, M2) per row and 4096-column block
    assert _ws(_desc(**wide, kind=cf.EPI_BIAS_GELU_RES_RMSNORM_MAX)) == (cf.OK, 256 * 2 * 8)
    assert _ws(_desc(N=8200, ldb=8200, ldr=8200, ldy=8200)) == (cf.OK, 256 * 33 * 8)   # not a multiple of 4096: 256-column tiles, a partial last one
    long_k = dict(K=1024, lda=1024)                                        # ... or, behind K >= 1024, in 256-column tiles
    assert _ws(_desc(**wide, **long_k)) == (cf.OK, 256 * 32 * 8)
    assert _ws(_desc(N=6144, ldb=6144, ldr=6144, ldy=6144, **long_k)) == (cf.OK, 256 * 24 * 8)
    assert _ws(_desc(N=6144, ldb=6144, ldr=6144, ldy=6144)) == (cf.OK, 256 * 24 * 8)   # no single-kernel form for this row length: any K
    assert _ws(_desc(N=1536, ldb=1536, ldr=1536, ldy=1536)) == (cf.OK, 0)   # K = 512: the on-chip form on a cluster of 6 CTAs
    assert _ws(_desc(N=1536, ldb=1536, ldr=1536, ldy=1536, K=2048, lda=2048)) == (cf.OK, 256 * 6 * 8)   # long K: two kernels
    assert _ws(_desc(N=2560, ldb=2560, ldr=2560, ldy=2560)) == (cf.OK, 256 * 10 * 8)
    assert _ws(_desc(N=1408, ldb=1408, ldr=1408, ldy=1408)) == (cf.OK, 256 * 6 * 8)    # not a multiple of 256: the last tile is partial
    assert _ws(_desc(N=4096, ldb=4096, ldr=4096, ldy=4096, **long_k)) == (cf.OK, 256 * 16 * 8)   # optional for rows that fit a cluster
    d = _desc()                                                            # A [256, 512], B [512, 768], R, Y [256, 768], dense
    n = ctypes.c_size_t(0)
    L = cf.lib()
    assert L.comfuse_host_staging_size(ctypes.byref(d), cf.HOST_A | cf.HOST_RESIDUAL | cf.HOST_Y, ctypes.byref(n)) == cf.OK
    assert n.value == 256 * 512 * 2 + 2 * 256 * 768 * 2                    # already multiples of the 256-byte slot alignment
    assert L.comfuse_host_staging_size(ctypes.byref(d), 0, ctypes.byref(n)) == cf.OK and n.value == 0
    assert L.comfuse_host_staging_size(ctypes.byref(d), 16, ctypes.byref(n)) == cf.ERR_INVALID_ARG      # unknown mask bit
    assert L.comfuse_host_staging_size(None, 1, ctypes.byref(n)) == cf.ERR_INVALID_ARG
    b = cf.make_b2b_desc(1000, 128, 512, 128, 1e-5, True)
    assert L.comfuse_b2b_host_staging_size(ctypes.byref(b), ctypes.byref(n)) == cf.OK
    assert n.value == 2 * 1000 * 128 * 2


def test_pattern_variant_flags_are_checked():
    assert _ws(_desc(flags=cf.FLAG_POST_RELU))[0] == cf.OK                                  # LayerNorm + ReLU
    assert _ws(_desc(flags=cf.FLAG_NO_ACTIVATION))[0] == cf.ERR_INVALID_ARG                 # belongs to the RMSNorm kind
    assert _ws(_desc(kind=cf.EPI_BIAS_GELU_RES_RMSNORM_MAX, flags=cf.FLAG_NO_ACTIVATION))[0] == cf.OK
    assert _ws(_desc(kind=cf.EPI_BIAS_GELU_RES_RMSNORM_MAX, flags=cf.FLAG_POST_RELU))[0] == cf.ERR_INVALID_ARG
    assert _ws(_desc(flags=8))[0] == cf.ERR_INVALID_ARG                                     # unknown bit
    assert _ws(_desc(softcap=30.0))[0] == cf.ERR_INVALID_ARG                                # soft-cap belongs to the softmax kind
    sm = dict(kind=cf.EPI_SCALE_MASK_SOFTMAX, N=2048, ldb=2048, ldr=2048, ldy=2048)
    assert _ws(_desc(**sm, softcap=30.0))[0] == cf.OK
    assert _ws(_desc(**sm, softcap=-1.0))[0] == cf.ERR_INVALID_ARG
    assert _ws(_desc(**sm, softcap=float("nan")))[0] == cf.ERR_INVALID_ARG


def test_gemm_epilogue_rejects_bad_arguments_before_any_launch():
    L = cf.lib()
    d = _desc()
    args = cf.EpilogueArgs(None, None, None, None, None, None, None)
    call = lambda dd, A, B, Y, a, ws, n: L.comfuse_gemm_epilogue(ctypes.byref(dd), A, B, Y, ctypes.byref(a), ws, n, None)
    before = cf.launch_count()
    assert call(d, None, FAKE, FAKE, args, None, 0) == cf.ERR_INVALID_ARG              # NULL operand
    assert call(d, ODD, FAKE, FAKE, args, None, 0) == cf.ERR_ALIGNMENT                 # misaligned operand
    bad = cf.EpilogueArgs(ODD, None, None, None, None, None, None)
    assert call(d, FAKE, FAKE, FAKE, bad, None, 0) == cf.ERR_ALIGNMENT                 # misaligned bias vector
    rms = _desc(kind=cf.EPI_BIAS_GELU_RES_RMSNORM_MAX)
    assert call(rms, FAKE, FAKE, FAKE, args, None, 0) == cf.ERR_INVALID_ARG            # row_max / row_argmax missing
    un = _desc(fused=0)
    assert call(un, FAKE, FAKE, FAKE, args, None, 0) == cf.ERR_WORKSPACE               # unfused without workspace
    assert call(un, FAKE, FAKE, FAKE, args, FAKE, 100) == cf.ERR_WORKSPACE             # ... or with too little
    assert cf.launch_count() == before


def test_b2b_validation():
    L = cf.lib()
    n = ctypes.c_size_t(0)
    ok = cf.make_b2b_desc(1024, 128, 512, 128, fused=True)
    assert L.comfuse_b2b_workspace_size(ctypes.byref(ok), ctypes.byref(n)) == cf.OK and n.value == 0
    un = cf.make_b2b_desc(1024, 128, 512, 128, fused=False)
    assert L.comfuse_b2b_workspace_size(ctypes.byref(un), ctypes.byref(n)) == cf.OK
    assert n.value == (1024 * 512 + 1024 * 128) * 2
    for bad, code in [(cf.make_b2b_desc(1024, 128, 512, 256), cf.ERR_INVALID_ARG),      # residual needs N2 == K
                      (cf.make_b2b_desc(1024, 256, 512, 256), cf.ERR_UNSUPPORTED),      # fused kernel: K = N2 = 128
                      (cf.make_b2b_desc(1024, 128, 4224, 128), cf.ERR_UNSUPPORTED),     # N1 <= 4096
                      (cf.make_b2b_desc(1024, 128, 516, 128), cf.ERR_ALIGNMENT),
                      (cf.make_b2b_desc(0, 128, 512, 128), cf.ERR_INVALID_ARG)]:
        assert L.comfuse_b2b_workspace_size(ctypes.byref(bad), ctypes.byref(n)) == code
    assert L.comfuse_b2b_gemm(ctypes.byref(ok), None, FAKE, FAKE, FAKE, FAKE, None, None, FAKE, None, 0, None) == cf.ERR_INVALID_ARG
    assert L.comfuse_b2b_gemm(ctypes.byref(ok), ODD, FAKE, FAKE, FAKE, FAKE, None, None, FAKE, None, 0, None) == cf.ERR_ALIGNMENT
    # attention form
    A = cf.B2B_SOFTMAX_ATTENTION
    att = cf.make_b2b_desc(4096, 128, 256, 128, 0.0, True, A, 32, 0.088)
    assert L.comfuse_b2b_workspace_size(ctypes.byref(att), ctypes.byref(n)) == cf.OK and n.value == 0
    attu = cf.make_b2b_desc(4096, 128, 256, 128, 0.0, False, A, 32, 0.088)
    assert L.comfuse_b2b_workspace_size(ctypes.byref(attu), ctypes.byref(n)) == cf.OK and n.value == 32 * 4096 * 256 * 2
    for bad, code in [(cf.make_b2b_desc(4096, 128, 512, 128, 0.0, True, A, 2, 0.1), cf.OK),                # fused: N1 <= 512, a multiple of 8
                      (cf.make_b2b_desc(4096, 128, 200, 128, 0.0, True, A, 2, 0.1), cf.OK),                # (positions from N1 on are masked)
                      (cf.make_b2b_desc(4096, 128, 1024, 128, 0.0, True, A, 2, 0.1), cf.ERR_UNSUPPORTED),
                      (cf.make_b2b_desc(4096, 128, 1024, 128, 0.0, False, A, 2, 0.1), cf.OK),              # unfused takes it
                      (cf.make_b2b_desc(4096, 64, 256, 64, 0.0, False, A, 2, 0.1), cf.OK),                  # N2 != K is fine here
                      (cf.make_b2b_desc(4096, 128, 256, 128, 0.0, True, A, 2, 0.0), cf.ERR_INVALID_ARG),   # alpha must be > 0
                      (cf.make_b2b_desc(4096, 128, 256, 128, 0.0, True, A, 0, 0.1), cf.ERR_INVALID_ARG),   # batch >= 1
                      (cf.make_b2b_desc(4096, 128, 256, 128, 0.0, True, 7, 1, 0.1), cf.ERR_INVALID_ARG),   # unknown kind
                      (cf.make_b2b_desc(1024, 128, 512, 128, 1e-5, True, cf.B2B_MLP_GELU_LAYERNORM, 2, 1.0), cf.ERR_INVALID_ARG)]:
        assert L.comfuse_b2b_workspace_size(ctypes.byref(bad), ctypes.byref(n)) == code
    # the attention form has no bias / affine vectors
    assert L.comfuse_b2b_gemm(ctypes.byref(att), FAKE, FAKE, FAKE, FAKE, None, None, None, FAKE, None, 0, None) == cf.ERR_INVALID_ARG
    # the two-layer ReLU MLP kind: K and N2 independent; fused for N2 = 128, N1 <= 512, any K that is a multiple of 8
    R = cf.B2B_MLP_RELU
    relu = cf.make_b2b_desc(32768, 1024, 512, 128, 0.0, True, R)
    assert L.comfuse_b2b_workspace_size(ctypes.byref(relu), ctypes.byref(n)) == cf.OK and n.value == 0
    reluu = cf.make_b2b_desc(32768, 1024, 512, 128, 0.0, False, R)
    assert L.comfuse_b2b_workspace_size(ctypes.byref(reluu), ctypes.byref(n)) == cf.OK and n.value == 32768 * 512 * 2
    for bad, code in [(cf.make_b2b_desc(1024, 8, 256, 128, 0.0, True, R), cf.OK),
                      (cf.make_b2b_desc(1024, 1024, 384, 128, 0.0, True, R), cf.OK),                 # N1: any multiple of 8 up to 512
                      (cf.make_b2b_desc(1024, 1024, 520, 128, 0.0, True, R), cf.ERR_UNSUPPORTED),
                      (cf.make_b2b_desc(1024, 1024, 1024, 128, 0.0, True, R), cf.ERR_UNSUPPORTED),
                      (cf.make_b2b_desc(1024, 1024, 512, 256, 0.0, True, R), cf.ERR_UNSUPPORTED),    # N2: 128
                      (cf.make_b2b_desc(1024, 1024, 1024, 256, 0.0, False, R), cf.OK),               # unfused takes any shape
                      (cf.make_b2b_desc(1024, 1020, 512, 128, 0.0, True, R), cf.ERR_ALIGNMENT),
                      (cf.make_b2b_desc(1024, 1024, 512, 128, 0.0, True, R, 2), cf.ERR_INVALID_ARG)]:  # batch must be 1
        assert L.comfuse_b2b_workspace_size(ctypes.byref(bad), ctypes.byref(n)) == code
    # no LayerNorm vectors in this kind
    assert L.comfuse_b2b_gemm(ctypes.byref(relu), FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, None, FAKE, None, 0, None) == cf.ERR_INVALID_ARG


def test_valid_call_without_a_usable_gpu_fails_cleanly():
    """On a machine with no CUDA device a well-formed call must come back with an error code, not crash and not fall
    back to anything else."""
    import torch
    if torch.cuda.is_available():
        return
    L = cf.lib()
    d = _desc()
    args = cf.EpilogueArgs(None, None, None, None, None, None, None)
    st = L.comfuse_gemm_epilogue(ctypes.byref(d), FAKE, FAKE, FAKE, ctypes.byref(args), None, 0, None)
    assert st in (cf.ERR_CUDA, cf.ERR_ARCH)
    assert cf.lib().comfuse_last_device_status(None) in (cf.ERR_CUDA, cf.ERR_ARCH)


def test_b2b_flags_are_checked():
    """The attention kind's layout flag: unknown bits and the flag on another kind are refused on the host."""
    L = cf.lib()
    n = ctypes.c_size_t(0)
    att = cf.make_b2b_desc(256, 128, 256, 128, 0.0, True, cf.B2B_SOFTMAX_ATTENTION, 2, 0.1, cf.B2B_FLAG_KEYS_ROW_MAJOR)
    assert L.comfuse_b2b_workspace_size(ctypes.byref(att), ctypes.byref(n)) == cf.OK and n.value == 0
    att.fused = 0
    assert L.comfuse_b2b_workspace_size(ctypes.byref(att), ctypes.byref(n)) == cf.OK
    assert n.value == 2 * 256 * 256 * 2                              # the scores; the keys are read in place
    att.flags = 2
    assert L.comfuse_b2b_workspace_size(ctypes.byref(att), ctypes.byref(n)) == cf.ERR_INVALID_ARG
    mlp = cf.make_b2b_desc(256, 128, 512, 128, 1e-5, True, cf.B2B_MLP_GELU_LAYERNORM, 1, 1.0, cf.B2B_FLAG_KEYS_ROW_MAJOR)
    assert L.comfuse_b2b_workspace_size(ctypes.byref(mlp), ctypes.byref(n)) == cf.ERR_INVALID_ARG


def test_second_operand_layout_flag_rules():
    """COMFUSE_FLAG_B_ROW_MAJOR_NK: ldb counts contraction elements, every kind takes it fused and unfused with the usual
    workspace, the host-buffer form stages the operand with its own extent."""
    nk = dict(flags=cf.FLAG_B_ROW_MAJOR_NK, ldb=512)                       # B [768, 512]: ldb >= K
    assert _ws(_desc(**nk)) == (cf.OK, 0)                                   # LayerNorm kind, fused
    assert _ws(_desc(fused=0, **nk)) == (cf.OK, 256 * 768 * 2)
    assert _ws(_desc(fused=0, flags=cf.FLAG_B_ROW_MAJOR_NK, ldb=504))[0] == cf.ERR_INVALID_ARG   # ldb < K
    sm = dict(kind=cf.EPI_SCALE_MASK_SOFTMAX, N=2048, ldr=2048, ldy=2048, K=64, lda=64, flags=cf.FLAG_B_ROW_MAJOR_NK, ldb=64)
    assert _ws(_desc(**sm)) == (cf.OK, 0)
    assert _ws(_desc(**dict(sm, K=512, lda=512, ldb=512))) == (cf.OK, 0)   # long K: still the row kernel
    assert _ws(_desc(flags=8))[0] == cf.ERR_INVALID_ARG                     # unknown bit
    n = ctypes.c_size_t(0)
    d = _desc(**sm)
    assert cf.lib().comfuse_host_staging_size(ctypes.byref(d), cf.HOST_B, ctypes.byref(n)) == cf.OK
    assert n.value == 2048 * 64 * 2                                         # the operand's own extent, [N, K]
