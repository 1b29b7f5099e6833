"""Python binding of libcomfuse.so -- argument marshalling only.

Every step of the hot path (GEMM, epilogue subgraph, reductions, stores) runs inside the CUDA library; this
module turns torch tensors into the plain pointers and sizes of the C ABI declared in include/comfuse.h and
raises if the library reports an error.  There is no CPU fallback: if the shared library is missing the
import of :func:`lib` fails loudly.

Functions mirror the C entry points:
    gemm_epilogue(...)      -> comfuse_gemm_epilogue      (GEMM -> elementwise/reduction subgraph, Sec. 3)
    gemm_epilogue_static_scratch(...) -> comfuse_gemm_epilogue_static_scratch (unfused path, no caller workspace)
    gemm_epilogue_host(...) -> comfuse_gemm_epilogue_host (per-step tensors in host memory, staged through a device buffer)
    b2b_gemm_host(...)      -> comfuse_b2b_gemm_host
    b2b_gemm(...)           -> comfuse_b2b_gemm           (GEMM -> F -> GEMM -> post-norm tail, Sec. 4)
    workspace_size(...)     -> comfuse_workspace_size
    b2b_workspace_size(...) -> comfuse_b2b_workspace_size
    last_device_status()    -> comfuse_last_device_status
    selftest_bounded_wait() -> comfuse_selftest_bounded_wait
    launch_count()          -> comfuse_launch_count
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_float, c_int32, c_int64, c_size_t, c_uint64, c_void_p

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("COMFUSE_LIB") or os.path.join(_PKG_DIR, "libcomfuse.so")   # COMFUSE_LIB: e.g. the checked build

# status codes / enums of include/comfuse.h
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_ARCH, ERR_CUDA, ERR_TIMEOUT = range(8)
ERR_BOUNDS = 8   # checked build only: a bounds predicate failed, the access was skipped
EPI_BIAS_RES_LAYERNORM, EPI_BIAS_GELU_RES_RMSNORM_MAX, EPI_SCALE_MASK_SOFTMAX = 0, 1, 2
EPI_BIAS_ACTIVATION = 3   # reduction-free epilogue; reached through gemm_spec only
MASK_NONE, MASK_CAUSAL, MASK_ADDITIVE = 0, 1, 2
HOST_A, HOST_B, HOST_RESIDUAL, HOST_Y = 1, 2, 4, 8
FLAG_POST_RELU, FLAG_NO_ACTIVATION, FLAG_B_ROW_MAJOR_NK = 1, 2, 4
B2B_MLP_GELU_LAYERNORM, B2B_SOFTMAX_ATTENTION, B2B_MLP_RELU = 0, 1, 2
B2B_FLAG_KEYS_ROW_MAJOR = 1   # attention kind: W1 is [batch, N1, K] (one key per row)

EXPORTED_SYMBOLS = (
    "comfuse_workspace_size",
    "comfuse_gemm_epilogue",
    "comfuse_gemm_epilogue_static_scratch",
    "comfuse_b2b_workspace_size",
    "comfuse_b2b_gemm",
    "comfuse_host_staging_size",
    "comfuse_gemm_epilogue_host",
    "comfuse_b2b_host_staging_size",
    "comfuse_b2b_gemm_host",
    "comfuse_spec_plan",
    "comfuse_gemm_spec_workspace_size",
    "comfuse_gemm_spec",
    "comfuse_gemm_spec_prepare",
    "comfuse_program_compiler_status",
    "comfuse_selftest_bounds_predicate",
    "comfuse_last_device_status",
    "comfuse_launch_count",
    "comfuse_selftest_bounded_wait",
    "comfuse_status_string",
)


class GemmDesc(Structure):
    _fields_ = [
        ("batch", c_int32), ("M", c_int32), ("N", c_int32), ("K", c_int32),
        ("lda", c_int64), ("ldb", c_int64), ("ldr", c_int64), ("ldy", c_int64),
        ("batch_stride_a", c_int64), ("batch_stride_b", c_int64), ("batch_stride_r", c_int64), ("batch_stride_y", c_int64),
        ("kind", c_int32), ("mask", c_int32), ("alpha", c_float), ("eps", c_float),
        ("fused", c_int32), ("flags", ctypes.c_uint32), ("softcap", c_float), ("reserved", c_int32),
    ]


class EpilogueArgs(Structure):
    _fields_ = [
        ("bias", c_void_p), ("residual", c_void_p), ("gamma", c_void_p), ("beta", c_void_p), ("mask", c_void_p),
        ("row_max", c_void_p), ("row_argmax", c_void_p),
    ]


class B2bDesc(Structure):
    _fields_ = [("M", c_int32), ("K", c_int32), ("N1", c_int32), ("N2", c_int32), ("eps", c_float), ("fused", c_int32),
                ("kind", c_int32), ("batch", c_int32), ("alpha", c_float), ("flags", c_int32)]


# Epilogue programs as data: the node vocabulary (comfuse_op_t), by name
OPS = {
    "acc": 0, "const": 1, "rowvec": 2, "tensor": 3, "causal_mask": 4,
    "neg": 16, "abs": 17, "square": 18, "sqrt": 19, "rsqrt": 20, "recip": 21, "exp": 22, "log": 23, "tanh": 24,
    "relu": 25, "gelu_tanh": 26, "sigmoid": 27,
    "add": 32, "sub": 33, "mul": 34, "div": 35, "max": 36, "min": 37,
    "sum": 48, "mean": 49, "rmax": 50, "rmin": 51, "prod": 52, "argmax": 53, "topk_values": 54, "topk_indices": 55,
}
SPEC_PATH_FUSED_KERNEL = 0
SPEC_PATH_ROW_PROGRAM = 1
SPEC_PATH_FUSED_PROGRAM = 2


class SpecNode(Structure):
    _fields_ = [("op", c_int32), ("in0", c_int32), ("in1", c_int32), ("param", c_int32), ("imm", c_float)]


class FusionSpec(Structure):
    _fields_ = [("n_nodes", c_int32), ("nodes", POINTER(SpecNode)), ("terminal", c_int32), ("n_params", c_int32),
                ("n_row_outputs", c_int32), ("row_outputs", POINTER(c_int32))]


class GemmShape(Structure):
    _fields_ = [("batch", c_int32), ("M", c_int32), ("N", c_int32), ("K", c_int32),
                ("lda", c_int64), ("ldb", c_int64), ("ldy", c_int64),
                ("batch_stride_a", c_int64), ("batch_stride_b", c_int64), ("batch_stride_y", c_int64), ("flags", ctypes.c_uint32)]


class SpecPlan(Structure):
    _fields_ = [("n_stages", c_int32), ("n_reductions", c_int32), ("n_live_nodes", c_int32), ("path", c_int32),
                ("program_path", c_int32), ("n_passes", c_int32),
                ("fused_kind", c_int32), ("fused_flags", ctypes.c_uint32), ("alpha", c_float), ("eps", c_float),
                ("softcap", c_float), ("causal", c_int32), ("n_instructions", c_int32), ("n_slots", c_int32)]


class ComfuseError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        msg = lib().comfuse_status_string(self.status).decode()
        super().__init__(f"{where}: {msg} (status {self.status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load libcomfuse.so (built by ``python -m paper_2608_03537_b200.build``).  Fails loudly if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} not found: build the CUDA library first (python -m paper_2608_03537_b200.build). "
                "There is no CPU fallback."
            )
        L = ctypes.CDLL(LIB_PATH)
        L.comfuse_workspace_size.argtypes = [POINTER(GemmDesc), POINTER(c_size_t)]
        L.comfuse_workspace_size.restype = c_int32
        L.comfuse_gemm_epilogue.argtypes = [POINTER(GemmDesc), c_void_p, c_void_p, c_void_p, POINTER(EpilogueArgs),
                                            c_void_p, c_size_t, c_void_p]
        L.comfuse_gemm_epilogue.restype = c_int32
        L.comfuse_gemm_epilogue_static_scratch.argtypes = [POINTER(GemmDesc), c_void_p, c_void_p, c_void_p, POINTER(EpilogueArgs), c_void_p]
        L.comfuse_gemm_epilogue_static_scratch.restype = c_int32
        L.comfuse_b2b_workspace_size.argtypes = [POINTER(B2bDesc), POINTER(c_size_t)]
        L.comfuse_b2b_workspace_size.restype = c_int32
        L.comfuse_b2b_gemm.argtypes = [POINTER(B2bDesc)] + [c_void_p] * 8 + [c_void_p, c_size_t, c_void_p]
        L.comfuse_b2b_gemm.restype = c_int32
        L.comfuse_host_staging_size.argtypes = [POINTER(GemmDesc), ctypes.c_uint32, POINTER(c_size_t)]
        L.comfuse_host_staging_size.restype = c_int32
        L.comfuse_gemm_epilogue_host.argtypes = [POINTER(GemmDesc), c_void_p, c_void_p, c_void_p, POINTER(EpilogueArgs),
                                                 ctypes.c_uint32, c_void_p, c_size_t, c_void_p, c_size_t, c_void_p]
        L.comfuse_gemm_epilogue_host.restype = c_int32
        L.comfuse_b2b_host_staging_size.argtypes = [POINTER(B2bDesc), POINTER(c_size_t)]
        L.comfuse_b2b_host_staging_size.restype = c_int32
        L.comfuse_b2b_gemm_host.argtypes = [POINTER(B2bDesc)] + [c_void_p] * 8 + [c_void_p, c_size_t, c_void_p, c_size_t, c_void_p]
        L.comfuse_b2b_gemm_host.restype = c_int32
        L.comfuse_spec_plan.argtypes = [POINTER(FusionSpec), POINTER(GemmShape), POINTER(SpecPlan)]
        L.comfuse_spec_plan.restype = c_int32
        L.comfuse_gemm_spec_workspace_size.argtypes = [POINTER(FusionSpec), POINTER(GemmShape), c_int32, POINTER(c_size_t)]
        L.comfuse_gemm_spec_workspace_size.restype = c_int32
        L.comfuse_gemm_spec.argtypes = [POINTER(FusionSpec), POINTER(GemmShape), c_void_p, c_void_p, c_void_p, POINTER(c_void_p),
                                        POINTER(c_int64), POINTER(c_void_p), c_int32, c_void_p, c_size_t, c_void_p]
        L.comfuse_gemm_spec.restype = c_int32
        L.comfuse_gemm_spec_prepare.argtypes = [POINTER(FusionSpec), POINTER(GemmShape), c_int32]
        L.comfuse_gemm_spec_prepare.restype = c_int32
        L.comfuse_program_compiler_status.argtypes = [POINTER(ctypes.c_char_p)]
        L.comfuse_program_compiler_status.restype = c_int32
        L.comfuse_last_device_status.argtypes = [c_void_p]
        L.comfuse_last_device_status.restype = c_int32
        L.comfuse_selftest_bounded_wait.argtypes = [ctypes.c_uint32, c_void_p, POINTER(ctypes.c_uint32)]
        L.comfuse_selftest_bounded_wait.restype = c_int32
        L.comfuse_selftest_bounds_predicate.argtypes = [c_void_p, POINTER(c_int32)]
        L.comfuse_selftest_bounds_predicate.restype = c_int32
        L.comfuse_launch_count.argtypes = []
        L.comfuse_launch_count.restype = c_uint64
        L.comfuse_status_string.argtypes = [c_int32]
        L.comfuse_status_string.restype = ctypes.c_char_p
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return c_void_p(s.cuda_stream)


def make_gemm_desc(A, B, Y, kind, *, residual=None, alpha=1.0, eps=1e-5, mask=MASK_NONE, fused=True, flags=0,
                   softcap=0.0) -> GemmDesc:
    """Describe A [b, M, K] (or [M, K]), B [b, K, N] (or [K, N]; with FLAG_B_ROW_MAJOR_NK in ``flags``: [b, N, K]),
    Y [b, M, N] from torch tensors' shapes and strides."""
    batched = A.dim() == 3
    batch = A.shape[0] if batched else 1
    M, K = A.shape[-2], A.shape[-1]
    b_nk = bool(int(flags) & FLAG_B_ROW_MAJOR_NK)
    N = B.shape[-2] if b_nk else B.shape[-1]
    assert (B.shape[-1] if b_nk else B.shape[-2]) == K and Y.shape[-2] == M and Y.shape[-1] == N
    assert A.stride(-1) == 1 and B.stride(-1) == 1 and Y.stride(-1) == 1
    d = GemmDesc()
    d.batch, d.M, d.N, d.K = batch, M, N, K
    d.lda, d.ldb, d.ldy = A.stride(-2), B.stride(-2), Y.stride(-2)
    d.ldr = residual.stride(-2) if residual is not None else N
    d.batch_stride_a = A.stride(0) if batched else M * d.lda
    d.batch_stride_b = B.stride(0) if batched else (N if b_nk else K) * d.ldb
    d.batch_stride_y = Y.stride(0) if batched else M * d.ldy
    d.batch_stride_r = (residual.stride(0) if batched else M * d.ldr) if residual is not None else M * N
    d.kind, d.mask, d.alpha, d.eps, d.fused, d.reserved = int(kind), int(mask), float(alpha), float(eps), int(bool(fused)), 0
    d.flags, d.softcap = int(flags), float(softcap)
    return d


def workspace_size(desc: GemmDesc) -> int:
    n = c_size_t(0)
    st = lib().comfuse_workspace_size(byref(desc), byref(n))
    if st != OK:
        raise ComfuseError(st, "comfuse_workspace_size")
    return int(n.value)


def gemm_epilogue(A, B, Y, kind, *, bias=None, residual=None, gamma=None, beta=None, mask_tensor=None, row_max=None,
                  row_argmax=None, alpha=1.0, eps=1e-5, mask=MASK_NONE, fused=True, workspace=None, stream=None, flags=0,
                  softcap=0.0):
    """Enqueue Y = subgraph(alpha * A.B) on the current (or given) stream.  Tensors are CUDA bf16 (row_max fp32,
    row_argmax int32).  ``workspace`` is a CUDA uint8 tensor of at least workspace_size(desc) bytes (unfused path, and fused LayerNorm /
    RMSNorm rows wider than 4096 columns)."""
    d = make_gemm_desc(A, B, Y, kind, residual=residual, alpha=alpha, eps=eps, mask=mask, fused=fused, flags=flags, softcap=softcap)
    args = EpilogueArgs(_ptr(bias), _ptr(residual), _ptr(gamma), _ptr(beta), _ptr(mask_tensor), _ptr(row_max), _ptr(row_argmax))
    ws_ptr, ws_bytes = (None, 0) if workspace is None else (c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size())
    st = lib().comfuse_gemm_epilogue(byref(d), _ptr(A), _ptr(B), _ptr(Y), byref(args), ws_ptr, ws_bytes, _stream(stream))
    if st != OK:
        raise ComfuseError(st, "comfuse_gemm_epilogue")
    return Y


STATIC_SCRATCH_BYTES = 16 << 20


def gemm_epilogue_static_scratch(A, B, Y, kind, *, bias=None, residual=None, gamma=None, beta=None, mask_tensor=None,
                                 row_max=None, row_argmax=None, alpha=1.0, eps=1e-5, mask=MASK_NONE, flags=0, softcap=0.0,
                                 stream=None):
    """The unfused GEMM -> row-kernel path for callers that cannot allocate a workspace (a loop in which cudaMalloc is not
    allowed, a plug-in without access to the host framework's allocator): the intermediate lives in a fixed
    STATIC_SCRATCH_BYTES array inside the library.  batch*M*N*2 bytes must fit; calls that may overlap on the GPU race
    on that array; the first call on a device sets the array up and should come before any stream capture."""
    d = make_gemm_desc(A, B, Y, kind, residual=residual, alpha=alpha, eps=eps, mask=mask, fused=False, flags=flags, softcap=softcap)
    args = EpilogueArgs(_ptr(bias), _ptr(residual), _ptr(gamma), _ptr(beta), _ptr(mask_tensor), _ptr(row_max), _ptr(row_argmax))
    st = lib().comfuse_gemm_epilogue_static_scratch(byref(d), _ptr(A), _ptr(B), _ptr(Y), byref(args), _stream(stream))
    if st != OK:
        raise ComfuseError(st, "comfuse_gemm_epilogue_static_scratch")
    return Y


def make_b2b_desc(M, K, N1, N2, eps=1e-5, fused=True, kind=B2B_MLP_GELU_LAYERNORM, batch=1, alpha=1.0, flags=0) -> B2bDesc:
    return B2bDesc(int(M), int(K), int(N1), int(N2), float(eps), int(bool(fused)), int(kind), int(batch), float(alpha), int(flags))


def b2b_attention(Q, Kt, V, O, *, alpha, fused=True, workspace=None, stream=None, keys_row_major=False):
    """Enqueue O = softmax(alpha * Q.Kt).V per batch (the attention form of the back-to-back GEMM).  Dense CUDA bf16
    tensors Q [b, M, d], Kt [b, d, S] (keys already transposed) or, with ``keys_row_major``, the keys as [b, S, d];
    V [b, S, d2], O [b, M, d2]."""
    nb, M, K = Q.shape
    N1, N2 = V.shape[1], V.shape[2]
    assert Kt.shape == ((nb, N1, K) if keys_row_major else (nb, K, N1)) and V.shape == (nb, N1, N2) and O.shape == (nb, M, N2)
    for t in (Q, Kt, V, O):
        assert t.is_contiguous()
    d = make_b2b_desc(M, K, N1, N2, 0.0, fused, B2B_SOFTMAX_ATTENTION, nb, alpha, B2B_FLAG_KEYS_ROW_MAJOR if keys_row_major else 0)
    ws_ptr, ws_bytes = (None, 0) if workspace is None else (c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size())
    st = lib().comfuse_b2b_gemm(byref(d), _ptr(Q), _ptr(Kt), None, _ptr(V), None, None, None, _ptr(O), ws_ptr, ws_bytes, _stream(stream))
    if st != OK:
        raise ComfuseError(st, "comfuse_b2b_gemm")
    return O


def host_staging_size(desc: GemmDesc, host_mask: int) -> int:
    n = c_size_t(0)
    st = lib().comfuse_host_staging_size(byref(desc), int(host_mask), byref(n))
    if st != OK:
        raise ComfuseError(st, "comfuse_host_staging_size")
    return int(n.value)


def gemm_epilogue_host(A, B, Y, kind, *, staging, host_mask, bias=None, residual=None, gamma=None, beta=None,
                       mask_tensor=None, row_max=None, row_argmax=None, alpha=1.0, eps=1e-5, mask=MASK_NONE, fused=True,
                       workspace=None, stream=None, flags=0):
    """gemm_epilogue with the tensors named in ``host_mask`` (HOST_A | HOST_B | HOST_RESIDUAL | HOST_Y) living in host
    memory (CPU tensors, pinned for asynchronous copies); ``staging`` is a CUDA uint8 tensor of at least
    host_staging_size(desc, host_mask) bytes.  Copies and kernels are enqueued on the stream; nothing synchronises."""
    d = make_gemm_desc(A, B, Y, kind, residual=residual, alpha=alpha, eps=eps, mask=mask, fused=fused, flags=flags)
    args = EpilogueArgs(_ptr(bias), _ptr(residual), _ptr(gamma), _ptr(beta), _ptr(mask_tensor), _ptr(row_max), _ptr(row_argmax))
    ws_ptr, ws_bytes = (None, 0) if workspace is None else (c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size())
    st = lib().comfuse_gemm_epilogue_host(byref(d), _ptr(A), _ptr(B), _ptr(Y), byref(args), int(host_mask),
                                          c_void_p(staging.data_ptr()), staging.numel() * staging.element_size(),
                                          ws_ptr, ws_bytes, _stream(stream))
    if st != OK:
        raise ComfuseError(st, "comfuse_gemm_epilogue_host")
    return Y


def b2b_workspace_size(desc: B2bDesc) -> int:
    n = c_size_t(0)
    st = lib().comfuse_b2b_workspace_size(byref(desc), byref(n))
    if st != OK:
        raise ComfuseError(st, "comfuse_b2b_workspace_size")
    return int(n.value)


def b2b_gemm(X, W1, b1, W2, b2, O, *, gamma=None, beta=None, eps=1e-5, fused=True, workspace=None, stream=None):
    """Enqueue O = LayerNorm(GELU_tanh(X.W1 + b1).W2 + b2 + X) * gamma + beta.  Dense row-major CUDA bf16 tensors."""
    M, K = X.shape
    N1, N2 = W1.shape[1], W2.shape[1]
    for t in (X, W1, W2, O):
        assert t.is_contiguous()
    d = make_b2b_desc(M, K, N1, N2, eps, fused)
    ws_ptr, ws_bytes = (None, 0) if workspace is None else (c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size())
    st = lib().comfuse_b2b_gemm(byref(d), _ptr(X), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), _ptr(gamma), _ptr(beta), _ptr(O),
                                ws_ptr, ws_bytes, _stream(stream))
    if st != OK:
        raise ComfuseError(st, "comfuse_b2b_gemm")
    return O


def b2b_mlp_relu(X, W1, b1, W2, b2, O, *, fused=True, workspace=None, stream=None):
    """Enqueue O = ReLU(ReLU(X.W1 + b1).W2 + b2) (the two-layer ReLU MLP form of the back-to-back GEMM).  Dense row-major
    CUDA bf16 tensors X [M, K], W1 [K, N1], W2 [N1, N2], O [M, N2]; b1, b2 may be None."""
    M, K = X.shape
    N1, N2 = W1.shape[1], W2.shape[1]
    assert W1.shape == (K, N1) and W2.shape == (N1, N2) and O.shape == (M, N2)
    for t in (X, W1, W2, O):
        assert t.is_contiguous()
    d = make_b2b_desc(M, K, N1, N2, 0.0, fused, B2B_MLP_RELU)
    ws_ptr, ws_bytes = (None, 0) if workspace is None else (c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size())
    st = lib().comfuse_b2b_gemm(byref(d), _ptr(X), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), None, None, _ptr(O),
                                ws_ptr, ws_bytes, _stream(stream))
    if st != OK:
        raise ComfuseError(st, "comfuse_b2b_gemm")
    return O


def b2b_mlp_relu_host(X, W1, b1, W2, b2, O, *, staging, fused=True, workspace=None, stream=None):
    """b2b_mlp_relu with X and O in host memory (dense CPU tensors, pinned for asynchronous copies)."""
    M, K = X.shape
    N1, N2 = W1.shape[1], W2.shape[1]
    for t in (X, W1, W2, O):
        assert t.is_contiguous()
    d = make_b2b_desc(M, K, N1, N2, 0.0, fused, B2B_MLP_RELU)
    ws_ptr, ws_bytes = (None, 0) if workspace is None else (c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size())
    st = lib().comfuse_b2b_gemm_host(byref(d), _ptr(X), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), None, None, _ptr(O),
                                     c_void_p(staging.data_ptr()), staging.numel() * staging.element_size(),
                                     ws_ptr, ws_bytes, _stream(stream))
    if st != OK:
        raise ComfuseError(st, "comfuse_b2b_gemm_host")
    return O


def b2b_host_staging_size(desc: B2bDesc) -> int:
    n = c_size_t(0)
    st = lib().comfuse_b2b_host_staging_size(byref(desc), byref(n))
    if st != OK:
        raise ComfuseError(st, "comfuse_b2b_host_staging_size")
    return int(n.value)


def b2b_gemm_host(X, W1, b1, W2, b2, O, *, staging, gamma=None, beta=None, eps=1e-5, fused=True, workspace=None, stream=None):
    """b2b_gemm with X and O in host memory (dense CPU tensors, pinned for asynchronous copies); weights and vectors are
    CUDA tensors; ``staging`` is a CUDA uint8 tensor of at least b2b_host_staging_size(desc) bytes."""
    M, K = X.shape
    N1, N2 = W1.shape[1], W2.shape[1]
    for t in (X, W1, W2, O):
        assert t.is_contiguous()
    d = make_b2b_desc(M, K, N1, N2, eps, fused)
    ws_ptr, ws_bytes = (None, 0) if workspace is None else (c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size())
    st = lib().comfuse_b2b_gemm_host(byref(d), _ptr(X), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), _ptr(gamma), _ptr(beta), _ptr(O),
                                     c_void_p(staging.data_ptr()), staging.numel() * staging.element_size(),
                                     ws_ptr, ws_bytes, _stream(stream))
    if st != OK:
        raise ComfuseError(st, "comfuse_b2b_gemm_host")
    return O


def b2b_attention_host(Q, Kt, V, O, *, staging, alpha, fused=True, workspace=None, stream=None, keys_row_major=False):
    """b2b_attention with Q, Kt, V and O in host memory (dense CPU tensors, pinned for asynchronous copies); ``staging`` is a
    CUDA uint8 tensor of at least b2b_host_staging_size(desc) bytes."""
    nb, M, K = Q.shape
    N1, N2 = V.shape[1], V.shape[2]
    for t in (Q, Kt, V, O):
        assert t.is_contiguous()
    d = make_b2b_desc(M, K, N1, N2, 0.0, fused, B2B_SOFTMAX_ATTENTION, nb, alpha, B2B_FLAG_KEYS_ROW_MAJOR if keys_row_major else 0)
    ws_ptr, ws_bytes = (None, 0) if workspace is None else (c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size())
    st = lib().comfuse_b2b_gemm_host(byref(d), _ptr(Q), _ptr(Kt), None, _ptr(V), None, None, None, _ptr(O),
                                     c_void_p(staging.data_ptr()), staging.numel() * staging.element_size(),
                                     ws_ptr, ws_bytes, _stream(stream))
    if st != OK:
        raise ComfuseError(st, "comfuse_b2b_gemm_host")
    return O


def make_spec(nodes, terminal, n_params=0, row_outputs=()) -> FusionSpec:
    """Pack a node list ``[(op name or code, in0, in1, param, imm), ...]`` into the C structure (host arrays are kept
    alive by the returned object)."""
    arr = (SpecNode * len(nodes))()
    for k, (op, a, b, prm, imm) in enumerate(nodes):
        arr[k] = SpecNode(OPS[op] if isinstance(op, str) else int(op), int(a), int(b), int(prm), float(imm))
    ro = (c_int32 * max(1, len(row_outputs)))(*[int(r) for r in row_outputs])
    spec = FusionSpec(len(nodes), ctypes.cast(arr, POINTER(SpecNode)), int(terminal), int(n_params), len(row_outputs),
                      ctypes.cast(ro, POINTER(c_int32)))
    spec._keep = (arr, ro)
    return spec


def make_gemm_shape(batch, M, N, K, lda=None, ldb=None, ldy=None, batch_stride_a=None, batch_stride_b=None,
                    batch_stride_y=None, flags=0) -> GemmShape:
    """Dense shapes by default; ``flags=FLAG_B_ROW_MAJOR_NK``: B is stored [batch, N, K]."""
    b_nk = bool(int(flags) & FLAG_B_ROW_MAJOR_NK)
    lda, ldb, ldy = lda or K, ldb or (K if b_nk else N), ldy or N
    return GemmShape(batch, M, N, K, lda, ldb, ldy, batch_stride_a or M * lda, batch_stride_b or (N if b_nk else K) * ldb,
                     batch_stride_y or M * ldy, int(flags))


def spec_plan(spec: FusionSpec, shape: GemmShape) -> SpecPlan:
    """Host-side analysis of a program on a shape (needs no GPU): stages, path, recovered constants."""
    plan = SpecPlan()
    st = lib().comfuse_spec_plan(byref(spec), byref(shape), byref(plan))
    if st != OK:
        raise ComfuseError(st, "comfuse_spec_plan")
    return plan


def gemm_spec_workspace_size(spec: FusionSpec, shape: GemmShape, fused=True) -> int:
    n = c_size_t(0)
    st = lib().comfuse_gemm_spec_workspace_size(byref(spec), byref(shape), int(fused), byref(n))
    if st != OK:
        raise ComfuseError(st, "comfuse_gemm_spec_workspace_size")
    return int(n.value)


GENERATED = 3   # `fused` value of the spec calls: the kernel generated (compiled at run time) for the program


def program_compiler_status():
    """(status, reason): OK and "" when programs can be compiled at run time on this machine (needs no GPU)."""
    why = ctypes.c_char_p()
    st = int(lib().comfuse_program_compiler_status(byref(why)))
    return st, (why.value or b"").decode()


def gemm_spec_prepare(spec: FusionSpec, shape: GemmShape, fused=GENERATED) -> None:
    """Compile ahead of the first launch what gemm_spec(..., fused=fused) would compile on it (needs no GPU)."""
    st = lib().comfuse_gemm_spec_prepare(byref(spec), byref(shape), int(fused))
    if st != OK:
        raise ComfuseError(st, "comfuse_gemm_spec_prepare")


def gemm_spec(A, B, Y, spec: FusionSpec, *, params=(), row_out=(), fused=True, workspace=None, stream=None, b_nk=False):
    """Enqueue Y = program(A.B): ``spec`` from make_spec, ``params`` the CUDA bf16 tensors of the parameter table
    (row vectors [N], tensors [batch, M, N]), ``row_out`` the per-row output tensors (fp32, int32 for an arg max);
    ``b_nk``: B is stored [batch, N, K].  ``fused``: 1 best path, 2 on-chip interpreter, 0 row program, GENERATED (3) the
    kernel compiled for this program (the first call compiles it: seconds)."""
    batched = A.dim() == 3
    batch = A.shape[0] if batched else 1
    M, K = A.shape[-2], A.shape[-1]
    N = B.shape[-2] if b_nk else B.shape[-1]
    shape = make_gemm_shape(batch, M, N, K, A.stride(-2), B.stride(-2), Y.stride(-2),
                            A.stride(0) if batched else None, B.stride(0) if batched else None, Y.stride(0) if batched else None,
                            flags=FLAG_B_ROW_MAJOR_NK if b_nk else 0)
    n = max(1, len(params))
    pp = (c_void_p * n)(*[None if t is None else t.data_ptr() for t in params])
    ld = (c_int64 * n)(*[0 if (t is None or t.dim() < 2) else t.stride(-2) for t in params])
    ro = (c_void_p * max(1, len(row_out)))(*[t.data_ptr() for t in row_out])
    ws_ptr, ws_bytes = (None, 0) if workspace is None else (c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size())
    st = lib().comfuse_gemm_spec(byref(spec), byref(shape), _ptr(A), _ptr(B), _ptr(Y), pp, ld, ro, int(fused),
                                 ws_ptr, ws_bytes, _stream(stream))
    if st != OK:
        raise ComfuseError(st, "comfuse_gemm_spec")
    return Y


def last_device_status(stream=None) -> int:
    """Synchronise the stream and return (and clear) the device status word: OK, ERR_TIMEOUT, or (checked build) ERR_BOUNDS."""
    return int(lib().comfuse_last_device_status(_stream(stream)))


def selftest_bounded_wait(timeout_ms: int = 20, stream=None) -> int:
    """Run the bounded-wait self-test kernel; returns how many of its 64 threads saw an expired or aborted wait.  The
    device status word reads ERR_TIMEOUT afterwards (last_device_status() returns and clears it)."""
    n = ctypes.c_uint32(0)
    st = lib().comfuse_selftest_bounded_wait(int(timeout_ms), _stream(stream), byref(n))
    if st != OK:
        raise ComfuseError(st, "comfuse_selftest_bounded_wait")
    return int(n.value)


def selftest_bounds_predicate(stream=None) -> bool:
    """Run the bounds-predicate self-test kernel; returns whether the loaded library is the checked build.  In that build
    the device status word reads ERR_BOUNDS afterwards, in the ordinary build OK; no access is out of bounds in either."""
    flag = ctypes.c_int32(-1)
    st = lib().comfuse_selftest_bounds_predicate(_stream(stream), byref(flag))
    if st != OK:
        raise ComfuseError(st, "comfuse_selftest_bounds_predicate")
    return bool(flag.value)


def launch_count() -> int:
    return int(lib().comfuse_launch_count())
