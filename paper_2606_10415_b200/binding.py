"""ctypes binding of the C-ABI library (``include/lt_attn.h``), same names as the C entry points.

Argument marshalling only: torch is used to hold device memory and streams; every
step of the attention path runs inside the library's kernels.  There is no CPU
fallback -- if ``liblt_attn.so`` is missing the import fails.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "liblt_attn.so"

LT_OK = 0
LT_ERR_INVALID_ARG = 1
LT_ERR_UNSUPPORTED = 2
LT_ERR_WORKSPACE = 3
LT_ERR_CUDA = 4
LT_ERR_DEVICE_TIMEOUT = 5

EXPORTS = (
    "lt_attn_fwd_workspace_bytes", "lt_attn_bwd_workspace_bytes", "lt_attn_fwd", "lt_attn_bwd",
    "lt_attn_bwd_profiled", "lt_attn_bwd_noalloc", "lt_attn_fwd_strided", "lt_attn_bwd_strided",
    "lt_attn_fwd_bf16", "lt_attn_bwd_bf16", "lt_attn_p_store_bytes", "lt_attn_save_p", "lt_attn_bwd_saved_p",
    "lt_gemm_f16", "lt_gemm_bf16", "lt_gemm_f16_workspace_bytes",
    "lt_attn_host_arena_bytes", "lt_attn_fwd_bwd_host", "lt_attn_check_status", "lt_status_string",
    "lt_last_cuda_error", "lt_attn_bwd_num_launches", "lt_attn_fwd_num_launches", "lt_attn_bwd_noalloc_check_status",
)
# test-support entry points (include/lt_attn_debug.h)
DEBUG_EXPORTS = ("lt_dbg_tile_gemm", "lt_dbg_wait_timeout")


class TensorStrides(ctypes.Structure):
    """Element strides of the batch, head and row indices (``lt_tensor_strides``)."""
    _fields_ = [("batch", ctypes.c_longlong), ("head", ctypes.c_longlong), ("row", ctypes.c_longlong)]


class AttnLayout(ctypes.Structure):
    """``lt_attn_layout``: strides of q, k, v, o, d_o, dq, dk, dv in that order."""
    _fields_ = [(n, TensorStrides) for n in ("q", "k", "v", "o", "d_o", "dq", "dk", "dv")]


class LtError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn} failed: {status_string(status)} (status {status}); last CUDA error: "
                         f"{last_cuda_error()}")


def _load() -> ctypes.CDLL:
    if not LIB_PATH.exists():
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2606_10415_b200.build` "
            "(there is no fallback path)")
    lib = ctypes.CDLL(str(LIB_PATH))
    vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.lt_attn_fwd_workspace_bytes.argtypes = [i] * 5
    lib.lt_attn_fwd_workspace_bytes.restype = sz
    lib.lt_attn_bwd_workspace_bytes.argtypes = [i] * 5
    lib.lt_attn_bwd_workspace_bytes.restype = sz
    lib.lt_attn_host_arena_bytes.argtypes = [i] * 5
    lib.lt_attn_host_arena_bytes.restype = sz
    lib.lt_attn_fwd.argtypes = [vp] * 5 + [i] * 6 + [f, vp, sz, vp]
    lib.lt_attn_fwd.restype = i
    lib.lt_attn_bwd.argtypes = [vp] * 9 + [i] * 6 + [f, vp, sz, vp]
    lib.lt_attn_bwd.restype = i
    lib.lt_attn_bwd_profiled.argtypes = [vp] * 9 + [i] * 6 + [f, vp, sz, vp, vp, vp]
    lib.lt_attn_bwd_profiled.restype = i
    lib.lt_attn_fwd_strided.argtypes = [vp] * 5 + [ctypes.POINTER(AttnLayout)] + [i] * 6 + [f, vp, sz, vp]
    lib.lt_attn_fwd_strided.restype = i
    lib.lt_attn_bwd_strided.argtypes = [vp] * 9 + [ctypes.POINTER(AttnLayout)] + [i] * 6 + [f, vp, sz, vp]
    lib.lt_attn_bwd_strided.restype = i
    lib.lt_attn_fwd_bf16.argtypes = lib.lt_attn_fwd_strided.argtypes
    lib.lt_attn_fwd_bf16.restype = i
    lib.lt_attn_bwd_bf16.argtypes = lib.lt_attn_bwd_strided.argtypes
    lib.lt_attn_bwd_bf16.restype = i
    lib.lt_attn_p_store_bytes.argtypes = [i] * 5
    lib.lt_attn_p_store_bytes.restype = sz
    lib.lt_attn_save_p.argtypes = [vp] * 4 + [i] * 6 + [f, vp, sz, vp]
    lib.lt_attn_save_p.restype = i
    lib.lt_attn_bwd_saved_p.argtypes = [vp] * 9 + [i] * 6 + [f, vp, sz, vp]
    lib.lt_attn_bwd_saved_p.restype = i
    lib.lt_gemm_f16_workspace_bytes.argtypes = []
    lib.lt_gemm_f16_workspace_bytes.restype = sz
    lib.lt_gemm_f16.argtypes = [vp] * 3 + [i] * 3 + [vp, sz, vp]
    lib.lt_gemm_f16.restype = i
    lib.lt_gemm_bf16.argtypes = lib.lt_gemm_f16.argtypes
    lib.lt_gemm_bf16.restype = i
    lib.lt_attn_bwd_noalloc.argtypes = [vp] * 9 + [i] * 6 + [f, vp]
    lib.lt_attn_bwd_noalloc.restype = i
    lib.lt_attn_fwd_bwd_host.argtypes = [vp] * 9 + [i] * 6 + [f, vp, sz, vp]
    lib.lt_attn_fwd_bwd_host.restype = i
    lib.lt_attn_check_status.argtypes = [vp, vp]
    lib.lt_attn_check_status.restype = i
    lib.lt_status_string.argtypes = [i]
    lib.lt_status_string.restype = ctypes.c_char_p
    lib.lt_last_cuda_error.argtypes = []
    lib.lt_last_cuda_error.restype = ctypes.c_char_p
    lib.lt_attn_bwd_num_launches.argtypes = [i] * 6
    lib.lt_attn_bwd_num_launches.restype = i
    lib.lt_attn_bwd_noalloc_check_status.argtypes = [vp]
    lib.lt_attn_bwd_noalloc_check_status.restype = i
    lib.lt_attn_fwd_num_launches.restype = i
    lib.lt_dbg_tile_gemm.argtypes = [vp, vp, vp, i, vp, sz, vp]
    lib.lt_dbg_tile_gemm.restype = i
    lib.lt_dbg_wait_timeout.argtypes = [vp, sz, vp]
    lib.lt_dbg_wait_timeout.restype = i
    return lib


_lib = _load()


def status_string(status: int) -> str:
    return _lib.lt_status_string(int(status)).decode()


def last_cuda_error() -> str:
    return _lib.lt_last_cuda_error().decode()


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _dims(Q: torch.Tensor, K: torch.Tensor):
    B, Hq, S, D = Q.shape
    return int(B), int(Hq), int(K.shape[1]), int(S), int(D)


def _check_layout(*tensors):
    for t in tensors:
        if t is not None and not t.is_contiguous():
            raise ValueError("tensors must be contiguous [B, H, S, D]")


def lt_attn_fwd_workspace_bytes(B, Hq, Hkv, S, D) -> int:
    return int(_lib.lt_attn_fwd_workspace_bytes(B, Hq, Hkv, S, D))


def lt_attn_bwd_workspace_bytes(B, Hq, Hkv, S, D) -> int:
    return int(_lib.lt_attn_bwd_workspace_bytes(B, Hq, Hkv, S, D))


def lt_attn_host_arena_bytes(B, Hq, Hkv, S, D) -> int:
    return int(_lib.lt_attn_host_arena_bytes(B, Hq, Hkv, S, D))


def lt_attn_bwd_num_launches(B, Hq, Hkv, S, D, causal) -> int:
    """Kernels one backward call enqueues for this shape (3, or 4 when groups are split over work items)."""
    return int(_lib.lt_attn_bwd_num_launches(B, Hq, Hkv, S, D, int(bool(causal))))


def lt_attn_fwd_num_launches() -> int:
    return int(_lib.lt_attn_fwd_num_launches())


def lt_attn_fwd_raw(*args) -> int:
    """Direct call with integer pointers; returns the status code (for boundary tests)."""
    return int(_lib.lt_attn_fwd(*args))


def lt_attn_bwd_raw(*args) -> int:
    return int(_lib.lt_attn_bwd(*args))


def lt_attn_fwd(Q, K, V, O, LSE, causal, scale, workspace, stream=None) -> None:
    """O (fp16) and LSE (fp32) from Q, K, V; device tensors; asynchronous on ``stream``."""
    _check_layout(Q, K, V, O, LSE)
    B, Hq, Hkv, S, D = _dims(Q, K)
    rc = _lib.lt_attn_fwd(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(LSE), B, Hq, Hkv, S, D, int(bool(causal)),
                          float(scale), _ptr(workspace), workspace.numel() * workspace.element_size(),
                          _stream_ptr(stream))
    if rc != LT_OK:
        raise LtError("lt_attn_fwd", rc)


def lt_attn_bwd(Q, K, V, O, dO, LSE, dQ, dK, dV, causal, scale, workspace, stream=None) -> None:
    """dQ, dK, dV (fp16) from Q, K, V, O, dO, LSE; device tensors; asynchronous on ``stream``."""
    _check_layout(Q, K, V, O, dO, LSE, dQ, dK, dV)
    B, Hq, Hkv, S, D = _dims(Q, K)
    rc = _lib.lt_attn_bwd(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO), _ptr(LSE), _ptr(dQ), _ptr(dK), _ptr(dV),
                          B, Hq, Hkv, S, D, int(bool(causal)), float(scale), _ptr(workspace),
                          workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != LT_OK:
        raise LtError("lt_attn_bwd", rc)


def lt_attn_p_store_bytes(B: int, Hq: int, Hkv: int, S: int, D: int) -> int:
    """Bytes of the saved-probability store of lt_attn_save_p (0 for an unsupported shape)."""
    return int(_lib.lt_attn_p_store_bytes(B, Hq, Hkv, S, D))


def lt_attn_save_p(Q, K, LSE, P, causal, scale, workspace, stream=None) -> None:
    """Write the forward's probability tiles (fp16, transposed 128 x 128 tiles) into ``P``, a device
    buffer of at least lt_attn_p_store_bytes() bytes; asynchronous on ``stream``."""
    _check_layout(Q, K, LSE, P)
    B, Hq, Hkv, S, D = _dims(Q, K)
    if P.numel() * P.element_size() < lt_attn_p_store_bytes(B, Hq, Hkv, S, D):
        raise ValueError("P is smaller than lt_attn_p_store_bytes()")
    rc = _lib.lt_attn_save_p(_ptr(Q), _ptr(K), _ptr(LSE), _ptr(P), B, Hq, Hkv, S, D, int(bool(causal)), float(scale),
                             _ptr(workspace), workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != LT_OK:
        raise LtError("lt_attn_save_p", rc)


def lt_attn_bwd_saved_p(Q, K, V, O, dO, P, dQ, dK, dV, causal, scale, workspace, stream=None) -> None:
    """lt_attn_bwd with the saved probability tiles ``P`` of lt_attn_save_p in place of LSE."""
    _check_layout(Q, K, V, O, dO, P, dQ, dK, dV)
    B, Hq, Hkv, S, D = _dims(Q, K)
    if P.numel() * P.element_size() < lt_attn_p_store_bytes(B, Hq, Hkv, S, D):
        raise ValueError("P is smaller than lt_attn_p_store_bytes()")
    rc = _lib.lt_attn_bwd_saved_p(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO), _ptr(P), _ptr(dQ), _ptr(dK),
                                  _ptr(dV), B, Hq, Hkv, S, D, int(bool(causal)), float(scale), _ptr(workspace),
                                  workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != LT_OK:
        raise LtError("lt_attn_bwd_saved_p", rc)


def _strides_of(t: torch.Tensor) -> TensorStrides:
    """Strides of a logical ``[B, H, S, D]`` view (any permutation or slice with unit D stride)."""
    if t.dim() != 4 or t.stride(3) != 1:
        raise ValueError("expected a [B, H, S, D] view whose last dimension is contiguous")
    return TensorStrides(int(t.stride(0)), int(t.stride(1)), int(t.stride(2)))


def lt_attn_fwd_strided(Q, K, V, O, LSE, causal, scale, workspace, stream=None) -> None:
    """lt_attn_fwd on ``[B, H, S, D]`` *views* (e.g. a permuted [B,S,H,D] tensor or slices of a fused
    QKV buffer); the strides are taken from the tensors.  LSE must be contiguous."""
    _check_layout(LSE)
    B, Hq, Hkv, S, D = _dims(Q, K)
    lay = AttnLayout()
    lay.q, lay.k, lay.v, lay.o = (_strides_of(t) for t in (Q, K, V, O))
    rc = _lib.lt_attn_fwd_strided(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(LSE), ctypes.byref(lay), B, Hq, Hkv, S, D,
                                  int(bool(causal)), float(scale), _ptr(workspace),
                                  workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != LT_OK:
        raise LtError("lt_attn_fwd_strided", rc)


def lt_attn_bwd_strided(Q, K, V, O, dO, LSE, dQ, dK, dV, causal, scale, workspace, stream=None) -> None:
    """lt_attn_bwd on ``[B, H, S, D]`` views; the strides are taken from the tensors.  LSE contiguous."""
    _check_layout(LSE)
    B, Hq, Hkv, S, D = _dims(Q, K)
    lay = AttnLayout()
    lay.q, lay.k, lay.v, lay.o, lay.d_o, lay.dq, lay.dk, lay.dv = (
        _strides_of(t) for t in (Q, K, V, O, dO, dQ, dK, dV))
    rc = _lib.lt_attn_bwd_strided(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO), _ptr(LSE), _ptr(dQ), _ptr(dK),
                                  _ptr(dV), ctypes.byref(lay), B, Hq, Hkv, S, D, int(bool(causal)), float(scale),
                                  _ptr(workspace), workspace.numel() * workspace.element_size(),
                                  _stream_ptr(stream))
    if rc != LT_OK:
        raise LtError("lt_attn_bwd_strided", rc)


def lt_gemm_f16_workspace_bytes() -> int:
    return int(_lib.lt_gemm_f16_workspace_bytes())


def lt_gemm_f16(A, W, C, workspace, stream=None) -> None:
    """C[M,N] = A[M,K] W[N,K]^T, fp16 (or, all three, bfloat16) device tensors, contiguous; asynchronous
    on ``stream``."""
    _check_layout(A, W, C)
    fn = _lib.lt_gemm_bf16 if A.dtype == torch.bfloat16 else _lib.lt_gemm_f16
    _require_dtype(A.dtype, W, C)
    M, K = (int(x) for x in A.shape)
    N = int(W.shape[0])
    if W.shape[1] != K or tuple(C.shape) != (M, N):
        raise ValueError("expected A [M, K], W [N, K], C [M, N]")
    rc = fn(_ptr(A), _ptr(W), _ptr(C), M, N, K, _ptr(workspace),
                          workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != LT_OK:
        raise LtError("lt_gemm_f16", rc)


def _require_dtype(dtype, *tensors):
    for t in tensors:
        if t.dtype != dtype:
            raise ValueError(f"expected {dtype} tensors, got {t.dtype}")


def lt_attn_fwd_bf16(Q, K, V, O, LSE, causal, scale, workspace, stream=None) -> None:
    """lt_attn_fwd with bfloat16 Q, K, V, O ([B, H, S, D] views; strides are taken from the tensors)."""
    _require_dtype(torch.bfloat16, Q, K, V, O)
    _check_layout(LSE)
    B, Hq, Hkv, S, D = _dims(Q, K)
    lay = AttnLayout()
    lay.q, lay.k, lay.v, lay.o = (_strides_of(t) for t in (Q, K, V, O))
    rc = _lib.lt_attn_fwd_bf16(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(LSE), ctypes.byref(lay), B, Hq, Hkv, S, D,
                               int(bool(causal)), float(scale), _ptr(workspace),
                               workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != LT_OK:
        raise LtError("lt_attn_fwd_bf16", rc)


def lt_attn_bwd_bf16(Q, K, V, O, dO, LSE, dQ, dK, dV, causal, scale, workspace, stream=None) -> None:
    """lt_attn_bwd with bfloat16 tensors ([B, H, S, D] views; strides are taken from the tensors)."""
    _require_dtype(torch.bfloat16, Q, K, V, O, dO, dQ, dK, dV)
    _check_layout(LSE)
    B, Hq, Hkv, S, D = _dims(Q, K)
    lay = AttnLayout()
    lay.q, lay.k, lay.v, lay.o, lay.d_o, lay.dq, lay.dk, lay.dv = (
        _strides_of(t) for t in (Q, K, V, O, dO, dQ, dK, dV))
    rc = _lib.lt_attn_bwd_bf16(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO), _ptr(LSE), _ptr(dQ), _ptr(dK), _ptr(dV),
                               ctypes.byref(lay), B, Hq, Hkv, S, D, int(bool(causal)), float(scale), _ptr(workspace),
                               workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != LT_OK:
        raise LtError("lt_attn_bwd_bf16", rc)


def lt_attn_bwd_profiled(Q, K, V, O, dO, LSE, dQ, dK, dV, causal, scale, workspace, stream=None,
                         main_begin=None, main_end=None) -> None:
    """lt_attn_bwd with torch CUDA events recorded around the main kernel (events created with
    ``enable_timing=True`` and recorded once beforehand so that their handles exist)."""
    _check_layout(Q, K, V, O, dO, LSE, dQ, dK, dV)
    B, Hq, Hkv, S, D = _dims(Q, K)
    e0 = 0 if main_begin is None else int(main_begin.cuda_event)
    e1 = 0 if main_end is None else int(main_end.cuda_event)
    rc = _lib.lt_attn_bwd_profiled(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO), _ptr(LSE), _ptr(dQ), _ptr(dK),
                                   _ptr(dV), B, Hq, Hkv, S, D, int(bool(causal)), float(scale), _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), _stream_ptr(stream), e0, e1)
    if rc != LT_OK:
        raise LtError("lt_attn_bwd_profiled", rc)


NOALLOC_MAX_SCRATCH_BYTES = 18 * 1024 * 1024


def lt_attn_bwd_noalloc(Q, K, V, O, dO, LSE, dQ, dK, dV, causal, scale, stream=None) -> None:
    """lt_attn_bwd without a workspace argument, for callers that may not allocate device memory:
    the scratch is a fixed array inside the library (``NOALLOC_MAX_SCRATCH_BYTES``).  Raises
    ``LtError`` with status ``LT_ERR_WORKSPACE`` when the shape needs more than that.  Calls on one
    device share the array, so do not let two of them overlap on the GPU."""
    _check_layout(Q, K, V, O, dO, LSE, dQ, dK, dV)
    B, Hq, Hkv, S, D = _dims(Q, K)
    rc = _lib.lt_attn_bwd_noalloc(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO), _ptr(LSE), _ptr(dQ), _ptr(dK),
                                  _ptr(dV), B, Hq, Hkv, S, D, int(bool(causal)), float(scale), _stream_ptr(stream))
    if rc != LT_OK:
        raise LtError("lt_attn_bwd_noalloc", rc)


def lt_attn_bwd_noalloc_check_status(stream=None) -> int:
    """Status of the last lt_attn_bwd_noalloc call on the current device (synchronises ``stream``)."""
    return int(_lib.lt_attn_bwd_noalloc_check_status(_stream_ptr(stream)))


def lt_attn_fwd_bwd_host(Q, K, V, dO, O, LSE, dQ, dK, dV, causal, scale, arena, stream=None) -> None:
    """Host tensors in and out (pinned for asynchronous copies); ``arena`` is a device buffer."""
    _check_layout(Q, K, V, dO, O, LSE, dQ, dK, dV)
    for t in (Q, K, V, dO, O, LSE, dQ, dK, dV):
        if t is not None and t.is_cuda:
            raise ValueError("lt_attn_fwd_bwd_host takes host tensors")
    B, Hq, Hkv, S, D = _dims(Q, K)
    rc = _lib.lt_attn_fwd_bwd_host(_ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(O), _ptr(LSE), _ptr(dQ), _ptr(dK),
                                   _ptr(dV), B, Hq, Hkv, S, D, int(bool(causal)), float(scale), _ptr(arena),
                                   arena.numel() * arena.element_size(), _stream_ptr(stream))
    if rc != LT_OK:
        raise LtError("lt_attn_fwd_bwd_host", rc)


def lt_attn_check_status(workspace, stream=None) -> int:
    return int(_lib.lt_attn_check_status(_ptr(workspace), _stream_ptr(stream)))


def lt_dbg_tile_gemm(A, B, C, mode, workspace, stream=None) -> None:
    rc = _lib.lt_dbg_tile_gemm(_ptr(A), _ptr(B), _ptr(C), int(mode), _ptr(workspace),
                               workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != LT_OK:
        raise LtError("lt_dbg_tile_gemm", rc)


def lt_dbg_wait_timeout(workspace, stream=None) -> None:
    rc = _lib.lt_dbg_wait_timeout(_ptr(workspace), workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != LT_OK:
        raise LtError("lt_dbg_wait_timeout", rc)


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A 256-byte aligned device byte buffer (torch's allocator aligns to 512 bytes)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
