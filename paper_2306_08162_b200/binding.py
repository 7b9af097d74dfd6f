"""ctypes binding of the C ABI in include/qlora.h.  Same names, same argument order; tensors are passed as their
device pointers and `stream=None` means torch's current CUDA stream.  No arithmetic happens here."""
from __future__ import annotations

import ctypes
import os

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG_DIR, "libqlora_b200.so")
_lib = None


class QloraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where} failed: {qlora_status_string(status)} ({status})")


class _Desc(ctypes.Structure):
    _fields_ = [("bits", ctypes.c_int), ("group_size", ctypes.c_int), ("K", ctypes.c_int), ("N", ctypes.c_int),
                ("r", ctypes.c_int), ("alpha", ctypes.c_float)]


def desc(bits: int, group_size: int, K: int, N: int, r: int, alpha: float) -> _Desc:
    """Layer descriptor (qlora_desc)."""
    return _Desc(int(bits), int(group_size), int(K), int(N), int(r), float(alpha))


def library_path() -> str:
    return _LIB_PATH


def library() -> ctypes.CDLL:
    """Load the CUDA library (built in-tree by paper_2306_08162_b200.build).  Raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2306_08162_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    dp = ctypes.POINTER(_Desc)
    lib.qlora_status_string.restype = ctypes.c_char_p
    lib.qlora_status_string.argtypes = [i32]
    lib.qlora_workspace_bytes.argtypes = [dp, i32, ctypes.POINTER(sz)]
    lib.qlora_fwd.argtypes = [dp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.qlora_bwd_input.argtypes = [dp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.qlora_bwd_lora.argtypes = [dp, i32, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, sz, vp]
    lib.qlora_bwd_input_db_on_producers.argtypes = [dp, i32]
    lib.qlora_bwd_input_db_on_producers.restype = i32
    lib.qlora_bwd_input_db.argtypes = [dp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, sz, vp]
    f32 = ctypes.c_float
    lib.qlora_fwd_dropout.argtypes = [dp, i32, vp, vp, f32, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.qlora_bwd_input_dropout.argtypes = [dp, i32, vp, vp, f32, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.qlora_bwd_lora_dropout.argtypes = [dp, i32, vp, vp, f32, vp, vp, vp, vp, vp, vp, vp, i32, vp, sz, vp]
    lib.qlora_bwd_lora_static.argtypes = [dp, i32, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp]
    lib.qlora_pack.argtypes = [i32, i32, i32, vp, vp, vp]
    lib.qlora_unpack.argtypes = [i32, i32, i32, vp, vp, vp]
    lib.qlora_dequant.argtypes = [dp, vp, vp, vp, vp, vp]
    lib.qlora_quantize_rtn.argtypes = [dp, vp, vp, vp, vp, vp]
    lib.qlora_gather_columns.argtypes = [i32, i32, i32, vp, vp, vp, vp]
    lib.qlora_lrec_loss.argtypes = [i32, i32, vp, vp, vp, ctypes.c_float, ctypes.c_float, ctypes.c_float, vp, vp, vp]
    lib.qlora_device_status.argtypes = [ctypes.POINTER(ctypes.c_uint), i32]
    lib.qlora_selftest_bounded_wait.argtypes = [i32, vp]
    for name in ("qlora_workspace_bytes", "qlora_fwd", "qlora_bwd_input", "qlora_bwd_input_db", "qlora_bwd_lora", "qlora_bwd_lora_static", "qlora_fwd_dropout", "qlora_bwd_input_dropout",
                 "qlora_bwd_lora_dropout", "qlora_pack",
                 "qlora_unpack", "qlora_dequant", "qlora_quantize_rtn", "qlora_gather_columns", "qlora_lrec_loss", "qlora_device_status", "qlora_selftest_bounded_wait"):
        getattr(lib, name).restype = i32
    _lib = lib
    return lib


def _ptr(t):
    """Device pointer of a torch tensor; None -> NULL; an int is passed through (tests of the error paths)."""
    if t is None:
        return None
    if isinstance(t, int):
        return ctypes.c_void_p(t)
    if not t.is_contiguous():
        raise ValueError("tensors must be contiguous (dense row-major)")
    return ctypes.c_void_p(t.data_ptr())


def _nbytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def _stream(stream):
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return ctypes.c_void_p(stream)
    return ctypes.c_void_p(stream.cuda_stream)


def _check(status: int, where: str):
    if status != 0:
        raise QloraError(status, where)


def qlora_status_string(status: int) -> str:
    return library().qlora_status_string(int(status)).decode()


def qlora_workspace_bytes(d: _Desc, M: int) -> int:
    out = ctypes.c_size_t(0)
    _check(library().qlora_workspace_bytes(ctypes.byref(d), int(M), ctypes.byref(out)), "qlora_workspace_bytes")
    return int(out.value)


def qlora_fwd(d, M, X, Q, scales, zeros, A, B, Y, H_out, workspace, stream=None, workspace_bytes=None):
    wb = _nbytes(workspace) if workspace_bytes is None else int(workspace_bytes)
    _check(library().qlora_fwd(ctypes.byref(d), int(M), _ptr(X), _ptr(Q), _ptr(scales), _ptr(zeros), _ptr(A), _ptr(B),
                               _ptr(Y), _ptr(H_out), _ptr(workspace), wb, _stream(stream)), "qlora_fwd")


def qlora_bwd_input(d, M, dY, Q, scales, zeros, A, B, dX, G_out, workspace, stream=None, workspace_bytes=None):
    wb = _nbytes(workspace) if workspace_bytes is None else int(workspace_bytes)
    _check(library().qlora_bwd_input(ctypes.byref(d), int(M), _ptr(dY), _ptr(Q), _ptr(scales), _ptr(zeros), _ptr(A),
                                     _ptr(B), _ptr(dX), _ptr(G_out), _ptr(workspace), wb, _stream(stream)),
           "qlora_bwd_input")


def qlora_bwd_input_db(d, M, dY, Q, scales, zeros, A, B, H, dX, G_out, dB, accumulate, workspace, stream=None, workspace_bytes=None):
    wb = _nbytes(workspace) if workspace_bytes is None else int(workspace_bytes)
    _check(library().qlora_bwd_input_db(ctypes.byref(d), int(M), _ptr(dY), _ptr(Q), _ptr(scales), _ptr(zeros), _ptr(A),
                                        _ptr(B), _ptr(H), _ptr(dX), _ptr(G_out), _ptr(dB), int(accumulate), _ptr(workspace), wb,
                                        _stream(stream)), "qlora_bwd_input_db")


def qlora_bwd_input_db_on_producers(d, M) -> bool:
    rc = library().qlora_bwd_input_db_on_producers(ctypes.byref(d), int(M))
    if rc < 0:
        _check(rc, "qlora_bwd_input_db_on_producers")
    return rc == 1


def qlora_bwd_lora(d, M, X, dY, A, B, H, G, dA, dB, accumulate, workspace, stream=None, workspace_bytes=None):
    wb = _nbytes(workspace) if workspace_bytes is None else int(workspace_bytes)
    _check(library().qlora_bwd_lora(ctypes.byref(d), int(M), _ptr(X), _ptr(dY), _ptr(A), _ptr(B), _ptr(H), _ptr(G),
                                    _ptr(dA), _ptr(dB), int(accumulate), _ptr(workspace), wb, _stream(stream)),
           "qlora_bwd_lora")


def qlora_fwd_dropout(d, M, X, mask, keep_scale, Q, scales, zeros, A, B, Y, H_out, workspace, stream=None, workspace_bytes=None):
    wb = _nbytes(workspace) if workspace_bytes is None else int(workspace_bytes)
    _check(library().qlora_fwd_dropout(ctypes.byref(d), int(M), _ptr(X), _ptr(mask), float(keep_scale), _ptr(Q), _ptr(scales),
                                       _ptr(zeros), _ptr(A), _ptr(B), _ptr(Y), _ptr(H_out), _ptr(workspace), wb, _stream(stream)),
           "qlora_fwd_dropout")


def qlora_bwd_input_dropout(d, M, dY, mask, keep_scale, Q, scales, zeros, A, B, dX, G_out, workspace, stream=None,
                            workspace_bytes=None):
    wb = _nbytes(workspace) if workspace_bytes is None else int(workspace_bytes)
    _check(library().qlora_bwd_input_dropout(ctypes.byref(d), int(M), _ptr(dY), _ptr(mask), float(keep_scale), _ptr(Q), _ptr(scales),
                                             _ptr(zeros), _ptr(A), _ptr(B), _ptr(dX), _ptr(G_out), _ptr(workspace), wb,
                                             _stream(stream)), "qlora_bwd_input_dropout")


def qlora_bwd_lora_dropout(d, M, X, mask, keep_scale, dY, A, B, H, G, dA, dB, accumulate, workspace, stream=None,
                           workspace_bytes=None):
    wb = _nbytes(workspace) if workspace_bytes is None else int(workspace_bytes)
    _check(library().qlora_bwd_lora_dropout(ctypes.byref(d), int(M), _ptr(X), _ptr(mask), float(keep_scale), _ptr(dY), _ptr(A),
                                            _ptr(B), _ptr(H), _ptr(G), _ptr(dA), _ptr(dB), int(accumulate), _ptr(workspace), wb,
                                            _stream(stream)), "qlora_bwd_lora_dropout")


STATIC_SCRATCH_BYTES = 16 << 20   # QLORA_STATIC_SCRATCH_BYTES


def qlora_bwd_lora_static(d, M, X, dY, A, B, H, G, dA, dB, accumulate, stream=None):
    """qlora_bwd_lora for callers that may not allocate device memory: no workspace argument, the scratch is an array
    inside the library (STATIC_SCRATCH_BYTES).  Raises QloraError(-7) when the shape needs more than that."""
    _check(library().qlora_bwd_lora_static(ctypes.byref(d), int(M), _ptr(X), _ptr(dY), _ptr(A), _ptr(B), _ptr(H), _ptr(G),
                                           _ptr(dA), _ptr(dB), int(accumulate), _stream(stream)),
           "qlora_bwd_lora_static")


def qlora_pack(bits, K, N, codes, Q, stream=None):
    _check(library().qlora_pack(int(bits), int(K), int(N), _ptr(codes), _ptr(Q), _stream(stream)), "qlora_pack")


def qlora_unpack(bits, K, N, Q, codes, stream=None):
    _check(library().qlora_unpack(int(bits), int(K), int(N), _ptr(Q), _ptr(codes), _stream(stream)), "qlora_unpack")


def qlora_lrec_loss(student_logits, teacher_logits, labels, lambda_kl, lambda_ce, grad_scale, loss_tokens, dlogits, stream=None):
    """Fused KL + cross-entropy loss of the error-correction objective and its gradient; logits bf16 [T, V]."""
    T, V = student_logits.shape
    _check(library().qlora_lrec_loss(int(T), int(V), _ptr(student_logits), _ptr(teacher_logits), _ptr(labels), float(lambda_kl),
                                     float(lambda_ce), float(grad_scale), _ptr(loss_tokens), _ptr(dlogits), _stream(stream)),
           "qlora_lrec_loss")


def qlora_gather_columns(inp, perm, out, stream=None):
    """out[m, j] = inp[m, perm[j]] for 2-D bf16 / fp16 / fp32 tensors; perm int32 [cols]."""
    rows, cols = inp.shape
    _check(library().qlora_gather_columns(inp.element_size(), int(rows), int(cols), _ptr(inp), _ptr(perm), _ptr(out),
                                          _stream(stream)), "qlora_gather_columns")


def qlora_dequant(d, Q, scales, zeros, W, stream=None):
    _check(library().qlora_dequant(ctypes.byref(d), _ptr(Q), _ptr(scales), _ptr(zeros), _ptr(W), _stream(stream)),
           "qlora_dequant")


def qlora_quantize_rtn(d, W, Q, scales, zeros, stream=None):
    """Min-max round-to-nearest quantization of W fp32 [N, K] into packed Q, fp16 scales and zeros [K/g, N]."""
    _check(library().qlora_quantize_rtn(ctypes.byref(d), _ptr(W), _ptr(Q), _ptr(scales), _ptr(zeros), _stream(stream)),
           "qlora_quantize_rtn")


def qlora_selftest_bounded_wait(limit_us: int, stream=None):
    """Enqueue a wait that is known to run out after limit_us microseconds (sets the device's sticky status word)."""
    _check(library().qlora_selftest_bounded_wait(int(limit_us), _stream(stream)), "qlora_selftest_bounded_wait")


def qlora_device_status(clear: bool = True) -> int:
    """Synchronise the device and return its sticky health word (0 = healthy).  Raises QloraError on a recorded timeout."""
    out = ctypes.c_uint(0)
    rc = library().qlora_device_status(ctypes.byref(out), 1 if clear else 0)
    if rc != 0:
        raise QloraError(rc, f"qlora_device_status (word {out.value:#x})")
    return int(out.value)
