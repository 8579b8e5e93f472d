"""Thin ctypes binding over liblords.so: argument marshalling only.

Every function has the name of the C entry point it calls (include/lords.h).  Tensors
are torch CUDA tensors used purely as device-memory handles; their ``data_ptr()`` and the
current CUDA stream are passed through.  There is no CPU fallback: if the library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import numpy as np

_PKG = Path(__file__).resolve().parent
_LIBPATH = _PKG / "liblords.so"
_lib = None


class LordsError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {lords_strerror(status)} (status {status})")


def _load():
    global _lib
    if _lib is not None:
        return _lib
    if not _LIBPATH.exists():
        raise ImportError(
            f"{_LIBPATH} is missing: build it with `python -m paper_2601_22716_b200.build` "
            "(nvcc, sm_100a).  There is no fallback path.")
    lib = ctypes.CDLL(str(_LIBPATH))
    i64, ci, p, sz = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t
    cs = ctypes.c_char_p
    sig = {
        "lords_version": (ci, []),
        "lords_strerror": (cs, [ci]),
        "lords_equivalent_rank": (i64, [i64, i64, i64]),
        "lords_packed_bytes": (i64, [i64, i64, ci]),
        "lords_pack_codes": (ci, [p, i64, i64, ci, p]),
        "lords_unpack_codes": (ci, [p, i64, i64, ci, p]),
        "lords_init": (ci, [ci, sz]),
        "lords_shutdown": (ci, []),
        "lords_linear_forward": (ci, [p, p, p, p, p, ci, ci, ci, ci, p, p]),
        "lords_linear_forward_bits": (ci, [p, p, p, p, p, ci, ci, ci, ci, ci, p, p]),
        "lords_linear_forward_f32": (ci, [p, p, p, p, p, ci, ci, ci, ci, ci, p, p]),
        "lords_linear_forward_host": (ci, [p, p, p, p, p, ci, ci, ci, ci, ci, p, p]),
        "lords_linear_forward_noalloc": (ci, [p, p, p, p, p, ci, ci, ci, ci, ci, p, p]),
        "lords_quantize_codes": (ci, [p, p, p, p, ci, ci, ci, ci, p, p]),
        "lords_transpose_codes": (ci, [p, ci, ci, ci, p, p]),
        "lords_linear_backward_input": (ci, [p, p, p, p, p, ci, ci, ci, ci, ci, p, p]),
        "lords_linear_backward_input_f32": (ci, [p, p, p, p, p, ci, ci, ci, ci, ci, p, p]),
        "lords_linear_backward_factors": (ci, [p, p, p, p, p, p, ci, ci, ci, ci, ci, p, p, p]),
        "lords_linear_backward_qat": (ci, [p, p, p, p, p, p, p, ci, ci, ci, ci, ci, p, p, p, p]),
        "lords_blockscale_forward": (ci, [p, p, p, p, ci, ci, ci, ci, ci, p, p]),
        "lords_blockscale_forward_f32": (ci, [p, p, p, p, ci, ci, ci, ci, ci, p, p]),
        "lords_adapter_forward": (ci, [p, p, p, p, p, p, ci, ci, ci, ci, ci, ci, p, p]),
        "lords_adapter_forward_f32": (ci, [p, p, p, p, p, p, ci, ci, ci, ci, ci, ci, p, p]),
        "lords_poll_status": (ci, [p]),
        "lords_read_status_detail": (ci, [p]),
        "lords_last_cuda_error": (ci, []),
        "lords_set_option": (ci, [cs, cs]),
        "lords_last_path": (cs, []),
        "lords_last_launch_count": (ci, []),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def library_path() -> Path:
    return _LIBPATH


def exported_symbols():
    """Names this binding expects the library to export (all of include/lords.h)."""
    return ["lords_version", "lords_strerror", "lords_equivalent_rank", "lords_packed_bytes",
            "lords_pack_codes", "lords_unpack_codes", "lords_init", "lords_shutdown",
            "lords_linear_forward", "lords_linear_forward_bits", "lords_linear_forward_f32",
            "lords_linear_forward_host", "lords_linear_forward_noalloc", "lords_quantize_codes", "lords_transpose_codes",
            "lords_linear_backward_input", "lords_linear_backward_input_f32", "lords_linear_backward_factors",
            "lords_linear_backward_qat", "lords_blockscale_forward", "lords_blockscale_forward_f32", "lords_adapter_forward", "lords_adapter_forward_f32", "lords_poll_status", "lords_read_status_detail", "lords_last_cuda_error", "lords_set_option", "lords_last_path",
            "lords_last_launch_count"]


def _check(status: int, what: str):
    if status != 0:
        raise LordsError(status, what)


def lords_version() -> int:
    return int(_load().lords_version())


def lords_strerror(status: int) -> str:
    return _load().lords_strerror(int(status)).decode()


def lords_equivalent_rank(rows: int, cols: int, blk: int) -> int:
    v = int(_load().lords_equivalent_rank(rows, cols, blk))
    if v < 0:
        raise LordsError(v, "lords_equivalent_rank")
    return v


def lords_packed_bytes(m: int, n: int, bits: int) -> int:
    v = int(_load().lords_packed_bytes(m, n, bits))
    if v < 0:
        raise LordsError(v, "lords_packed_bytes")
    return v


def lords_pack_codes(codes: np.ndarray, bits: int) -> np.ndarray:
    """Host: uint8 codes [m, n] -> packed uint8 [m, n*bits/8]."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    m, n = codes.shape
    nbytes = lords_packed_bytes(m, n, bits)
    out = np.empty((m, nbytes // m if m else 0), dtype=np.uint8)
    _check(_load().lords_pack_codes(codes.ctypes.data, m, n, bits, out.ctypes.data), "lords_pack_codes")
    return out


def lords_unpack_codes(packed: np.ndarray, m: int, n: int, bits: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    if packed.size != lords_packed_bytes(m, n, bits):
        raise ValueError("packed buffer has the wrong size")
    out = np.empty((m, n), dtype=np.uint8)
    _check(_load().lords_unpack_codes(packed.ctypes.data, m, n, bits, out.ctypes.data), "lords_unpack_codes")
    return out


def lords_init(device: int = 0, workspace_bytes: int = 0) -> None:
    _check(_load().lords_init(int(device), int(workspace_bytes)), "lords_init")


def lords_shutdown() -> None:
    _check(_load().lords_shutdown(), "lords_shutdown")


def _stream_ptr(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(int(stream.cuda_stream))


def _cb_ptr(codebook, bits):
    cb = np.ascontiguousarray(codebook, dtype=np.float32)
    if cb.size != 2**bits:
        raise ValueError("codebook must hold 2**bits floats")
    return cb


def lords_linear_forward(x, Qpacked, B, A, codebook, M, m, n, r, y, stream=None) -> None:
    """4-bit entry point: device tensors x[M,n], Qpacked[m,n/2], B[m,r], A[r,n] -> y[M,m] (bf16)."""
    cb = _cb_ptr(codebook, 4)
    _check(_load().lords_linear_forward(x.data_ptr(), Qpacked.data_ptr(), B.data_ptr(), A.data_ptr(),
                                        cb.ctypes.data, M, m, n, r, y.data_ptr(), _stream_ptr(stream)),
           "lords_linear_forward")


def lords_linear_forward_bits(x, Qpacked, B, A, codebook, bits, M, m, n, r, y, stream=None) -> None:
    cb = _cb_ptr(codebook, bits)
    _check(_load().lords_linear_forward_bits(x.data_ptr(), Qpacked.data_ptr(), B.data_ptr(), A.data_ptr(),
                                             cb.ctypes.data, bits, M, m, n, r, y.data_ptr(),
                                             _stream_ptr(stream)), "lords_linear_forward_bits")


def lords_linear_forward_f32(x, Qpacked, B, A, codebook, bits, M, m, n, r, y32, stream=None) -> None:
    cb = _cb_ptr(codebook, bits)
    _check(_load().lords_linear_forward_f32(x.data_ptr(), Qpacked.data_ptr(), B.data_ptr(), A.data_ptr(),
                                            cb.ctypes.data, bits, M, m, n, r, y32.data_ptr(),
                                            _stream_ptr(stream)), "lords_linear_forward_f32")


def lords_linear_forward_host(x_host, Qpacked, B, A, codebook, bits, M, m, n, r, y_host, stream=None) -> None:
    """x_host / y_host are CPU tensors (pinned for asynchronous copies); weights are device tensors."""
    cb = _cb_ptr(codebook, bits)
    if x_host.is_cuda or y_host.is_cuda:
        raise ValueError("x_host and y_host must be host tensors")
    _check(_load().lords_linear_forward_host(x_host.data_ptr(), Qpacked.data_ptr(), B.data_ptr(), A.data_ptr(),
                                             cb.ctypes.data, bits, M, m, n, r, y_host.data_ptr(),
                                             _stream_ptr(stream)), "lords_linear_forward_host")


def lords_linear_forward_noalloc(x, Qpacked, B, A, codebook, bits, M, m, n, r, y, stream=None) -> None:
    """Forward that never allocates and needs no lords_init (scratch lives in the library image)."""
    cb = _cb_ptr(codebook, bits)
    _check(_load().lords_linear_forward_noalloc(x.data_ptr(), Qpacked.data_ptr(), B.data_ptr(), A.data_ptr(),
                                                cb.ctypes.data, bits, M, m, n, r, y.data_ptr(),
                                                _stream_ptr(stream)), "lords_linear_forward_noalloc")


def lords_quantize_codes(W, B, A, codebook, bits, m, n, r, Qpacked, stream=None) -> None:
    """Alg. 1 step 2.1 on the device: packed codes of the nearest levels of W / (B A)."""
    cb = _cb_ptr(codebook, bits)
    _check(_load().lords_quantize_codes(W.data_ptr(), B.data_ptr(), A.data_ptr(), cb.ctypes.data, bits, m, n, r,
                                        Qpacked.data_ptr(), _stream_ptr(stream)), "lords_quantize_codes")


def lords_transpose_codes(Qpacked, bits, m, n, Qt_packed, stream=None) -> None:
    """Packed codes of Q^T (n rows of m codes) from the packed codes of Q, on the device."""
    _check(_load().lords_transpose_codes(Qpacked.data_ptr(), bits, m, n, Qt_packed.data_ptr(), _stream_ptr(stream)),
           "lords_transpose_codes")


def lords_linear_backward_input(dy, Qt_packed, B, A, codebook, bits, M, m, n, r, dx, stream=None) -> None:
    """dx = dy W^ (bf16 [M, n]) for a layer whose transposed codes Qt_packed were made by lords_transpose_codes."""
    cb = _cb_ptr(codebook, bits)
    _check(_load().lords_linear_backward_input(dy.data_ptr(), Qt_packed.data_ptr(), B.data_ptr(), A.data_ptr(), cb.ctypes.data,
                                               bits, M, m, n, r, dx.data_ptr(), _stream_ptr(stream)),
           "lords_linear_backward_input")


def lords_linear_backward_input_f32(dy, Qt_packed, B, A, codebook, bits, M, m, n, r, dx32, stream=None) -> None:
    """The same with the fp32 accumulator stored (float [M, n])."""
    cb = _cb_ptr(codebook, bits)
    _check(_load().lords_linear_backward_input_f32(dy.data_ptr(), Qt_packed.data_ptr(), B.data_ptr(), A.data_ptr(),
                                                   cb.ctypes.data, bits, M, m, n, r, dx32.data_ptr(), _stream_ptr(stream)),
           "lords_linear_backward_input_f32")


def lords_linear_backward_factors(dy, x, Qpacked, B, A, codebook, bits, M, m, n, r, dB, dA, stream=None) -> None:
    """dB (float [m, r]) and dA (float [r, n]) of the layer with the codes fixed; either may be None."""
    cb = _cb_ptr(codebook, bits)
    _check(_load().lords_linear_backward_factors(dy.data_ptr(), x.data_ptr(), Qpacked.data_ptr(), B.data_ptr(), A.data_ptr(),
                                                 cb.ctypes.data, bits, M, m, n, r,
                                                 None if dB is None else dB.data_ptr(), None if dA is None else dA.data_ptr(),
                                                 _stream_ptr(stream)), "lords_linear_backward_factors")


def lords_linear_backward_qat(dy, x, W, Qpacked, B, A, codebook, bits, M, m, n, r, dW, dB, dA, stream=None) -> None:
    """Straight-through gradients of quantisation-aware training (Eq. 4-5); any of dW, dB, dA may be None."""
    cb = _cb_ptr(codebook, bits)
    ptr = lambda t: None if t is None else t.data_ptr()
    _check(_load().lords_linear_backward_qat(dy.data_ptr(), x.data_ptr(), W.data_ptr(), Qpacked.data_ptr(), B.data_ptr(),
                                             A.data_ptr(), cb.ctypes.data, bits, M, m, n, r, ptr(dW), ptr(dB), ptr(dA),
                                             _stream_ptr(stream)), "lords_linear_backward_qat")


def lords_blockscale_forward(x, Qpacked, scales, codebook, bits, blk, M, m, n, y, stream=None, f32=False) -> None:
    """Comparator (Eq. 2): y = x (L[Q] (.) (s (x) 1))^T; y is bf16 [M, m], or float with f32=True."""
    cb = _cb_ptr(codebook, bits)
    fn = _load().lords_blockscale_forward_f32 if f32 else _load().lords_blockscale_forward
    _check(fn(x.data_ptr(), Qpacked.data_ptr(), scales.data_ptr(), cb.ctypes.data, bits, blk, M, m, n, y.data_ptr(),
              _stream_ptr(stream)), "lords_blockscale_forward")


def lords_adapter_forward(x, Qpacked, scales, A_l, B_l, codebook, bits, blk, M, m, n, r, y, stream=None, f32=False) -> None:
    """Comparator (Sec. 3.4 / 4.4): the block-scaled layer plus an additive rank-r adapter, three launches."""
    cb = _cb_ptr(codebook, bits)
    fn = _load().lords_adapter_forward_f32 if f32 else _load().lords_adapter_forward
    _check(fn(x.data_ptr(), Qpacked.data_ptr(), scales.data_ptr(), A_l.data_ptr(), B_l.data_ptr(), cb.ctypes.data, bits, blk,
              M, m, n, r, y.data_ptr(), _stream_ptr(stream)), "lords_adapter_forward")


def lords_poll_status(stream=None) -> int:
    return int(_load().lords_poll_status(_stream_ptr(stream)))


def lords_read_status_detail():
    """The two 64-bit words of the first expired wait's record (both 0 if none), read and cleared."""
    buf = (ctypes.c_uint64 * 2)()
    _check(_load().lords_read_status_detail(ctypes.cast(buf, ctypes.c_void_p)), "lords_read_status_detail")
    return int(buf[0]), int(buf[1])


def lords_last_cuda_error() -> int:
    return int(_load().lords_last_cuda_error())


def lords_set_option(key: str, value: str) -> None:
    _check(_load().lords_set_option(key.encode(), str(value).encode()), f"lords_set_option({key}={value})")


def lords_last_path() -> str:
    return _load().lords_last_path().decode()


def lords_last_launch_count() -> int:
    return int(_load().lords_last_launch_count())
