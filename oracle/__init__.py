"""ctypes loader for the fp64 CPU oracle (``lords_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's
CPU-baseline leg import this; the product package never does.  The oracle is
compiled with gcc on first use into ``oracle/liblords_oracle.so``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "lords_oracle.c"
_LIB = _HERE / "liblords_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle (gcc -O2 -fopenmp; no fast-math, so fp64 sums stay in index order)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-Wall", "-Wextra",
               str(_SRC), "-o", str(tmp), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        i64, p, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        lib.lords_oracle_packed_bytes.restype = i64
        lib.lords_oracle_packed_bytes.argtypes = [i64, i64, ci]
        lib.lords_oracle_pack_codes.restype = ci
        lib.lords_oracle_pack_codes.argtypes = [p, i64, i64, ci, p]
        lib.lords_oracle_unpack_codes.restype = ci
        lib.lords_oracle_unpack_codes.argtypes = [p, i64, i64, ci, p]
        lib.lords_oracle_dequant_rows.restype = ci
        lib.lords_oracle_dequant_rows.argtypes = [p, p, p, p, ci, i64, i64, i64, p, i64, p]
        lib.lords_oracle_forward.restype = ci
        lib.lords_oracle_forward.argtypes = [p, p, p, p, p, ci, i64, i64, i64, i64, p, i64, p, ci]
        lib.lords_oracle_round_bf16.restype = None
        lib.lords_oracle_round_bf16.argtypes = [p, i64, p]
        lib.lords_oracle_quantize.restype = ci
        lib.lords_oracle_quantize.argtypes = [p, p, p, p, ci, i64, i64, i64, p, p, p, p]
        lib.lords_oracle_backward.restype = ci
        lib.lords_oracle_backward.argtypes = [p, p, p, p, p, p, ci, i64, i64, i64, i64, p, p, p]
        lib.lords_oracle_backward_qat.restype = ci
        lib.lords_oracle_backward_qat.argtypes = [p, p, p, p, p, p, p, ci, i64, i64, i64, i64, p, p, p]
        lib.lords_oracle_equivalent_rank.restype = i64
        lib.lords_oracle_equivalent_rank.argtypes = [i64, i64, i64]
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def packed_bytes(m: int, n: int, bits: int) -> int:
    v = _load().lords_oracle_packed_bytes(m, n, bits)
    if v < 0:
        raise ValueError(f"oracle: bad shape for packing (m={m}, n={n}, bits={bits})")
    return int(v)


def pack_codes(codes: np.ndarray, bits: int) -> np.ndarray:
    """codes uint8 [m, n] -> packed uint8 [m, n*bits/8] in the written layout."""
    codes = _c(codes, np.uint8)
    m, n = codes.shape
    out = np.empty((m, packed_bytes(m, n, bits) // max(m, 1)), dtype=np.uint8)
    rc = _load().lords_oracle_pack_codes(_ptr(codes), m, n, bits, _ptr(out))
    if rc != 0:
        raise ValueError(f"oracle pack failed: {rc}")
    return out


def unpack_codes(packed: np.ndarray, m: int, n: int, bits: int) -> np.ndarray:
    packed = _c(packed, np.uint8)
    if packed.size != packed_bytes(m, n, bits):
        raise ValueError("oracle unpack: wrong packed size")
    out = np.empty((m, n), dtype=np.uint8)
    rc = _load().lords_oracle_unpack_codes(_ptr(packed), m, n, bits, _ptr(out))
    if rc != 0:
        raise ValueError(f"oracle unpack failed: {rc}")
    return out


def dequant_rows(qpacked, B, A, codebook, bits: int, rows=None) -> np.ndarray:
    """Rows of W^ = L[Q] (.) (B A) as fp64 [nrows, n]."""
    B = _c(B, np.uint16); A = _c(A, np.uint16)
    qpacked = _c(qpacked, np.uint8); codebook = _c(codebook, np.float32)
    m, r = B.shape
    n = A.shape[1]
    assert A.shape[0] == r and codebook.size == 2**bits and qpacked.size == packed_bytes(m, n, bits)
    if rows is None:
        rows_p, nrows = None, m
    else:
        rows = _c(rows, np.int64); rows_p, nrows = _ptr(rows), rows.size
    W = np.empty((nrows, n), dtype=np.float64)
    rc = _load().lords_oracle_dequant_rows(_ptr(qpacked), _ptr(B), _ptr(A), _ptr(codebook), bits,
                                           m, n, r, rows_p, nrows, _ptr(W))
    if rc != 0:
        raise ValueError(f"oracle dequant failed: {rc}")
    return W


def forward(x, qpacked, B, A, codebook, bits: int, rows=None, threads: int = 0, return_threads=False):
    """y64[t, q] = sum_j x[t, j] * W^[rows[q], j]  (fp64 [M, nrows]); rows=None -> all m rows."""
    x = _c(x, np.uint16); B = _c(B, np.uint16); A = _c(A, np.uint16)
    qpacked = _c(qpacked, np.uint8); codebook = _c(codebook, np.float32)
    M, n = x.shape
    m, r = B.shape
    assert A.shape == (r, n) and codebook.size == 2**bits and qpacked.size == packed_bytes(m, n, bits)
    if rows is None:
        rows_p, nrows = None, m
    else:
        rows = _c(rows, np.int64); rows_p, nrows = _ptr(rows), rows.size
    y = np.empty((M, nrows), dtype=np.float64)
    rc = _load().lords_oracle_forward(_ptr(x), _ptr(qpacked), _ptr(B), _ptr(A), _ptr(codebook), bits,
                                      M, m, n, r, rows_p, nrows, _ptr(y), threads)
    if rc < 0:
        raise ValueError(f"oracle forward failed: {rc}")
    return (y, rc) if return_threads else y


def round_bf16(v: np.ndarray) -> np.ndarray:
    """fp64 array -> bf16 bit patterns (uint16), one round-to-nearest-even step."""
    v = _c(v, np.float64)
    out = np.empty(v.shape, dtype=np.uint16)
    _load().lords_oracle_round_bf16(_ptr(v), v.size, _ptr(out))
    return out


def equivalent_rank(rows: int, cols: int, blk: int) -> int:
    return int(_load().lords_oracle_equivalent_rank(rows, cols, blk))


def quantize(W, B, A, codebook, bits: int, details: bool = False):
    """Alg. 1 step 2.1: codes uint8 [m, n] = argmin_c (S * L[c] - W)^2 with S = B A, lowest code on ties.
    W, B, A are bf16 bit patterns.  With details=True also returns (runner-up codes, gap, magnitude)."""
    W = _c(W, np.uint16); B = _c(B, np.uint16); A = _c(A, np.uint16); codebook = _c(codebook, np.float32)
    m, n = W.shape
    r = B.shape[1]
    assert B.shape == (m, r) and A.shape == (r, n) and codebook.size == 2**bits
    codes = np.empty((m, n), dtype=np.uint8)
    if details:
        runner = np.empty((m, n), dtype=np.uint8)
        gap = np.empty((m, n), dtype=np.float64)
        mag = np.empty((m, n), dtype=np.float64)
        rc = _load().lords_oracle_quantize(_ptr(W), _ptr(B), _ptr(A), _ptr(codebook), bits, m, n, r,
                                           _ptr(codes), _ptr(runner), _ptr(gap), _ptr(mag))
    else:
        rc = _load().lords_oracle_quantize(_ptr(W), _ptr(B), _ptr(A), _ptr(codebook), bits, m, n, r,
                                           _ptr(codes), None, None, None)
    if rc != 0:
        raise ValueError(f"oracle quantize failed: {rc}")
    return (codes, runner, gap, mag) if details else codes


def backward(g, x, qpacked, B, A, codebook, bits: int):
    """Gradients of sum(g * y) for y = x W^T with the codes fixed (Sec. 3.4): (dx [M, n], dB [m, r], dA [r, n]), fp64.

    g and x are bf16 bit patterns [M, m] and [M, n]."""
    g = _c(g, np.uint16); x = _c(x, np.uint16); B = _c(B, np.uint16); A = _c(A, np.uint16)
    qpacked = _c(qpacked, np.uint8); codebook = _c(codebook, np.float32)
    M, n = x.shape
    m, r = B.shape
    assert g.shape == (M, m) and A.shape == (r, n) and codebook.size == 2**bits and qpacked.size == packed_bytes(m, n, bits)
    dx = np.empty((M, n), dtype=np.float64)
    dB = np.empty((m, r), dtype=np.float64)
    dA = np.empty((r, n), dtype=np.float64)
    rc = _load().lords_oracle_backward(_ptr(g), _ptr(x), _ptr(qpacked), _ptr(B), _ptr(A), _ptr(codebook), bits,
                                       M, m, n, r, _ptr(dx), _ptr(dB), _ptr(dA))
    if rc != 0:
        raise ValueError(f"oracle backward failed: {rc}")
    return dx, dB, dA


def backward_qat(g, x, W, qpacked, B, A, codebook, bits: int):
    """Straight-through gradients of quantisation-aware training (Eq. 4-5): (dW [m, n], dB [m, r], dA [r, n]), fp64.

    dW = g^T x (Eq. 4); dS = dW * (L[Q] - W / S) (Eq. 5), zero where S is zero; dB = dS A^T, dA = B^T dS."""
    g = _c(g, np.uint16); x = _c(x, np.uint16); W = _c(W, np.uint16); B = _c(B, np.uint16); A = _c(A, np.uint16)
    qpacked = _c(qpacked, np.uint8); codebook = _c(codebook, np.float32)
    M, n = x.shape
    m, r = B.shape
    assert g.shape == (M, m) and W.shape == (m, n) and A.shape == (r, n) and codebook.size == 2**bits
    assert qpacked.size == packed_bytes(m, n, bits)
    dW = np.empty((m, n), dtype=np.float64)
    dB = np.empty((m, r), dtype=np.float64)
    dA = np.empty((r, n), dtype=np.float64)
    rc = _load().lords_oracle_backward_qat(_ptr(g), _ptr(x), _ptr(W), _ptr(qpacked), _ptr(B), _ptr(A), _ptr(codebook), bits,
                                           M, m, n, r, _ptr(dW), _ptr(dB), _ptr(dA))
    if rc != 0:
        raise ValueError(f"oracle QAT backward failed: {rc}")
    return dW, dB, dA


def adapter_forward(x, qpacked, s, blk: int, A_l, B_l, codebook, bits: int) -> np.ndarray:
    """The comparator of Sec. 4.4 / Table 6 in fp64: a block-scaled layer (Eq. 2, one scale s[i, j // blk]
    per row and block) plus an additive low-rank adapter that stays separate (Sec. 3.4),

        y = x W_block^T + (x A_l^T) B_l^T,      W_block = L[Q] (.) (s (x) 1).

    The block-scaled term is the forward above with B = s and A = the 0/1 block indicator (the
    special case that the block-wise pin checks against an independent Eq. 2 dequantiser); the adapter
    term is two library matmuls.  All inputs are bf16 bit patterns except the codes and the level table."""
    s = _c(s, np.uint16); x = _c(x, np.uint16); A_l = _c(A_l, np.uint16); B_l = _c(B_l, np.uint16)
    m, nblk = s.shape
    M, n = x.shape
    assert nblk * blk >= n and (nblk - 1) * blk < n and A_l.shape[1] == n and B_l.shape == (m, A_l.shape[0])
    ind = np.zeros((nblk, n), dtype=np.uint16)
    for b in range(nblk):
        ind[b, b * blk:(b + 1) * blk] = 0x3F80                      # bf16 1.0
    y = forward(x, qpacked, s, ind, codebook, bits)

    def f64(bits16):
        return (bits16.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return y + (f64(x) @ f64(A_l).T) @ f64(B_l).T
