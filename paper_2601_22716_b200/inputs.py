"""Seeded synthetic inputs for the LoRDS dequant-GEMM path.

This module only *draws data*: codes, low-rank factors, activations and the level
table that is handed to the path as a runtime argument.  It contains none of the
method's arithmetic (no packing, no scale reconstruction, no dequantisation, no
matmul), so both the CPU oracle's tests and the CUDA path's tests can take their
inputs from here without sharing any computation.

All floating-point tensors are returned as numpy ``uint16`` arrays holding bf16 bit
patterns (the exact bytes both sides consume); ``codes`` holds one code per byte.

Draw order is fixed: codes, B, A, x, outlier columns.  Shapes follow the letters
used for the kernel interface: ``m`` = out-features (rows of Q and B), ``n`` =
in-features (columns of Q and A, the reduction axis), ``M`` = tokens.  The layer
shapes mirror the paper's Llama3-8B modules (Table 7 lists them as out x in).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

__all__ = [
    "LayerInputs",
    "nf_codebook",
    "int_codebook",
    "bf16_bits",
    "bf16_to_f32",
    "make_layer",
    "make_blockwise_layer",
    "make_integer_layer",
    "LLAMA3_8B_SHAPES",
]

# out-features x in-features of one Llama3-8B decoder block (paper Table 7).
LLAMA3_8B_SHAPES = {
    "q": (4096, 4096),
    "k": (1024, 4096),
    "v": (1024, 4096),
    "o": (4096, 4096),
    "gate": (14336, 4096),
    "up": (14336, 4096),
    "down": (4096, 14336),
}


@dataclass
class LayerInputs:
    """One linear layer's operands, as the bytes handed to either implementation."""

    m: int
    n: int
    r: int
    M: int
    bits: int
    codes: np.ndarray      # uint8 [m, n], values in [0, 2**bits)
    B: np.ndarray          # uint16 (bf16 bits) [m, r]
    A: np.ndarray          # uint16 (bf16 bits) [r, n]
    x: np.ndarray          # uint16 (bf16 bits) [M, n]
    codebook: np.ndarray   # float32 [2**bits], ascending
    meta: dict = field(default_factory=dict)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """fp32 tensor -> bf16 (round to nearest even) -> uint16 bit patterns."""
    return t.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16).copy()


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float32 values (exact widening)."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def nf_codebook(bits: int) -> np.ndarray:
    """NormalFloat-k level table: 2**bits ascending levels in [-1, 1], exactly one 0.

    Construction (the published NormalFloat recipe, restated): 2**(k-1) evenly spaced
    probabilities from delta up to 1/2 on the negative side and 2**(k-1)+1 from 1/2
    up to 1-delta on the positive side are mapped through the inverse normal CDF;
    the shared zero is kept once, and everything is divided by the largest
    magnitude.  delta = (1/(2*2**k) + 1/(2*(2**k-1))) / 2.
    """
    from scipy.stats import norm

    if bits < 2 or bits > 8:
        raise ValueError("bits must be in 2..8")
    half = 2 ** (bits - 1)
    delta = 0.5 * (1.0 / (2 * 2**bits) + 1.0 / (2 * (2**bits - 1)))
    neg = norm.ppf(np.linspace(delta, 0.5, half, dtype=np.float64))[:-1]       # half-1 values < 0
    pos = norm.ppf(np.linspace(0.5, 1.0 - delta, half + 1, dtype=np.float64))[1:]  # half values > 0
    levels = np.concatenate([neg, [0.0], pos])
    # both sides start the same distance delta from their tail, so the extremes are +-1
    levels = np.sort(levels / np.max(np.abs(levels)))
    out = levels.astype(np.float32)
    assert out.shape[0] == 2**bits
    return out


def int_codebook(bits: int) -> np.ndarray:
    """Signed-integer level table -2**(bits-1) .. 2**(bits-1)-1 (the INT-k data type)."""
    half = 2 ** (bits - 1)
    return np.arange(-half, half, dtype=np.float32)


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def make_layer(
    m: int,
    n: int,
    r: int,
    M: int,
    bits: int = 4,
    seed: int = 0,
    *,
    scale_gain: float = 0.05,
    scale_shift: float = 0.01,
    mixed_sign: bool = False,
    outlier_frac: float = 0.0,
    outlier_gain: float = 20.0,
    codebook: np.ndarray | None = None,
) -> LayerInputs:
    """Random layer in the recipe of the benchmark configurations.

    codes ~ uniform over the 2**bits levels; B, A = bf16(|N(0,1)|*gain + shift)
    (signs flipped at random when ``mixed_sign``); x = bf16(N(0,1)), with a fraction
    ``outlier_frac`` of the in-feature columns multiplied by ``outlier_gain``.
    """
    g = _gen(seed)
    codes = torch.randint(0, 2**bits, (m, n), generator=g, dtype=torch.int64).to(torch.uint8).numpy()
    Bf = torch.randn(m, r, generator=g).abs() * scale_gain + scale_shift
    Af = torch.randn(r, n, generator=g).abs() * scale_gain + scale_shift
    xf = torch.randn(M, n, generator=g)
    n_out = int(round(outlier_frac * n))
    cols = None
    if n_out > 0:
        cols = torch.randperm(n, generator=g)[:n_out]
        xf[:, cols] *= outlier_gain
    if mixed_sign:
        Bf = Bf * (torch.randint(0, 2, (m, r), generator=g).float() * 2 - 1)
        Af = Af * (torch.randint(0, 2, (r, n), generator=g).float() * 2 - 1)
    cb = nf_codebook(bits) if codebook is None else np.asarray(codebook, dtype=np.float32)
    return LayerInputs(
        m=m, n=n, r=r, M=M, bits=bits, codes=codes,
        B=bf16_bits(Bf), A=bf16_bits(Af), x=bf16_bits(xf), codebook=cb,
        meta={"seed": seed, "outlier_cols": None if cols is None else cols.numpy()},
    )


def make_blockwise_layer(m: int, n: int, blk: int, M: int, bits: int = 4, seed: int = 0,
                         *, scale_gain: float = 0.1, scale_shift: float = 0.05):
    """Block-wise special case: B = block scales s (m x n/blk), A = 0/1 block indicator.

    Blocks are runs of ``blk`` consecutive in-feature columns inside one output row,
    so r = n/blk.  Returns (LayerInputs, s) with s the bf16 bit patterns of the scales.
    """
    if n % blk:
        raise ValueError("n must be a multiple of blk")
    r = n // blk
    g = _gen(seed)
    codes = torch.randint(0, 2**bits, (m, n), generator=g, dtype=torch.int64).to(torch.uint8).numpy()
    sf = torch.randn(m, r, generator=g).abs() * scale_gain + scale_shift
    ind = torch.zeros(r, n)
    for k in range(r):
        ind[k, k * blk:(k + 1) * blk] = 1.0
    xf = torch.randn(M, n, generator=g)
    s = bf16_bits(sf)
    lay = LayerInputs(m=m, n=n, r=r, M=M, bits=bits, codes=codes, B=s.copy(), A=bf16_bits(ind),
                      x=bf16_bits(xf), codebook=nf_codebook(bits), meta={"seed": seed, "blk": blk})
    return lay, s


def make_integer_layer(m: int, n: int, r: int, M: int, bits: int = 4, seed: int = 0,
                       *, nnz_per_token: int = 6) -> LayerInputs:
    """Inputs for which every intermediate of the path is a small exact integer.

    Levels are the signed integers of the bit width; B holds 0/1 entries with exactly
    one 1 per row and A entries are in {1, 2}, so S = B*A has entries in {1, 2}; x has
    ``nnz_per_token`` non-zeros per token drawn from {-2, -1, 1, 2}.  Then |y| <=
    nnz * 2 * 2 * 2**(bits-1) <= 256 for the defaults, every partial sum is an integer
    below 2**24, and fp16/bf16/fp32 all represent every value exactly.
    """
    g = _gen(seed)
    codes = torch.randint(0, 2**bits, (m, n), generator=g, dtype=torch.int64).to(torch.uint8).numpy()
    Bf = torch.zeros(m, r)
    Bf[torch.arange(m), torch.randint(0, r, (m,), generator=g)] = 1.0
    Af = torch.randint(1, 3, (r, n), generator=g).float()
    xf = torch.zeros(M, n)
    vals = torch.tensor([-2.0, -1.0, 1.0, 2.0])
    for t in range(M):
        cols = torch.randperm(n, generator=g)[:nnz_per_token]
        xf[t, cols] = vals[torch.randint(0, 4, (nnz_per_token,), generator=g)]
    return LayerInputs(m=m, n=n, r=r, M=M, bits=bits, codes=codes, B=bf16_bits(Bf), A=bf16_bits(Af),
                       x=bf16_bits(xf), codebook=int_codebook(bits), meta={"seed": seed, "integer": True})


def make_weight(m: int, n: int, seed: int = 0, *, sigma: float = 0.05) -> np.ndarray:
    """A weight matrix to quantise: bf16 bit patterns of N(0, sigma^2), m x n (out x in).

    With the scale factors of ``make_layer`` (S = B*A around 0.1 for r = 32) the ratios W / S spread over
    and a little beyond the level range [-1, 1], as weights divided by their block scales do.
    """
    g = _gen(seed)
    return bf16_bits(torch.randn(m, n, generator=g) * sigma)

