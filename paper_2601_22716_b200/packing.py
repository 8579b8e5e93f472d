"""Layers that read the same activations, laid out as one layer (no arithmetic: concatenation only).

Projections that share their input (the q, k and v projections of an attention block; gate and up of
an MLP) can be handed to the forward calls as ONE layer, which saves the fixed cost of a launch per
projection: the rows of the code matrices are stacked, the rank axes of the factors are stacked, and B
becomes block-diagonal, so that S = B A of Eq. 3 keeps every layer's own scales on its own rows,

    Q = [Q_1; Q_2; ...]     A = [A_1; A_2; ...]     B = diag(B_1, B_2, ...)  (zero elsewhere).

The output of the combined layer is the concatenation of the layers' outputs.  All layers must have
the same code width and in-features; the combined rank is the sum of the ranks.  The saving is there
where the combined rank still fits the decode kernels (rank <= 64, up to 16 tokens); beyond that the
call falls to a slower path.
"""
from __future__ import annotations

import numpy as np

__all__ = ["concat_layers"]


def concat_layers(codes, B, A):
    """codes: list of uint8 [m_i, n]; B: list of uint16 (bf16 bits) [m_i, r_i]; A: list of uint16 [r_i, n].

    Returns (codes [sum m_i, n], B [sum m_i, sum r_i], A [sum r_i, n]) of the combined layer."""
    if not (len(codes) == len(B) == len(A)) or not codes:
        raise ValueError("concat_layers: need the same, non-zero number of code, B and A arrays")
    n = codes[0].shape[1]
    for c, b, a in zip(codes, B, A):
        if c.ndim != 2 or b.ndim != 2 or a.ndim != 2 or c.shape[1] != n or a.shape[1] != n:
            raise ValueError("concat_layers: every layer needs the same in-features")
        if b.shape[0] != c.shape[0] or b.shape[1] != a.shape[0]:
            raise ValueError("concat_layers: B is [m, r] and A is [r, n] of the same layer")
        if b.dtype != np.uint16 or a.dtype != np.uint16 or c.dtype != np.uint8:
            raise ValueError("concat_layers: codes are uint8, factors are bf16 bit patterns (uint16)")
    m_total = sum(c.shape[0] for c in codes)
    r_total = sum(a.shape[0] for a in A)
    Bc = np.zeros((m_total, r_total), dtype=np.uint16)           # 0x0000 is bf16 +0.0
    row = col = 0
    for b in B:
        Bc[row:row + b.shape[0], col:col + b.shape[1]] = b
        row += b.shape[0]
        col += b.shape[1]
    return np.concatenate(codes, axis=0), Bc, np.concatenate(A, axis=0)
