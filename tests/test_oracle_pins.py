"""Pins for the fp64 oracle: everything here checks the oracle against something
other than itself -- paper-printed values, the block-wise special case written as an
independent Eq. 2 dequantiser, brute force, closed forms and invariants."""
import os

import numpy as np
import pytest

import oracle
from paper_2601_22716_b200 import inputs as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _f64(bits16):
    return gen.bf16_to_f32(bits16).astype(np.float64)


def _oracle_forward(lay, rows=None):
    qp = oracle.pack_codes(lay.codes, lay.bits)
    return oracle.forward(lay.x, qp, lay.B, lay.A, lay.codebook, lay.bits, rows=rows)


# ---------------------------------------------------------------- packing (P7)

def _numpy_pack(codes, bits):
    """Independent packer: Python big integers, one per row."""
    m, n = codes.shape
    out = np.zeros((m, n * bits // 8), dtype=np.uint8)
    for i in range(m):
        v = 0
        for j in range(n):
            v |= int(codes[i, j]) << (bits * j)
        out[i] = np.frombuffer(v.to_bytes(n * bits // 8, "little"), dtype=np.uint8)
    return out


def test_pack_known_answers():
    with open(os.path.join(GOLDEN, "pack_known_answers.txt")) as fh:
        rows = [ln for ln in fh if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 4
    for ln in rows:
        bits_s, codes_s, bytes_s = [p.strip() for p in ln.split("|")]
        bits = int(bits_s)
        codes = np.array([int(c) for c in codes_s.split()], dtype=np.uint8)[None, :]
        want = np.array([int(b, 16) for b in bytes_s.split()], dtype=np.uint8)[None, :]
        got = oracle.pack_codes(codes, bits)
        assert np.array_equal(got, want), (bits, got, want)
        assert np.array_equal(oracle.unpack_codes(want, 1, codes.shape[1], bits), codes)


@pytest.mark.parametrize("bits,n", [(4, 64), (4, 2), (3, 32), (3, 96), (2, 8)])
def test_pack_matches_bigint_and_roundtrips(bits, n):
    rng = np.random.default_rng(bits * 100 + n)
    codes = rng.integers(0, 2**bits, size=(5, n), dtype=np.uint8)
    packed = oracle.pack_codes(codes, bits)
    assert np.array_equal(packed, _numpy_pack(codes, bits))
    assert np.array_equal(oracle.unpack_codes(packed, 5, n, bits), codes)


def test_pack_rejects_bad_input():
    with pytest.raises(ValueError):
        oracle.pack_codes(np.full((1, 32), 8, dtype=np.uint8), 3)      # code out of range
    with pytest.raises(ValueError):
        oracle.pack_codes(np.zeros((1, 31), dtype=np.uint8), 3)        # n not a multiple of 32
    with pytest.raises(ValueError):
        oracle.pack_codes(np.zeros((1, 3), dtype=np.uint8), 4)


# ------------------------------------------------- block-wise equivalence (P1)

def _block_dequant(codes, s_bits, codebook, blk):
    """Eq. 2 written directly: W_b = Q_b * s_b, blocks of blk consecutive in-features per row."""
    s = _f64(s_bits)
    levels = codebook.astype(np.float64)[codes]
    return levels * np.repeat(s, blk, axis=1)


@pytest.mark.parametrize("m,n,blk,M,bits", [(256, 256, 64, 4, 4), (48, 128, 32, 3, 3), (24, 96, 32, 2, 3)])
def test_blockwise_special_case_is_reproduced_exactly(m, n, blk, M, bits):
    lay, s = gen.make_blockwise_layer(m, n, blk, M, bits=bits, seed=0)
    W_blk = _block_dequant(lay.codes, s, lay.codebook, blk)
    qp = oracle.pack_codes(lay.codes, bits)
    W = oracle.dequant_rows(qp, lay.B, lay.A, lay.codebook, bits)
    # products with 0/1 and sums of zeros are exact, so equality is bit-for-bit
    assert np.array_equal(W, W_blk)
    y = oracle.forward(lay.x, qp, lay.B, lay.A, lay.codebook, bits)
    y_lib = _f64(lay.x) @ W_blk.T
    np.testing.assert_allclose(y, y_lib, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------ brute force (P2)

@pytest.mark.parametrize("m,n,r,M,bits", [(5, 32, 1, 1, 3), (7, 64, 3, 2, 4), (16, 32, 8, 4, 3), (3, 8, 5, 3, 2)])
def test_brute_force_elementwise(m, n, r, M, bits):
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=m + n + r, mixed_sign=True)
    Bf, Af, xf = _f64(lay.B), _f64(lay.A), _f64(lay.x)
    L = lay.codebook.astype(np.float64)
    want = np.zeros((M, m))
    for t in range(M):
        for i in range(m):
            acc = 0.0
            for j in range(n):
                s = 0.0
                for k in range(r):
                    s += Bf[i, k] * Af[k, j]
                acc += xf[t, j] * (L[lay.codes[i, j]] * s)
            want[t, i] = acc
    got = _oracle_forward(lay)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-14)


def test_row_subset_matches_full():
    lay = gen.make_layer(40, 64, 6, 3, bits=4, seed=3)
    full = _oracle_forward(lay)
    rows = np.array([39, 0, 17, 17, 5], dtype=np.int64)
    sub = _oracle_forward(lay, rows=rows)
    assert np.array_equal(sub, full[:, rows])


def test_thread_count_does_not_change_results():
    lay = gen.make_layer(64, 64, 4, 2, bits=4, seed=9)
    qp = oracle.pack_codes(lay.codes, 4)
    y1 = oracle.forward(lay.x, qp, lay.B, lay.A, lay.codebook, 4, threads=1)
    y4 = oracle.forward(lay.x, qp, lay.B, lay.A, lay.codebook, 4, threads=4)
    assert np.array_equal(y1, y4)


# --------------------------------------------------------------- linearity (P3)

def test_linearity_in_x():
    m, n, r = 33, 128, 7
    lay = gen.make_layer(m, n, r, 2, bits=4, seed=11, mixed_sign=True)
    x = gen.bf16_to_f32(lay.x).copy()
    x[0, n // 2:] = 0.0       # disjoint supports: the combination below is bf16-exact
    x[1, :n // 2] = 0.0
    combo = 4.0 * x[0] - 0.5 * x[1]
    import torch
    xs = gen.bf16_bits(torch.from_numpy(np.stack([x[0], x[1], combo])))
    assert np.array_equal(gen.bf16_to_f32(xs)[2], combo)
    qp = oracle.pack_codes(lay.codes, 4)
    y = oracle.forward(xs, qp, lay.B, lay.A, lay.codebook, 4)
    np.testing.assert_allclose(y[2], 4.0 * y[0] - 0.5 * y[1], rtol=1e-12, atol=1e-13)
    assert np.abs(y[2]).max() > 0


# ------------------------------------------------------ rank-1 reduction (P4)

def test_rank_one_reduces_to_scaled_matmul():
    m, n, M = 29, 96, 3
    lay = gen.make_layer(m, n, 1, M, bits=3, seed=5, mixed_sign=True)
    b = _f64(lay.B)[:, 0]
    a = _f64(lay.A)[0]
    Lq = lay.codebook.astype(np.float64)[lay.codes]
    want = ((_f64(lay.x) * a[None, :]) @ Lq.T) * b[None, :]
    np.testing.assert_allclose(_oracle_forward(lay), want, rtol=1e-12, atol=1e-14)


# ------------------------------------------------------- exact integers (P5)

@pytest.mark.parametrize("bits,n", [(4, 128), (3, 96)])
def test_integer_case_closed_form(bits, n):
    m, r, M = 37, 5, 4
    lay = gen.make_integer_layer(m, n, r, M, bits=bits, seed=2)
    Bi = _f64(lay.B).astype(np.int64)
    Ai = _f64(lay.A).astype(np.int64)
    xi = _f64(lay.x).astype(np.int64)
    Li = lay.codebook.astype(np.int64)[lay.codes]
    want = xi @ (Li * (Bi @ Ai)).T                       # int64, exact
    got = _oracle_forward(lay)
    assert np.array_equal(got, want.astype(np.float64))
    assert np.abs(want).max() <= 256 and np.abs(want).max() > 0
    # exactly representable in bf16, so the rounded output carries the same integers
    assert np.array_equal(gen.bf16_to_f32(oracle.round_bf16(got)).astype(np.int64), want)


# ------------------------------------------- reassociated form identity (P6)

def test_reassociated_form_equals_definition():
    m, n, r, M = 21, 64, 6, 3
    lay = gen.make_layer(m, n, r, M, bits=4, seed=8, mixed_sign=True)
    Bf, Af, xf = _f64(lay.B), _f64(lay.A), _f64(lay.x)
    Lq = lay.codebook.astype(np.float64)[lay.codes]
    # z[t,i,k] = sum_j L[Q_ij] A_kj x_tj ; y[t,i] = sum_k B_ik z[t,i,k]
    z = np.einsum("ij,kj,tj->tik", Lq, Af, xf)
    want = np.einsum("ik,tik->ti", Bf, z)
    np.testing.assert_allclose(_oracle_forward(lay), want, rtol=1e-11, atol=1e-13)


# ------------------------------------------------------ Table 7 rank rule (P8)

def test_equivalent_rank_reproduces_table7():
    n_rows = 0
    with open(os.path.join(GOLDEN, "table7_ranks.txt")) as fh:
        for ln in fh:
            if not ln.strip() or ln.startswith("#"):
                continue
            parts = ln.split()
            rows, cols, r128, r256 = (int(v) for v in parts[-4:])
            assert oracle.equivalent_rank(rows, cols, 128) == r128, ln
            assert oracle.equivalent_rank(rows, cols, 256) == r256, ln
            n_rows += 1
    assert n_rows == 13
    # parameter parity at block size 64 for the 4096 x 4096 projection: 32*(4096+4096) = 4096*4096/64
    assert oracle.equivalent_rank(4096, 4096, 64) == 32


# --------------------------------------------------------- bf16 rounding helper

def test_round_bf16_is_single_rne_step():
    v = np.array([
        1.0, -2.5, 0.0, 3.140625,             # exactly representable
        1.0 + 2.0**-8,                         # tie -> even (1.0)
        1.0 + 3 * 2.0**-8,                     # tie -> even (1 + 2^-6)
        1.0 + 2.0**-8 + 2.0**-40,              # just above the tie: must go up (double rounding via fp32 would not)
        -(1.0 + 2.0**-8 + 2.0**-40),
        255.5, 1e-3,
    ])
    got = gen.bf16_to_f32(oracle.round_bf16(v)).astype(np.float64)
    want = np.array([1.0, -2.5, 0.0, 3.140625, 1.0, 1.0 + 2.0**-6, 1.0 + 2.0**-7, -(1.0 + 2.0**-7), 256.0,
                     0.00099945068359375])
    assert np.array_equal(got, want)
    # agrees with the torch fp32->bf16 cast wherever the input is an fp32 value
    import torch
    f = torch.randn(4096, dtype=torch.float32)
    assert np.array_equal(oracle.round_bf16(f.double().numpy()), gen.bf16_bits(f))


# --------------------------------------------------------------- level tables

@pytest.mark.parametrize("bits", [2, 3, 4])
def test_nf_codebook_properties(bits):
    cb = gen.nf_codebook(bits)
    assert cb.dtype == np.float32 and cb.shape == (2**bits,)
    assert np.all(np.diff(cb) > 0)
    assert cb[0] == -1.0 and cb[-1] == 1.0
    assert np.count_nonzero(cb == 0.0) == 1
    assert np.count_nonzero(cb < 0) == 2 ** (bits - 1) - 1 and np.count_nonzero(cb > 0) == 2 ** (bits - 1)


# ---------------------------------------------------------------- quantisation step (Alg. 1, step 2.1)

def test_quantize_recovers_the_codes_of_a_representable_weight():
    """W = L[Q] * S exactly (small integers everywhere): the error of the true code is zero and every
    other level is off by at least |S|, so the codes come back -- except where S = 0, where every level
    ties and the lowest code wins."""
    import torch
    lay = gen.make_integer_layer(48, 96, 5, 1, bits=4, seed=3)
    S = _f64(lay.B) @ _f64(lay.A)
    S[::7, ::5] = 0.0                                   # some exact zeros in S: knock out the rows of B that feed them
    Bz = _f64(lay.B).copy()
    Bz[::7, :] = 0.0
    S = Bz @ _f64(lay.A)
    W = lay.codebook.astype(np.float64)[lay.codes] * S
    Wb = gen.bf16_bits(torch.from_numpy(W.astype(np.float32)))
    assert np.array_equal(_f64(Wb), W)                  # representable: nothing was rounded
    got = oracle.quantize(Wb, gen.bf16_bits(torch.from_numpy(Bz.astype(np.float32))), lay.A, lay.codebook, 4)
    want = np.where(S != 0.0, lay.codes, 0)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("bits,r,mixed", [(4, 7, True), (3, 16, False), (2, 3, True)])
def test_quantize_is_the_array_wise_argmin(bits, r, mixed):
    """Independent statement with library routines: S by a matmul, the errors of all levels as one
    array, numpy's argmin (which returns the first, i.e. lowest, index of the minimum)."""
    lay = gen.make_layer(40, 64, r, 1, bits=bits, seed=11 + bits, mixed_sign=mixed)
    Wb = gen.make_weight(40, 64, seed=5 + bits)
    S = _f64(lay.B) @ _f64(lay.A)
    E = (S[:, :, None] * lay.codebook.astype(np.float64)[None, None, :] - _f64(Wb)[:, :, None]) ** 2
    codes, runner, gap, mag = oracle.quantize(Wb, lay.B, lay.A, lay.codebook, bits, details=True)
    clear = gap > 1e-12 * mag                            # the two summation orders may differ in the last bits
    assert clear.mean() > 0.999
    assert np.array_equal(codes[clear], E.argmin(axis=2)[clear])
    assert (gap >= 0).all() and (runner != codes).all()


def test_quantize_ties_go_to_the_lower_code_and_signs_cancel():
    import torch
    levels = gen.int_codebook(3)                         # -4 .. 3
    n = 32
    B1 = gen.bf16_bits(torch.ones(1, 1))
    A1 = gen.bf16_bits(torch.full((1, n), 2.0))          # S = 2 everywhere
    mids = (levels[:-1] + levels[1:]) / 2.0              # exact midpoints between neighbouring levels
    w = np.zeros((1, n), dtype=np.float32)
    w[0, :mids.size] = 2.0 * mids                        # W / S on a midpoint: both neighbours are equally far
    w[0, mids.size:mids.size + 2] = [100.0, -100.0]      # far outside the table: the end levels
    Wb = gen.bf16_bits(torch.from_numpy(w))
    got = oracle.quantize(Wb, B1, A1, levels, 3)
    assert np.array_equal(got[0, :mids.size], np.arange(mids.size))            # the lower of the two codes
    assert got[0, mids.size] == 7 and got[0, mids.size + 1] == 0
    # S < 0: the products S * L[c] run downwards, ties still go to the lower code
    Bn = gen.bf16_bits(-torch.ones(1, 1))
    gotn = oracle.quantize(gen.bf16_bits(torch.from_numpy(-w)), Bn, A1, levels, 3)
    assert np.array_equal(gotn, got)                     # (-S) * v - (-W) = -(S v - W): same errors


def test_quantize_is_monotone_in_the_weight_for_positive_scales():
    import torch
    lay = gen.make_layer(8, 64, 4, 1, bits=4, seed=2)     # positive B, A
    base = np.linspace(-0.2, 0.2, 8 * 64, dtype=np.float32).reshape(8, 64)
    cols = np.sort(base, axis=0)                         # every column increases down the rows ...
    Bsame = np.repeat(lay.B[:1], 8, axis=0)              # ... while S is the same in all rows
    got = oracle.quantize(gen.bf16_bits(torch.from_numpy(cols)), Bsame, lay.A, lay.codebook, 4)
    assert (np.diff(got.astype(np.int32), axis=0) >= 0).all()
    assert got.min() == 0 and got.max() == 15            # the grid reaches both ends of the table



# ---- backward with the codes fixed (Sec. 3.4; chain rule of Eq. 5 through S = BA) ------------------------

def _loss(g, y64):
    """The scalar whose gradients the backward returns: sum(g * y), g widened exactly."""
    return float(np.sum(gen.bf16_to_f32(g).astype(np.float64) * y64))


def _replace_entry(bits16, idx, factor=1.5):
    """A copy of a bf16 array with one entry multiplied by 1.5 (exact in bf16 for these inputs' few
    significand bits or not -- the returned difference is the exact one either way)."""
    import torch
    out = bits16.copy()
    old = float(gen.bf16_to_f32(bits16[idx:idx + 1] if bits16.ndim == 1 else np.array([bits16[idx]], dtype=np.uint16))[0])
    new_bits = gen.bf16_bits(torch.tensor([old * factor + 0.25]))
    out[idx] = new_bits[0]
    new = float(gen.bf16_to_f32(new_bits)[0])
    return out, new - old


@pytest.mark.parametrize("bits,m,n,r,M,mixed", [(4, 24, 64, 5, 3, True), (3, 16, 96, 3, 2, True), (2, 20, 40, 4, 4, False)])
def test_backward_matches_exact_differences_of_the_forward(bits, m, n, r, M, mixed):
    """y is linear in every single entry of x, of B and of A.  Replacing one entry by another bf16
    value therefore changes sum(g * y) by exactly (new - old) * (that entry of the gradient), up to
    fp64 rounding: a finite difference with no truncation error, through the forward oracle only."""
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=11 * m + n, mixed_sign=mixed)
    packed = oracle.pack_codes(lay.codes, bits)
    g = gen.make_layer(m, m, 1, M, bits=4, seed=5).x[:, :m].copy()          # any bf16 numbers, M x m
    dx, dB, dA = oracle.backward(g, lay.x, packed, lay.B, lay.A, lay.codebook, bits)
    base = _loss(g, oracle.forward(lay.x, packed, lay.B, lay.A, lay.codebook, bits))
    rng = np.random.default_rng(m + n)
    scale = max(1.0, abs(base))
    for _ in range(12):
        t, j = int(rng.integers(M)), int(rng.integers(n))
        x2, d = _replace_entry(lay.x.reshape(-1), t * n + j)
        l2 = _loss(g, oracle.forward(x2.reshape(M, n), packed, lay.B, lay.A, lay.codebook, bits))
        assert abs((l2 - base) - d * dx[t, j]) <= 1e-11 * scale * max(1.0, abs(d))
        i, k = int(rng.integers(m)), int(rng.integers(r))
        B2, d = _replace_entry(lay.B.reshape(-1), i * r + k)
        l2 = _loss(g, oracle.forward(lay.x, packed, B2.reshape(m, r), lay.A, lay.codebook, bits))
        assert abs((l2 - base) - d * dB[i, k]) <= 1e-11 * scale * max(1.0, abs(d))
        k, j = int(rng.integers(r)), int(rng.integers(n))
        A2, d = _replace_entry(lay.A.reshape(-1), k * n + j)
        l2 = _loss(g, oracle.forward(lay.x, packed, lay.B, A2.reshape(r, n), lay.codebook, bits))
        assert abs((l2 - base) - d * dA[k, j]) <= 1e-11 * scale * max(1.0, abs(d))


def test_backward_euler_identities():
    """y is homogeneous of degree one in x, in B and in A separately, so each gradient paired with its
    own argument gives back the loss: <dx, x> = <dB, B> = <dA, A> = sum(g * y)."""
    lay = gen.make_layer(40, 128, 6, 5, bits=4, seed=3, mixed_sign=True)
    packed = oracle.pack_codes(lay.codes, 4)
    g = gen.make_layer(40, 64, 1, 5, bits=4, seed=8).x[:, :40].copy()
    dx, dB, dA = oracle.backward(g, lay.x, packed, lay.B, lay.A, lay.codebook, 4)
    loss = _loss(g, oracle.forward(lay.x, packed, lay.B, lay.A, lay.codebook, 4))
    f64 = lambda b: gen.bf16_to_f32(b).astype(np.float64)
    for got in (np.sum(dx * f64(lay.x)), np.sum(dB * f64(lay.B)), np.sum(dA * f64(lay.A))):
        assert abs(got - loss) <= 1e-10 * max(1.0, abs(loss))


def test_backward_input_gradient_is_g_times_the_dequantised_weight():
    """dx = g W^: a library matmul with the oracle's own dequantised rows (pinned by P1/P2)."""
    lay = gen.make_layer(48, 96, 7, 3, bits=3, seed=21, mixed_sign=True)
    packed = oracle.pack_codes(lay.codes, 3)
    g = gen.make_layer(48, 64, 1, 3, bits=4, seed=9).x[:, :48].copy()
    dx, _, _ = oracle.backward(g, lay.x, packed, lay.B, lay.A, lay.codebook, 3)
    What = oracle.dequant_rows(packed, lay.B, lay.A, lay.codebook, 3)
    want = gen.bf16_to_f32(g).astype(np.float64) @ What
    assert np.allclose(dx, want, rtol=1e-12, atol=1e-12 * np.abs(want).max())


# ---- the additive-adapter comparator (Sec. 3.4, Sec. 4.4 / Table 6) --------------------------------------

def test_adapter_comparator_against_brute_force():
    """Four nested loops on a tiny problem: block scale times level times x, plus the adapter's two sums."""
    import torch
    m, n, blk, M, r, bits = 6, 64, 32, 2, 3, 4
    lay, s = gen.make_blockwise_layer(m, n, blk, M, bits=bits, seed=4)
    g = torch.Generator().manual_seed(9)
    Al = gen.bf16_bits(torch.randn(r, n, generator=g) * 0.1)
    Bl = gen.bf16_bits(torch.randn(m, r, generator=g) * 0.1)
    qp = oracle.pack_codes(lay.codes, bits)
    got = oracle.adapter_forward(lay.x, qp, s, blk, Al, Bl, lay.codebook, bits)
    xf, sf, af, bf = _f64(lay.x), _f64(s), _f64(Al), _f64(Bl)
    for t in range(M):
        for i in range(m):
            acc = 0.0
            for j in range(n):
                acc += xf[t, j] * float(lay.codebook[lay.codes[i, j]]) * sf[i, j // blk]
            for k in range(r):
                u = 0.0
                for j in range(n):
                    u += xf[t, j] * af[k, j]
                acc += u * bf[i, k]
            assert abs(got[t, i] - acc) <= 1e-12 * max(1.0, abs(acc))
    # without an adapter it is the block-wise forward itself
    zero = np.zeros_like(Al)
    assert np.array_equal(oracle.adapter_forward(lay.x, qp, s, blk, zero, Bl, lay.codebook, bits),
                          oracle.forward(lay.x, qp, lay.B, lay.A, lay.codebook, bits))


# ---- straight-through gradients of quantisation-aware training (Eq. 4-5) --------------------------------

def test_qat_backward_pins():
    import torch
    m, n, r, M, bits = 24, 64, 5, 3, 4
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=31, mixed_sign=True)
    packed = oracle.pack_codes(lay.codes, bits)
    g = gen.make_layer(m, 64, 1, M, bits=4, seed=6).x[:, :m].copy()
    Wb = gen.make_weight(m, n, seed=7, sigma=0.02)
    dW, dB, dA = oracle.backward_qat(g, lay.x, Wb, packed, lay.B, lay.A, lay.codebook, bits)
    gf, xf, Wf, Bf, Af = _f64(g), _f64(lay.x), _f64(Wb), _f64(lay.B), _f64(lay.A)
    # Eq. 4: dL/dW is dL/dW^ = g^T x, a library matmul
    assert np.allclose(dW, gf.T @ xf, rtol=1e-13, atol=1e-13)
    # Eq. 5 against the fine-tuning gradients (pinned above): dS_qat = dS_peft - dW^ (.) (W / S)
    _, dB_p, dA_p = oracle.backward(g, lay.x, packed, lay.B, lay.A, lay.codebook, bits)
    S = Bf @ Af
    assert (S != 0).all()
    extra = dW * (Wf / S)
    assert np.allclose(dB, dB_p - extra @ Af.T, rtol=1e-10, atol=1e-10 * np.abs(dB_p).max())
    assert np.allclose(dA, dA_p - Bf.T @ extra, rtol=1e-10, atol=1e-10 * np.abs(dA_p).max())
    # a weight that its codes represent exactly has Q - W / S = 0: no gradient reaches S
    What = oracle.dequant_rows(packed, lay.B, lay.A, lay.codebook, bits)
    Wexact = gen.bf16_bits(torch.from_numpy(What.astype(np.float32)))
    if np.array_equal(gen.bf16_to_f32(Wexact).astype(np.float64), What):     # only when W^ is bf16-representable
        _, dB0, dA0 = oracle.backward_qat(g, lay.x, Wexact, packed, lay.B, lay.A, lay.codebook, bits)
        assert np.abs(dB0).max() <= 1e-12 and np.abs(dA0).max() <= 1e-12
    # linear in g
    g2 = gen.make_layer(m, 64, 1, M, bits=4, seed=8).x[:, :m].copy()
    gsum = gen.bf16_bits(torch.from_numpy((gen.bf16_to_f32(g) * 2.0).astype(np.float32)))      # 2 g is exact in bf16
    dW2, dB2, dA2 = oracle.backward_qat(gsum, lay.x, Wb, packed, lay.B, lay.A, lay.codebook, bits)
    assert np.allclose(dW2, 2 * dW, rtol=1e-13) and np.allclose(dB2, 2 * dB, rtol=1e-12, atol=1e-15) and np.allclose(dA2, 2 * dA, rtol=1e-12, atol=1e-15)
    del g2


def test_qat_backward_exactly_representable_weight_and_zero_scale():
    """Integers: W = L[Q] * S exactly, so dB = dA = 0; rows with S = 0 contribute nothing either."""
    import torch
    lay = gen.make_integer_layer(32, 64, 4, 2, bits=4, seed=3)
    packed = oracle.pack_codes(lay.codes, 4)
    S = _f64(lay.B) @ _f64(lay.A)
    W = lay.codebook.astype(np.float64)[lay.codes] * S
    Bz = lay.B.copy(); Bz[::5, :] = 0                       # S = 0 in every fifth row
    Wb = gen.bf16_bits(torch.from_numpy(W.astype(np.float32)))
    g = gen.bf16_bits(torch.randint(-2, 3, (2, 32), generator=torch.Generator().manual_seed(1)).float())
    dW, dB, dA = oracle.backward_qat(g, lay.x, Wb, packed, lay.B, lay.A, lay.codebook, 4)
    assert np.array_equal(dB, np.zeros_like(dB)) and np.array_equal(dA, np.zeros_like(dA))
    assert np.array_equal(dW, _f64(g).T @ _f64(lay.x))
    dWz, dBz, dAz = oracle.backward_qat(g, lay.x, Wb, packed, Bz, lay.A, lay.codebook, 4)
    assert np.isfinite(dBz).all() and np.isfinite(dAz).all()
    assert np.array_equal(dBz[::5], np.zeros_like(dBz[::5]))
