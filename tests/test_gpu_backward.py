"""GPU backward with the codes fixed (Sec. 3.4) against the fp64 oracle, through the C ABI.

dx runs on the forward kernels (the transposed layer), so it is held to the forward's criteria: the
fp32 accumulator within the normwise and per-element tolerances, the bf16 output the RNE rounding of
that accumulator and within one bf16 ulp of the rounded oracle value.  dB and dA are fp32 sums on the
CUDA cores over exactly widened bf16 inputs: a sum of K products carries a relative rounding error of
the order of sqrt(K) * 2^-24 (K up to a few million here: about 1e-4 of the norm at worst), so they are
held to 1e-4 normwise and 1e-3 per element (relative to max(|value|, rms)); integer inputs are exact.
The transposition of the packed codes is integer work: bit-exact."""
import numpy as np
import pytest

import oracle
from paper_2601_22716_b200 import inputs as gen
from _util import check_against_oracle, error_metrics

pytestmark = pytest.mark.gpu

FACTOR_NORMWISE_TOL = 1e-4
FACTOR_ELEMENT_TOL = 1e-3


@pytest.fixture(scope="module")
def lords():
    import torch
    from paper_2601_22716_b200 import binding
    assert torch.cuda.is_available()
    binding.lords_init(0, 0)
    yield binding
    binding.lords_set_option("path", "auto")
    binding.lords_shutdown()


def _dev(a16):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a16).view(np.int16)).to("cuda:0")


def _grad_out(M, m, seed, integer=False):
    """g = dL/dy as bf16 bit patterns: N(0, 1), or small integers for the exact cases."""
    import torch
    g = torch.Generator().manual_seed(1000 + seed)
    if integer:
        v = torch.randint(-2, 3, (M, m), generator=g).float()
    else:
        v = torch.randn(M, m, generator=g)
    return gen.bf16_bits(v)


@pytest.mark.parametrize("bits,m,n", [(4, 64, 96), (4, 38, 70), (3, 96, 64), (3, 160, 352), (2, 44, 132), (2, 256, 64),
                                      (4, 1000, 2048)])
def test_transposed_codes_are_bit_exact(lords, bits, m, n):
    import torch
    rng = np.random.default_rng(m * n + bits)
    codes = rng.integers(0, 1 << bits, size=(m, n), dtype=np.uint8)
    q = torch.from_numpy(oracle.pack_codes(codes, bits)).to("cuda:0")
    qt = torch.full((lords.lords_packed_bytes(n, m, bits),), 0xA5, dtype=torch.uint8, device="cuda:0")
    lords.lords_transpose_codes(q, bits, m, n, qt)
    torch.cuda.synchronize()
    want = oracle.pack_codes(np.ascontiguousarray(codes.T), bits)
    assert np.array_equal(qt.cpu().numpy().reshape(want.shape), want)


BACKWARD_SHAPES = [
    # bits, m, n, r, M, mixed, path the input gradient is expected to take
    (4, 512, 384, 32, 1, True, "decode"),        # the transposed layer has 512 in-features
    (4, 1024, 300, 12, 2, True, "decode"),       # ragged out-features of the transposed layer
    (3, 256, 544, 48, 8, True, "decode16"),
    (2, 320, 256, 6, 5, False, "decode16"),
    (4, 384, 256, 32, 200, True, "umma"),
    (3, 512, 160, 16, 40, False, "umma"),
    (4, 38, 66, 5, 3, True, "simt"),             # nothing a multiple of a tile
    (3, 96, 64, 100, 4, False, "simt"),          # a rank the tensor-core paths decline
]


@pytest.mark.parametrize("bits,m,n,r,M,mixed,path", BACKWARD_SHAPES)
def test_backward_against_the_oracle(lords, bits, m, n, r, M, mixed, path):
    import torch
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=7 * m + n + r + M, mixed_sign=mixed)
    g = _grad_out(M, m, m + n)
    packed = oracle.pack_codes(lay.codes, bits)
    dx64, dB64, dA64 = oracle.backward(g, lay.x, packed, lay.B, lay.A, lay.codebook, bits)

    q = torch.from_numpy(packed).to("cuda:0")
    qt = torch.empty(lords.lords_packed_bytes(n, m, bits), dtype=torch.uint8, device="cuda:0")
    lords.lords_transpose_codes(q, bits, m, n, qt)
    gd, xd, Bd, Ad = _dev(g), _dev(lay.x), _dev(lay.B), _dev(lay.A)
    dx32 = torch.zeros((M, n), dtype=torch.float32, device="cuda:0")
    dxbf = torch.zeros((M, n), dtype=torch.int16, device="cuda:0")
    lords.lords_linear_backward_input_f32(gd, qt, Bd, Ad, lay.codebook, bits, M, m, n, r, dx32)
    lords.lords_linear_backward_input(gd, qt, Bd, Ad, lay.codebook, bits, M, m, n, r, dxbf)
    assert lords.lords_last_path() == path
    check_against_oracle(dx32.cpu().numpy(), dxbf.cpu().numpy().view(np.uint16), dx64)
    # the three schedules of the factor gradients: the tile product on the tensor cores (taken when the row
    # pitches of g and x suit TMA), one CTA per tile of W on the CUDA cores -- both with the tiles'
    # contributions summed by a second kernel (one launch for dB and dA) --, and the walk that needs no scratch memory.  (Any forced
    # tensor-core forward path switches the tensor schedule off, "simt" leaves only the walk.)
    first = "backward_tensor" if m % 8 == 0 and n % 8 == 0 else "backward_tiles"
    for option, schedule, launches in (("auto", first, 2), ("decode", "backward_tiles", 2), ("simt", "backward_walk", 2)):
        dB = torch.full((m, r), float("nan"), dtype=torch.float32, device="cuda:0")
        dA = torch.full((r, n), float("nan"), dtype=torch.float32, device="cuda:0")
        lords.lords_set_option("path", option)
        try:
            lords.lords_linear_backward_factors(gd, xd, q, Bd, Ad, lay.codebook, bits, M, m, n, r, dB, dA)
        finally:
            lords.lords_set_option("path", "auto")
        assert lords.lords_last_path() == schedule and lords.lords_last_launch_count() == launches
        torch.cuda.synchronize()
        assert lords.lords_poll_status() == 0
        for name, got, want in (("dB", dB.cpu().numpy(), dB64), ("dA", dA.cpu().numpy(), dA64)):
            assert np.isfinite(got).all(), (schedule, name)
            nw, el = error_metrics(got, want)
            assert nw <= FACTOR_NORMWISE_TOL and el <= FACTOR_ELEMENT_TOL, (schedule, name, nw, el)


@pytest.mark.parametrize("bits,m,n,r,M", [(4, 256, 384, 8, 3), (3, 160, 128, 5, 20), (2, 128, 320, 40, 2)])
def test_backward_integer_case_is_bit_exact(lords, bits, m, n, r, M):
    """Small integers everywhere: every product and partial sum is an exact integer below 2^24."""
    import torch
    lay = gen.make_integer_layer(m, n, r, M, bits=bits, seed=bits + m)
    g = _grad_out(M, m, m, integer=True)
    packed = oracle.pack_codes(lay.codes, bits)
    dx64, dB64, dA64 = oracle.backward(g, lay.x, packed, lay.B, lay.A, lay.codebook, bits)
    q = torch.from_numpy(packed).to("cuda:0")
    qt = torch.empty(lords.lords_packed_bytes(n, m, bits), dtype=torch.uint8, device="cuda:0")
    lords.lords_transpose_codes(q, bits, m, n, qt)
    gd, xd, Bd, Ad = _dev(g), _dev(lay.x), _dev(lay.B), _dev(lay.A)
    dx32 = torch.zeros((M, n), dtype=torch.float32, device="cuda:0")
    dB = torch.zeros((m, r), dtype=torch.float32, device="cuda:0")
    dA = torch.zeros((r, n), dtype=torch.float32, device="cuda:0")
    lords.lords_linear_backward_input_f32(gd, qt, Bd, Ad, lay.codebook, bits, M, m, n, r, dx32)
    torch.cuda.synchronize()
    assert np.array_equal(dx32.cpu().numpy().astype(np.float64), dx64)
    for option in ("auto", "decode", "simt"):
        dB.fill_(float("nan")); dA.fill_(float("nan"))
        lords.lords_set_option("path", option)
        try:
            lords.lords_linear_backward_factors(gd, xd, q, Bd, Ad, lay.codebook, bits, M, m, n, r, dB, dA)
        finally:
            lords.lords_set_option("path", "auto")
        torch.cuda.synchronize()
        assert lords.lords_poll_status() == 0
        assert np.array_equal(dB.cpu().numpy().astype(np.float64), dB64), option
        assert np.array_equal(dA.cpu().numpy().astype(np.float64), dA64), option


def test_backward_factors_one_at_a_time_and_bad_arguments(lords):
    import torch
    lay = gen.make_layer(128, 128, 8, 2, bits=4, seed=1)
    g = _grad_out(2, 128, 3)
    packed = oracle.pack_codes(lay.codes, 4)
    _, dB64, dA64 = oracle.backward(g, lay.x, packed, lay.B, lay.A, lay.codebook, 4)
    q = torch.from_numpy(packed).to("cuda:0")
    gd, xd, Bd, Ad = _dev(g), _dev(lay.x), _dev(lay.B), _dev(lay.A)
    dB = torch.zeros((128, 8), dtype=torch.float32, device="cuda:0")
    dA = torch.zeros((8, 128), dtype=torch.float32, device="cuda:0")
    lords.lords_linear_backward_factors(gd, xd, q, Bd, Ad, lay.codebook, 4, 2, 128, 128, 8, dB, None)
    assert lords.lords_last_path() == "backward_tensor" and lords.lords_last_launch_count() == 2    # the tile kernel and one sum
    lords.lords_linear_backward_factors(gd, xd, q, Bd, Ad, lay.codebook, 4, 2, 128, 128, 8, None, dA)
    torch.cuda.synchronize()
    assert error_metrics(dB.cpu().numpy(), dB64)[0] <= FACTOR_NORMWISE_TOL
    assert error_metrics(dA.cpu().numpy(), dA64)[0] <= FACTOR_NORMWISE_TOL
    with pytest.raises(lords.LordsError) as ei:
        lords.lords_linear_backward_factors(gd, xd, q, Bd, Ad, lay.codebook, 4, 2, 128, 128, 8, None, None)
    assert ei.value.status == -1
    with pytest.raises(lords.LordsError) as ei:        # m = 127 is not a multiple of the 4-bit pack group
        lords.lords_transpose_codes(q, 4, 127, 128, torch.empty(128 * 64, dtype=torch.uint8, device="cuda:0"))
    assert ei.value.status == -2


# ---- straight-through gradients of quantisation-aware training (Eq. 4-5) --------------------------------
# dW is the tile product itself (fp32 accumulation of exactly widened bf16 products: as dB, dA above).  dS
# carries the factor L[Q] - W / S with S (r products) and the quotient in fp32: its rounding error is a few
# 2^-24 of the two terms, far below the fp32 summation error of the folds, so the same tolerances hold
# (measured: 1e-7 to 3e-7 normwise).
QAT_NORMWISE_TOL = FACTOR_NORMWISE_TOL
QAT_ELEMENT_TOL = FACTOR_ELEMENT_TOL


# ranks that are multiples of 8 up to 64 take S from a scale MMA on the tensor schedule, the others rebuild it on the CUDA cores
@pytest.mark.parametrize("bits,m,n,r,M,mixed", [(4, 512, 384, 32, 64, False), (3, 256, 544, 48, 8, True), (2, 320, 256, 6, 5, False),
                                                (4, 136, 200, 12, 130, True), (4, 264, 320, 64, 16, True), (3, 384, 256, 8, 40, False),
                                                (4, 200, 136, 24, 9, True), (4, 128, 64, 72, 3, False)])
def test_qat_backward_against_the_oracle(lords, bits, m, n, r, M, mixed):
    import torch
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=m + 3 * n + r, mixed_sign=mixed)
    Wb = gen.make_weight(m, n, seed=m + r, sigma=0.05 * (r / 32.0))
    codes = oracle.quantize(Wb, lay.B, lay.A, lay.codebook, bits)      # the codes of the current rounding
    packed = oracle.pack_codes(codes, bits)
    g = _grad_out(M, m, n)
    dW64, dB64, dA64 = oracle.backward_qat(g, lay.x, Wb, packed, lay.B, lay.A, lay.codebook, bits)
    q = torch.from_numpy(packed).to("cuda:0")
    # both schedules: the tile product on the tensor cores, and the walk on the CUDA cores that any forced
    # forward path other than "auto" selects (no scratch memory, one launch per factor gradient)
    for option, schedule, launches in (("auto", "backward_qat_tensor", 2), ("simt", "backward_qat_walk", 2)):
        dW = torch.full((m, n), float("nan"), dtype=torch.float32, device="cuda:0")
        dB = torch.full((m, r), float("nan"), dtype=torch.float32, device="cuda:0")
        dA = torch.full((r, n), float("nan"), dtype=torch.float32, device="cuda:0")
        lords.lords_set_option("path", option)
        try:
            lords.lords_linear_backward_qat(_dev(g), _dev(lay.x), _dev(Wb), q, _dev(lay.B), _dev(lay.A), lay.codebook, bits,
                                            M, m, n, r, dW, dB, dA)
        finally:
            lords.lords_set_option("path", "auto")
        assert lords.lords_last_path() == schedule and lords.lords_last_launch_count() == launches
        torch.cuda.synchronize()
        assert lords.lords_poll_status() == 0
        nw, el = error_metrics(dW.cpu().numpy(), dW64)
        assert nw <= FACTOR_NORMWISE_TOL and el <= FACTOR_ELEMENT_TOL, (schedule, "dW", nw, el)
        for name, got, want in (("dB", dB.cpu().numpy(), dB64), ("dA", dA.cpu().numpy(), dA64)):
            assert np.isfinite(got).all(), (schedule, name)
            nw, el = error_metrics(got, want)
            print(f"qat {schedule} {name} bits={bits} m={m} n={n} r={r} M={M}: normwise={nw:.2e} element={el:.2e}")
            assert nw <= QAT_NORMWISE_TOL and el <= QAT_ELEMENT_TOL, (schedule, name, nw, el)


def test_qat_backward_exactly_representable_weight_is_exact(lords):
    """Integers: W = L[Q] S exactly, so the factor L[Q] - W / S is exactly zero and no gradient reaches B or
    A; rows whose S is zero contribute nothing; dW is the exact integer product."""
    import torch
    m, n, r, M = 256, 384, 8, 3
    lay = gen.make_integer_layer(m, n, r, M, bits=4, seed=13)
    Bz = lay.B.copy(); Bz[::9, :] = 0
    S = gen.bf16_to_f32(Bz).astype(np.float64) @ gen.bf16_to_f32(lay.A).astype(np.float64)
    W = lay.codebook.astype(np.float64)[lay.codes] * S
    Wb = gen.bf16_bits(torch.from_numpy(W.astype(np.float32)))
    assert np.array_equal(gen.bf16_to_f32(Wb).astype(np.float64), W)
    packed = oracle.pack_codes(lay.codes, 4)
    g = _grad_out(M, m, 5, integer=True)
    dW64, dB64, dA64 = oracle.backward_qat(g, lay.x, Wb, packed, Bz, lay.A, lay.codebook, 4)
    assert not dB64.any() and not dA64.any()
    q = torch.from_numpy(packed).to("cuda:0")
    dW = torch.full((m, n), float("nan"), dtype=torch.float32, device="cuda:0")
    dB = torch.full((m, r), float("nan"), dtype=torch.float32, device="cuda:0")
    dA = torch.full((r, n), float("nan"), dtype=torch.float32, device="cuda:0")
    lords.lords_linear_backward_qat(_dev(g), _dev(lay.x), _dev(Wb), q, _dev(Bz), _dev(lay.A), lay.codebook, 4, M, m, n, r, dW, dB, dA)
    torch.cuda.synchronize()
    assert lords.lords_poll_status() == 0
    assert np.array_equal(dW.cpu().numpy().astype(np.float64), dW64)
    assert not dB.cpu().numpy().any() and not dA.cpu().numpy().any()


@pytest.mark.parametrize("bits,m,n,r,M,ask", [(4, 36, 64, 4, 2, "WBA"), (3, 75, 96, 7, 19, "WBA"), (2, 130, 68, 33, 1, "BA"),
                                              (4, 100, 70, 17, 5, "W"), (4, 61, 130, 3, 33, "WA"), (3, 67, 64, 128, 4, "B")])
def test_qat_backward_walk_takes_shapes_outside_the_tensor_schedule(lords, bits, m, n, r, M, ask):
    """Row or column counts that are not multiples of 8 (the row pitches of g and x do not suit TMA): the
    walk runs, with any subset of the three gradients asked for; what is not asked for is not touched."""
    import torch
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=5 * m + n + r, mixed_sign=(r % 2 == 1))
    Wb = gen.make_weight(m, n, seed=m + r, sigma=0.05 * (r / 32.0))
    codes = oracle.quantize(Wb, lay.B, lay.A, lay.codebook, bits)
    packed = oracle.pack_codes(codes, bits)
    g = _grad_out(M, m, n + 1)
    want = dict(zip("WBA", oracle.backward_qat(g, lay.x, Wb, packed, lay.B, lay.A, lay.codebook, bits)))
    q = torch.from_numpy(packed).to("cuda:0")
    shapes = {"W": (m, n), "B": (m, r), "A": (r, n)}
    out = {k: torch.full(shapes[k], float("nan"), dtype=torch.float32, device="cuda:0") for k in "WBA"}
    args = [out[k] if k in ask else None for k in "WBA"]
    lords.lords_linear_backward_qat(_dev(g), _dev(lay.x), _dev(Wb), q, _dev(lay.B), _dev(lay.A), lay.codebook, bits,
                                    M, m, n, r, *args)
    launches = (1 if ("B" in ask or "A" not in ask) else 0) + (1 if "A" in ask else 0)
    assert lords.lords_last_path() == "backward_qat_walk" and lords.lords_last_launch_count() == launches
    torch.cuda.synchronize()
    assert lords.lords_poll_status() == 0
    for k in "WBA":
        got = out[k].cpu().numpy()
        if k not in ask:
            assert np.isnan(got).all(), k
            continue
        assert np.isfinite(got).all(), k
        nw, el = error_metrics(got, want[k])
        assert nw <= QAT_NORMWISE_TOL and el <= QAT_ELEMENT_TOL, (k, nw, el)
