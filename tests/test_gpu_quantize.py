"""GPU quantisation step (Alg. 1, step 2.1) against the fp64 oracle, through the C ABI.

The kernel accumulates S = B A in fp32 and decides in fp32; the oracle does both in fp64.  A weight whose
two nearest levels are equally far to within fp32 rounding (of a sum of r products: proportional to
the sum of their absolute values) may therefore get either of the two.  The test asserts that the codes are equal wherever the oracle's choice was clear by more than
that rounding distance, that every other code is as good as the oracle's to within that distance, and
that such near ties are rare; then that the packed codes, fed to the forward path, reproduce the oracle's forward of
the oracle's codes up to the forward tolerances."""
import dataclasses

import numpy as np
import pytest

import oracle
from paper_2601_22716_b200 import inputs as gen
from _util import NORMWISE_TOL, error_metrics

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lords():
    import torch
    from paper_2601_22716_b200 import binding
    assert torch.cuda.is_available()
    binding.lords_init(0, 0)
    yield binding
    binding.lords_set_option("path", "auto")
    binding.lords_shutdown()


def _quantize_on_gpu(lords, Wb, lay, path="auto"):
    import torch
    dev = torch.device("cuda:0")
    W = torch.from_numpy(Wb.view(np.int16)).to(dev)
    B = torch.from_numpy(lay.B.view(np.int16)).to(dev)
    A = torch.from_numpy(lay.A.view(np.int16)).to(dev)
    nbytes = lords.lords_packed_bytes(lay.m, lay.n, lay.bits)
    Q = torch.full((nbytes,), 0xA5, dtype=torch.uint8, device=dev)
    lords.lords_set_option("path", path)
    try:
        lords.lords_quantize_codes(W, B, A, lay.codebook, lay.bits, lay.m, lay.n, lay.r, Q)
        torch.cuda.synchronize()
        used = lords.lords_last_path()
    finally:
        lords.lords_set_option("path", "auto")
    assert lords.lords_poll_status() == 0
    return Q, used


def _check_codes(lords, Q, Wb, lay):
    packed = Q.cpu().numpy().reshape(lay.m, -1)
    got = oracle.unpack_codes(packed, lay.m, lay.n, lay.bits)          # the oracle's own reader of the layout
    want, runner, gap, mag = oracle.quantize(Wb, lay.B, lay.A, lay.codebook, lay.bits, details=True)
    # fp32 accumulation of r products and one fused multiply-add: a few (r + 2) * 2^-24 of the magnitude,
    # which is that of the sum of the ABSOLUTE products B_ik A_kj (times the largest level) plus |W|:
    # with factors of mixed sign S cancels, and its rounding error does not
    slack = 8.0 * (lay.r + 2) * 2.0 ** -24 * mag
    clear = gap > slack
    assert np.array_equal(got[clear], want[clear]), "codes differ where the choice was clear"
    near = ~clear
    # a near tie may go to any level that is as good as the best one to within the slack (with a scale
    # near zero several levels are)
    S = gen.bf16_to_f32(lay.B).astype(np.float64) @ gen.bf16_to_f32(lay.A).astype(np.float64)
    Wf = gen.bf16_to_f32(Wb).astype(np.float64)
    L = lay.codebook.astype(np.float64)
    excess = np.abs(S * L[got] - Wf) - np.abs(S * L[want] - Wf)
    assert np.all(excess <= slack), "a near tie went to a level that is clearly worse"
    assert near.mean() < 1e-3 + 3e-5 * lay.r, f"too many near ties: {near.mean():.2e}"       # the slack grows with r
    return want


@pytest.mark.parametrize("bits,m,n,r,mixed", [
    (4, 256, 512, 32, False),
    (4, 300, 1088, 24, True),       # ragged rows, r padded to 32, mixed signs of S
    (3, 384, 1024, 48, False),
    (3, 130, 256, 7, True),
    (2, 128, 320, 5, True),
    (4, 129, 64, 64, False),        # one column step, the largest tensor-core rank
])
def test_quantize_tensor_core_path(lords, bits, m, n, r, mixed):
    lay = gen.make_layer(m, n, r, 1, bits=bits, seed=m + n + r, mixed_sign=mixed)
    Wb = gen.make_weight(m, n, seed=3 * m + r, sigma=0.05 * (r / 32.0))
    Q, used = _quantize_on_gpu(lords, Wb, lay)
    assert used == "quantize"
    _check_codes(lords, Q, Wb, lay)


@pytest.mark.parametrize("bits,m,n,r", [(4, 70, 66, 5), (3, 33, 96, 100), (2, 64, 132, 3), (4, 200, 512, 128),
                                        (4, 520, 2048, 128)])      # the last one: many ranks of mixed sign, S cancels heavily
def test_quantize_cuda_core_path(lords, bits, m, n, r):
    lay = gen.make_layer(m, n, r, 1, bits=bits, seed=m + n, mixed_sign=True)
    Wb = gen.make_weight(m, n, seed=m, sigma=0.05 * (r / 32.0))
    Q, used = _quantize_on_gpu(lords, Wb, lay)
    assert used == "quantize_simt"
    _check_codes(lords, Q, Wb, lay)


def test_quantize_integer_case_is_bit_exact(lords):
    """Small integers everywhere: no rounding anywhere, so the packed bytes equal the packed true codes."""
    import torch
    lay = gen.make_integer_layer(256, 512, 8, 1, bits=4, seed=9)
    S = gen.bf16_to_f32(lay.B).astype(np.float64) @ gen.bf16_to_f32(lay.A).astype(np.float64)
    W = lay.codebook.astype(np.float64)[lay.codes] * S
    Wb = gen.bf16_bits(torch.from_numpy(W.astype(np.float32)))
    assert np.array_equal(gen.bf16_to_f32(Wb).astype(np.float64), W)
    Q, used = _quantize_on_gpu(lords, Wb, lay)
    assert np.array_equal(Q.cpu().numpy().reshape(lay.m, -1), oracle.pack_codes(lay.codes, 4))
    assert np.array_equal(oracle.quantize(Wb, lay.B, lay.A, lay.codebook, 4), lay.codes)


def test_quantize_then_forward_matches_the_oracle(lords):
    """The step before the path feeds the path: codes quantised on the device, used by the forward
    kernels as they are, against the oracle's forward of the oracle's codes."""
    import torch
    m, n, r, M = 512, 1024, 32, 4
    lay = gen.make_layer(m, n, r, M, bits=4, seed=21)
    Wb = gen.make_weight(m, n, seed=22)
    Q, _ = _quantize_on_gpu(lords, Wb, lay)
    want_codes = _check_codes(lords, Q, Wb, lay)
    dev = torch.device("cuda:0")
    B = torch.from_numpy(lay.B.view(np.int16)).to(dev)
    A = torch.from_numpy(lay.A.view(np.int16)).to(dev)
    x = torch.from_numpy(lay.x.view(np.int16)).to(dev)
    y32 = torch.zeros((M, m), dtype=torch.float32, device=dev)
    lords.lords_linear_forward_f32(x, Q, B, A, lay.codebook, 4, M, m, n, r, y32)
    torch.cuda.synchronize()
    assert lords.lords_poll_status() == 0
    y64 = oracle.forward(lay.x, oracle.pack_codes(want_codes, 4), lay.B, lay.A, lay.codebook, 4)
    nw, _ = error_metrics(y32.cpu().numpy(), y64)
    assert nw <= 2 * NORMWISE_TOL          # a handful of near-tie codes may differ on top of the forward's own rounding
    # and the quantised layer approximates the weight it came from: mean squared error well below the weight's power
    What = oracle.dequant_rows(Q.cpu().numpy().reshape(m, -1), lay.B, lay.A, lay.codebook, 4)
    Wf = gen.bf16_to_f32(Wb).astype(np.float64)
    assert np.mean((What - Wf) ** 2) < 0.1 * np.mean(Wf ** 2)


@pytest.mark.parametrize("bits", [4, 3, 2])
def test_quantize_with_a_table_that_is_not_ascending(lords, bits):
    """An ascending table is searched by bisection over its midpoints, any other one level by level:
    a permuted table takes the second route and must give the oracle's codes just the same."""
    lay = gen.make_layer(256, 256, 16, 1, bits=bits, seed=70 + bits, mixed_sign=True)
    rng = np.random.default_rng(bits)
    lay = dataclasses.replace(lay, codebook=np.ascontiguousarray(lay.codebook[rng.permutation(1 << bits)]))
    Wb = gen.make_weight(256, 256, seed=80 + bits, sigma=0.025)
    Q, used = _quantize_on_gpu(lords, Wb, lay)
    assert used == "quantize"
    _check_codes(lords, Q, Wb, lay)


def test_quantize_exact_ties_and_zero_scale_take_the_lowest_code(lords):
    """Integers, so that nothing rounds: weights exactly half-way between two levels keep the lower
    code for either sign of S, and rows whose S is zero (every level equally good) get code 0."""
    import torch
    m, n, r = 128, 64, 2
    levels = np.array([-6, -4, -2, 0, 2, 4, 6, 8], dtype=np.float32)      # 3 bits, ascending
    rng = np.random.default_rng(5)
    Bf = np.zeros((m, r), dtype=np.float32)
    Bf[:, 0] = rng.choice([-2.0, -1.0, 1.0, 2.0], size=m)
    Bf[::7, 0] = 0.0                                     # rows with S = 0
    Af = np.zeros((r, n), dtype=np.float32)
    Af[0, :] = 1.0
    S = Bf @ Af
    lo = rng.integers(0, 7, size=(m, n))
    W = S * (levels[lo] + 1.0)                           # exactly between level lo and lo + 1 (in units of S)
    W[::7, :] = rng.integers(-5, 6, size=(len(range(0, m, 7)), n))
    lay = dataclasses.replace(gen.make_integer_layer(m, n, r, 1, bits=3, seed=1), B=gen.bf16_bits(torch.from_numpy(Bf)),
                              A=gen.bf16_bits(torch.from_numpy(Af)), codebook=levels)
    Wb = gen.bf16_bits(torch.from_numpy(W.astype(np.float32)))
    assert np.array_equal(gen.bf16_to_f32(Wb), W.astype(np.float32))
    want = oracle.quantize(Wb, lay.B, lay.A, lay.codebook, 3)
    expect = lo.copy()
    expect[::7, :] = 0
    assert np.array_equal(want, expect)                  # the oracle follows the tie rule ...
    Q, used = _quantize_on_gpu(lords, Wb, lay)
    assert used == "quantize"
    got = oracle.unpack_codes(Q.cpu().numpy().reshape(m, -1), m, n, 3)
    assert np.array_equal(got, expect)                   # ... and so does the kernel, bit for bit
