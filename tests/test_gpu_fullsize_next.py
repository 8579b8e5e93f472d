"""The quantisation step, the backward calls and the comparators at the sizes and in the launch
configurations that bench.py times (Llama-3-8B q_proj and gate shapes), against the fp64 oracle on
sampled outputs.

Every output of these calls is independent along at least one axis, so the oracle computes a sample
exactly from a slice of the inputs: codes of sampled rows from those rows of W and B; dx of sampled
tokens from those rows of g; dB of sampled rows from those rows of g^T, Q and B with all tokens; dA of
sampled column groups from those columns of x, Q and A with all rows and tokens; the comparators' y of
sampled rows from those rows of Q, the scales and the adapter's B.  Rows are stratified over every
128-row tile and 32-lane quadrant, column groups over every 64-column tile.  Criteria as in the
dedicated files."""
import numpy as np
import pytest

import oracle
from paper_2601_22716_b200 import inputs as gen
from _util import check_against_oracle, error_metrics

pytestmark = pytest.mark.gpu

GRADIENT_NORMWISE_TOL = 1e-4     # fp32 sums of exactly widened products (see test_gpu_backward.py)
GRADIENT_ELEMENT_TOL = 1e-3


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


def _sampled_rows(m, extra, seed):
    """One random row from every 32-row quadrant of every 128-row tile, the first and the last row, plus
    `extra` rows drawn uniformly."""
    rng = np.random.default_rng(seed)
    starts = np.arange(0, m, 32)
    strat = np.minimum(starts + rng.integers(0, 32, size=starts.size), m - 1)
    return np.unique(np.concatenate([[0, m - 1], strat, rng.integers(0, m, size=extra)])).astype(np.int64)


def _sampled_column_groups(n, width, seed):
    """Columns of one group of `width` consecutive columns out of every 64-column tile (width divides 64
    and is a multiple of the pack group), including the first and the last group of the matrix."""
    rng = np.random.default_rng(seed)
    per = 64 // width
    starts = np.arange(0, n, 64) + width * rng.integers(0, per, size=n // 64)
    starts = np.unique(np.concatenate([[0, n - width], starts]))
    return (starts[:, None] + np.arange(width)[None, :]).reshape(-1).astype(np.int64)


@pytest.mark.parametrize("m,n,r,bits", [(4096, 4096, 32, 4), (14336, 4096, 48, 3)])
def test_quantize_full_size_sampled(lords, m, n, r, bits):
    import torch
    lay = gen.make_layer(m, n, r, 1, bits=bits, seed=3)
    Wb = gen.make_weight(m, n, seed=9, sigma=0.05 * (r / 32.0))
    Q = torch.full((lords.lords_packed_bytes(m, n, bits),), 0xA5, dtype=torch.uint8, device="cuda:0")
    lords.lords_quantize_codes(_dev(Wb), _dev(lay.B), _dev(lay.A), lay.codebook, bits, m, n, r, Q)
    assert lords.lords_last_path() == "quantize"
    torch.cuda.synchronize()
    assert lords.lords_poll_status() == 0
    rows = _sampled_rows(m, 32, 17)
    got = oracle.unpack_codes(Q.cpu().numpy().reshape(m, -1)[rows], rows.size, n, bits)
    want, _, gap, mag = oracle.quantize(Wb[rows], lay.B[rows], lay.A, lay.codebook, bits, details=True)
    slack = 8.0 * (r + 2) * 2.0 ** -24 * mag                     # as in test_gpu_quantize.py
    clear = gap > slack
    assert np.array_equal(got[clear], want[clear]), "codes differ where the choice was clear"
    S = gen.bf16_to_f32(lay.B[rows]).astype(np.float64) @ gen.bf16_to_f32(lay.A).astype(np.float64)
    Wf = gen.bf16_to_f32(Wb[rows]).astype(np.float64)
    L = lay.codebook.astype(np.float64)
    excess = np.abs(S * L[got] - Wf) - np.abs(S * L[want] - Wf)
    assert np.all(excess <= slack), "a near tie went to a level that is clearly worse"
    assert (~clear).mean() < 1e-3 + 3e-5 * r
    print(f"quantize {m}x{n} bits={bits}: {rows.size} rows, near ties {(~clear).mean():.2e}, "
          f"differing codes {(got != want).mean():.2e}")


def _check_gradient(name, got, want):
    nw, el = error_metrics(got, want)
    print(f"  {name}: normwise={nw:.2e} element={el:.2e}")
    assert np.isfinite(got).all(), name
    assert nw <= GRADIENT_NORMWISE_TOL and el <= GRADIENT_ELEMENT_TOL, (name, nw, el)


def test_backward_full_size_sampled(lords):
    """q_proj, NF4, r = 32, 512 tokens: the input gradient, the factor gradients and the gradients of
    quantisation-aware training, each on the schedule the dispatcher picks at this size."""
    import torch
    m = n = 4096
    r, bits, M = 32, 4, 512
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=21)
    packed = oracle.pack_codes(lay.codes, bits)
    g = gen.bf16_bits(torch.randn(M, m, generator=torch.Generator().manual_seed(5)))
    Wb = gen.make_weight(m, n, seed=4)
    q = torch.from_numpy(packed).to("cuda:0")
    gd, xd, Bd, Ad = _dev(g), _dev(lay.x), _dev(lay.B), _dev(lay.A)

    qt = torch.empty(lords.lords_packed_bytes(n, m, bits), dtype=torch.uint8, device="cuda:0")
    lords.lords_transpose_codes(q, bits, m, n, qt)
    dx32 = torch.zeros((M, n), dtype=torch.float32, device="cuda:0")
    dxbf = torch.zeros((M, n), dtype=torch.int16, device="cuda:0")
    lords.lords_linear_backward_input_f32(gd, qt, Bd, Ad, lay.codebook, bits, M, m, n, r, dx32)
    lords.lords_linear_backward_input(gd, qt, Bd, Ad, lay.codebook, bits, M, m, n, r, dxbf)
    assert lords.lords_last_path() == "umma"
    dB = torch.full((m, r), float("nan"), dtype=torch.float32, device="cuda:0")
    dA = torch.full((r, n), float("nan"), dtype=torch.float32, device="cuda:0")
    lords.lords_linear_backward_factors(gd, xd, q, Bd, Ad, lay.codebook, bits, M, m, n, r, dB, dA)
    assert lords.lords_last_path() == "backward_tensor"
    dW = torch.full((m, n), float("nan"), dtype=torch.float32, device="cuda:0")
    dBq = torch.full((m, r), float("nan"), dtype=torch.float32, device="cuda:0")
    dAq = torch.full((r, n), float("nan"), dtype=torch.float32, device="cuda:0")
    lords.lords_linear_backward_qat(gd, xd, _dev(Wb), q, Bd, Ad, lay.codebook, bits, M, m, n, r, dW, dBq, dAq)
    assert lords.lords_last_path() == "backward_qat_tensor"
    torch.cuda.synchronize()
    assert lords.lords_poll_status() == 0

    # dx of sampled tokens: the whole layer, those rows of g
    toks = np.unique(np.concatenate([[0, M - 1], np.random.default_rng(1).integers(0, M, size=4)]))
    dx64, _, _ = oracle.backward(g[toks], lay.x[toks], packed, lay.B, lay.A, lay.codebook, bits)
    check_against_oracle(dx32.cpu().numpy()[toks], dxbf.cpu().numpy().view(np.uint16)[toks], dx64, label="dx q_proj 512 tokens")
    assert np.isfinite(dx32.cpu().numpy()).all()

    # dB (and the rows of dW) of sampled rows: all tokens, those rows of g^T, Q, W and B
    rows = _sampled_rows(m, 0, 2)
    gr = np.ascontiguousarray(g[:, rows])
    _, dB64, _ = oracle.backward(gr, lay.x, packed[rows], lay.B[rows], lay.A, lay.codebook, bits)
    _check_gradient("dB", dB.cpu().numpy()[rows], dB64)
    dW64, dBq64, _ = oracle.backward_qat(gr, lay.x, Wb[rows], packed[rows], lay.B[rows], lay.A, lay.codebook, bits)
    _check_gradient("dB qat", dBq.cpu().numpy()[rows], dBq64)
    _check_gradient("dW rows", dW.cpu().numpy()[rows], dW64)

    # dA (and the columns of dW) of sampled column groups: all rows and tokens, those columns of x, Q, W and A
    cols = _sampled_column_groups(n, 8, 3)
    xc = np.ascontiguousarray(lay.x[:, cols])
    Ac = np.ascontiguousarray(lay.A[:, cols])
    pc = oracle.pack_codes(np.ascontiguousarray(lay.codes[:, cols]), bits)
    _, _, dA64 = oracle.backward(g, xc, pc, lay.B, Ac, lay.codebook, bits)
    _check_gradient("dA", dA.cpu().numpy()[:, cols], dA64)
    dW64c, _, dAq64 = oracle.backward_qat(g, xc, np.ascontiguousarray(Wb[:, cols]), pc, lay.B, Ac, lay.codebook, bits)
    _check_gradient("dA qat", dAq.cpu().numpy()[:, cols], dAq64)
    _check_gradient("dW columns", dW.cpu().numpy()[:, cols], dW64c)
    assert np.isfinite(dW.cpu().numpy()).all() and np.isfinite(dB.cpu().numpy()).all() and np.isfinite(dA.cpu().numpy()).all()


@pytest.mark.parametrize("M", [1, 8])
def test_comparators_full_size_sampled(lords, M):
    """q_proj with block-64 NF4 scales, alone and with a rank-32 additive adapter."""
    import torch
    m = n = 4096
    bits, blk, r = 4, 64, 32
    lay, s = gen.make_blockwise_layer(m, n, blk, M, bits=bits, seed=12 + M)
    packed = oracle.pack_codes(lay.codes, bits)
    gg = torch.Generator().manual_seed(8)
    Al = gen.bf16_bits(torch.randn(r, n, generator=gg) * 0.05)
    Bl = gen.bf16_bits(torch.randn(m, r, generator=gg) * 0.05)
    q, xd, sd = torch.from_numpy(packed).to("cuda:0"), _dev(lay.x), _dev(s)
    y32 = torch.zeros((M, m), dtype=torch.float32, device="cuda:0")
    ybf = torch.zeros((M, m), dtype=torch.int16, device="cuda:0")
    lords.lords_blockscale_forward(xd, q, sd, lay.codebook, bits, blk, M, m, n, y32, f32=True)
    lords.lords_blockscale_forward(xd, q, sd, lay.codebook, bits, blk, M, m, n, ybf)
    assert lords.lords_last_path() == "blockscale16"
    a32 = torch.zeros((M, m), dtype=torch.float32, device="cuda:0")
    abf = torch.zeros((M, m), dtype=torch.int16, device="cuda:0")
    lords.lords_adapter_forward(xd, q, sd, _dev(Al), _dev(Bl), lay.codebook, bits, blk, M, m, n, r, a32, f32=True)
    lords.lords_adapter_forward(xd, q, sd, _dev(Al), _dev(Bl), lay.codebook, bits, blk, M, m, n, r, abf)
    assert lords.lords_last_path() == "blockscale16+adapter"
    torch.cuda.synchronize()
    assert lords.lords_poll_status() == 0
    rows = _sampled_rows(m, 32, 6)
    zero_B = np.zeros((rows.size, r), dtype=np.uint16)
    want_block = oracle.adapter_forward(lay.x, packed[rows], s[rows], blk, Al, zero_B, lay.codebook, bits)
    check_against_oracle(y32.cpu().numpy()[:, rows], ybf.cpu().numpy().view(np.uint16)[:, rows], want_block,
                         label=f"blockscale q_proj M={M}")
    want = oracle.adapter_forward(lay.x, packed[rows], s[rows], blk, Al, Bl[rows], lay.codebook, bits)
    check_against_oracle(a32.cpu().numpy()[:, rows], abf.cpu().numpy().view(np.uint16)[:, rows], want,
                         label=f"blockscale + adapter q_proj M={M}")
    assert np.isfinite(y32.cpu().numpy()).all() and np.isfinite(a32.cpu().numpy()).all()
