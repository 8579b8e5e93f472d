"""Seeded random shapes through every entry point, against the fp64 oracle.

The hand-picked cases of the other files aim at tile edges; this file draws shapes, ranks, token counts,
bit widths and sign patterns at random (fixed seeds) and runs, for each draw: the forward on the path
the dispatcher picks and on every forced path that accepts the shape; the input gradient and the factor
gradients; the quantisation-aware-training gradients; the block-scaled layer with an adapter; the
quantisation step.  Criteria are those of the dedicated files."""
import numpy as np
import pytest

import oracle
from paper_2601_22716_b200 import inputs as gen
from _util import DeviceLayer, check_against_oracle, error_metrics

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


def _draw(rng):
    bits = int(rng.choice([2, 3, 4]))
    grp = {2: 4, 3: 32, 4: 2}[bits]
    n = int(rng.choice([64, 128, 192, 256, 320, 512, 1024, 1088, 2048])) if rng.random() < 0.8 else int(grp * rng.integers(1, 40))
    m = int(rng.choice([8, 64, 100, 128, 130, 256, 384, 520, 1000])) if rng.random() < 0.8 else int(rng.integers(8, 300))
    r = int(rng.choice([1, 2, 3, 5, 6, 7, 8, 12, 15, 16, 24, 32, 33, 48, 64, 65, 100, 128]))
    M = int(rng.choice([1, 2, 3, 4, 7, 8, 15, 16, 17, 33, 64, 100, 129, 257, 300]))
    return bits, grp, m, n, r, M, bool(rng.random() < 0.5)


def _check_gradient(name, got, want):
    nw, el = error_metrics(got.cpu().numpy(), want)
    assert nw <= GRADIENT_NORMWISE_TOL and el <= GRADIENT_ELEMENT_TOL, (name, nw, el)


@pytest.mark.parametrize("seed", [101, 102, 103])
def test_random_shapes(lords, seed):
    import torch
    rng = np.random.default_rng(seed)
    for case in range(25):
        bits, grp, m, n, r, M, mixed = _draw(rng)
        tag = dict(seed=seed, case=case, bits=bits, m=m, n=n, r=r, M=M, mixed=mixed)
        lay = gen.make_layer(m, n, r, M, bits=bits, seed=seed * 1000 + case, mixed_sign=mixed)
        dl = DeviceLayer(lay)
        y64 = oracle.forward(lay.x, dl.packed_host, lay.B, lay.A, lay.codebook, bits)
        for path in ("auto", "decode", "decode16", "umma", "simt"):
            lords.lords_set_option("path", path)
            try:
                try:
                    y32, ybf = dl.forward()
                except lords.LordsError as e:
                    assert e.status == -11 and path != "auto" and path != "simt", (tag, path, e.status)
                    continue
            finally:
                lords.lords_set_option("path", "auto")
            check_against_oracle(y32, ybf, y64, label=f"random {tag} {path}")

        if M <= 64 and m % grp == 0:              # gradients of fine-tuning (Sec. 3.4)
            g = gen.bf16_bits(torch.randn(M, m, generator=torch.Generator().manual_seed(case)))
            dx64, dB64, dA64 = oracle.backward(g, lay.x, dl.packed_host, lay.B, lay.A, lay.codebook, bits)
            gd = _dev(g)
            qt = torch.empty(lords.lords_packed_bytes(n, m, bits), dtype=torch.uint8, device="cuda:0")
            lords.lords_transpose_codes(dl.q, bits, m, n, qt)
            dx32 = torch.zeros((M, n), dtype=torch.float32, device="cuda:0")
            dxb = torch.zeros((M, n), dtype=torch.int16, device="cuda:0")
            lords.lords_linear_backward_input_f32(gd, qt, dl.B, dl.A, lay.codebook, bits, M, m, n, r, dx32)
            lords.lords_linear_backward_input(gd, qt, dl.B, dl.A, lay.codebook, bits, M, m, n, r, dxb)
            dB = torch.zeros((m, r), dtype=torch.float32, device="cuda:0")
            dA = torch.zeros((r, n), dtype=torch.float32, device="cuda:0")
            lords.lords_linear_backward_factors(gd, dl.x, dl.q, dl.B, dl.A, lay.codebook, bits, M, m, n, r, dB, dA)
            torch.cuda.synchronize()
            assert lords.lords_poll_status() == 0, tag
            check_against_oracle(dx32.cpu().numpy(), dxb.cpu().numpy().view(np.uint16), dx64)
            _check_gradient(("dB", tag), dB, dB64)
            _check_gradient(("dA", tag), dA, dA64)
            # gradients of quantisation-aware training (Eq. 4-5), on whichever schedule takes the shape
            Wq = gen.make_weight(m, n, seed=case + 5, sigma=0.05 * max(r, 4) / 32.0)
            dW64, dBq64, dAq64 = oracle.backward_qat(g, lay.x, Wq, dl.packed_host, lay.B, lay.A, lay.codebook, bits)
            dW = torch.zeros((m, n), dtype=torch.float32, device="cuda:0")
            lords.lords_linear_backward_qat(gd, dl.x, _dev(Wq), dl.q, dl.B, dl.A, lay.codebook, bits, M, m, n, r, dW, dB, dA)
            torch.cuda.synchronize()
            assert lords.lords_poll_status() == 0, tag
            _check_gradient(("dW", tag), dW, dW64)
            _check_gradient(("dB qat", tag), dB, dBq64)
            _check_gradient(("dA qat", tag), dA, dAq64)

        if M <= 16 and n % 128 == 0:              # the comparators (Sec. 4.4)
            blk = int(rng.choice([64, 128]))
            bl, sc = gen.make_blockwise_layer(m, n, blk, M, bits=bits, seed=case)
            pk = oracle.pack_codes(bl.codes, bits)
            gg = torch.Generator().manual_seed(case)
            Al = gen.bf16_bits(torch.randn(8, n, generator=gg) * 0.05)
            Bl = gen.bf16_bits(torch.randn(m, 8, generator=gg) * 0.05)
            a32 = torch.zeros((M, m), dtype=torch.float32, device="cuda:0")
            abf = torch.zeros((M, m), dtype=torch.int16, device="cuda:0")
            args = (_dev(bl.x), torch.from_numpy(pk).to("cuda:0"), _dev(sc), _dev(Al), _dev(Bl), bl.codebook, bits, blk, M, m, n, 8)
            lords.lords_adapter_forward(*args, a32, f32=True)
            lords.lords_adapter_forward(*args, abf)
            torch.cuda.synchronize()
            assert lords.lords_poll_status() == 0, tag
            check_against_oracle(a32.cpu().numpy(), abf.cpu().numpy().view(np.uint16),
                                 oracle.adapter_forward(bl.x, pk, sc, blk, Al, Bl, bl.codebook, bits))

        if M <= 4:                                # the quantisation step (Alg. 1, step 2.1)
            Wb = gen.make_weight(m, n, seed=case, sigma=0.05 * max(r, 4) / 32.0)
            Q = torch.empty(lords.lords_packed_bytes(m, n, bits), dtype=torch.uint8, device="cuda:0")
            lords.lords_quantize_codes(_dev(Wb), dl.B, dl.A, lay.codebook, bits, m, n, r, Q)
            torch.cuda.synchronize()
            assert lords.lords_poll_status() == 0, tag
            got = oracle.unpack_codes(Q.cpu().numpy().reshape(m, -1), m, n, bits)
            want, _, gap, mag = oracle.quantize(Wb, lay.B, lay.A, lay.codebook, bits, details=True)
            slack = 8.0 * (r + 2) * 2.0 ** -24 * mag
            assert np.array_equal(got[gap > slack], want[gap > slack]), tag
            S = gen.bf16_to_f32(lay.B).astype(np.float64) @ gen.bf16_to_f32(lay.A).astype(np.float64)
            Wf = gen.bf16_to_f32(Wb).astype(np.float64)
            L = lay.codebook.astype(np.float64)
            assert np.all(np.abs(S * L[got] - Wf) - np.abs(S * L[want] - Wf) <= slack), tag
