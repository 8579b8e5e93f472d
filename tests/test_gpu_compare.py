"""The comparators of Sec. 4.4 / Table 6 on the GPU against the fp64 oracle, through the C ABI.

The block-scaled layer (Eq. 2) is the LoRDS layer with B = s and A = the block indicator, so the
oracle's forward of that special case is its reference (the block-wise pin ties it to an independent
Eq. 2 dequantiser); it is also compared with the library's own LoRDS kernels fed those factors, which
must agree with it to within the forward tolerance.  The adapter variant is held to the same forward
criteria against oracle.adapter_forward."""
import numpy as np
import pytest

import oracle
from paper_2601_22716_b200 import inputs as gen
from _util import check_against_oracle, error_metrics, NORMWISE_TOL

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


def _dev(a16):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a16).view(np.int16)).to("cuda:0")


CASES = [
    # bits, m, n, blk, M
    (4, 512, 1024, 64, 1),
    (4, 300, 1088, 64, 8),      # ragged rows, n = 8.5 k-steps
    (4, 256, 2048, 128, 16),
    (3, 384, 1024, 128, 3),
    (2, 200, 512, 64, 5),
    (4, 128, 4096, 256, 2),
]


@pytest.mark.parametrize("bits,m,n,blk,M", CASES)
def test_blockscale_and_adapter_against_the_oracle(lords, bits, m, n, blk, M):
    import torch
    if n % blk:
        pytest.skip("the generator wants whole blocks")
    lay, s = gen.make_blockwise_layer(m, n, blk, M, bits=bits, seed=m + n + blk)
    packed = oracle.pack_codes(lay.codes, bits)
    q, xd, sd = torch.from_numpy(packed).to("cuda:0"), _dev(lay.x), _dev(s)
    y64 = oracle.forward(lay.x, packed, lay.B, lay.A, lay.codebook, bits)

    y32 = torch.zeros((M, m), dtype=torch.float32, device="cuda:0")
    ybf = torch.zeros((M, m), dtype=torch.int16, device="cuda:0")
    lords.lords_blockscale_forward(xd, q, sd, lay.codebook, bits, blk, M, m, n, y32, f32=True)
    lords.lords_blockscale_forward(xd, q, sd, lay.codebook, bits, blk, M, m, n, ybf)
    assert lords.lords_last_path() == "blockscale16" and lords.lords_last_launch_count() == 1
    torch.cuda.synchronize()
    assert lords.lords_poll_status() == 0
    check_against_oracle(y32.cpu().numpy(), ybf.cpu().numpy().view(np.uint16), y64)

    # the same layer through the LoRDS kernels with B = s, A = indicator (whatever path takes r = n / blk)
    yl = torch.zeros((M, m), dtype=torch.float32, device="cuda:0")
    lords.lords_linear_forward_f32(xd, q, _dev(lay.B), _dev(lay.A), lay.codebook, bits, M, m, n, lay.r, yl)
    torch.cuda.synchronize()
    assert error_metrics(y32.cpu().numpy(), yl.cpu().numpy().astype(np.float64))[0] <= 2 * NORMWISE_TOL

    # with an additive rank-32 adapter on top
    g = torch.Generator().manual_seed(m)
    r = 32
    Al = gen.bf16_bits(torch.randn(r, n, generator=g) * 0.05)
    Bl = gen.bf16_bits(torch.randn(m, r, generator=g) * 0.05)
    want = oracle.adapter_forward(lay.x, packed, s, blk, Al, Bl, lay.codebook, bits)
    a32 = torch.zeros((M, m), dtype=torch.float32, device="cuda:0")
    abf = torch.zeros((M, m), dtype=torch.int16, device="cuda:0")
    lords.lords_adapter_forward(xd, q, sd, _dev(Al), _dev(Bl), lay.codebook, bits, blk, M, m, n, r, a32, f32=True)
    lords.lords_adapter_forward(xd, q, sd, _dev(Al), _dev(Bl), lay.codebook, bits, blk, M, m, n, r, abf)
    assert lords.lords_last_path() == "blockscale16+adapter" and lords.lords_last_launch_count() == 3
    torch.cuda.synchronize()
    assert lords.lords_poll_status() == 0
    check_against_oracle(a32.cpu().numpy(), abf.cpu().numpy().view(np.uint16), want)


def test_comparators_decline_what_they_cannot_run(lords):
    import torch
    lay, s = gen.make_blockwise_layer(128, 256, 64, 4, bits=4, seed=1)
    q = torch.from_numpy(oracle.pack_codes(lay.codes, 4)).to("cuda:0")
    y = torch.zeros((4, 128), dtype=torch.int16, device="cuda:0")
    with pytest.raises(lords.LordsError) as ei:       # blocks of 32 columns: a thread's 64 columns would span two
        lords.lords_blockscale_forward(_dev(lay.x), q, _dev(s), lay.codebook, 4, 32, 4, 128, 256, y)
    assert ei.value.status == -11
    x17 = torch.zeros((17, 256), dtype=torch.int16, device="cuda:0")
    y17 = torch.zeros((17, 128), dtype=torch.int16, device="cuda:0")
    with pytest.raises(lords.LordsError) as ei:       # more than 16 tokens
        lords.lords_blockscale_forward(x17, q, _dev(s), lay.codebook, 4, 64, 17, 128, 256, y17)
    assert ei.value.status == -11
