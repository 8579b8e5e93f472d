"""The allocation-free entry point against the regular one.

lords_linear_forward_noalloc serves callers that are not allowed to allocate device memory
(a plugin under a server whose pool owns all of HBM; a loop that cannot take cudaMalloc's
device-wide synchronisation).  It keeps its split-K partial sums in a fixed array inside the
library image instead of the lords_init workspace.  Here it is called twice in a row through
the C ABI -- a larger problem first, then a smaller one that reuses the same array with stale
contents in it -- and each result is compared with lords_linear_forward_bits.  The two entry
points may split the reduction differently, so the comparison uses the suite's tolerances
rather than bit equality.  The file name keeps it last in collection order.
"""
import numpy as np
import pytest

from paper_2601_22716_b200 import inputs as gen
from _util import NORMWISE_TOL, ELEMENT_TOL, error_metrics

pytestmark = pytest.mark.gpu


def _upload(lay, lords, torch):
    dev = torch.device("cuda:0")
    packed = lords.lords_pack_codes(lay.codes, lay.bits)
    return (torch.from_numpy(packed).to(dev), torch.from_numpy(lay.B.view(np.int16)).to(dev),
            torch.from_numpy(lay.A.view(np.int16)).to(dev), torch.from_numpy(lay.x.view(np.int16)).to(dev))


def test_noalloc_entry_matches_regular_entry_twice_in_a_row():
    import torch
    from paper_2601_22716_b200 import binding as lords
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)

    cases = [gen.make_layer(1024, 2048, 32, 8, bits=4, seed=31),
             gen.make_layer(200, 96, 5, 3, bits=3, seed=32, mixed_sign=True)]
    uploaded = [_upload(lay, lords, torch) for lay in cases]
    outs = []
    # the new entry point first, back to back, before the library is initialised at all
    for lay, (q, B, A, x) in zip(cases, uploaded):
        y = torch.full((lay.M, lay.m), 0x7FC0, dtype=torch.int16, device="cuda:0")
        lords.lords_linear_forward_noalloc(x, q, B, A, lay.codebook, lay.bits, lay.M, lay.m, lay.n, lay.r, y)
        outs.append(y)
    torch.cuda.synchronize()

    lords.lords_init(0, 0)
    try:
        for lay, (q, B, A, x), y_new in zip(cases, uploaded, outs):
            y_ref = torch.zeros((lay.M, lay.m), dtype=torch.int16, device="cuda:0")
            lords.lords_linear_forward_bits(x, q, B, A, lay.codebook, lay.bits, lay.M, lay.m, lay.n, lay.r, y_ref)
            torch.cuda.synchronize()
            got = gen.bf16_to_f32(y_new.cpu().numpy().view(np.uint16)).astype(np.float64)
            want = gen.bf16_to_f32(y_ref.cpu().numpy().view(np.uint16)).astype(np.float64)
            assert np.isfinite(got).all()
            # both are bf16 roundings of nearly equal fp32 sums: at most one bf16 step apart
            normwise, element = error_metrics(got, want)
            assert normwise <= 2 * NORMWISE_TOL and element <= 2 * ELEMENT_TOL, (normwise, element)
    finally:
        lords.lords_shutdown()


def test_noalloc_entry_rejects_oversized_problems():
    import ctypes
    from paper_2601_22716_b200 import binding as lords
    lib = ctypes.CDLL(str(lords.library_path()))
    f = lib.lords_linear_forward_noalloc
    f.restype = ctypes.c_int
    P = ctypes.c_void_p
    f.argtypes = [P, P, P, P, P, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, P, P]
    cb = (ctypes.c_float * 16)()
    ok = P(4096)   # aligned and never dereferenced: the size check comes first
    # 2 * M * m = 2 * 512 * 4096 floats > 2^20
    assert f(ok, ok, ok, ok, ctypes.cast(cb, P), 4, 512, 4096, 4096, 32, ok, None) == -9
