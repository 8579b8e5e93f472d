"""The allocation-free entry point against the fp64 oracle, and interleaved with the regular path.

lords_linear_forward_noalloc serves callers that are not allowed to allocate device memory
(a plugin under a server whose pool owns all of HBM; a loop that cannot take cudaMalloc's
device-wide synchronisation).  It keeps its split-K partial sums in a fixed array inside the
library image instead of the lords_init workspace.  Here it is called several times in a row
through the C ABI -- a larger problem first, then smaller ones that reuse the same array with stale
contents in it, one of them with a rank whose shared-memory need exceeds the default limit -- before
the library is initialised at all, and each bf16 result is compared with the oracle by the suite's
bf16 criteria (within one bf16 ulp of the rounded exact value; normwise error no larger than the
tolerance plus the error of a perfectly rounded result).  The file name keeps it last in collection
order.
"""
import numpy as np
import pytest

import oracle
from paper_2601_22716_b200 import inputs as gen
from _util import NORMWISE_TOL, bf16_ulp, error_metrics

pytestmark = pytest.mark.gpu


def _upload(lay, lords, torch):
    dev = torch.device("cuda:0")
    packed = lords.lords_pack_codes(lay.codes, lay.bits)
    return (packed, torch.from_numpy(packed).to(dev), torch.from_numpy(lay.B.view(np.int16)).to(dev),
            torch.from_numpy(lay.A.view(np.int16)).to(dev), torch.from_numpy(lay.x.view(np.int16)).to(dev))


def _check_bf16_against_oracle(ybits, lay, packed):
    y64 = oracle.forward(lay.x, packed, lay.B, lay.A, lay.codebook, lay.bits)
    got = gen.bf16_to_f32(ybits).astype(np.float64)
    assert np.isfinite(got).all()
    yhat = gen.bf16_to_f32(oracle.round_bf16(y64)).astype(np.float64)
    rms = np.sqrt(np.mean(y64 * y64, axis=1, keepdims=True))
    ulp = bf16_ulp(np.maximum(np.abs(y64), rms))
    worst = float(np.max(np.abs(got - yhat) / ulp))
    assert worst <= 1.0 + 1e-9, f"bf16 output {worst:.2f} ulp from the rounded oracle value"
    e_out, _ = error_metrics(got, y64)
    e_floor, _ = error_metrics(yhat, y64)
    assert e_out <= NORMWISE_TOL + e_floor, (e_out, e_floor)
    print(f"noalloc m={lay.m} n={lay.n} r={lay.r} M={lay.M} bits={lay.bits}: e_out={e_out:.3e} e_floor={e_floor:.3e} ulp={worst:.2f}")


def test_noalloc_entry_matches_oracle_on_calls_in_a_row():
    import torch
    from paper_2601_22716_b200 import binding as lords
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)

    cases = [gen.make_layer(1024, 2048, 32, 8, bits=4, seed=31),
             gen.make_layer(200, 96, 5, 3, bits=3, seed=32, mixed_sign=True),     # a single chunk of columns
             gen.make_layer(320, 1024, 96, 4, bits=4, seed=33, mixed_sign=True),  # shared memory above the default limit
             gen.make_layer(64, 512, 7, 2, bits=2, seed=34)]
    uploaded = [_upload(lay, lords, torch) for lay in cases]
    outs = []
    # back to back, before the library is initialised at all
    for lay, (packed, q, B, A, x) in zip(cases, uploaded):
        y = torch.full((lay.M, lay.m), 0x7FC0, dtype=torch.int16, device="cuda:0")
        lords.lords_linear_forward_noalloc(x, q, B, A, lay.codebook, lay.bits, lay.M, lay.m, lay.n, lay.r, y)
        outs.append(y)
    torch.cuda.synchronize()
    for lay, (packed, q, B, A, x), y in zip(cases, uploaded, outs):
        _check_bf16_against_oracle(y.cpu().numpy().view(np.uint16), lay, packed)


def test_noalloc_entry_interleaved_with_the_regular_cuda_core_path():
    """The two entry points launch the same kernel with different ranks in turn: neither may leave the
    kernel's shared-memory limit too small for the other."""
    import torch
    from paper_2601_22716_b200 import binding as lords
    torch.cuda.set_device(0)
    big = gen.make_layer(256, 1024, 128, 4, bits=4, seed=41)      # r = 128: the largest shared-memory need
    mid = gen.make_layer(256, 1024, 96, 4, bits=4, seed=42)
    up_big, up_mid = _upload(big, lords, torch), _upload(mid, lords, torch)
    lords.lords_init(0, 0)
    lords.lords_set_option("path", "simt")
    try:
        def regular(lay, up):
            _, q, B, A, x = up
            y = torch.full((lay.M, lay.m), 0x7FC0, dtype=torch.int16, device="cuda:0")
            lords.lords_linear_forward_bits(x, q, B, A, lay.codebook, lay.bits, lay.M, lay.m, lay.n, lay.r, y)
            return y

        def noalloc(lay, up):
            _, q, B, A, x = up
            y = torch.full((lay.M, lay.m), 0x7FC0, dtype=torch.int16, device="cuda:0")
            lords.lords_linear_forward_noalloc(x, q, B, A, lay.codebook, lay.bits, lay.M, lay.m, lay.n, lay.r, y)
            return y

        ys = [(big, up_big, regular(big, up_big)), (mid, up_mid, noalloc(mid, up_mid)), (big, up_big, regular(big, up_big)),
              (big, up_big, noalloc(big, up_big)), (mid, up_mid, regular(mid, up_mid))]
        torch.cuda.synchronize()
        assert lords.lords_poll_status() == 0
        for lay, up, y in ys:
            _check_bf16_against_oracle(y.cpu().numpy().view(np.uint16), lay, up[0])
    finally:
        lords.lords_set_option("path", "auto")
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


def test_reinitialising_on_the_same_device_keeps_every_path_working():
    """lords_shutdown followed by lords_init: the per-device launch attributes and occupancy figures are
    kept, the device buffers are new; every kernel path still runs and agrees with the oracle."""
    import torch
    from paper_2601_22716_b200 import binding as lords
    torch.cuda.set_device(0)
    cases = [(gen.make_layer(512, 1024, 32, 1, bits=4, seed=51), "decode"),
             (gen.make_layer(384, 1024, 32, 8, bits=4, seed=52), "decode16"),
             (gen.make_layer(256, 512, 16, 64, bits=4, seed=53), "umma")]
    uploaded = [_upload(lay, lords, torch) for lay, _ in cases]
    for round_ in range(2):
        lords.lords_init(0, 0)
        try:
            for (lay, path), (packed, q, B, A, x) in zip(cases, uploaded):
                y = torch.full((lay.M, lay.m), 0x7FC0, dtype=torch.int16, device="cuda:0")
                lords.lords_linear_forward_bits(x, q, B, A, lay.codebook, lay.bits, lay.M, lay.m, lay.n, lay.r, y)
                assert lords.lords_last_path() == path, (round_, path)
                torch.cuda.synchronize()
                assert lords.lords_poll_status() == 0
                _check_bf16_against_oracle(y.cpu().numpy().view(np.uint16), lay, packed)
        finally:
            lords.lords_shutdown()
