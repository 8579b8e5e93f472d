"""Host-side boundary tests (no GPU): exports, packing, argument validation."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2601_22716_b200 import binding as lords
from paper_2601_22716_b200 import build as lords_build


@pytest.fixture(scope="module", autouse=True)
def _built():
    lords_build.build()


def _declared_functions(repo_root):
    names = []
    inc = os.path.join(repo_root, "include")
    for fn in sorted(os.listdir(inc)):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(lords_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol(repo_root):
    declared = _declared_functions(repo_root)
    assert "lords_linear_forward" in declared and "lords_pack_codes" in declared
    lib = ctypes.CDLL(str(lords.library_path()))
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert sorted(lords.exported_symbols()) == declared


def test_version_and_strerror():
    assert lords.lords_version() == 100
    assert lords.lords_strerror(0) == "ok"
    for code in range(-11, 0):
        assert lords.lords_strerror(code) not in ("", "unknown status")
    assert lords.lords_strerror(-99) == "unknown status"


@pytest.mark.parametrize("bits,n", [(4, 2), (4, 4096), (3, 32), (3, 14336 // 32 * 32), (2, 4), (2, 128)])
def test_pack_is_bit_exact_with_the_written_layout(bits, n):
    rng = np.random.default_rng(1000 * bits + n)
    codes = rng.integers(0, 2**bits, size=(7, n), dtype=np.uint8)
    packed = lords.lords_pack_codes(codes, bits)
    assert packed.shape == (7, n * bits // 8)
    # the oracle's independent writer and reader of the layout agree byte for byte
    assert np.array_equal(packed, oracle.pack_codes(codes, bits))
    assert np.array_equal(oracle.unpack_codes(packed, 7, n, bits), codes)
    assert np.array_equal(lords.lords_unpack_codes(packed, 7, n, bits), codes)


def test_pack_known_answer_bytes():
    assert bytes(lords.lords_pack_codes(np.array([[1, 2]], dtype=np.uint8), 4)[0]) == b"\x21"
    c3 = (np.arange(32, dtype=np.uint8) % 8)[None]
    assert bytes(lords.lords_pack_codes(c3, 3)[0]) == bytes.fromhex("88c6fa") * 4


def test_pack_errors():
    with pytest.raises(lords.LordsError) as e:
        lords.lords_pack_codes(np.full((2, 32), 8, dtype=np.uint8), 3)
    assert e.value.status == -5
    with pytest.raises(lords.LordsError) as e:
        lords.lords_packed_bytes(4, 33, 3)
    assert e.value.status == -2
    with pytest.raises(lords.LordsError) as e:
        lords.lords_packed_bytes(4, 32, 5)
    assert e.value.status == -4
    assert lords.lords_packed_bytes(4096, 4096, 4) == 8388608
    assert lords.lords_packed_bytes(14336, 4096, 3) == 22020096


def test_rank_rule_matches_paper_rows():
    assert lords.lords_equivalent_rank(4096, 4096, 128) == 16
    assert lords.lords_equivalent_rank(14336, 4096, 128) == 24
    assert lords.lords_equivalent_rank(1024, 2560, 256) == 2
    assert lords.lords_equivalent_rank(4096, 4096, 64) == 32


def test_forward_validation_happens_before_any_launch():
    lib = ctypes.CDLL(str(lords.library_path()))
    f = lib.lords_linear_forward_bits
    f.restype = ctypes.c_int
    P = ctypes.c_void_p
    f.argtypes = [P, P, P, P, P, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, P, P]
    cb = (ctypes.c_float * 16)()
    cbp = ctypes.cast(cb, P)
    ok = P(4096)       # aligned, never dereferenced: every call below fails validation first
    odd = P(4100)
    assert f(None, ok, ok, ok, cbp, 4, 1, 64, 64, 4, ok, None) == -1
    assert f(ok, ok, ok, ok, None, 4, 1, 64, 64, 4, ok, None) == -1
    assert f(ok, ok, ok, ok, cbp, 5, 1, 64, 64, 4, ok, None) == -4
    assert f(ok, ok, ok, ok, cbp, 4, 0, 64, 64, 4, ok, None) == -2
    assert f(ok, ok, ok, ok, cbp, 4, 1, 64, 63, 4, ok, None) == -2
    assert f(ok, ok, ok, ok, cbp, 3, 1, 64, 48, 4, ok, None) == -2
    assert f(ok, ok, ok, ok, cbp, 4, 1, 64, 64, 129, ok, None) == -2
    assert f(ok, odd, ok, ok, cbp, 4, 1, 64, 64, 4, ok, None) == -3
    assert f(ok, ok, ok, ok, cbp, 4, 1, 64, 64, 4, ok, None) == -6   # valid arguments, library not initialised


def test_options():
    lords.lords_set_option("path", "simt")
    lords.lords_set_option("path", "auto")
    lords.lords_set_option("splitk", "0")
    with pytest.raises(lords.LordsError):
        lords.lords_set_option("path", "warp-drive")
    with pytest.raises(lords.LordsError):
        lords.lords_set_option("nonsense", "1")


def test_measurement_options_are_validated():
    # known keys with legal values
    for key, value in [("path", "auto"), ("path", "simt"), ("path", "decode"), ("path", "decode16"), ("path", "umma"), ("path", "prefill"),
                       ("splitk", "0"), ("splitk", "7"), ("bn", "0"), ("bn", "128")]:
        lords.lords_set_option(key, value)
    for key, value in [("path", "fast"), ("splitk", "-1"), ("splitk", "x"), ("bn", "48"), ("halves", "2"), ("colour", "blue")]:
        with pytest.raises(lords.LordsError) as ei:
            lords.lords_set_option(key, value)
        assert ei.value.status == -10
    for key, value in [("path", "auto"), ("splitk", "0"), ("bn", "0")]:
        lords.lords_set_option(key, value)


def test_concat_layers_is_the_concatenation_of_the_layers_outputs():
    """Host logic of packing.concat_layers, checked with the oracle: the combined layer (rows and ranks
    stacked, B block-diagonal) gives exactly the layers' outputs side by side -- the zero blocks of B add
    exact zeros to every scale -- and malformed input is refused."""
    from paper_2601_22716_b200 import inputs as gen
    from paper_2601_22716_b200 import packing
    shapes = [(96, 5), (32, 16), (40, 3)]
    lays = [gen.make_layer(m, 128, r, 3, bits=4, seed=10 + i, mixed_sign=(i == 1)) for i, (m, r) in enumerate(shapes)]
    x = lays[0].x
    codes, B, A = packing.concat_layers([l.codes for l in lays], [l.B for l in lays], [l.A for l in lays])
    assert codes.shape == (168, 128) and B.shape == (168, 24) and A.shape == (24, 128)
    assert not B[:96, 5:].any() and not B[96:128, :5].any() and not B[96:128, 21:].any() and not B[128:, :21].any()
    y = oracle.forward(x, oracle.pack_codes(codes, 4), B, A, lays[0].codebook, 4)
    parts = [oracle.forward(x, oracle.pack_codes(l.codes, 4), l.B, l.A, l.codebook, 4) for l in lays]
    assert np.array_equal(y, np.concatenate(parts, axis=1))
    with pytest.raises(ValueError):
        packing.concat_layers([lays[0].codes], [lays[0].B, lays[1].B], [lays[0].A])
    with pytest.raises(ValueError):
        packing.concat_layers([lays[0].codes, lays[1].codes[:, :64]], [lays[0].B, lays[1].B], [lays[0].A, lays[1].A[:, :64]])
    with pytest.raises(ValueError):
        packing.concat_layers([lays[0].codes], [lays[1].B], [lays[0].A])
