"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle."""
import numpy as np
import pytest

import oracle
from paper_2601_22716_b200 import inputs as gen
from _util import DeviceLayer, check_against_oracle, error_metrics, NORMWISE_TOL, ELEMENT_TOL

pytestmark = pytest.mark.gpu

PATHS = ["auto", "simt"]


@pytest.fixture(scope="module")
def lords():
    import torch
    from paper_2601_22716_b200 import binding
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.lords_init(0, 0)
    yield binding
    binding.lords_set_option("path", "auto")
    binding.lords_set_option("splitk", "0")
    binding.lords_set_option("bn", "0")
    binding.lords_shutdown()


def _oracle(lay, packed, rows=None):
    return oracle.forward(lay.x, packed, lay.B, lay.A, lay.codebook, lay.bits, rows=rows)


def _run(lords, lay, path="auto"):
    lords.lords_set_option("path", path)
    try:
        dl = DeviceLayer(lay)
        y32, ybf = dl.forward()
    finally:
        lords.lords_set_option("path", "auto")
    return dl, y32, ybf


@pytest.mark.parametrize("path", PATHS)
def test_config0_tiny_random(lords, path):
    lay = gen.make_layer(256, 256, 4, 4, bits=4, seed=0, scale_gain=0.1, scale_shift=0.05)
    dl, y32, ybf = _run(lords, lay, path)
    check_against_oracle(y32, ybf, _oracle(lay, dl.packed_host))


@pytest.mark.parametrize("path", PATHS)
def test_config0_blockwise_equivalence(lords, path):
    lay, s = gen.make_blockwise_layer(256, 256, 64, 4, bits=4, seed=0)
    dl, y32, ybf = _run(lords, lay, path)
    check_against_oracle(y32, ybf, _oracle(lay, dl.packed_host))


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("bits,m,n,r,M", [(4, 160, 256, 5, 3), (3, 131, 192, 7, 2), (4, 256, 512, 32, 16),
                                          (3, 256, 1024, 48, 1), (2, 64, 128, 3, 2)])
def test_integer_case_is_bit_exact(lords, path, bits, m, n, r, M):
    lay = gen.make_integer_layer(m, n, r, M, bits=bits, seed=bits + m)
    dl, y32, ybf = _run(lords, lay, path)
    y64 = _oracle(lay, dl.packed_host)
    assert np.array_equal(y32.astype(np.float64), y64)
    assert np.array_equal(ybf, oracle.round_bf16(y64))


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("bits,m,n,r,M,mixed", [
    (4, 37, 66, 5, 3, True),        # nothing a multiple of a tile; r odd
    (4, 300, 1000, 24, 19, False),  # several token tiles with a ragged tail
    (3, 129, 352, 12, 9, True),     # 3-bit stream, n = 11 groups of 32
    (3, 512, 2048, 48, 16, False),
    (2, 96, 260, 2, 5, True),
    (4, 64, 4096, 128, 2, False),   # largest rank
    (4, 1, 2, 1, 1, False),         # smallest legal problem
])
def test_odd_shapes(lords, path, bits, m, n, r, M, mixed):
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=7 * m + n, mixed_sign=mixed)
    dl, y32, ybf = _run(lords, lay, path)
    check_against_oracle(y32, ybf, _oracle(lay, dl.packed_host))


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("splitk", [1, 2, 5, 64])
def test_forced_splitk_is_deterministic_and_correct(lords, splitk, path):
    lay = gen.make_layer(200, 1536, 8, 3, bits=4, seed=4)
    lords.lords_set_option("splitk", str(splitk))
    lords.lords_set_option("path", path)
    try:
        dl = DeviceLayer(lay)
        y32, ybf = dl.forward()
        y32b, ybfb = dl.forward()
    finally:
        lords.lords_set_option("splitk", "0")
        lords.lords_set_option("path", "auto")
    assert np.array_equal(y32, y32b) and np.array_equal(ybf, ybfb)   # bit-identical run to run
    check_against_oracle(y32, ybf, _oracle(lay, dl.packed_host))


# ---- the decode kernel (reassociated form, M <= 2), forced so that a decline is an error -----------

DECODE_SHAPES = [
    # bits, m, n, r, M, mixed
    (4, 512, 4096, 32, 2, False),
    (4, 300, 1056, 8, 1, True),      # ragged rows; n = 8.25 k-steps; r padded to 16
    (4, 1000, 2048, 24, 2, True),    # r padded to 32, two tokens
    (4, 64, 8192, 64, 1, False),     # one tile, the largest cluster
    (4, 40000, 64, 16, 1, False),    # more tiles than resident clusters, half a k-step each
    (4, 256, 32, 8, 1, True),        # a quarter-filled k-step
    (3, 520, 1152, 48, 1, True),
    (3, 256, 128, 16, 2, False),
    (3, 2048, 4096, 32, 2, False),
    # 2-bit codes and ranks of the paper's Table 7 (6, 12, 15: rows of B that are not 16-byte multiples)
    (2, 512, 4096, 32, 2, False),
    (2, 300, 1088, 6, 1, True),      # ragged rows; n = 8.5 k-steps; r padded to 16
    (2, 1000, 2048, 15, 2, True),
    (2, 64, 8192, 64, 1, False),
    (2, 256, 64, 12, 1, True),       # half a k-step
    (4, 512, 1024, 12, 2, True),
    (3, 384, 1024, 15, 1, True),
]


@pytest.mark.parametrize("bits,m,n,r,M,mixed", DECODE_SHAPES)
def test_decode_kernel_shapes(lords, bits, m, n, r, M, mixed):
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=3 * m + n + r, mixed_sign=mixed)
    dl, y32, ybf = _run(lords, lay, "decode")
    assert lords.lords_last_path() == "decode" and lords.lords_last_launch_count() == 1
    y64 = _oracle(lay, dl.packed_host)
    check_against_oracle(y32, ybf, y64)


@pytest.mark.parametrize("bits,m,n,r,M", [(4, 700, 2048, 32, 1), (4, 256, 1024, 16, 2), (3, 384, 1024, 48, 1),
                                          (3, 131, 256, 8, 2), (2, 300, 1024, 6, 1), (2, 512, 320, 24, 2)])
def test_decode_kernel_integer_case_is_bit_exact(lords, bits, m, n, r, M):
    lay = gen.make_integer_layer(m, n, r, M, bits=bits, seed=bits + m)
    dl, y32, ybf = _run(lords, lay, "decode")
    assert lords.lords_last_path() == "decode"
    y64 = _oracle(lay, dl.packed_host)
    assert np.array_equal(y32.astype(np.float64), y64)
    assert np.array_equal(ybf, oracle.round_bf16(y64))


@pytest.mark.parametrize("cluster", [1, 3, 7, 100])
def test_decode_kernel_cluster_split_is_deterministic(lords, cluster):
    lay = gen.make_layer(600, 3072, 32, 2, bits=4, seed=17)
    lords.lords_set_option("splitk", str(cluster))
    lords.lords_set_option("path", "decode")
    try:
        dl = DeviceLayer(lay)
        y32, ybf = dl.forward()
        y32b, ybfb = dl.forward()
    finally:
        lords.lords_set_option("splitk", "0")
        lords.lords_set_option("path", "auto")
    assert np.array_equal(y32, y32b) and np.array_equal(ybf, ybfb)
    check_against_oracle(y32, ybf, _oracle(lay, dl.packed_host))


def test_two_tokens_with_a_large_rank_take_the_128_column_kernel(lords):
    lay = gen.make_layer(512, 1024, 48, 2, bits=3, seed=5)       # 2 * 48 accumulator columns: too many for the reassociated form
    dl, y32, ybf = _run(lords, lay, "auto")
    assert lords.lords_last_path() == "decode16"
    check_against_oracle(y32, ybf, _oracle(lay, dl.packed_host))


def test_decode_kernel_declines_what_it_cannot_run(lords):
    lay = gen.make_layer(256, 256, 4, 4, bits=4, seed=0)      # M = 4, r = 4
    lords.lords_set_option("path", "decode")
    try:
        with pytest.raises(lords.LordsError) as ei:
            DeviceLayer(lay).forward()
        assert ei.value.status == -11
    finally:
        lords.lords_set_option("path", "auto")


# ---- the decode kernel for 3 .. 16 tokens (scale-MMA form, 128-column k-steps), forced ----------------

DECODE16_SHAPES = [
    # bits, m, n, r, M, mixed
    (4, 384, 1024, 32, 5, True),
    (4, 512, 4096, 32, 8, False),
    (4, 300, 1088, 8, 3, True),       # ragged rows; n = 8.5 k-steps; r padded to 16
    (4, 1000, 2048, 24, 16, True),    # r padded to 32, a full token tile
    (4, 64, 8192, 16, 7, False),      # one tile, the largest cluster
    (4, 20000, 128, 16, 4, False),    # more tiles than resident clusters, one k-step each
    (4, 256, 64, 8, 9, True),         # half a k-step
    (3, 260, 1152, 48, 16, True),
    (3, 256, 128, 16, 3, False),
    (3, 2048, 4096, 32, 8, False),
    (3, 640, 2048, 48, 2, True),      # two tokens with a rank the reassociated kernel declines
    (4, 256, 512, 32, 1, False),
    # 2-bit codes and ranks of the paper's Table 7
    (2, 384, 1024, 32, 5, True),
    (2, 300, 1088, 6, 3, True),
    (2, 1000, 2048, 48, 16, True),
    (2, 256, 64, 12, 9, True),
    (4, 512, 1024, 15, 8, True),
    # 4-bit codes with ranks above 32 (a two-stage factor ring)
    (4, 384, 1024, 48, 8, True),
    (4, 300, 2112, 64, 16, False),
    (4, 128, 128, 33, 3, True),       # one k-step
    (4, 1024, 4096, 64, 5, True),
]


@pytest.mark.parametrize("bits,m,n,r,M,mixed", DECODE16_SHAPES)
def test_decode16_kernel_shapes(lords, bits, m, n, r, M, mixed):
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=3 * m + n + r + M, mixed_sign=mixed)
    dl, y32, ybf = _run(lords, lay, "decode16")
    assert lords.lords_last_path() == "decode16" and lords.lords_last_launch_count() == 1
    y64 = _oracle(lay, dl.packed_host)
    check_against_oracle(y32, ybf, y64)


@pytest.mark.parametrize("bits,m,n,r,M", [(4, 700, 2048, 32, 8), (4, 256, 512, 16, 16), (4, 260, 1024, 64, 7), (3, 384, 1024, 48, 3),
                                          (3, 131, 384, 7, 9), (2, 300, 1024, 5, 4), (2, 256, 192, 40, 16)])
def test_decode16_kernel_integer_case_is_bit_exact(lords, bits, m, n, r, M):
    lay = gen.make_integer_layer(m, n, r, M, bits=bits, seed=bits + m + M)
    dl, y32, ybf = _run(lords, lay, "decode16")
    assert lords.lords_last_path() == "decode16"
    y64 = _oracle(lay, dl.packed_host)
    assert np.array_equal(y32.astype(np.float64), y64)
    assert np.array_equal(ybf, oracle.round_bf16(y64))


@pytest.mark.parametrize("cluster", [1, 3, 7, 100])
def test_decode16_kernel_cluster_split_is_deterministic(lords, cluster):
    lay = gen.make_layer(600, 3072, 32, 6, bits=4, seed=19)
    lords.lords_set_option("splitk", str(cluster))
    lords.lords_set_option("path", "decode16")
    try:
        dl = DeviceLayer(lay)
        y32, ybf = dl.forward()
        y32b, ybfb = dl.forward()
    finally:
        lords.lords_set_option("splitk", "0")
        lords.lords_set_option("path", "auto")
    assert lords.lords_last_path() == "decode16"
    assert np.array_equal(y32, y32b) and np.array_equal(ybf, ybfb)
    check_against_oracle(y32, ybf, _oracle(lay, dl.packed_host))


def test_decode16_kernel_declines_what_it_cannot_run(lords):
    lords.lords_set_option("path", "decode16")
    try:
        for lay in (gen.make_layer(256, 256, 65, 4, bits=4, seed=0),      # r > 64
                    gen.make_layer(256, 256, 4, 17, bits=4, seed=0)):     # more than one token tile
            with pytest.raises(lords.LordsError) as ei:
                DeviceLayer(lay).forward()
            assert ei.value.status == -11
    finally:
        lords.lords_set_option("path", "auto")


# ---- the scale-MMA kernel, forced; token tiles forced too so that every instantiation runs ----------

UMMA_SHAPES = [
    # bits, m, n, r, M, bn, mixed
    (4, 384, 1024, 32, 5, 0, True),
    (3, 260, 1152, 48, 16, 0, True),
    (3, 128, 256, 16, 2, 0, False),
    (4, 130, 128, 64, 1, 0, False),      # one pair of k-steps, largest rank
    (4, 256, 2048, 24, 40, 32, True),
    (3, 200, 1024, 32, 70, 64, False),
    (4, 300, 1536, 16, 100, 128, True),
    (3, 384, 1280, 48, 300, 256, False),
    (4, 256, 1024, 8, 257, 256, True),   # a second token tile with one token in it
    (4, 1024, 512, 16, 600, 32, False),  # more tiles than resident CTAs: the last wave is filled with split tiles
    (3, 1100, 512, 32, 620, 32, True),
    # 2-bit codes (the paper's ultra-low-bit setting) and ranks of its Table 7
    (2, 384, 1024, 12, 5, 0, True),
    (2, 130, 192, 6, 1, 0, False),       # n = 1.5 code stages
    (2, 256, 2048, 15, 40, 32, True),
    (2, 200, 1024, 32, 70, 64, False),
    (2, 300, 1536, 24, 100, 128, True),
    (2, 384, 1280, 48, 300, 256, False),
]


@pytest.mark.parametrize("bits,m,n,r,M,bn,mixed", UMMA_SHAPES)
def test_umma_kernel_shapes(lords, bits, m, n, r, M, bn, mixed):
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=5 * m + n + r + M, mixed_sign=mixed)
    lords.lords_set_option("bn", str(bn))
    try:
        dl, y32, ybf = _run(lords, lay, "umma")
    finally:
        lords.lords_set_option("bn", "0")
    assert lords.lords_last_path() == "umma"
    check_against_oracle(y32, ybf, _oracle(lay, dl.packed_host))


@pytest.mark.parametrize("bits,m,n,r,M,bn", [(4, 256, 512, 32, 16, 0), (3, 131, 384, 7, 9, 0), (4, 140, 256, 16, 33, 32),
                                             (3, 256, 512, 48, 200, 256), (4, 1280, 256, 8, 500, 32),
                                             (2, 256, 512, 16, 4, 0), (2, 140, 320, 5, 130, 128)])
def test_umma_kernel_integer_case_is_bit_exact(lords, bits, m, n, r, M, bn):
    lay = gen.make_integer_layer(m, n, r, M, bits=bits, seed=bits + m + M)
    lords.lords_set_option("bn", str(bn))
    try:
        dl, y32, ybf = _run(lords, lay, "umma")
    finally:
        lords.lords_set_option("bn", "0")
    assert lords.lords_last_path() == "umma"
    y64 = _oracle(lay, dl.packed_host)
    assert np.array_equal(y32.astype(np.float64), y64)
    assert np.array_equal(ybf, oracle.round_bf16(y64))


def test_linearity_on_gpu(lords):
    import torch
    m, n, r = 128, 512, 16
    lay = gen.make_layer(m, n, r, 3, bits=4, seed=21, mixed_sign=True)
    x = gen.bf16_to_f32(lay.x).copy()
    x[0, n // 2:] = 0.0
    x[1, :n // 2] = 0.0
    x[2] = 4.0 * x[0] - 0.5 * x[1]
    lay.x = gen.bf16_bits(torch.from_numpy(x))
    dl, y32, ybf = _run(lords, lay)
    want = 4.0 * y32[0].astype(np.float64) - 0.5 * y32[1].astype(np.float64)
    nw, el = error_metrics(y32[2:3], want[None])
    assert nw <= NORMWISE_TOL and el <= ELEMENT_TOL


@pytest.mark.parametrize("M", [1, 8, 40])
@pytest.mark.parametrize("xscale,what", [(2.0 ** 10, "large activations"), (2.0 ** -6, "small activations")])
def test_operand_range_edges(lords, M, xscale, what):
    """The tensor-core paths keep x (or A*x) and the dequantised weight in fp16.  Inside the documented
    range -- |x| up to a few thousand with factors of the order 1e-2, and activations as small as 1e-2 --
    the tolerances still hold on every path (M = 1: reassociated form, 8: 128-column form A, 40: form A)."""
    import torch
    lay = gen.make_layer(384, 1024, 32, M, bits=4, seed=91 + M, scale_gain=0.005, scale_shift=0.01)
    x = gen.bf16_to_f32(lay.x) * np.float32(xscale)
    lay.x = gen.bf16_bits(torch.from_numpy(x))
    dl, y32, ybf = _run(lords, lay, "auto")
    assert lords.lords_last_path() in ("decode", "decode16", "umma")
    check_against_oracle(y32, ybf, _oracle(lay, dl.packed_host))


def _sampled_rows(m, count, seed):
    """Stratified sample of output rows: one random row from every 32-row quadrant of every 128-row
    tile (so that no row tile and no lane quadrant of any kernel goes unchecked), the first and the
    last row, plus `count` more rows drawn uniformly."""
    rng = np.random.default_rng(seed)
    starts = np.arange(0, m, 32)
    strat = np.minimum(starts + rng.integers(0, 32, size=starts.size), m - 1)
    rows = np.unique(np.concatenate([[0, m - 1], strat, rng.integers(0, m, size=count)]))
    return rows.astype(np.int64)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M", [1, 8])
def test_config1_qproj_decode_full_size(lords, path, M):
    lay = gen.make_layer(4096, 4096, 32, M, bits=4, seed=0)
    dl, y32, ybf = _run(lords, lay, path)
    y64 = _oracle(lay, dl.packed_host)            # the full layer: ~0.6 GFLOP fp64 per token
    check_against_oracle(y32, ybf, y64)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("m,n,M", [(14336, 4096, 1), (4096, 14336, 1), (4096, 14336, 16), (14336, 4096, 16)])
def test_config2_mlp_nf3_full_size(lords, path, m, n, M):
    lay = gen.make_layer(m, n, 48, M, bits=3, seed=0)
    dl, y32, ybf = _run(lords, lay, path)
    rows = _sampled_rows(m, 64, 5)
    y64 = _oracle(lay, dl.packed_host, rows=rows)
    check_against_oracle(y32[:, rows], ybf[:, rows], y64)
    assert np.isfinite(y32).all()


@pytest.mark.parametrize("path", ["auto"])
def test_config3_prefill_full_size_sampled(lords, path):
    lay = gen.make_layer(4096, 14336, 32, 2048, bits=4, seed=0, outlier_frac=0.01)
    dl, y32, ybf = _run(lords, lay, path)
    assert lords.lords_last_path() == "umma"
    rows = _sampled_rows(4096, 16, 6)
    y64 = _oracle(lay, dl.packed_host, rows=rows)
    check_against_oracle(y32[:, rows], ybf[:, rows], y64)
    assert np.isfinite(y32).all()


# ---- the remaining Llama-3-8B module shapes of the full linear stack (k/v with r = 16, o, gate/up at
# ---- 4 bits, M in {1, 8, 512}), full size, outputs sampled by row

@pytest.mark.parametrize("name,r,bits,M", [("k", 16, 4, 1), ("v", 16, 4, 8), ("o", 32, 4, 8), ("gate", 32, 4, 1),
                                            ("up", 32, 4, 8), ("down", 32, 4, 1), ("q", 32, 4, 512),
                                            ("down", 48, 3, 512), ("k", 16, 4, 512)])
def test_config4_stack_shapes_full_size_sampled(lords, name, r, bits, M):
    m, n = gen.LLAMA3_8B_SHAPES[name]
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=7 * len(name) + M)
    dl, y32, ybf = _run(lords, lay, "auto")
    assert lords.lords_last_path() in ("decode", "decode16", "umma")
    rows = _sampled_rows(m, 64 if M <= 8 else 0, 11)
    y64 = _oracle(lay, dl.packed_host, rows=rows)
    check_against_oracle(y32[:, rows], ybf[:, rows], y64)
    assert np.isfinite(y32).all()


def test_status_word_round_trip_and_recovery(lords):
    """A recorded give-up is reported once by lords_poll_status and cleared; while it stands, the
    kernels' waits end at once (no result is promised); afterwards everything works again."""
    import torch
    lay = gen.make_layer(512, 2048, 32, 1, bits=4, seed=77)
    dl = DeviceLayer(lay)
    y32, ybf = dl.forward()
    lords.lords_set_option("inject_status", "-8")
    assert lords.lords_poll_status() == -8
    assert lords.lords_poll_status() == 0
    lords.lords_set_option("inject_status", "-8")
    lords.lords_linear_forward_bits(dl.x, dl.q, dl.B, dl.A, lay.codebook, lay.bits, lay.M, lay.m, lay.n, lay.r, dl.y)
    torch.cuda.synchronize()                      # returns promptly: no wait runs to its own limit
    assert lords.lords_poll_status() == -8
    assert lords.lords_poll_status() == 0
    y32b, ybfb = dl.forward()
    assert np.array_equal(y32, y32b) and np.array_equal(ybf, ybfb)


@pytest.mark.parametrize("m,n,r,bits,M,path", [(14336, 4096, 48, 3, 1, "decode"), (6144, 4096, 64, 4, 8, "decode16")])
def test_many_back_to_back_launches_leave_no_status(lords, m, n, r, bits, M, path):
    """The 3-bit gate shape runs the two-half variant of the M <= 2 kernel, whose rings are three
    stages deep while its converter groups take the k-steps alternately; a 4-bit layer of rank 64 runs
    the 16-token kernel with a two-stage factor ring that its two scale issuers share.  Several thousand
    dependent launches over distinct weight copies (replayed from a CUDA graph, as a model's layers
    are) must leave the status word clear and reproduce the first result bit for bit: a barrier that
    two groups share by parity alone would show up here as a recorded give-up."""
    import torch
    lay = gen.make_layer(m, n, r, M, bits=bits, seed=91)
    dl = DeviceLayer(lay)
    copies = 6
    qs = [dl.q] + [torch.roll(dl.q, l, 0).contiguous() for l in range(1, copies)]
    ys = [torch.zeros((M, lay.m), dtype=torch.int16, device="cuda:0") for _ in range(copies)]

    def one_round():
        for q, y in zip(qs, ys):
            lords.lords_linear_forward_bits(dl.x, q, dl.B, dl.A, lay.codebook, bits, M, lay.m, lay.n, lay.r, y)

    one_round()
    torch.cuda.synchronize()
    assert lords.lords_last_path() == path
    first = [y.clone() for y in ys]
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        one_round()
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _ in range(20):
            one_round()
    for _ in range(40):                      # 40 x 20 x 6 = 4800 launches
        g.replay()
    torch.cuda.synchronize()
    assert lords.lords_poll_status() == 0
    for y, f in zip(ys, first):
        assert torch.equal(y, f)


@pytest.mark.parametrize("M,path", [(1, "auto"), (4, "auto"), (40, "auto"), (3, "simt"), (300, "auto")])
def test_host_buffer_entry_point_matches_device_entry(lords, M, path):
    """x from and y into pinned host memory (small buffers: y is stored by the kernels straight into the
    mapped host buffer; 300 tokens: staged copies), on every kind of kernel: bit-identical to the device entry."""
    import torch
    lay = gen.make_layer(520, 1024, 16, M, bits=4, seed=12 + M)
    dl, y32, ybf = _run(lords, lay, path)
    used = lords.lords_last_path()
    xh = torch.from_numpy(lay.x.view(np.int16)).pin_memory()
    yh = torch.full((lay.M, lay.m), 0x7FC0, dtype=torch.int16).pin_memory()
    lords.lords_set_option("path", path)
    try:
        lords.lords_linear_forward_host(xh, dl.q, dl.B, dl.A, lay.codebook, lay.bits, lay.M, lay.m, lay.n, lay.r, yh)
    finally:
        lords.lords_set_option("path", "auto")
    assert lords.lords_last_path() == used
    torch.cuda.synchronize()
    assert lords.lords_poll_status() == 0
    assert np.array_equal(yh.numpy().view(np.uint16), ybf)


def test_four_bit_entry_point_and_launch_count(lords):
    import torch
    lay = gen.make_layer(256, 256, 4, 4, bits=4, seed=0)
    dl, y32, ybf = _run(lords, lay)
    y = torch.zeros_like(dl.y)
    lords.lords_linear_forward(dl.x, dl.q, dl.B, dl.A, lay.codebook, lay.M, lay.m, lay.n, lay.r, y)
    torch.cuda.synchronize()
    assert np.array_equal(y.cpu().numpy().view(np.uint16), ybf)
    assert lords.lords_last_launch_count() >= 1
    assert lords.lords_last_path() in ("simt", "decode", "decode16", "umma")


@pytest.mark.parametrize("M", [1, 8])
def test_qkv_as_one_layer_full_size(lords, M):
    """The q, k and v projections of a Llama-3-8B block (NF4, r = 32 / 16 / 16) as one 6144 x 4096 layer
    of rank 64 with a block-diagonal B (packing.concat_layers): against the oracle on stratified rows,
    and against the three separate calls."""
    import dataclasses
    import torch
    from paper_2601_22716_b200 import packing
    parts = [gen.make_layer(m, 4096, r, M, bits=4, seed=40 + i) for i, (m, r) in enumerate([(4096, 32), (1024, 16), (1024, 16)])]
    codes, B, A = packing.concat_layers([p.codes for p in parts], [p.B for p in parts], [p.A for p in parts])
    lay = dataclasses.replace(parts[0], m=6144, r=64, codes=codes, B=B, A=A)
    dl, y32, ybf = _run(lords, lay, "auto")
    # rank 64: one token fits the reassociated decode kernel (M * r <= 64), eight go to the 16-token kernel
    assert lords.lords_last_path() == ("decode" if M == 1 else "decode16")
    rows = _sampled_rows(6144, 32, 9)
    check_against_oracle(y32[:, rows], ybf[:, rows], _oracle(lay, dl.packed_host, rows=rows), label=f"qkv as one layer M={M}")
    assert np.isfinite(y32).all()
    separate = []
    for p in parts:
        p.x = lay.x
        separate.append(_run(lords, p, "auto")[1])
    assert error_metrics(y32, np.concatenate(separate, axis=1).astype(np.float64))[0] <= 1e-5
