"""Parity of the CUDA library with the CPU oracle, element by element and bit-exact, through the C ABI."""
from __future__ import annotations

import numpy as np
import pytest

from paper_2011_10680_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hq():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2011_10680_b200 import binding, build
    build.build()
    h = binding.Handle(0)
    yield h
    h.close()


def oracle():
    from oracle import hqref
    return hqref


def host(t, like: np.ndarray) -> np.ndarray:
    return t.cpu().numpy().view(like.dtype).reshape(like.shape)


def run_conv_and_compare(hq, case, path):
    from paper_2011_10680_b200 import binding
    hq.set_conv_path(path)
    try:
        st, out = hq.conv_case(case)
        assert st == binding.HQ_OK, binding.status_string(st)
        hq.sync()
    finally:
        hq.set_conv_path(0)
    ref = oracle().conv_case(case)
    got = host(out, ref)
    if not np.array_equal(got, ref):
        bad = np.argwhere(got != ref)
        raise AssertionError(f"{len(bad)} of {ref.size} outputs differ; first at {bad[0]}: got {got[tuple(bad[0])]} want {ref[tuple(bad[0])]}")


@pytest.mark.parametrize("shape", [
    (1, 136, 136, 32, 8, 131, 1, 0),      # a filter wider than an im2col tensor map's corner range (kw > pad + 129)
    (1, 8, 8, 32, 19072, 1, 1, 0),        # more channel tiles than a persistent grid has CTAs
])
def test_automatic_path_falls_back_when_the_tensor_core_launcher_declines(hq, shape):
    """Shapes that pass the tensor-core path's argument checks but that its launcher declines before launching anything:
    the automatic path must still return the right integers (CUDA-core kernel), not the launcher's status."""
    n, h, w, cin, cout, k, stride, pad = shape
    case = inputs.conv_case(311, n, h, w, cin, cout, k, stride, pad, c_range=(40, 46))
    run_conv_and_compare(hq, case, 0)


def _random_conv_configs(count, seed):
    """Seeded random single-layer configurations over everything the dispatch looks at: channel counts the direct
    kernel takes or not, filter sizes, strides, padding, operand and output widths, residual kinds, signs, shift
    ranges on both sides of 32."""
    g = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        bits = int(g.choice([8, 8, 4]))
        cin = int(g.choice([3, 8, 16, 32, 48, 64, 96, 128]))
        if bits == 4 and cin % 2:
            continue
        cout = int(g.choice([8, 16, 24, 64, 100, 128, 192]))
        k = int(g.choice([1, 1, 3, 3, 5]))
        stride = int(g.choice([1, 1, 2]))
        pad = int(g.choice([0, k // 2]))
        h, w = int(g.integers(5, 21)), int(g.integers(5, 21))
        if h + 2 * pad < k or w + 2 * pad < k:
            continue
        out_bits = int(g.choice([8, 8, 4, 32]))
        if out_bits == 4 and cout % 2:
            continue
        res = None if out_bits == 32 else g.choice([None, None, 8, 32])
        lo = int(g.integers(24, 41))
        out.append(dict(n=int(g.integers(1, 4)), h=h, w=w, cin=cin, cout=cout, k=k, stride=stride, pad=pad, bits=bits,
                        out_bits=out_bits, residual=res is not None, res_bits=int(res) if res is not None else 8,
                        relu=bool(g.integers(0, 2)), in_signed=bool(g.integers(0, 2)), c_range=(lo, lo + int(g.integers(0, 9)))))
    return out


@pytest.mark.parametrize("order", [0, 1])
@pytest.mark.parametrize("path", [0, 3])
def test_conv_random_configurations(hq, path, order):
    """48 seeded random layers through hq_conv2d on the automatic path and with the tensor-core launch shapes chosen by
    what a layer allows rather than by its size: every dispatch branch (direct, lowered, widened, first-layer form,
    CUDA cores) must return the oracle's integers, whichever end of the tensor the pixel tiles start from."""
    from paper_2011_10680_b200 import binding
    hq.set_tile_order(order)
    try:
        _random_configurations_body(hq, path)
    finally:
        hq.set_tile_order(0)


def _random_configurations_body(hq, path):
    from paper_2011_10680_b200 import binding
    for i, cfg in enumerate(_random_conv_configs(48, 20260 + path)):
        case = inputs.conv_case(7000 + i, cfg["n"], cfg["h"], cfg["w"], cfg["cin"], cfg["cout"], cfg["k"], cfg["stride"],
                                cfg["pad"], bits=cfg["bits"], out_bits=cfg["out_bits"], residual=cfg["residual"],
                                res_bits=cfg["res_bits"], relu=cfg["relu"], in_signed=cfg["in_signed"], c_range=cfg["c_range"])
        hq.set_conv_path(path)
        try:
            st, out = hq.conv_case(case)
            if path == 3 and st == binding.HQ_ERR_UNSUPPORTED:
                continue                                   # tensor cores demanded for a shape they do not take
            assert st == binding.HQ_OK, (cfg, binding.status_string(st))
            hq.sync()
        finally:
            hq.set_conv_path(0)
        ref = oracle().conv_case(case)
        got = host(out, ref)
        assert np.array_equal(got, ref), (i, cfg, int((got != ref).sum()))


def test_conv_random_midsize_layers_reach_every_launch_shape(hq):
    """16 seeded random layers of 20-60 thousand output pixels with the channel counts of ResNet stages: large enough for
    im2col maps, 256-pixel tiles, resident weights, the strip form, the fragment epilogue and the two-CTA shape, small
    enough for the oracle; shift ranges on both sides of 32, with and without an 8-bit residual, 8- and 4-bit operands."""
    from paper_2011_10680_b200 import binding
    g = np.random.default_rng(20261)
    for i in range(16):
        hw = int(g.choice([14, 28, 56]))
        n = max(1, int(g.integers(20000, 60000)) // (hw * hw))
        cin, cout = int(g.choice([64, 128, 256, 512])), int(g.choice([64, 128, 256, 512]))
        k = int(g.choice([1, 1, 3]))
        if k == 3 and cin * cout > 256 * 256:
            cin = 128
        bits = int(g.choice([8, 8, 4]))
        lo = int(g.integers(26, 41))
        residual = bool(g.integers(0, 2))
        case = inputs.conv_case(7100 + i, n, hw, hw, cin, cout, k, 1, k // 2, bits=bits, residual=residual,
                                in_signed=bool(g.integers(0, 2)), c_range=(lo, lo + 6))
        for path, order in ((0, 0), (3, 0), (0, 1), (3, 1)):         # order 1: pixel tiles from the last to the first
            hq.set_conv_path(path)
            hq.set_tile_order(order)
            try:
                st, out = hq.conv_case(case)
                assert st == binding.HQ_OK, (i, path, binding.status_string(st))
                hq.sync()
            finally:
                hq.set_conv_path(0)
                hq.set_tile_order(0)
            if path == 0 and order == 0:
                ref = oracle().conv_case(case)
            got = host(out, ref)
            assert np.array_equal(got, ref), (i, path, order, hw, n, cin, cout, k, bits, residual, int((got != ref).sum()))
            del out
        binding.check_guards()


# ------------------------------------------------------------------ CUDA-core conv path --------
CORE_CASES = [
    # n, h, w, cin, cout, k, stride, pad, bits, out_bits, residual, res_bits, relu
    (2, 9, 11, 3, 8, 7, 2, 3, 8, 8, False, 8, True),        # stem-like, odd channels
    (1, 8, 8, 16, 12, 3, 1, 1, 8, 8, True, 8, True),
    (2, 7, 6, 8, 10, 3, 2, 1, 8, 32, False, 8, False),
    (1, 6, 6, 8, 8, 1, 1, 0, 4, 4, False, 8, True),
    (2, 5, 7, 16, 6, 3, 1, 1, 4, 8, True, 32, True),
    (1, 6, 6, 6, 4, 3, 1, 1, 4, 8, False, 8, False),         # 4-bit, cin not a multiple of 8
]


@pytest.mark.parametrize("cfg", CORE_CASES)
def test_conv_cuda_core_path(hq, cfg):
    n, h, w, cin, cout, k, stride, pad, bits, out_bits, residual, res_bits, relu = cfg
    case = inputs.conv_case(101, n, h, w, cin, cout, k, stride, pad, bits=bits, out_bits=out_bits,
                            residual=residual, res_bits=res_bits, relu=relu, c_range=(38, 44))
    run_conv_and_compare(hq, case, path=1)


def test_conv_cuda_core_signed_input(hq):
    case = inputs.conv_case(102, 1, 6, 6, 8, 8, 3, 1, 1, in_signed=True, c_range=(38, 44))
    run_conv_and_compare(hq, case, path=1)


# ------------------------------------------------------------------ tensor-core conv path ------
TC_CASES = [
    # n, h, w, cin, cout, k, stride, pad, out_bits, residual, res_bits, relu
    (1, 56, 56, 64, 64, 3, 1, 1, 8, False, 8, True),         # benchmark config 1 geometry (ragged last M tile)
    (2, 16, 16, 128, 128, 1, 1, 0, 8, False, 8, True),       # 1x1, 128-byte K blocks, 4 M tiles
    (2, 14, 14, 256, 64, 3, 1, 1, 8, False, 8, True),        # several K chunks per tap
    (3, 15, 13, 64, 96, 3, 2, 1, 8, False, 8, True),         # stride 2, odd extents, N not a multiple of the tile
    (2, 28, 28, 64, 128, 1, 2, 0, 8, False, 8, False),       # strided 1x1 (shortcut conv), signed output
    (2, 14, 14, 64, 256, 1, 1, 0, 8, True, 8, True),         # residual, N = 256
    (1, 14, 14, 128, 512, 1, 1, 0, 8, True, 32, True),       # INT32 residual, two N tiles
    (2, 10, 10, 32, 72, 3, 1, 1, 32, False, 8, False),       # 32-byte K blocks, INT32 output, N tail
    (1, 9, 9, 96, 40, 5, 1, 2, 8, False, 8, True),           # 5x5, cin = 3 x 32
    (2, 12, 12, 64, 64, 3, 1, 1, 4, False, 8, True),         # uint4 output
    (1, 7, 7, 512, 1000, 1, 1, 0, 32, False, 8, False),      # classifier-like N = 1000
    (2, 9, 9, 64, 40, 3, 1, 1, 8, True, 8, True),            # N = 40: rows not 16-byte multiples, direct stores
    (2, 13, 13, 64, 96, 1, 1, 0, 8, True, 8, True),          # residual tile clipped in N by the TMA box
    (1, 20, 20, 128, 256, 3, 1, 1, 8, True, 8, True),        # residual + 3x3 + two N tiles of 128
    (3, 8, 8, 64, 64, 1, 1, 0, 4, True, 8, True),            # uint4 output with residual
    (2, 16, 16, 32, 128, 1, 1, 0, 4, False, 8, True),        # uint4 output, 64-byte store boxes
    # the same kinds of geometry on tensors of at least 128 KiB, which the direct kernel fetches through im2col-mode
    # tensor maps (smaller ones, above, take the patch-matrix form); the last two straddle the threshold
    (6, 30, 26, 64, 96, 3, 2, 1, 8, False, 8, True),         # stride 2, odd extents, N tail
    (3, 28, 28, 64, 128, 1, 2, 0, 8, False, 8, False),       # strided 1x1, signed output
    (8, 24, 24, 32, 72, 3, 1, 1, 32, False, 8, False),       # 32-byte K blocks, INT32 output
    (4, 19, 19, 96, 40, 5, 1, 2, 8, False, 8, True),         # 5x5, pad 2, direct stores
    (4, 24, 24, 64, 64, 3, 1, 1, 4, False, 8, True),         # uint4 output
    (3, 20, 20, 128, 256, 3, 1, 1, 8, True, 8, True),        # residual + 3x3 + two N tiles
    (2, 32, 32, 64, 64, 3, 1, 1, 8, False, 8, True),         # exactly 128 KiB: im2col mode
    (2, 32, 31, 64, 64, 3, 1, 1, 8, False, 8, True),         # 124 KiB: patch-matrix form
    # large enough for the benchmark's launch shapes (the pixel tile grows with the number of tiles per SM)
    (33, 56, 56, 64, 64, 1, 1, 0, 8, False, 8, True),        # 256-pixel tiles, folded 64-channel tile, ragged last tile
    (13, 56, 56, 64, 64, 3, 1, 1, 8, True, 8, True),         # 128-pixel tiles, four accumulator buffers, folded, residual
    (17, 56, 56, 64, 256, 1, 1, 0, 8, True, 8, True),        # two CTAs per SM (fused residual, short K), ragged last tile
    (21, 28, 28, 128, 512, 1, 1, 0, 8, True, 8, False),      # two CTAs per SM with 64-byte K blocks cut from cin = 128, signed out
    (9, 28, 28, 128, 128, 3, 1, 1, 8, False, 8, True),       # 256-pixel tiles, long K, one CTA per SM
    (9, 28, 28, 128, 256, 3, 1, 1, 8, True, 8, True),        # 256-pixel tiles, long K, residual through a single staging tile
]


@pytest.mark.parametrize("cfg", TC_CASES)
def test_conv_tensor_core_path(hq, cfg):
    n, h, w, cin, cout, k, stride, pad, out_bits, residual, res_bits, relu = cfg
    kk = k * k * cin
    lo = 36 + int(np.log2(kk)) // 2
    case = inputs.conv_case(201, n, h, w, cin, cout, k, stride, pad, bits=8, out_bits=out_bits, residual=residual,
                            res_bits=res_bits, relu=relu, c_range=(lo, lo + 4) if out_bits != 4 else (lo + 4, lo + 8))
    run_conv_and_compare(hq, case, path=2)


STRIP_CASES = [
    # n, h, w, cin, cout: 3x3 / stride 1 / pad 1 through the strip form (one input patch per cin chunk for all nine taps)
    (2, 14, 14, 128, 128),     # pitch 16, a whole image per tile (two scratch rows), weights through the stage ring
    (3, 14, 14, 256, 192),     # two cin chunks, ragged channel tile
    (2, 28, 28, 128, 128),     # pitch 32, eight rows per tile, a partly filled last tile per image
    (1, 56, 56, 64, 64),       # pitch 64, 64-byte K blocks, resident weights, folded channel tile
    (2, 56, 56, 64, 128),      # the same with a full channel tile
    (2, 12, 11, 64, 96),       # narrower and lower than the pitch / the tile
    (1, 30, 25, 128, 64),      # width 25 on pitch 32, 30 rows (last tile of six rows), folded
    (2, 50, 62, 64, 64),       # width 62: the padded row fills the pitch of 64 exactly
]


@pytest.mark.parametrize("cfg", STRIP_CASES)
@pytest.mark.parametrize("signed_in", [0, 1])
def test_conv_tensor_core_strip_form(hq, cfg, signed_in):
    n, h, w, cin, cout = cfg
    kk = 9 * cin
    lo = 36 + int(np.log2(kk)) // 2
    case = inputs.conv_case(209, n, h, w, cin, cout, 3, 1, 1, bits=8, relu=not signed_in, in_signed=bool(signed_in),
                            c_range=(lo, lo + 4))
    run_conv_and_compare(hq, case, path=3)


@pytest.mark.parametrize("cin,cout,k,hw,out_bits,residual", [
    (512, 128, 1, 56, 8, False), (640, 128, 1, 56, 8, False), (1024, 256, 1, 28, 8, False), (128, 128, 3, 28, 8, False),
    (64, 64, 3, 56, 8, False), (256, 64, 1, 56, 8, False),
    (64, 256, 1, 56, 8, True),       # two CTAs per SM, residual pairs worked out ahead of the single large call
    (256, 256, 3, 28, 4, False),     # 4-bit output through the pipelined epilogue
    (1024, 256, 1, 28, 4, False),
    (256, 256, 3, 28, 8, False),     # long reductions with 256 | cout: two CTAs share every MMA (cta_group::2)
    (1024, 256, 1, 28, 8, True),
    (512, 512, 3, 14, 8, False),
    (128, 512, 1, 28, 8, True),      # sixteen epilogue warps working in place in the residual tiles
    (256, 1024, 1, 28, 8, True),
    (512, 2048, 1, 14, 8, True),     # the same with two operand stages beside a 64 KiB weight slab
])
def test_conv_many_tiles_per_cta_repeated_images(hq, cin, cout, k, hw, out_bits, residual):
    """Benchmark-sized launches (several tiles per CTA: every accumulator buffer, operand stage and issuer warp is
    reused many times, with K block counts that do and do not divide among the issuers) at an oracle cost of two
    images: the batch repeats two distinct images, and every copy must equal the oracle's result for its image."""
    from paper_2011_10680_b200 import binding
    n = 64
    lo = 36 + int(np.log2(k * k * cin)) // 2
    if out_bits == 4:
        lo += 4
    case = inputs.conv_case(210, 2, hw, hw, cin, cout, k, 1, k // 2, bits=8, out_bits=out_bits, residual=residual,
                            c_range=(lo - 6, lo + 4) if out_bits == 4 else (lo, lo + 4))
    ref = oracle().conv_case(case)
    big = dict(case)
    big["x"] = np.ascontiguousarray(np.tile(case["x"], (n // 2, 1, 1, 1)))
    if residual:
        big["res"] = np.ascontiguousarray(np.tile(case["res"], (n // 2, 1, 1, 1)))
    big["n"] = n
    hq.set_conv_path(2)
    try:
        st, out = hq.conv_case(big)
        assert st == binding.HQ_OK
        hq.sync()
    finally:
        hq.set_conv_path(0)
    got = out.cpu().numpy().view(ref.dtype).reshape((n // 2, 2) + ref.shape[1:])
    for i in range(n // 2):
        assert np.array_equal(got[i], ref), f"copy {i} differs"


@pytest.mark.parametrize("variant", ["small_residual_shift", "clamp_and_small_c", "signed_residual", "ragged_channels"])
def test_conv_in_place_residual_shape_variants(hq, variant):
    """The launch shape that overwrites the prefetched residual tile with its outputs (256-pixel tiles, 8-bit residual,
    short reduction), in the cases that leave its common loop: residual shifts below 9 (64-bit tile loop, direct
    stores), clamp bounds inside the type with main shifts below 32, a signed residual with every shift, and a
    channel count that leaves the last channel tile ragged.  Two distinct images repeated over a batch of 16."""
    from paper_2011_10680_b200 import binding
    n, cout = 16, 256
    kw = dict(residual=True, c_range=(39, 43))
    if variant == "clamp_and_small_c":
        kw["c_range"] = (28, 43)
    if variant == "signed_residual":
        kw["relu"] = False
    if variant == "ragged_channels":
        cout = 208
    case = inputs.conv_case(212, 2, 56, 56, 64, cout, 1, 1, 0, **kw)
    if variant == "small_residual_shift":
        case["rc"][::3] = 5
    if variant == "clamp_and_small_c":
        case["qmin"], case["qmax"] = 3, 200
    if variant == "signed_residual":
        case["res"] = case["res"].view(np.int8)
        case["res_signed"] = 1
        case["rc"][:] = np.arange(cout) % 36 + 9
    ref = oracle().conv_case(case)
    big = dict(case)
    big["x"] = np.ascontiguousarray(np.tile(case["x"], (n // 2, 1, 1, 1)))
    big["res"] = np.ascontiguousarray(np.tile(case["res"], (n // 2, 1, 1, 1)))
    big["n"] = n
    hq.set_conv_path(2)
    try:
        st, out = hq.conv_case(big)
        assert st == binding.HQ_OK
        hq.sync()
    finally:
        hq.set_conv_path(0)
    got = out.cpu().numpy().view(ref.dtype).reshape((n // 2, 2) + ref.shape[1:])
    for i in range(n // 2):
        assert np.array_equal(got[i], ref), f"copy {i} differs"


def test_conv_tensor_core_config1_exact_distribution(hq):
    run_conv_and_compare(hq, inputs.config1_case(), path=2)


def test_conv_tensor_core_signed_input_and_small_c(hq):
    case = inputs.conv_case(203, 1, 12, 12, 64, 64, 3, 1, 1, in_signed=True, relu=False, c_range=(41, 45))
    run_conv_and_compare(hq, case, path=2)
    # shifts below 32 and very large shifts both take the general 64-bit path
    case = inputs.conv_case(204, 1, 12, 12, 64, 64, 1, 1, 0, relu=True, c_range=(20, 62))
    run_conv_and_compare(hq, case, path=2)


@pytest.mark.parametrize("residual,big", [(False, False), (True, False), (True, True), (False, True)])
def test_conv_small_shifts_pre_shift_form_and_its_bounds(hq, residual, big):
    """Shifts below 32 (common with 4-bit operands): where accumulator and bias are known to stay below 2^(c-2) the
    epilogue shifts the accumulator left first and uses the plain form; elsewhere the exact funnel-shift form.  K = 64
    bounds |acc| by 64 * 255 * 128 < 2^21, so c >= 23 qualifies; activations and weights at their extremes, biases
    just inside the bound for channels 0-127 and just outside it for channels 128-255 (whole warps fall back).
    The large case reaches the 256-pixel tiles and, with a residual, the fragment epilogue."""
    n, hw = (40, 56) if big else (2, 12)
    case = inputs.conv_case(312, n, hw, hw, 64, 256, 1, 1, 0, residual=residual, c_range=(23, 35))
    case["x"][0, :2] = 255
    case["x"][-1, -1] = 0
    case["wgt"][0:32] = 127
    case["wgt"][32:64] = -128
    case["wgt"][128:160] = 127
    sign = np.where(np.arange(256) % 2 == 0, 1, -1)
    edge = (1 << (np.minimum(case["c"].astype(np.int64), 31) - 2))
    bias = np.where(np.arange(256) < 128, edge - 1, edge + 5) * sign
    case["bias"] = bias.astype(np.int32)
    run_conv_and_compare(hq, case, 2)


def test_conv_tensor_core_general_tiles_with_residual(hq):
    # residual shifts below 9 and main shifts below 32 force the 64-bit tile path, staged and direct
    for cout in (64, 40):
        case = inputs.conv_case(205, 2, 10, 10, 64, cout, 1, 1, 0, residual=True, c_range=(30, 44))
        case["rc"][::3] = 5
        run_conv_and_compare(hq, case, path=2)


def test_conv_tensor_core_clamp_variants(hq):
    # clamp bounds inside the type's range (explicit min/max instead of the saturating pack), signed
    # residual operand, signed output with residual
    case = inputs.conv_case(207, 2, 12, 12, 64, 128, 1, 1, 0, residual=True, c_range=(39, 43))
    case["qmin"], case["qmax"] = 3, 200
    run_conv_and_compare(hq, case, path=2)
    case = inputs.conv_case(208, 2, 12, 12, 64, 128, 1, 1, 0, residual=True, relu=False, c_range=(39, 43))
    case["res"] = case["res"].view(np.int8)
    case["res_signed"] = 1
    case["rc"][:] = np.arange(128) % 36 + 9          # every residual shift from 9 to 44
    run_conv_and_compare(hq, case, path=2)
    case = inputs.conv_case(209, 1, 12, 12, 64, 64, 3, 1, 1, residual=True, relu=True, c_range=(39, 43))
    case["rc"][:] = np.arange(64) % 36 + 9
    case["c"][:] = np.arange(64) % 30 + 32            # main shifts from 32 to 61
    run_conv_and_compare(hq, case, path=2)


INT4_TC_CASES = [
    # n, h, w, cin, cout, k, stride, pad, out_bits, residual
    (2, 14, 14, 128, 128, 3, 1, 1, 4, False),      # uint4 in, uint4 out (conv inside a 4-bit block)
    (2, 14, 14, 64, 256, 1, 1, 0, 8, True),        # uint4 in, uint8 stream out with residual (block's last conv)
    (1, 14, 14, 256, 64, 1, 2, 0, 8, False),       # strided shortcut conv
    (3, 7, 7, 32, 48, 3, 1, 1, 4, False),
]


@pytest.mark.parametrize("cfg", INT4_TC_CASES)
def test_conv_int4_on_tensor_cores(hq, cfg):
    n, h, w, cin, cout, k, stride, pad, out_bits, residual = cfg
    case = inputs.conv_case(210, n, h, w, cin, cout, k, stride, pad, bits=4, out_bits=out_bits, residual=residual,
                            c_range=(42, 46) if out_bits == 8 else (46, 50))
    run_conv_and_compare(hq, case, path=2)          # 4-bit operands widened, contraction on tcgen05


def test_conv_int4_signed_activations(hq):
    case = inputs.conv_case(211, 2, 10, 10, 64, 64, 3, 1, 1, bits=4, in_signed=True, relu=False, c_range=(42, 46))
    run_conv_and_compare(hq, case, path=2)


LOWERED_CASES = [
    # n, h, w, cin, cout, k, stride, pad
    (2, 32, 32, 3, 64, 7, 2, 3),
    (1, 17, 19, 3, 32, 7, 2, 3),
    (2, 9, 9, 5, 16, 3, 1, 1),
    (1, 12, 12, 16, 48, 3, 2, 1),
]


@pytest.mark.parametrize("cfg", LOWERED_CASES)
def test_conv_lowered_first_layer_path(hq, cfg):
    n, h, w, cin, cout, k, stride, pad = cfg
    case = inputs.conv_case(206, n, h, w, cin, cout, k, stride, pad, c_range=(38, 42))
    run_conv_and_compare(hq, case, path=0)     # automatic choice: patch matrix + tensor-core kernel


def test_linear_matches_oracle_and_conv(hq):
    from paper_2011_10680_b200 import binding
    g = inputs.rng(7, 1)
    x = g.integers(0, 256, size=(8, 1, 1, 512), dtype=np.int64).astype(np.uint8)
    w = g.integers(-127, 128, size=(1000, 1, 1, 512), dtype=np.int64).astype(np.int8)
    bias = g.integers(-(1 << 15), 1 << 15, size=1000, dtype=np.int64).astype(np.int32)
    ref = oracle().linear(x.reshape(8, 512), 512, 8, 0, w, 1000, bias, None, None, 0, -(1 << 31), (1 << 31) - 1, 32, 1)
    out = binding.alloc_out(8, 1, 1, 1000, 32, 1)
    st = hq.conv2d(binding.to_device(x), 8, 0, 512, binding.to_device(w), 1000, 1, 1, 1, 0, binding.to_device(bias),
                   None, None, out, 32, 1, relu=0, qmin=-(1 << 31), qmax=(1 << 31) - 1, linear=True)
    assert st == binding.HQ_OK
    hq.sync()
    assert np.array_equal(host(out, ref), ref)


# ------------------------------------------------------------------ memory-bound kernels -------
@pytest.mark.parametrize("main_bits,res_bits,out_bits,ch", [
    (32, 8, 8, 64), (8, 8, 8, 256), (8, 0, 4, 64), (32, 32, 8, 48), (4, 8, 8, 32), (8, 8, 8, 10), (32, 0, 4, 6),
])
def test_residual_add(hq, main_bits, res_bits, out_bits, ch):
    from paper_2011_10680_b200 import binding
    g = inputs.rng(301, main_bits, res_bits, out_bits, ch)
    shape = (3, 7, 9, ch)

    def draw(bits):
        if bits == 32:
            return g.integers(-(1 << 22), 1 << 22, size=shape, dtype=np.int64).astype(np.int32), 1
        if bits == 8:
            return g.integers(0, 256, size=shape, dtype=np.int64).astype(np.uint8), 0
        return inputs.pack4(g.integers(0, 16, size=shape, dtype=np.int64)), 0

    main, main_signed = draw(main_bits)
    mb = g.integers(1 << 30, 1 << 31, size=ch, dtype=np.int64).astype(np.int32)
    mc = g.integers(45, 50, size=ch).astype(np.int32) if main_bits == 32 else g.integers(29, 34, size=ch).astype(np.int32)
    res = rb = rc = None
    res_signed = 0
    if res_bits:
        res, res_signed = draw(res_bits)
        rb = g.integers(1 << 30, 1 << 31, size=ch, dtype=np.int64).astype(np.int32)
        rc = g.integers(45, 50, size=ch).astype(np.int32) if res_bits == 32 else g.integers(29, 34, size=ch).astype(np.int32)
    qmax = 255 if out_bits == 8 else 15
    ref = oracle().residual_add(main, main_bits, main_signed, mb, mc, res, res_bits, res_signed, rb, rc, ch, 1, 0, qmax,
                                out_bits, 0)
    out = binding.alloc_out(*shape[:3], ch, out_bits, 0)
    st = hq.residual_add(binding.to_device(main), main_bits, main_signed, binding.to_device(mb), binding.to_device(mc),
                         binding.to_device(res), res_bits, res_signed, binding.to_device(rb), binding.to_device(rc),
                         ch, 1, 0, qmax, out, out_bits, 0)
    assert st == binding.HQ_OK
    hq.sync()
    assert np.array_equal(host(out, ref), ref)


@pytest.mark.parametrize("ch,res_signed,out_signed,shifts", [
    (64, None, 0, "wide"), (256, 0, 0, "wide"), (128, 1, 1, "every"), (1024, 0, 0, "every"), (4, None, 1, "every"),
    (64, 0, 0, "clamp"),
])
def test_residual_add_int32_main_flat_kernel(hq, ch, res_signed, out_signed, shifts):
    """INT32 main operand -> 8-bit output on the flat kernel: full-range accumulators, shifts 1..62 (threads with a
    shift below 32 take the 64-bit form), signed / unsigned residual and output, clamp bounds inside the range."""
    from paper_2011_10680_b200 import binding
    g = inputs.rng(307, ch, out_signed)
    shape = (1, 83, 61, ch)                    # 5063 pixels: several block trips and a ragged last one
    main = g.integers(-(1 << 31), 1 << 31, size=shape, dtype=np.int64).astype(np.int32)
    main[0, :4] >>= 12                         # some rows of moderate size, so that not everything saturates
    mb, rb = (g.integers(1 << 30, 1 << 31, size=ch, dtype=np.int64).astype(np.int32) for _ in range(2))
    if shifts == "every":
        mc = (np.arange(ch) % 62 + 1).astype(np.int32)
        rc = ((np.arange(ch) * 7) % 62 + 1).astype(np.int32)
    else:
        mc = g.integers(50, 58, size=ch).astype(np.int32)
        rc = g.integers(29, 34, size=ch).astype(np.int32)
    res = None
    if res_signed is not None:
        res = (g.integers(-128, 128, size=shape, dtype=np.int64).astype(np.int8) if res_signed else
               g.integers(0, 256, size=shape, dtype=np.int64).astype(np.uint8))
    qmin, qmax = (-128, 127) if out_signed else (0, 255)
    if shifts == "clamp":
        qmin, qmax = 7, 201
    relu = 0 if out_signed else 1
    ref = oracle().residual_add(main, 32, 1, mb, mc, res, 8 if res is not None else 0, res_signed or 0,
                                rb if res is not None else None, rc if res is not None else None, ch, relu, qmin, qmax,
                                8, out_signed)
    out = binding.alloc_out(*shape[:3], ch, 8, out_signed)
    st = hq.residual_add(binding.to_device(main), 32, 1, binding.to_device(mb), binding.to_device(mc),
                         binding.to_device(res), 8 if res is not None else 0, res_signed or 0,
                         binding.to_device(rb) if res is not None else None, binding.to_device(rc) if res is not None else None,
                         ch, relu, qmin, qmax, out, 8, out_signed)
    assert st == binding.HQ_OK
    hq.sync()
    assert np.array_equal(host(out, ref), ref)


def test_residual_add_8bit_fast_kernel_every_shift(hq):
    """8-bit operands take the 32-bit kernel; shifts from 1 to 62, signed and unsigned, both outputs."""
    from paper_2011_10680_b200 import binding
    g = inputs.rng(305)
    ch, shape = 128, (2, 9, 7, 128)
    for main_signed, res_signed, out_bits in ((0, 0, 8), (1, 1, 8), (0, 1, 4), (1, 0, 8)):
        main = g.integers(-128, 128, size=shape, dtype=np.int64).astype(np.int8) if main_signed else \
            g.integers(0, 256, size=shape, dtype=np.int64).astype(np.uint8)
        res = g.integers(-128, 128, size=shape, dtype=np.int64).astype(np.int8) if res_signed else \
            g.integers(0, 256, size=shape, dtype=np.int64).astype(np.uint8)
        mb, rb = (g.integers(1 << 30, 1 << 31, size=ch, dtype=np.int64).astype(np.int32) for _ in range(2))
        mc = (np.arange(ch) % 62 + 1).astype(np.int32)
        rc = ((np.arange(ch) * 7) % 62 + 1).astype(np.int32)
        qmin, qmax = (0, 15) if out_bits == 4 else (-128, 127)
        out_signed = int(out_bits == 8)
        ref = oracle().residual_add(main, 8, main_signed, mb, mc, res, 8, res_signed, rb, rc, ch, 0, qmin, qmax, out_bits, out_signed)
        out = binding.alloc_out(*shape[:3], ch, out_bits, out_signed)
        st = hq.residual_add(binding.to_device(main), 8, main_signed, binding.to_device(mb), binding.to_device(mc),
                             binding.to_device(res), 8, res_signed, binding.to_device(rb), binding.to_device(rc),
                             ch, 0, qmin, qmax, out, out_bits, out_signed)
        assert st == binding.HQ_OK
        hq.sync()
        assert np.array_equal(host(out, ref), ref)


LARGE_ELT_CASES = [
    # pixels (h x w of one image, n = 1), ch, main_signed, res (None / signed flag), out_bits, shifts
    ((157, 131), 256, 0, 0, 8, "fast"),        # 20567 pixels of 64 words: a ragged last trip
    ((157, 131), 256, 0, None, 8, "fast"),     # plain requantization (eight words in flight per thread)
    ((211, 97), 64, 1, 1, 8, "fast"),          # signed operands and output
    ((157, 131), 128, 0, 1, 4, "fast"),        # packed 4-bit output, clamp [0, 15]
    ((95, 83), 1024, 0, 0, 8, "fast"),         # 256 words: one pixel per block step
    ((157, 131), 256, 0, 0, 8, "every"),       # shifts 1..62: threads with a shift below 9 take the 64-bit form
    ((301, 211), 32, 0, 0, 8, "fast"),         # 8 words per pixel
    ((157, 131), 4, 0, 0, 8, "fast"),          # a single word per pixel
    ((101, 67), 192, 0, 0, 8, "fast"),         # 48 words: not a power of two
    ((157, 131), 128, 1, None, 4, "fast"),     # 4-bit output from signed input
    # more than eight chunks per SM: the bulk-copy pipeline, with words left over after the last full chunk
    ((331, 251), 128, 0, 0, 8, "fast"),
    ((331, 251), 128, 0, None, 8, "fast"),
    ((331, 251), 128, 1, 1, 4, "every"),
    ((499, 333), 64, 0, 1, 8, "every"),
    ((331, 251), 128, 0, None, 4, "fast"),     # 4-bit output packed from high nibbles (shifts reduced by four)
    ((331, 251), 128, 1, None, 4, "every"),    # the same with shifts below four in some warps (plain clamp there)
    ((157, 131), 128, 0, None, 4, "every"),
    # more than 256 words per pixel that do not divide into blocks of 256 (the 17x17 Inception module's 1088 channels)
    ((53, 41), 1088, 0, None, 4, "fast"),
    ((53, 41), 1088, 0, 1, 8, "every"),
    ((37, 29), 2052, 1, None, 8, "fast"),
]


@pytest.mark.parametrize("main_signed,res_signed,out_bits", [(1, 1, 8), (1, None, 8), (0, 1, 8), (1, 0, 8), (1, None, 4)])
def test_residual_add_narrow_pairs_with_signed_operands(hq, main_signed, res_signed, out_bits):
    """A single call on at least 2^25 values works out narrow multiply-add pairs first and then reads every byte
    through the one-instruction extraction; signed bytes must come out sign-extended.  Negative operands on both
    branches, every stored value compared."""
    from paper_2011_10680_b200 import binding
    h, w, ch = 727, 723, 64
    assert h * w * ch >= 1 << 25
    g = inputs.rng(307, main_signed, 2 if res_signed is None else res_signed, out_bits)
    shape = (1, h, w, ch)
    draw = lambda sg: (g.integers(-128, 128, size=shape, dtype=np.int64).astype(np.int8) if sg else
                       g.integers(0, 256, size=shape, dtype=np.int64).astype(np.uint8))
    main = draw(main_signed)
    res = draw(res_signed) if res_signed is not None else None
    mb, rb = (g.integers(1 << 30, 1 << 31, size=ch, dtype=np.int64).astype(np.int32) for _ in range(2))
    mc = g.integers(31, 34, size=ch).astype(np.int32)
    rc = g.integers(31, 34, size=ch).astype(np.int32)
    out_signed = int(out_bits == 8)
    qmin, qmax = (0, 15) if out_bits == 4 else (-128, 127)
    ref = oracle().residual_add(main, 8, main_signed, mb, mc, res, 8 if res is not None else 0, res_signed or 0,
                                rb if res is not None else None, rc if res is not None else None, ch, 0, qmin, qmax,
                                out_bits, out_signed)
    if out_bits == 8:
        assert np.count_nonzero((ref > qmin) & (ref < 0)) > ref.size // 8        # negative results that are not clamped
    out = binding.alloc_out(*shape[:3], ch, out_bits, out_signed)
    st = hq.residual_add(binding.to_device(main), 8, main_signed, binding.to_device(mb), binding.to_device(mc),
                         binding.to_device(res), 8 if res is not None else 0, res_signed or 0,
                         binding.to_device(rb) if res is not None else None, binding.to_device(rc) if res is not None else None,
                         ch, 0, qmin, qmax, out, out_bits, out_signed)
    assert st == binding.HQ_OK
    hq.sync()
    assert np.array_equal(host(out, ref), ref)


@pytest.mark.parametrize("cfg", LARGE_ELT_CASES)
def test_residual_add_large_tensors(hq, cfg):
    """Tensors of many block trips with a ragged last trip: the flat word-array kernel (channel words a power of two),
    every output form, and a channel count that keeps the pixel-row kernel (192 = 48 words)."""
    from paper_2011_10680_b200 import binding
    (h, w), ch, main_signed, res_signed, out_bits, shifts = cfg
    g = inputs.rng(306, h, w, ch, main_signed, out_bits)
    shape = (1, h, w, ch)
    draw = lambda sg: (g.integers(-128, 128, size=shape, dtype=np.int64).astype(np.int8) if sg else
                       g.integers(0, 256, size=shape, dtype=np.int64).astype(np.uint8))
    main = draw(main_signed)
    res = draw(res_signed) if res_signed is not None else None
    mb, rb = (g.integers(1 << 30, 1 << 31, size=ch, dtype=np.int64).astype(np.int32) for _ in range(2))
    if shifts == "every":
        mc = (np.arange(ch) % 62 + 1).astype(np.int32)
        rc = ((np.arange(ch) * 7) % 62 + 1).astype(np.int32)
    else:
        mc = g.integers(29, 34, size=ch).astype(np.int32)
        rc = g.integers(29, 34, size=ch).astype(np.int32)
    out_signed = int(out_bits == 8 and main_signed == 1)
    qmin, qmax = (0, 15) if out_bits == 4 else ((-128, 127) if out_signed else (0, 255))
    relu = 0 if out_signed else 1
    ref = oracle().residual_add(main, 8, main_signed, mb, mc, res, 8 if res is not None else 0, res_signed or 0,
                                rb if res is not None else None, rc if res is not None else None, ch, relu, qmin, qmax,
                                out_bits, out_signed)
    out = binding.alloc_out(*shape[:3], ch, out_bits, out_signed)
    st = hq.residual_add(binding.to_device(main), 8, main_signed, binding.to_device(mb), binding.to_device(mc),
                         binding.to_device(res), 8 if res is not None else 0, res_signed or 0,
                         binding.to_device(rb) if res is not None else None, binding.to_device(rc) if res is not None else None,
                         ch, relu, qmin, qmax, out, out_bits, out_signed)
    assert st == binding.HQ_OK
    hq.sync()
    assert np.array_equal(host(out, ref), ref)


@pytest.mark.parametrize("n,hw,ch,in_bits", [(4, 7, 64, 8), (2, 7, 2048, 8), (3, 5, 6, 8), (2, 4, 16, 32), (2, 3, 8, 4)])
def test_avgpool_requant(hq, n, hw, ch, in_bits):
    from paper_2011_10680_b200 import binding
    g = inputs.rng(302, n, hw, ch, in_bits)
    if in_bits == 8:
        x = g.integers(0, 256, size=(n, hw, hw, ch), dtype=np.int64).astype(np.uint8)
    elif in_bits == 32:
        x = g.integers(-(1 << 16), 1 << 16, size=(n, hw, hw, ch), dtype=np.int64).astype(np.int32)
    else:
        x = inputs.pack4(g.integers(0, 16, size=(n, hw, hw, ch), dtype=np.int64))
    scale = np.exp(g.uniform(np.log(0.2), np.log(2.0), size=ch)) / (hw * hw) / (256.0 if in_bits == 32 else 1.0)
    b, c = inputs.dyadic_from_scale(scale)
    ref = oracle().avgpool_requant(x, ch, in_bits, int(in_bits == 32), b, c, 0, 255)
    out = binding.alloc_out(n, 1, 1, ch, 8, 0)
    st = hq.avgpool_requant(binding.to_device(x), ch, in_bits, int(in_bits == 32), binding.to_device(b),
                            binding.to_device(c), 0, 255, out, 8, 0)
    assert st == binding.HQ_OK
    hq.sync()
    assert np.array_equal(host(out, ref), ref)


@pytest.mark.parametrize("n,h,w,ch", [(2, 112, 112, 64), (3, 9, 11, 16), (2, 8, 7, 5)])
def test_maxpool(hq, n, h, w, ch):
    from paper_2011_10680_b200 import binding
    x = inputs.rng(303, n, h, w, ch).integers(0, 256, size=(n, h, w, ch), dtype=np.int64).astype(np.uint8)
    ref = oracle().maxpool(x, 3, 2, 1)
    out = binding.alloc_out(n, ref.shape[1], ref.shape[2], ch, 8, 0)
    st = hq.maxpool(binding.to_device(x), ch, 0, 3, 2, 1, out)
    assert st == binding.HQ_OK
    hq.sync()
    assert np.array_equal(host(out, ref), ref)


@pytest.mark.parametrize("k,stride,pad", [(3, 2, 1), (3, 1, 1), (3, 2, 0), (3, 3, 1), (2, 2, 0), (5, 2, 2), (3, 1, 2)])
@pytest.mark.parametrize("signed", [0, 1])
def test_maxpool_windows_and_signedness(hq, k, stride, pad, signed):
    # every window form of the vector kernel (unrolled 3x3 with replaced border taps, general loop), on odd
    # extents, with values that include both ends of the type's range
    from paper_2011_10680_b200 import binding
    n, h, w, ch = 2, 13, 10, 48
    g = inputs.rng(304, k, stride, pad, signed)
    x = g.integers(0, 256, size=(n, h, w, ch), dtype=np.int64).astype(np.uint8)
    x[0, :3] = 0x80 if signed else 0            # whole windows at the type's minimum
    x[1, -3:] = 0x7F if signed else 0xFF
    xs = x.view(np.int8) if signed else x
    ref = oracle().maxpool(xs, k, stride, pad, signed)
    out = binding.alloc_out(n, ref.shape[1], ref.shape[2], ch, 8, signed)
    st = hq.maxpool(binding.to_device(xs), ch, signed, k, stride, pad, out)
    assert st == binding.HQ_OK
    hq.sync()
    assert np.array_equal(host(out, ref), ref)


@pytest.mark.parametrize("n,hw,ch,signed", [(3, 16, 48, 0), (2, 7, 528, 0), (2, 16, 64, 1), (5, 7, 2048, 1), (2, 9, 20, 1),
                                            (2, 17, 32, 0), (2, 17, 1664, 1), (2, 35, 288, 0), (2, 45, 48, 1), (2, 46, 32, 0)])
def test_avgpool_requant_8bit_kernels(hq, n, hw, ch, signed):
    # the 16-channel kernel with a partly filled block, two blocks per image, 256 pixels at the maximum value
    # (16-bit lane sums at their limit), signed bytes; the 4-channel kernel (ch = 20); more than 257 pixels: slices of the
    # 16-channel kernel added at full width (Inception's 17x17 and 35x35 maps, 45x45 = 2025 pixels with every slice at
    # its limit), and beyond 2056 pixels the 4-channel kernel again
    from paper_2011_10680_b200 import binding
    g = inputs.rng(305, n, hw, ch, signed)
    x = g.integers(0, 256, size=(n, hw, hw, ch), dtype=np.int64).astype(np.uint8)
    x[0] = 0x80 if signed else 0xFF
    x[1, :, :, ::3] = 0x7F if signed else 0xFF
    xs = x.view(np.int8) if signed else x
    scale = np.exp(g.uniform(np.log(0.2), np.log(2.0), size=ch)) / (hw * hw)
    b, c = inputs.dyadic_from_scale(scale)
    lo, hi = (-128, 127) if signed else (0, 255)
    ref = oracle().avgpool_requant(xs, ch, 8, signed, b, c, lo, hi, 8, signed)
    out = binding.alloc_out(n, 1, 1, ch, 8, signed)
    st = hq.avgpool_requant(binding.to_device(xs), ch, 8, signed, binding.to_device(b), binding.to_device(c), lo, hi, out, 8, signed)
    assert st == binding.HQ_OK
    hq.sync()
    assert np.array_equal(host(out, ref), ref)


@pytest.mark.parametrize("path", [1, 2])
def test_conv_degenerate_and_extreme_cases(hq, path):
    """Extreme operands and degenerate geometry on both conv paths: every activation and weight at the end of its
    range with the longest ResNet reduction (largest accumulators the workloads can produce, both signs, clamped at
    both ends), all-zero operands (bias only), a filter as large as its input (one output pixel), a single pixel."""
    def extreme(sign, relu):
        case = inputs.conv_case(212, 1, 7, 7, 512, 64, 3, 1, 1, relu=relu, c_range=(44, 48))
        case["x"][:] = 255
        case["wgt"][:] = 127 * sign
        case["bias"][:] = (1 << 15) * sign
        return case
    run_conv_and_compare(hq, extreme(+1, True), path)          # acc = 9 * 512 * 255 * 127 at the centre: saturates high
    run_conv_and_compare(hq, extreme(-1, True), path)          # most negative accumulators: ReLU clamps to 0
    neg = extreme(-1, False)
    neg["qmin"], neg["qmax"], neg["out_signed"] = -128, 127, 1
    run_conv_and_compare(hq, neg, path)                        # ... and to -128 without ReLU
    zero = inputs.conv_case(213, 2, 9, 9, 64, 96, 3, 1, 1, c_range=(20, 24))
    zero["x"][:] = 0
    run_conv_and_compare(hq, zero, path)                       # bias * b >> c only; shifts below 32
    run_conv_and_compare(hq, inputs.conv_case(214, 3, 7, 7, 64, 64, 7, 1, 0), path)    # one output pixel per image
    run_conv_and_compare(hq, inputs.conv_case(215, 1, 1, 1, 64, 32, 1, 1, 0), path)    # a single pixel
    run_conv_and_compare(hq, inputs.conv_case(216, 1, 1, 1, 32, 8, 3, 1, 1), path)     # all taps but the centre are padding


def test_bounded_wait_expires_and_context_stays_usable(hq):
    """A device-side wait that nothing ever satisfies gives up after its budget, hq_sync reports it once, and the
    same handle then runs a convolution bit-exactly (no trap, no hang, no lost context)."""
    from paper_2011_10680_b200 import binding
    import time
    assert hq.expire_wait_selftest(0) == binding.HQ_ERR_INVALID_ARG
    t0 = time.time()
    assert hq.expire_wait_selftest(300) == binding.HQ_OK
    with pytest.raises(binding.HqError) as err:
        hq.sync()
    assert err.value.code == binding.HQ_ERR_TIMEOUT
    assert 0.25 < time.time() - t0 < 5.0
    hq.sync()                                     # the status word was cleared by the report
    case = inputs.conv_case(211, 2, 12, 12, 64, 64, 3, 1, 1)
    run_conv_and_compare(hq, case, path=2)


# ------------------------------------------------------------------ argument errors ------------
def test_invalid_arguments_return_codes_not_crashes(hq):
    from paper_2011_10680_b200 import binding
    case = inputs.conv_case(401, 1, 8, 8, 32, 32, 3, 1, 1)
    dev = binding.upload_case(case)
    out = binding.alloc_out(1, 8, 8, 32, 8, 0)
    args = dict(res=None, relu=1, qmin=0, qmax=255)
    ok = hq.conv2d(dev["x"], 8, 0, 32, dev["wgt"], 32, 3, 3, 1, 1, dev["bias"], dev["b"], dev["c"], out, 8, 0, **args)
    assert ok == binding.HQ_OK
    bad_shape = binding.alloc_out(1, 7, 8, 32, 8, 0)
    assert hq.conv2d(dev["x"], 8, 0, 32, dev["wgt"], 32, 3, 3, 1, 1, dev["bias"], dev["b"], dev["c"], bad_shape, 8, 0,
                     **args) == binding.HQ_ERR_INVALID_ARG
    assert hq.conv2d(dev["x"], 8, 0, 32, dev["wgt"], 32, 3, 3, 1, 1, dev["bias"], None, None, out, 8, 0,
                     **args) == binding.HQ_ERR_INVALID_ARG
    assert hq.conv2d(dev["x"], 8, 0, 32, dev["wgt"], 32, 3, 3, 1, 1, dev["bias"], dev["b"], dev["c"], out, 8, 0,
                     res=None, relu=1, qmin=0, qmax=256) == binding.HQ_ERR_INVALID_ARG
    off = dev["x"].view(-1)[1:1 + 4 * 4 * 32].view(1, 4, 4, 32)      # data pointer is 1 byte past alignment
    assert hq.maxpool(off, 32, 0, 3, 2, 1, binding.alloc_out(1, 2, 2, 32, 8, 0)) == binding.HQ_ERR_ALIGNMENT
    hq.set_conv_path(2)
    try:
        c3 = inputs.conv_case(402, 1, 6, 6, 3, 8, 3, 1, 1)
        st, _ = hq.conv_case(c3)
        assert st == binding.HQ_ERR_UNSUPPORTED          # no silent fallback when tensor cores are demanded
    finally:
        hq.set_conv_path(0)
    hq.sync()


# ------------------------------------------------------------------ networks -------------------
def run_network_and_compare(hq, table, batch, seed):
    from oracle.network import run_network
    from paper_2011_10680_b200 import binding
    images = inputs.random_images(seed, batch, table["image_hw"])
    ref = run_network(table, images)
    net = binding.Network(hq, table, batch)
    try:
        d_img = binding.to_device(images)
        logits = binding.alloc_out(*net.logits_shape, 32, 1)
        taps = net.alloc_taps()
        assert net.run(d_img, logits, taps) == binding.HQ_OK
        hq.sync()
        net.check_guards()           # no kernel wrote outside a buffer the network owns
        for i, (t, r) in enumerate(zip(taps, ref)):
            got = t.cpu().numpy().view(r.dtype).reshape(r.shape)
            assert np.array_equal(got, r), f"layer {i} ({table['layers'][i]['op']}) differs in {(got != r).sum()} of {r.size}"
        assert np.array_equal(host(logits, ref[-1]), ref[-1])
        # graph replay path (no taps) must give the same logits, twice in a row
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            for _ in range(2):
                logits.zero_()
                assert net.run(d_img, logits, None) == binding.HQ_OK
                hq.sync()
                assert np.array_equal(host(logits, ref[-1]), ref[-1])
        net.check_guards()
    finally:
        net.close()
    return ref


def test_reduced_resnet18_and_resnet50_every_layer(hq):
    for depth, mixed in ((18, False), (50, False), (50, True)):
        t = inputs.resnet_table(depth, seed=5, image_hw=64, classes=24, width=32, mixed=mixed)
        run_network_and_compare(hq, t, batch=3, seed=depth)


@pytest.mark.parametrize("depth,pattern", [(18, "alternate"), (18, "random"), (50, "alternate"), (50, "random"),
                                           (50, "all4")])
def test_network_per_conv_bit_widths(hq, depth, pattern):
    """Bit-width tables as the ILP of Section 3.4 emits them: 4 or 8 bit chosen per block conv, so that 8-bit convs
    write 4-bit outputs for a 4-bit successor and the other way round, blocks requantize their input only when
    their first conv is 4-bit, and a shortcut conv follows the block's first conv.  Every layer bit for bit."""
    units = inputs.resnet_choice_units(depth)
    g = inputs.rng(21, depth, len(pattern))
    if pattern == "alternate":
        bits = [8 if i % 2 == 0 else 4 for i in range(units)]
    elif pattern == "random":
        bits = [int(b) for b in g.choice([4, 8], size=units)]
    else:
        bits = [4] * units
    t = inputs.resnet_table(depth, seed=6, image_hw=64, classes=24, width=32, conv_bits=bits)
    run_network_and_compare(hq, t, batch=3, seed=depth + 1)


def test_network_residual_shifts_per_channel(hq):
    """Fused residual adds inside a network with a different dyadic pair on every channel: shifts from 9 to
    45 (terms that vanish, terms with and without a narrow 32-bit form), unsigned and signed residual
    operands.  Every layer must still match the oracle bit for bit."""
    t = inputs.resnet_table(50, seed=11, image_hw=64, classes=24, width=32)
    g = inputs.rng(11, 3)
    n_res = 0
    for l in t["layers"]:
        if l["op"] == "conv" and l["in1"] >= 0:
            c = l["cout"]
            l["rb"] = g.integers(1 << 30, 1 << 31, size=c, dtype=np.int64).astype(np.int32)
            l["rc"] = g.integers(9, 46, size=c, dtype=np.int64).astype(np.int32)
            if n_res % 2 == 0:          # a few layers with shifts in the common range only
                l["rc"] = g.integers(28, 36, size=c, dtype=np.int64).astype(np.int32)
            n_res += 1
    assert n_res >= 8
    run_network_and_compare(hq, t, batch=2, seed=12)


@pytest.mark.parametrize("depth,mixed", [(18, False), (50, False), (50, True)])
def test_network_with_int32_residual_stream_every_layer(hq, depth, mixed):
    """The dataflow of Fig. 2 as the paper draws it: INT32 residual stream between blocks, one requantization per
    block input, raw INT32 accumulators of the block's last conv and of the shortcut conv into an element-wise add
    with an INT32 result.  Every layer equals the oracle."""
    t = inputs.resnet_table(depth, seed=8, image_hw=64, classes=24, width=32, mixed=mixed, int32_stream=True)
    assert sum(1 for l in t["layers"] if l["op"] == "add" and l["out_bits"] == 32) == {18: 8, 50: 16}[depth]
    run_network_and_compare(hq, t, batch=3, seed=depth + 2)


def test_residual_add_int32_result(hq):
    """hq_residual_add with out bits 32 on its own: INT32 + INT32 and INT32 + 8-bit operands, every shift."""
    from paper_2011_10680_b200 import binding
    g = inputs.rng(43, 1)
    n, hw, ch = 2, 9, 40
    main = g.integers(-(1 << 24), 1 << 24, size=(n, hw, hw, ch), dtype=np.int64).astype(np.int32)
    mb = g.integers(1 << 30, 1 << 31, size=ch, dtype=np.int64).astype(np.int32)
    mc = (np.arange(ch) % 62 + 1).astype(np.int32)
    for res_bits in (32, 8):
        res = (g.integers(-(1 << 20), 1 << 20, size=main.shape, dtype=np.int64).astype(np.int32) if res_bits == 32
               else g.integers(0, 256, size=main.shape, dtype=np.int64).astype(np.uint8))
        rb = g.integers(1 << 30, 1 << 31, size=ch, dtype=np.int64).astype(np.int32)
        rc = ((np.arange(ch) * 7) % 62 + 1).astype(np.int32)
        ref = oracle().residual_add(main, 32, 1, mb, mc, res, res_bits, int(res_bits == 32), rb, rc, ch, 0,
                                    -(1 << 31), (1 << 31) - 1, 32, 1)
        out = binding.alloc_out(n, hw, hw, ch, 32, 1)
        st = hq.residual_add(binding.to_device(main), 32, 1, binding.to_device(mb), binding.to_device(mc),
                             binding.to_device(res), res_bits, int(res_bits == 32), binding.to_device(rb), binding.to_device(rc),
                             ch, 0, -(1 << 31), (1 << 31) - 1, out, 32, 1)
        assert st == binding.HQ_OK
        hq.sync()
        assert np.array_equal(host(out, ref), ref)


@pytest.mark.parametrize("conv_bits", [4, 8])
def test_inception_modules_every_layer(hq, conv_bits):
    """Inception modules as Appendix E draws them, through hq_run_network: requantized input for the convolution
    branches, INT32 window sums of the module input as the pooling branch, per-branch DN, concatenation; 35x35 and
    17x17 module shapes at reduced width.  Every layer equals the oracle."""
    t = inputs.inception_table(7, conv_bits=conv_bits, image_hw=71, classes=24, width=32, modules35=2, modules17=1)
    ops = [l["op"] for l in t["layers"]]
    assert ops.count("concat") == 3 and ops.count("sumpool") == 3
    run_network_and_compare(hq, t, batch=2, seed=31)


def test_maxpool_int32(hq):
    from paper_2011_10680_b200 import binding
    g = inputs.rng(44, 2)
    x = g.integers(-(1 << 30), 1 << 30, size=(2, 11, 9, 20), dtype=np.int64).astype(np.int32)
    ref = oracle().maxpool(x, 3, 2, 1)
    out = binding.alloc_out(2, ref.shape[1], ref.shape[2], 20, 32, 1)
    assert hq.maxpool(binding.to_device(x), 20, 1, 3, 2, 1, out, bits=32) == binding.HQ_OK
    hq.sync()
    assert np.array_equal(host(out, ref), ref)


def test_table_from_the_offline_tool_runs_bit_exact(hq):
    """Float network (batch norm, a residual block, pooling, classifier) -> the offline tool (BN fold, channel-wise
    weight quantizer, INT32 bias, DN pairs, static calibration) -> hq_run_network: every layer equals the oracle."""
    from paper_2011_10680_b200 import offline
    g = np.random.default_rng(17)
    n, hw, c1, classes = 3, 16, 32, 12
    images = g.integers(0, 256, size=(n, hw, hw, 3)).astype(np.uint8)

    def bn(ch):
        return (g.uniform(0.8, 1.2, ch), g.normal(0, 0.1, ch), g.normal(0, 0.1, ch), g.uniform(0.8, 1.2, ch))

    layers = [
        dict(op="conv", in0=-1, in1=-1, w=g.normal(size=(c1, 3, 3, 3)) * 0.4, bn=bn(c1), stride=1, pad=1, bits=8, relu=True),
        dict(op="maxpool", in0=0, k=3, stride=2, pad=1),
        dict(op="conv", in0=1, in1=-1, w=g.normal(size=(c1, 3, 3, c1)) * 0.08, bn=bn(c1), stride=1, pad=1, bits=8, relu=True),
        dict(op="conv", in0=2, in1=1, w=g.normal(size=(c1, 1, 1, c1)) * 0.2, bn=bn(c1), stride=1, pad=0, bits=8, relu=True),
        dict(op="avgpool", in0=3, hw=(hw // 2) ** 2, channels=c1),
        dict(op="linear", in0=4, in1=-1, w=g.normal(size=(classes, 1, 1, c1)) * 0.3, bn=None, bias=np.full(classes, -0.1),
             bits=8, relu=False, s_out=None),
    ]
    s_img = 1.0 / 255.0
    table = offline.quantize_network(offline.calibrate(layers, images * s_img), s_img, image_hw=hw)
    for l in table["layers"]:
        if l["op"] == "maxpool":
            l["cout"] = c1
    # run_network_and_compare draws its own images from the table's image size; same shapes as the calibration batch
    ref = run_network_and_compare(hq, table, batch=n, seed=3)
    assert ref[-1].dtype == np.int32 and len(np.unique(ref[-1])) > classes


def test_resnet18_imagenet_shape_batch8_every_layer(hq):
    """Benchmark config 2: ResNet-18, 224x224x3, 1000 classes, batch 8, all layers INT8."""
    t = inputs.resnet_table(18, seed=2)
    ref = run_network_and_compare(hq, t, batch=8, seed=2)
    sat = [float(np.mean((r == 0) | (r == 255))) for r, l in zip(ref, t["layers"]) if l["op"] == "conv" and l["out_bits"] == 8]
    assert min(sat) < 0.9, "every layer is saturated: the workload would not exercise the requantization"


def test_resnet50_batch256_benchmark_configuration_every_image(hq):
    """The benchmark workloads themselves (ResNet-50, 224x224, batch 256, INT8 and mixed INT4/8), in the launch
    configuration bench.py times: tile sizes, folded channel tiles, the two-CTA shape and the number of
    accumulator buffers all depend on the batch.  Images are independent, so the batch is made of four distinct
    images dealt over the 256 positions in an irregular order; the oracle runs the four, and EVERY layer's output
    for EVERY one of the 256 positions must equal the oracle's output for the image at that position (compared
    on the device), as must the logits of the graph-replay path that the benchmark times."""
    from oracle.network import run_network
    from paper_2011_10680_b200 import binding
    batch, distinct = 256, 4
    order = np.array([(7 * i + i // 5 + (i * i) // 11) % distinct for i in range(batch)])
    assert len(set(order.tolist())) == distinct and order[0] != order[1] and order[-1] != order[-2]
    order_d = torch.from_numpy(order).cuda()
    for mixed, seed in ((False, 3), (True, 4)):
        t = inputs.resnet_table(50, seed, mixed=mixed)
        base = inputs.random_images(seed, distinct, t["image_hw"])
        ref = run_network(t, base)
        net = binding.Network(hq, t, batch)
        try:
            d_img = binding.to_device(base[order])
            logits = binding.alloc_out(*net.logits_shape, 32, 1)
            taps = net.alloc_taps()
            assert net.run(d_img, logits, taps) == binding.HQ_OK
            hq.sync()
            net.check_guards()
            for i, (tap, r) in enumerate(zip(taps, ref)):
                per_image = tap.numel() // batch
                want = torch.from_numpy(np.ascontiguousarray(r).view(np.uint8).reshape(distinct, per_image)).cuda()
                got = tap.view(batch, per_image)
                if not torch.equal(got, want[order_d]):
                    bad = (got != want[order_d]).any(dim=1).nonzero().flatten().tolist()
                    raise AssertionError(f"mixed={mixed} layer {i} ({t['layers'][i]['op']}) differs at batch positions {bad[:8]} ({len(bad)} of {batch})")
                del want
            # the graph-replay path that the benchmark times
            logits.zero_()
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                assert net.run(d_img, logits, None) == binding.HQ_OK
                hq.sync()
            want = ref[-1].reshape(distinct, -1)[order]
            assert np.array_equal(logits.cpu().numpy().reshape(batch, -1), want)
            net.check_guards()
            del taps
        finally:
            net.close()
        binding.check_guards()
        torch.cuda.empty_cache()
