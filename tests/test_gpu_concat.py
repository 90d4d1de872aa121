"""Parity of hq_concat_requant (Inception concatenation, Appendix E) with the CPU oracle: bit-exact, through the C ABI."""
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


def run_and_compare(hq, case):
    from oracle import hqref
    from paper_2011_10680_b200 import binding
    dev = [{**br, "x": binding.to_device(br["x"]), "b": binding.to_device(br["b"]), "c": binding.to_device(br["c"])}
           for br in case["branches"]]
    out = binding.alloc_out(case["n"], case["hw"], case["hw"], case["out_ch"], case["out_bits"], case["out_signed"])
    out.fill_(0x5A)                                             # stale bytes must all be overwritten
    st = hq.concat_requant(dev, case["relu"], case["qmin"], case["qmax"], out, case["out_bits"], case["out_signed"])
    assert st == binding.HQ_OK, binding.status_string(st)
    hq.sync()
    ref = hqref.concat_requant(case["branches"], case["relu"], case["qmin"], case["qmax"], case["out_bits"], case["out_signed"])
    got = out.cpu().numpy().view(ref.dtype).reshape(ref.shape)
    if not np.array_equal(got, ref):
        bad = np.argwhere(got != ref)
        raise AssertionError(f"{len(bad)} of {ref.size} stored values differ; first at {bad[0]}: got {got[tuple(bad[0])]} want {ref[tuple(bad[0])]}")
    return ref


# (channels, bits, signed) per branch
INCEPTION_A = [(64, 8, 0), (64, 8, 0), (96, 8, 0), (32, 32, 1)]            # 35x35 module: 1x1, 5x5, double 3x3, pool (INT32)
INCEPTION_C = [(192, 8, 0), (192, 8, 0), (192, 8, 0), (192, 32, 1)]        # 17x17 module
RAGGED = [(6, 8, 1), (20, 32, 1), (10, 4, 0), (48, 8, 0), (2, 32, 1), (16, 4, 1)]   # odd group sizes, unaligned offsets
VERY_WIDE = [(192, 8, 0), (1088, 32, 1), (2120, 8, 1), (64, 8, 0)]         # branches of more than 1024 channels: entered in pieces
TOO_MANY_PIECES = [(8, 8, 0)] * 6 + [(3080, 8, 0), (16, 32, 1)]            # no entries left for pieces: sixteen-channel form


@pytest.mark.parametrize("branches,n,hw", [(INCEPTION_A, 3, 35), (INCEPTION_C, 2, 17), (RAGGED, 2, 9), (VERY_WIDE, 2, 9),
                                          (TOO_MANY_PIECES, 1, 7)])
@pytest.mark.parametrize("out_bits,out_signed,relu", [(8, 0, 1), (8, 1, 0), (4, 0, 1)])
def test_concat_matches_the_oracle(hq, branches, n, hw, out_bits, out_signed, relu):
    case = inputs.concat_case(401, n, hw, branches, out_bits, out_signed, relu)
    ref = run_and_compare(hq, case)
    hq.set_tile_order(1)                     # the same pixels walked from the last to the first
    try:
        run_and_compare(hq, case)
    finally:
        hq.set_tile_order(0)
    if branches is INCEPTION_A and out_bits == 8:
        # the draw must exercise the arithmetic: not everything saturated
        inner = np.count_nonzero((ref > case["qmin"]) & (ref < case["qmax"]))
        assert inner > ref.size // 4


def test_concat_large_call_with_narrow_pairs(hq):
    """Above 2^22 outputs the 8- and 4-bit branches run on narrow multiply-add pairs worked out by a first launch;
    shifts from 9 to 45 across the channels so that channels with and without a pair (and with a zero term) mix."""
    g = inputs.rng(405)
    n, hw = 12, 35
    branches = []
    for ch, bits, signed in [(64, 8, 0), (64, 8, 1), (96, 4, 0), (64, 32, 1)]:
        if bits == 32:
            x = g.integers(-(1 << 22), 1 << 22, size=(n, hw, hw, ch), dtype=np.int64).astype(np.int32)
            c = g.integers(44, 48, size=ch).astype(np.int32)
        else:
            lo, hi = ((-128, 128) if signed else (0, 256)) if bits == 8 else ((-8, 8) if signed else (0, 16))
            x = g.integers(lo, hi, size=(n, hw, hw, ch), dtype=np.int64)
            x = inputs.pack4(x) if bits == 4 else x.astype(np.int8 if signed else np.uint8)
            c = (9 + (np.arange(ch) * 3) % 37).astype(np.int32)
            c[:16] = g.integers(29, 33, size=16)                 # one group of sixteen that surely has pairs
        b = g.integers(1 << 30, 1 << 31, size=ch, dtype=np.int64).astype(np.int32)
        branches.append({"x": x, "bits": bits, "signed": signed, "ch": ch, "b": b, "c": c})
    for out_bits, out_signed, relu, lo, hi in ((8, 0, 1, 0, 255), (8, 1, 0, -128, 127), (8, 0, 0, 3, 200), (4, 0, 1, 0, 15)):
        case = {"branches": branches, "relu": relu, "qmin": lo, "qmax": hi, "out_bits": out_bits, "out_signed": out_signed,
                "n": n, "hw": hw, "out_ch": 288}
        run_and_compare(hq, case)
        hq.set_tile_order(1)
        try:
            run_and_compare(hq, case)
        finally:
            hq.set_tile_order(0)


def _uniform_branch(g, n, hw, ch, bits, signed, b, c, uniform=True):
    """One branch whose channels all share the pair (b, c) (or, with uniform=False, all but the last channel)."""
    if bits == 32:
        x = g.integers(-(1 << 22), 1 << 22, size=(n, hw, hw, ch), dtype=np.int64).astype(np.int32)
    else:
        x = g.integers(-128 if signed else 0, 128 if signed else 256, size=(n, hw, hw, ch), dtype=np.int64)
        x = x.astype(np.int8 if signed else np.uint8)
    bb = np.full(ch, b, np.int32)
    cc = np.full(ch, c, np.int32)
    if not uniform:
        bb[-1] = b - 12345
    return {"x": x, "bits": bits, "signed": signed, "ch": ch, "b": bb, "c": cc}


@pytest.mark.parametrize("layout", ["module_35", "module_17", "signed_mix", "pieces", "unaligned_offset"])
def test_concat_branches_with_one_pair_per_branch(hq, layout):
    """Per-tensor activation scales give ONE pair DN(S_i / S_a) per branch (Appendix E); such 8-bit branches are walked
    in 16-byte pieces.  Cases: the two module shapes, signed operands beside unsigned ones, a branch that is uniform
    except for its last channel (must stay on the per-channel form), a branch wider than 1024 channels entered in
    pieces, an output offset that is not a multiple of sixteen (per-channel form), and pixel counts that leave a
    ragged last group of pixels; each with the saturating and the explicit clamp and a signed output."""
    g = inputs.rng(411)
    pair = lambda lo_c, hi_c: (int(g.integers(1 << 30, 1 << 31)), int(g.integers(lo_c, hi_c)))
    if layout == "module_35":
        n, hw = 15, 35
        spec = [(64, 8, 0, True), (64, 8, 0, True), (96, 8, 0, True), (64, 32, 1, True)]
    elif layout == "module_17":
        n, hw = 25, 17
        spec = [(192, 8, 0, True)] * 3 + [(192, 8, 0, False)]
    elif layout == "signed_mix":
        n, hw = 31, 19
        spec = [(48, 8, 1, True), (80, 8, 0, True), (16, 8, 1, True), (112, 8, 1, False), (128, 8, 0, True)]
    elif layout == "pieces":
        n, hw = 5, 23
        spec = [(64, 8, 0, True), (2064, 8, 0, True), (32, 32, 1, True)]
    else:
        n, hw = 40, 21
        spec = [(8, 8, 0, True), (64, 8, 0, True), (120, 8, 1, True), (64, 8, 0, True)]
    branches = []
    for ch, bits, signed, uniform in spec:
        b, c = pair(44, 48) if bits == 32 else pair(29, 33)
        branches.append(_uniform_branch(g, n, hw, ch, bits, signed, b, c, uniform))
    out_ch = sum(s[0] for s in spec)
    assert n * hw * hw * out_ch >= 1 << 22                          # large enough for the narrow pairs
    for out_signed, relu, lo, hi in ((0, 1, 0, 255), (1, 0, -128, 127), (0, 0, 3, 200)):
        case = {"branches": branches, "relu": relu, "qmin": lo, "qmax": hi, "out_bits": 8, "out_signed": out_signed,
                "n": n, "hw": hw, "out_ch": out_ch}
        ref = run_and_compare(hq, case)
        inner = np.count_nonzero((ref > lo) & (ref < hi))
        assert inner > ref.size // 8
        hq.set_tile_order(1)
        try:
            run_and_compare(hq, case)
        finally:
            hq.set_tile_order(0)
    # a pair whose shift has no narrow form (c = 40) and one whose term is always zero (c = 45)
    for c in (40, 45):
        odd = [_uniform_branch(g, n, hw, ch, bits, signed, (1 << 31) - 7, c if bits == 8 else 46, True)
               for ch, bits, signed, _ in spec]
        run_and_compare(hq, {"branches": odd, "relu": 1, "qmin": 0, "qmax": 255, "out_bits": 8, "out_signed": 0,
                             "n": n, "hw": hw, "out_ch": out_ch})


def test_concat_at_the_benchmark_size(hq):
    """The 35x35 module at batch 256, as `bench.py --membound` times it (90 M outputs): every stored value."""
    case = inputs.concat_case(406, 256, 35, [(64, 8, 0), (64, 8, 0), (96, 8, 0), (64, 32, 1)])
    run_and_compare(hq, case)


def test_concat_every_shift_and_extreme_operands(hq):
    """Shifts 1..62 across the channels (both forms of the arithmetic), full-range INT32 and 8-bit operands."""
    g = inputs.rng(402)
    n, hw = 1, 12
    branches = []
    for ch, bits, signed in [(64, 32, 1), (62, 8, 1), (64, 8, 0)]:
        if bits == 32:
            x = g.integers(-(1 << 31), 1 << 31, size=(n, hw, hw, ch), dtype=np.int64).astype(np.int32)
            x[0, 0, :4] = [[-(1 << 31)] * ch, [(1 << 31) - 1] * ch, [0] * ch, [-1] * ch]
        else:
            x = g.integers(-128 if signed else 0, 128 if signed else 256, size=(n, hw, hw, ch), dtype=np.int64)
            x = x.astype(np.int8 if signed else np.uint8)
        b = g.integers(1 << 30, 1 << 31, size=ch, dtype=np.int64).astype(np.int32)
        b[:3] = [(1 << 31) - 1, 1 << 30, 0]
        c = ((np.arange(ch) * 5) % 62 + 1).astype(np.int32)
        branches.append({"x": x, "bits": bits, "signed": signed, "ch": ch, "b": b, "c": c})
    for out_signed, relu in ((1, 0), (0, 1)):
        lo, hi = (-128, 127) if out_signed else (0, 255)
        case = {"branches": branches, "relu": relu, "qmin": lo, "qmax": hi, "out_bits": 8, "out_signed": out_signed,
                "n": n, "hw": hw, "out_ch": 190}
        run_and_compare(hq, case)


def test_concat_single_branch_equals_residual_add_and_rejects_bad_arguments(hq):
    from paper_2011_10680_b200 import binding
    case = inputs.concat_case(403, 2, 8, [(32, 32, 1)])
    ref = run_and_compare(hq, case)
    br = case["branches"][0]
    x, b, c = (binding.to_device(br[k]) for k in ("x", "b", "c"))
    out = binding.alloc_out(2, 8, 8, 32, 8, 0)
    st = hq.residual_add(x, 32, 1, b, c, None, 0, 0, None, None, 32, 1, 0, 255, out, 8, 0)
    assert st == binding.HQ_OK
    hq.sync()
    assert np.array_equal(out.cpu().numpy(), ref)
    dev = [{**br, "x": x, "b": b, "c": c}]
    # channel counts must sum to the output's; 4-bit outputs need even branches; at most eight branches
    wrong = binding.alloc_out(2, 8, 8, 48, 8, 0)
    assert hq.concat_requant(dev, 1, 0, 255, wrong, 8, 0) == binding.HQ_ERR_INVALID_ARG
    assert hq.concat_requant(dev * 9, 1, 0, 255, out, 8, 0) == binding.HQ_ERR_INVALID_ARG
    assert hq.concat_requant(dev, 1, 0, 300, out, 8, 0) == binding.HQ_ERR_INVALID_ARG
    odd = inputs.concat_case(404, 1, 4, [(5, 8, 0), (3, 8, 0)])
    odd_dev = [{**o, "x": binding.to_device(o["x"]), "b": binding.to_device(o["b"]), "c": binding.to_device(o["c"])}
               for o in odd["branches"]]
    out4 = binding.alloc_out(1, 4, 4, 8, 4, 0)
    assert hq.concat_requant(odd_dev, 1, 0, 15, out4, 4, 0) == binding.HQ_ERR_UNSUPPORTED


def test_concat_empty_batch_is_a_no_op(hq):
    from paper_2011_10680_b200 import binding
    x = torch.empty((0, 5, 5, 16), dtype=torch.uint8, device="cuda")
    keep = torch.zeros(16, dtype=torch.uint8, device="cuda")        # a valid pointer for the empty tensors
    b = binding.to_device(np.full(16, 1 << 30, np.int32))
    c = binding.to_device(np.full(16, 30, np.int32))
    tin = binding.hq_tensor(keep.data_ptr(), 0, 5, 5, 16, 8, 0)
    tout = binding.hq_tensor(keep.data_ptr(), 0, 5, 5, 16, 8, 0)
    import ctypes as C
    ts = (binding.hq_tensor * 1)(tin)
    ds = (binding.hq_dyadic * 1)(binding.hq_dyadic(b.data_ptr(), c.data_ptr()))
    st = binding.lib().hq_concat_requant(hq._h, 1, ts, ds, 1, 0, 255, C.byref(tout), None)
    assert st == binding.HQ_OK
    hq.sync()
    assert x.numel() == 0 and int(keep.sum()) == 0


# ------------------------------------------------------------------ INT32 window sums (pooling branch) ----
@pytest.mark.parametrize("n,h,w,ch,bits,signed,k,stride,pad", [
    (2, 35, 35, 64, 32, 1, 3, 1, 1),        # the 35x35 module's pooling branch
    (3, 17, 17, 192, 32, 1, 3, 1, 1),
    (2, 9, 7, 6, 32, 1, 3, 2, 1),           # channel count not a multiple of 4, stride 2, H != W
    (2, 8, 8, 10, 8, 0, 3, 1, 1),
    (1, 6, 5, 8, 4, 1, 2, 2, 0),
    (1, 7, 7, 4, 8, 1, 5, 1, 2),
    (3, 35, 35, 288, 8, 0, 3, 1, 1),        # the layer-table form: 8-bit module input, four channels per thread
    (2, 17, 19, 64, 8, 1, 3, 1, 1),         # signed bytes, H != W, several strips of rows
    (1, 1, 1, 8, 8, 1, 3, 1, 1),            # a single pixel: every neighbour is padding
    (2, 3, 40, 12, 32, 1, 3, 1, 1),         # fewer rows than a strip
])
def test_sumpool_matches_the_oracle(hq, n, h, w, ch, bits, signed, k, stride, pad):
    from oracle import hqref
    from paper_2011_10680_b200 import binding
    g = inputs.rng(407, n, h, ch, bits)
    if bits == 32:
        x = g.integers(-(1 << 26), 1 << 26, size=(n, h, w, ch), dtype=np.int64).astype(np.int32)
    elif bits == 8:
        x = g.integers(-128 if signed else 0, 128 if signed else 256, size=(n, h, w, ch), dtype=np.int64).astype(np.int8 if signed else np.uint8)
    else:
        x = inputs.pack4(g.integers(-8 if signed else 0, 8 if signed else 16, size=(n, h, w, ch), dtype=np.int64))
    ref = hqref.sumpool(x, ch, bits, signed, k, stride, pad)
    out = torch.full(ref.shape, 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    st = hq.sumpool(binding.to_device(x), ch, bits, signed, k, stride, pad, out)
    assert st == binding.HQ_OK, binding.status_string(st)
    hq.sync()
    assert np.array_equal(out.cpu().numpy(), ref)


def test_pooling_branch_then_concat_is_an_inception_module_tail(hq):
    """INT32 feature map -> 3x3 window sums (INT32) -> concatenated with 8-bit branches, 1/9 inside the pooling
    branch's dyadic pairs: both calls chained on the device against the oracle's chain."""
    from oracle import hqref
    from paper_2011_10680_b200 import binding
    g = inputs.rng(408)
    n, hw = 2, 35
    fmap = g.integers(-(1 << 18), 1 << 18, size=(n, hw, hw, 32), dtype=np.int64).astype(np.int32)
    pb, pc = inputs.dyadic_from_scale(np.exp2(g.uniform(-12.0, -10.0, size=32)) / 9.0)
    case = inputs.concat_case(409, n, hw, [(64, 8, 0), (96, 8, 0)])
    pooled_ref = hqref.sumpool(fmap, 32, 32, 1, 3, 1, 1)
    branches_ref = case["branches"] + [{"x": pooled_ref, "bits": 32, "signed": 1, "ch": 32, "b": pb, "c": pc}]
    ref = hqref.concat_requant(branches_ref, 1, 0, 255, 8, 0)
    pooled = torch.empty((n, hw, hw, 32), dtype=torch.int32, device="cuda")
    assert hq.sumpool(binding.to_device(fmap), 32, 32, 1, 3, 1, 1, pooled) == binding.HQ_OK
    dev = [{**br, "x": binding.to_device(br["x"]), "b": binding.to_device(br["b"]), "c": binding.to_device(br["c"])}
           for br in case["branches"]]
    dev.append({"x": pooled, "bits": 32, "signed": 1, "ch": 32, "b": binding.to_device(pb), "c": binding.to_device(pc)})
    out = binding.alloc_out(n, hw, hw, 192, 8, 0)
    assert hq.concat_requant(dev, 1, 0, 255, out, 8, 0) == binding.HQ_OK
    hq.sync()
    assert np.array_equal(out.cpu().numpy(), ref)
    assert np.count_nonzero((ref[..., 160:] > 0) & (ref[..., 160:] < 255)) > ref[..., 160:].size // 4
