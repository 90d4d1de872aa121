"""Pins for the CPU oracle: every exported function is checked against something other than itself.

What fixes the values: exact rational arithmetic (Python big integers / fractions), brute-force
loops on tiny shapes, an independently written im2col + matrix-product formulation, special cases
that reduce to the identity or to a closed form, the worked example of the paper's Appendix G and
the cost columns of its Table 1.
"""
from __future__ import annotations

import os
import re
from fractions import Fraction

import numpy as np
import pytest

from oracle import build as oracle_build
from oracle import hqref
from oracle.network import run_network
from paper_2011_10680_b200 import inputs


# ---------------------------------------------------------------- P1: rounding shift ------------
def exact_round_half_up(num: int, c: int) -> int:
    """floor(num / 2^c + 1/2) in exact rational arithmetic."""
    q = Fraction(num, 1 << c) + Fraction(1, 2)
    return q.numerator // q.denominator


def test_rshift_round_ties_and_signs():
    # x*b / 2^c = +-0.5, +-1.5: ties go toward +infinity
    assert hqref.dn(1, 1 << 30, 31) == 1
    assert hqref.dn(-1, 1 << 30, 31) == 0
    assert hqref.dn(3, 1 << 30, 31) == 2
    assert hqref.dn(-3, 1 << 30, 31) == -1
    assert hqref.rshift_round(5, 1) == 3 and hqref.rshift_round(-5, 1) == -2
    assert hqref.rshift_round(0, 62) == 0


def test_rshift_round_matches_exact_rational():
    g = np.random.default_rng(1)
    for c in list(range(1, 63)):
        for _ in range(40):
            x = int(g.integers(-(1 << 31), 1 << 31))
            b = int(g.integers(0, 1 << 31))
            assert hqref.dn(x, b, c) == exact_round_half_up(x * b, c), (x, b, c)
    # dense range around zero for a few pairs
    for b, c in [(1 << 30, 31), ((1 << 31) - 1, 33), (1518500250, 36), (3, 2)]:
        for x in range(-300, 301):
            assert hqref.dn(x, b, c) == exact_round_half_up(x * b, c)
    # extremes of the argument range
    for x in (-(1 << 31), (1 << 31) - 1):
        for b in (0, 1, (1 << 31) - 1):
            for c in (1, 31, 62):
                assert hqref.dn(x, b, c) == exact_round_half_up(x * b, c)


# ---------------------------------------------------------------- P2/P3: DN and its error -------
def test_dyadic_from_scale_bound_and_range():
    g = np.random.default_rng(2)
    s = np.exp(g.uniform(np.log(2.0 ** -30), np.log(2.0 ** 20), size=200000))
    s = np.concatenate([s, 2.0 ** np.arange(-30, 21), np.nextafter(2.0 ** np.arange(-30, 21), 0)])
    b, c = inputs.dyadic_from_scale(s)
    assert b.dtype == np.int32 and c.dtype == np.int32
    assert np.all(b >= 1 << 30) and np.all(b.astype(np.int64) < 1 << 31)
    assert np.all(c >= 1) and np.all(c <= 62)
    for i in g.integers(0, len(s), size=3000):       # exact check of |b/2^c - s| <= 2^-(c+1)
        err = abs(Fraction(int(b[i]), 1 << int(c[i])) - Fraction(float(s[i])))
        assert err <= Fraction(1, 1 << (int(c[i]) + 1)), (s[i], b[i], c[i])
    err = np.abs(b.astype(np.float64) / 2.0 ** c - s)
    assert np.all(err <= 2.0 ** -(c.astype(np.float64) + 1) * (1 + 1e-9))
    # c = 30 + ceil(log2(1/s)) away from exact powers of two
    s2 = np.array([0.1, 0.3, 0.75, 3.0, 1e-4])
    _, c2 = inputs.dyadic_from_scale(s2)
    assert np.array_equal(c2, 30 + np.ceil(np.log2(1 / s2)).astype(np.int32))


def test_requant_error_bound_against_real_scale():
    g = np.random.default_rng(3)
    for _ in range(2000):
        s = float(np.exp(g.uniform(np.log(2.0 ** -20), np.log(4.0))))
        t = int(g.integers(-(1 << 24), 1 << 24))
        b, c = inputs.dyadic_from_scale(s)
        q = hqref.dn(t, int(b[0]), int(c[0]))
        bound = Fraction(1, 2) + abs(t) * Fraction(1, 1 << (int(c[0]) + 1))
        assert abs(Fraction(q) - Fraction(t) * Fraction(s)) <= bound


# ---------------------------------------------------------------- P4: convolution ---------------
def brute_conv(x, w, stride, pad):
    """Direct convolution with Python integers.  x: (n,h,w,ci) w: (co,kh,kw,ci)."""
    n, h, wd, ci = x.shape
    co, kh, kw, _ = w.shape
    ho = (h + 2 * pad - kh) // stride + 1
    wo = (wd + 2 * pad - kw) // stride + 1
    out = np.zeros((n, ho, wo, co), dtype=object)
    xl, wl = x.tolist(), w.tolist()
    for b in range(n):
        for oh in range(ho):
            for ow in range(wo):
                for oc in range(co):
                    acc = 0
                    for r in range(kh):
                        ih = oh * stride + r - pad
                        if not 0 <= ih < h:
                            continue
                        for s in range(kw):
                            iw = ow * stride + s - pad
                            if not 0 <= iw < wd:
                                continue
                            px, pw = xl[b][ih][iw], wl[oc][r][s]
                            for k in range(ci):
                                acc += px[k] * pw[k]
                    out[b, oh, ow, oc] = acc
    return out


def im2col_conv(x, w, stride, pad):
    """Independent formulation: explicit zero padding, patch matrix, one int64 matrix product."""
    n, h, wd, ci = x.shape
    co, kh, kw, _ = w.shape
    xp = np.zeros((n, h + 2 * pad, wd + 2 * pad, ci), np.int64)
    xp[:, pad:pad + h, pad:pad + wd] = x
    ho = (h + 2 * pad - kh) // stride + 1
    wo = (wd + 2 * pad - kw) // stride + 1
    cols = np.empty((n, ho, wo, kh, kw, ci), np.int64)
    for r in range(kh):
        for s in range(kw):
            cols[:, :, :, r, s] = xp[:, r:r + stride * ho:stride, s:s + stride * wo:stride]
    return (cols.reshape(n * ho * wo, -1) @ w.astype(np.int64).reshape(co, -1).T).reshape(n, ho, wo, co)


def epilogue_exact(acc, bias, b, c, res, rb, rc, relu, qmin, qmax):
    """Bias + dyadic requant + residual + ReLU + clamp with Python integers (Eq. 4, Section 3.3)."""
    out = np.zeros(acc.shape, np.int64)
    it = np.nditer(out, flags=["multi_index"])
    for _ in it:
        idx = it.multi_index
        oc = idx[-1]
        y = exact_round_half_up((int(acc[idx]) + int(bias[oc])) * int(b[oc]), int(c[oc]))
        if res is not None:
            y += exact_round_half_up(int(res[idx]) * int(rb[oc]), int(rc[oc]))
        if relu:
            y = max(y, 0)
        out[idx] = min(max(y, qmin), qmax)
    return out


CONV_SHAPES = [
    # n, h, w, cin, cout, k, stride, pad
    (1, 5, 5, 4, 3, 1, 1, 0),
    (2, 6, 5, 4, 5, 3, 1, 1),
    (1, 9, 11, 2, 4, 7, 2, 3),
    (2, 7, 8, 6, 4, 3, 2, 1),
    (1, 8, 8, 8, 2, 1, 2, 0),
    (3, 4, 6, 2, 7, 3, 1, 0),
]


@pytest.mark.parametrize("shape", CONV_SHAPES)
@pytest.mark.parametrize("bits", [8, 4])
def test_conv_raw_accumulator_vs_bruteforce_and_im2col(shape, bits):
    n, h, w, cin, cout, k, stride, pad = shape
    case = inputs.conv_case(11, n, h, w, cin, cout, k, stride, pad, bits=bits, out_bits=32, relu=False)
    got = hqref.conv_case(case)
    x = inputs.unpack4(case["x"], False) if bits == 4 else case["x"]
    wt = inputs.unpack4(case["wgt"], True) if bits == 4 else case["wgt"]
    x, wt = x.astype(np.int64), wt.astype(np.int64)
    ref = brute_conv(x, wt, stride, pad) + case["bias"].astype(object)
    assert np.array_equal(got.astype(object), ref)
    assert np.array_equal(got.astype(np.int64), im2col_conv(x, wt, stride, pad) + case["bias"].astype(np.int64))


@pytest.mark.parametrize("residual,res_bits,relu,out_bits", [
    (False, 8, True, 8), (True, 8, True, 8), (True, 32, True, 8), (True, 8, False, 8), (False, 8, True, 4),
])
def test_conv_fused_epilogue_vs_exact_integers(residual, res_bits, relu, out_bits):
    case = inputs.conv_case(5, 2, 6, 7, 8, 6, 3, 1, 1, bits=8, out_bits=out_bits, residual=residual,
                            res_bits=res_bits, relu=relu, c_range=(43, 47) if out_bits == 4 else (39, 43))
    got = hqref.conv_case(case)
    if out_bits == 4:
        got = inputs.unpack4(got, bool(case["out_signed"]))
    acc = im2col_conv(case["x"].astype(np.int64), case["wgt"].astype(np.int64), 1, 1)
    ref = epilogue_exact(acc, case["bias"], case["b"], case["c"], case["res"], case["rb"], case["rc"],
                         case["relu"], case["qmin"], case["qmax"])
    assert np.array_equal(got.astype(np.int64), ref)
    frac_mid = np.mean((ref > case["qmin"]) & (ref < case["qmax"]))
    assert frac_mid > 0.2, "case degenerate: almost everything saturates"


# ---------------------------------------------------------------- P5: special cases -------------
def test_identity_1x1_and_centre_delta_3x3_return_the_input():
    g = np.random.default_rng(4)
    x = g.integers(0, 256, size=(2, 5, 6, 4)).astype(np.uint8)
    eye = np.zeros((4, 1, 1, 4), np.int8)
    delta = np.zeros((4, 3, 3, 4), np.int8)
    for i in range(4):
        eye[i, 0, 0, i] = 1
        delta[i, 1, 1, i] = 1
    one_b, one_c = np.full(4, 1 << 30, np.int32), np.full(4, 30, np.int32)   # b/2^c == 1
    y = hqref.conv2d(x, 4, 8, 0, eye, 4, 1, 1, 1, 0, None, one_b, one_c)
    assert np.array_equal(y, x)
    y = hqref.conv2d(x, 4, 8, 0, delta, 4, 3, 3, 1, 1, None, one_b, one_c)
    assert np.array_equal(y, x)


def test_all_ones_3x3_counts_the_taps_inside_the_image():
    v = 7
    x = np.full((1, 5, 6, 1), v, np.uint8)   # odd channel count is fine at 8 bit
    w = np.ones((1, 3, 3, 1), np.int8)
    y = hqref.conv2d(x, 1, 8, 0, w, 1, 3, 3, 1, 1, None, None, None, out_bits=32, out_signed=1,
                     qmin=-(1 << 31), qmax=(1 << 31) - 1)[0, :, :, 0]
    assert y[2, 3] == 9 * v and y[0, 2] == 6 * v and y[3, 0] == 6 * v
    assert y[0, 0] == 4 * v and y[4, 5] == 4 * v and y[0, 5] == 4 * v


def test_linear_is_conv_on_a_1x1_image_and_matches_a_matrix_product():
    g = np.random.default_rng(6)
    x = g.integers(0, 256, size=(5, 32)).astype(np.uint8)
    w = g.integers(-127, 128, size=(10, 1, 1, 32)).astype(np.int8)
    bias = g.integers(-1000, 1000, size=10).astype(np.int32)
    y = hqref.linear(x, 32, 8, 0, w, 10, bias, None, None, 0, -(1 << 31), (1 << 31) - 1, 32, 1)
    assert np.array_equal(y.reshape(5, 10), x.astype(np.int64) @ w.reshape(10, 32).astype(np.int64).T + bias)
    y2 = hqref.conv2d(x.reshape(5, 1, 1, 32), 32, 8, 0, w, 10, 1, 1, 1, 0, bias, None, None,
                      out_bits=32, out_signed=1, qmin=-(1 << 31), qmax=(1 << 31) - 1)
    assert np.array_equal(y, y2)


def test_relu_before_or_after_requant_is_the_same():
    # max(Int(x s), 0) == Int(max(x, 0) s) for a positive scale: checked through the oracle itself
    g = np.random.default_rng(8)
    t = g.integers(-(1 << 20), 1 << 20, size=(1, 1, 64, 8)).astype(np.int32)
    b = g.integers(1 << 30, 1 << 31, size=8).astype(np.int32)
    c = g.integers(40, 46, size=8).astype(np.int32)
    after = hqref.residual_add(t, 32, 1, b, c, None, 0, 0, None, None, 8, 1, -128, 127, 8, 1)
    before = hqref.residual_add(np.maximum(t, 0), 32, 1, b, c, None, 0, 0, None, None, 8, 0, -128, 127, 8, 1)
    assert np.array_equal(after, before)


# ---------------------------------------------------------------- P6: the paper's example -------
def test_appendix_g_example_two_roundings_then_add(golden_dir):
    rows = [l.split() for l in open(os.path.join(golden_dir, "appendix_g_residual_example.txt"))
            if l.strip() and not l.startswith("#")]
    m, r, fake, integer_only = float(rows[0][0]), float(rows[0][1]), int(rows[0][2]), int(rows[0][3])
    # represent m and r as integers at scale 0.1 and rescale both branches by DN(0.1) to S_a = 1
    q_m, q_r = round(m * 10), round(r * 10)
    b, c = inputs.dyadic_from_scale(0.1)
    main = np.full((1, 1, 1, 2), q_m, np.int32)
    res = np.full((1, 1, 1, 2), q_r, np.int32)
    bb, cc = np.full(2, b[0], np.int32), np.full(2, c[0], np.int32)
    y = hqref.residual_add(main, 32, 1, bb, cc, res, 32, 1, bb, cc, 2, 0, -128, 127, 8, 1)
    assert int(y.ravel()[0]) == integer_only == 6
    # adding first and rounding once (what fake quantization does) gives the other value
    y1 = hqref.residual_add(main + res, 32, 1, bb, cc, None, 0, 0, None, None, 2, 0, -128, 127, 8, 1)
    assert int(y1.ravel()[0]) == fake == 7


# ---------------------------------------------------------------- P7: 4-bit packing -------------
def test_int4_equals_int8_on_widened_values_and_nibble_order():
    case4 = inputs.conv_case(21, 2, 5, 6, 8, 6, 3, 1, 1, bits=4, out_bits=4, residual=True, c_range=(39, 43))
    y4 = hqref.conv_case(case4)
    wide = dict(case4)
    wide.update(bits=8, x=inputs.unpack4(case4["x"], False), wgt=inputs.unpack4(case4["wgt"], True), out_bits=8)
    y8 = hqref.conv_case(wide)
    assert np.array_equal(inputs.unpack4(y4, False), y8)
    # element 2j is the low nibble of byte j: a delta weight on channel 1 must read the high nibble
    x = np.array([[[[0x21, 0x43]]]], np.uint8)          # channels 0..3 = 1, 2, 3, 4
    for ch in range(4):
        w = np.zeros((2, 1, 1, 4), np.int64)
        w[0, 0, 0, ch] = 1
        w[1, 0, 0, ch] = -8                               # most negative nibble must sign-extend
        y = hqref.conv2d(x, 4, 4, 0, inputs.pack4(w), 2, 1, 1, 1, 0, None, None, None, out_bits=32,
                         out_signed=1, qmin=-(1 << 31), qmax=(1 << 31) - 1)
        assert y.ravel().tolist() == [ch + 1, -8 * (ch + 1)]
    a = np.arange(-8, 8).reshape(1, 16)
    assert np.array_equal(inputs.unpack4(inputs.pack4(a), True), a)
    assert inputs.pack4(np.array([1, 2]))[0] == 0x21


# ---------------------------------------------------------------- P8: pooling -------------------
def test_avgpool_of_a_constant_returns_it_and_matches_exact_mean():
    b, c = inputs.dyadic_from_scale(1.0 / 49.0)
    for v in range(256):
        x = np.full((1, 7, 7, 2), v, np.uint8)
        y = hqref.avgpool_requant(x, 2, 8, 0, np.full(2, b[0]), np.full(2, c[0]), 0, 255)
        assert int(y.ravel()[0]) == v
    g = np.random.default_rng(9)
    x = g.integers(0, 256, size=(3, 7, 7, 6)).astype(np.uint8)
    bb, cc = inputs.dyadic_from_scale(np.full(6, 0.37 / 49.0))
    y = hqref.avgpool_requant(x, 6, 8, 0, bb, cc, 0, 255).reshape(3, 6)
    s = x.astype(np.int64).sum(axis=(1, 2))
    for n in range(3):
        for k in range(6):
            assert int(y[n, k]) == min(255, max(0, exact_round_half_up(int(s[n, k]) * int(bb[k]), int(cc[k]))))


def test_maxpool_matches_padded_numpy_max():
    g = np.random.default_rng(10)
    x = g.integers(0, 256, size=(2, 9, 10, 3)).astype(np.uint8)
    y = hqref.maxpool(x, 3, 2, 1)
    xp = np.zeros((2, 11, 12, 3), np.uint8)
    xp[:, 1:10, 1:11] = x
    ref = np.zeros_like(y)
    for oh in range(y.shape[1]):
        for ow in range(y.shape[2]):
            ref[:, oh, ow] = xp[:, 2 * oh:2 * oh + 3, 2 * ow:2 * ow + 3].max(axis=(1, 2))
    assert np.array_equal(y, ref)


def test_residual_add_elementwise_vs_exact():
    g = np.random.default_rng(12)
    main = g.integers(-(1 << 22), 1 << 22, size=(2, 3, 4, 6)).astype(np.int32)
    res = g.integers(-128, 128, size=(2, 3, 4, 6)).astype(np.int8)
    mb, rb = (g.integers(1 << 30, 1 << 31, size=6).astype(np.int32) for _ in range(2))
    mc = g.integers(44, 50, size=6).astype(np.int32)
    rc = g.integers(28, 34, size=6).astype(np.int32)
    y = hqref.residual_add(main, 32, 1, mb, mc, res, 8, 1, rb, rc, 6, 1, 0, 255, 8, 0)
    ref = epilogue_exact(main.astype(np.int64), np.zeros(6, np.int64), mb, mc, res, rb, rc, 1, 0, 255)
    assert np.array_equal(y.astype(np.int64), ref)


# ---------------------------------------------------------------- concat (Appendix E) -----------
def _concat_branches(g):
    n, h, w = 2, 3, 5
    specs = [(6, 8, 0), (4, 32, 1), (10, 8, 1), (2, 32, 1)]      # (channels, bits, signed)
    branches = []
    for ch, bits, signed in specs:
        if bits == 32:
            x = g.integers(-(1 << 20), 1 << 20, size=(n, h, w, ch)).astype(np.int32)
            c = g.integers(40, 46, size=ch).astype(np.int32)
        else:
            x = g.integers(-128 if signed else 0, 128 if signed else 256, size=(n, h, w, ch)).astype(np.int8 if signed else np.uint8)
            c = g.integers(29, 33, size=ch).astype(np.int32)
        b = g.integers(1 << 30, 1 << 31, size=ch).astype(np.int32)
        branches.append({"x": x, "bits": bits, "signed": signed, "ch": ch, "b": b, "c": c})
    return branches


def test_concat_places_every_branch_at_its_offset_with_exact_rounding():
    """Each output channel range holds clamp(floor(q*b/2^c + 1/2)) of its own branch, in exact rationals."""
    branches = _concat_branches(np.random.default_rng(21))
    y = hqref.concat_requant(branches, 0, -128, 127, 8, 1).astype(np.int64)
    off = 0
    for br in branches:
        x = br["x"].astype(np.int64)
        for k in range(br["ch"]):
            want = np.array([min(max(exact_round_half_up(int(q) * int(br["b"][k]), int(br["c"][k])), -128), 127)
                             for q in x[..., k].ravel()]).reshape(x.shape[:3])
            assert np.array_equal(y[..., off + k], want)
        off += br["ch"]
    assert off == y.shape[-1]


def test_concat_with_unit_scales_is_numpy_concatenate_and_relu_clamps():
    g = np.random.default_rng(22)
    xs = [g.integers(-100, 100, size=(1, 4, 4, ch)).astype(np.int8) for ch in (2, 6, 4)]
    branches = [{"x": x, "bits": 8, "signed": 1, "ch": x.shape[-1], "b": np.full(x.shape[-1], 1 << 30, np.int32),
                 "c": np.full(x.shape[-1], 30, np.int32)} for x in xs]
    cat = np.concatenate(xs, axis=-1)
    assert np.array_equal(hqref.concat_requant(branches, 0, -128, 127, 8, 1), cat)
    assert np.array_equal(hqref.concat_requant(branches, 1, 0, 15, 8, 0), np.clip(cat, 0, 15).astype(np.uint8))
    packed = hqref.concat_requant(branches, 1, 0, 15, 4, 0)                  # 4-bit output: same values, two per byte
    assert np.array_equal(inputs.unpack4(packed, False), np.clip(cat, 0, 15).astype(np.uint8))


def test_concat_of_one_branch_is_the_plain_requantization():
    g = np.random.default_rng(23)
    x = g.integers(-(1 << 21), 1 << 21, size=(2, 2, 3, 8)).astype(np.int32)
    b = g.integers(1 << 30, 1 << 31, size=8).astype(np.int32)
    c = g.integers(42, 48, size=8).astype(np.int32)
    one = hqref.concat_requant([{"x": x, "bits": 32, "signed": 1, "ch": 8, "b": b, "c": c}], 1, 0, 255, 8, 0)
    assert np.array_equal(one, hqref.residual_add(x, 32, 1, b, c, None, 0, 0, None, None, 8, 1, 0, 255, 8, 0))


def test_sumpool_counts_taps_and_matches_padded_window_sums():
    """Constant input: 9v inside, 6v on edges, 4v in corners (zero padding); random input: numpy window sums."""
    v = np.full((1, 5, 6, 2), 7, np.int32)
    y = hqref.sumpool(v, 2, 32, 1, 3, 1, 1)
    assert y[0, 2, 3, 0] == 63 and y[0, 0, 2, 1] == 42 and y[0, 4, 5, 0] == 28 and y.shape == (1, 5, 6, 2)
    g = np.random.default_rng(31)
    for bits, k, stride, pad in ((32, 3, 1, 1), (8, 3, 2, 1), (32, 2, 2, 0), (8, 5, 1, 2)):
        x = (g.integers(-(1 << 20), 1 << 20, size=(2, 7, 9, 4)).astype(np.int32) if bits == 32
             else g.integers(-128, 128, size=(2, 7, 9, 4)).astype(np.int8))
        y = hqref.sumpool(x, 4, bits, 1, k, stride, pad)
        xp = np.pad(x.astype(np.int64), ((0, 0), (pad, pad), (pad, pad), (0, 0)))
        ref = np.zeros(y.shape, np.int64)
        for oh in range(y.shape[1]):
            for ow in range(y.shape[2]):
                ref[:, oh, ow] = xp[:, oh * stride:oh * stride + k, ow * stride:ow * stride + k].sum(axis=(1, 2))
        assert np.array_equal(y.astype(np.int64), ref)
    # an average pool without division: window sum, then DN(1/9): a constant v comes back in the interior
    b, c = inputs.dyadic_from_scale(1.0 / 9)
    s9 = hqref.sumpool(np.full((1, 5, 5, 1), 100, np.int32), 1, 32, 1, 3, 1, 1)
    avg = hqref.residual_add(s9, 32, 1, b, c, None, 0, 0, None, None, 1, 0, -128, 127, 8, 1)
    assert avg[0, 2, 2, 0] == 100 and avg[0, 0, 0, 0] == 44          # corner: round(400 / 9)


# ---------------------------------------------------------------- P9: topology ------------------
def test_table_cost_matches_the_papers_table1(golden_dir):
    want = {}
    for l in open(os.path.join(golden_dir, "table1_cost_columns.txt")):
        if l.strip() and not l.startswith("#"):
            model, prec, size, bops = l.split()
            want[(model, prec)] = (float(size), float(bops))
    for depth in (18, 50):
        t = inputs.resnet_table(depth, seed=depth, image_hw=224)
        for prec, force in (("w8a8", None), ("w4a4", 4)):
            cost = inputs.table_cost(t, force)
            size_mb, bops_g = cost["weight_bytes"] / 2 ** 20, cost["bops"] / 1e9
            w_size, w_bops = want[(f"resnet{depth}", prec)]
            assert abs(bops_g - w_bops) <= 1.0, (depth, prec, bops_g)   # printed as whole G
            assert abs(size_mb - w_size) <= 0.25, (depth, prec, size_mb)
    # the other stride placement does not reproduce the ResNet50 column
    alt = inputs.table_cost(inputs.resnet_table(50, seed=50, stride_on_3x3=True))
    assert abs(alt["bops"] / 1e9 - 247) > 5


# ---------------------------------------------------------------- P10: no float, no division ----
def test_oracle_source_has_no_float_and_no_division():
    src = open(oracle_build.SRC).read()
    code = re.sub(r"//[^\n]*", "", src)
    assert not re.search(r"\b(float|double|long double)\b", code)
    assert not re.search(r"[^/*]/[^/*]", code) and "%" not in code
    oracle_build.check_no_float_codegen()


def test_no_float_compile_pass_rejects_a_double(tmp_path):
    """The compile pass above is not vacuous: the same command refuses a translation unit that touches a
    floating-point register, and accepts the same function written with integers."""
    import subprocess
    bad = tmp_path / "uses_double.cpp"
    bad.write_text("extern \"C\" long long scale(long long x) { return (long long)((double)x * 0.5); }\n")
    with pytest.raises(subprocess.CalledProcessError):
        oracle_build.check_no_float_codegen(str(bad))
    good = tmp_path / "integers_only.cpp"
    good.write_text("extern \"C\" long long scale(long long x) { return x >> 1; }\n")
    oracle_build.check_no_float_codegen(str(good))


# ---------------------------------------------------------------- P11: fused == unfused ---------
def test_fused_conv_residual_equals_int32_conv_then_residual_add():
    case = inputs.conv_case(31, 2, 6, 6, 8, 8, 3, 1, 1, bits=8, residual=True, c_range=(39, 43))
    fused = hqref.conv_case(case)
    raw = dict(case)
    raw.update(out_bits=32, out_signed=1, res=None, qmin=-(1 << 31), qmax=(1 << 31) - 1)
    t = hqref.conv_case(raw)
    two_step = hqref.residual_add(t, 32, 1, case["b"], case["c"], case["res"], 8, 0, case["rb"], case["rc"],
                                  8, case["relu"], case["qmin"], case["qmax"], 8, 0)
    assert np.array_equal(fused, two_step)


def test_range_error_is_reported_not_wrapped():
    x = np.full((1, 1, 1, 4), 255, np.uint8)
    w = np.full((1, 1, 1, 4), 127, np.int8)
    bias = np.array([(1 << 31) - 1], np.int32)
    with pytest.raises(hqref.OracleError) as e:
        hqref.conv2d(x, 4, 8, 0, w, 1, 1, 1, 1, 0, bias, None, None, out_bits=32, out_signed=1,
                     qmin=-(1 << 31), qmax=(1 << 31) - 1)
    assert e.value.code == hqref.HQREF_ERR_RANGE


# ---------------------------------------------------------------- network walk ------------------
def hand_walk(table, images):
    """Every layer of a table applied by hand, without oracle.network: the operands are looked up from the
    table's own wiring (in0, in1, and the bits / sign the PRODUCING layer declares), the arithmetic is the
    independent formulations above (patch matrix + int64 product, exact rational rounding, exact mean, padded
    numpy maximum).  Returns the list of outputs as int64 arrays of logical (unpacked) values."""
    layers = table["layers"]
    vals = {-1: images.astype(np.int64)}

    def kind(i):                                   # (bits, signed) of tensor i as its producer states them
        return (8, 0) if i == -1 else (layers[i]["out_bits"], layers[i]["out_signed"])

    def dn_exact(x, b, c):
        return exact_round_half_up(int(x) * int(b), int(c))

    for li, l in enumerate(layers):
        op, x = l["op"], vals[l["in0"]]
        if op in ("conv", "linear"):
            bits_in, _ = kind(l["in0"])
            assert bits_in == l["bits"], "Section 3.4: weights and activations of a layer share the bit-width"
            wt = (inputs.unpack4(l["wgt"], True) if l["bits"] == 4 else l["wgt"]).astype(np.int64)
            if op == "linear":
                x = x.reshape(x.shape[0], 1, 1, -1)
            acc = im2col_conv(x, wt, l["stride"], l["pad"])
            if l["out_bits"] == 32:
                y = acc + l["bias"].astype(np.int64)
            else:
                res = vals[l["in1"]] if l["in1"] >= 0 else None
                y = epilogue_exact(acc, l["bias"], l["b"], l["c"], res, l["rb"], l["rc"], l["relu"], l["qmin"], l["qmax"])
        elif op == "maxpool":
            k, st, pad = l["pool_k"], l["pool_stride"], l["pool_pad"]
            lowest = -128 if kind(l["in0"])[1] else 0
            xp = np.pad(x, ((0, 0), (pad, pad), (pad, pad), (0, 0)), constant_values=lowest)
            ho, wo = (x.shape[1] + 2 * pad - k) // st + 1, (x.shape[2] + 2 * pad - k) // st + 1
            y = np.stack([np.stack([xp[:, oh * st:oh * st + k, ow * st:ow * st + k].max(axis=(1, 2))
                                    for ow in range(wo)], axis=1) for oh in range(ho)], axis=1)
        elif op == "avgpool":
            s = x.sum(axis=(1, 2))
            y = np.zeros((x.shape[0], 1, 1, x.shape[3]), np.int64)
            for n in range(x.shape[0]):
                for ch in range(x.shape[3]):
                    y[n, 0, 0, ch] = min(max(dn_exact(s[n, ch], l["b"][ch], l["c"][ch]), l["qmin"]), l["qmax"])
        elif op in ("requant", "add"):
            y = np.zeros(x.shape, np.int64)
            r = vals[l["in1"]] if l["in1"] >= 0 else None
            it = np.nditer(y, flags=["multi_index"])
            for _ in it:
                idx = it.multi_index
                ch = idx[-1]
                v = dn_exact(x[idx], l["b"][ch], l["c"][ch])
                if r is not None:
                    v += dn_exact(r[idx], l["rb"][ch], l["rc"][ch])
                if l["relu"]:
                    v = max(v, 0)
                y[idx] = min(max(v, l["qmin"]), l["qmax"])
        elif op == "sumpool":
            k, st, pad = l["pool_k"], l["pool_stride"], l["pool_pad"]
            xp = np.pad(x, ((0, 0), (pad, pad), (pad, pad), (0, 0)))
            ho, wo = (x.shape[1] + 2 * pad - k) // st + 1, (x.shape[2] + 2 * pad - k) // st + 1
            y = np.stack([np.stack([xp[:, oh * st:oh * st + k, ow * st:ow * st + k].sum(axis=(1, 2))
                                    for ow in range(wo)], axis=1) for oh in range(ho)], axis=1)
        elif op == "concat":
            parts = []
            for tid, b, c in zip(l["ins"], l["bs"], l["cs"]):
                src = vals[tid]
                part = np.zeros(src.shape, np.int64)
                it = np.nditer(part, flags=["multi_index"])
                for _ in it:
                    idx = it.multi_index
                    v = dn_exact(src[idx], b[idx[-1]], c[idx[-1]])
                    if l["relu"]:
                        v = max(v, 0)
                    part[idx] = min(max(v, l["qmin"]), l["qmax"])
                parts.append(part)
            y = np.concatenate(parts, axis=-1)
        else:
            raise AssertionError(op)
        vals[li] = y
    return [vals[i] for i in range(len(layers))]


def logical(y, layer):
    """An oracle output as int64 logical values (4-bit tensors unpacked)."""
    if layer["out_bits"] == 4:
        return inputs.unpack4(y, bool(layer["out_signed"])).astype(np.int64)
    return y.astype(np.int64)


def test_residual_add_with_int32_result_matches_exact_rational():
    """The add of Section 3.3 with its sum kept in INT32 (the wide residual stream of Fig. 2): a raw INT32 main branch
    with a pair per channel plus an INT32 or 8-bit second branch, every value against exact rational rounding."""
    g = np.random.default_rng(41)
    ch = 6
    main = g.integers(-(1 << 22), 1 << 22, size=(2, 3, 4, ch)).astype(np.int32)
    b, c = inputs.dyadic_from_scale(np.exp(g.uniform(np.log(2.0 ** -9), np.log(2.0 ** -5), ch)))
    for res_bits in (32, 8):
        res = (g.integers(0, 1 << 17, size=main.shape).astype(np.int32) if res_bits == 32
               else g.integers(0, 256, size=main.shape).astype(np.uint8))
        rb, rc = inputs.dyadic_from_scale(np.full(ch, 0.37 if res_bits == 32 else 181.0))
        y = hqref.residual_add(main, 32, 1, b, c, res, res_bits, int(res_bits == 32), rb, rc, ch, 1, 0, (1 << 31) - 1, 32, 1)
        assert y.dtype == np.int32
        for idx in np.ndindex(main.shape):
            k = idx[-1]
            want = exact_round_half_up(int(main[idx]) * int(b[k]), int(c[k])) + exact_round_half_up(int(res[idx]) * int(rb[k]), int(rc[k]))
            assert int(y[idx]) == max(want, 0), idx
    # the clamp applies to the wide result too
    y = hqref.residual_add(main, 32, 1, b, c, None, 0, 0, None, None, ch, 0, -100, 100, 32, 1)
    assert y.min() == -100 and y.max() == 100


@pytest.mark.parametrize("depth,mixed,hw,wide", [(18, False, 32, False), (18, True, 32, False), (50, True, 32, False),
                                                  (50, False, 32, False), (50, False, 32, True), (18, True, 32, True)])
def test_network_walk_equals_layers_applied_by_hand(depth, mixed, hw, wide):
    """EVERY layer of reduced ResNet-18 / ResNet-50 tables (uniform and mixed 4/8 bit): the oracle's walk against
    the hand-applied layers.  A wrong residual operand, a swapped bits / sign lookup for in0 and in1, or a slip
    in the requant / add / pooling / linear branches of the walk changes some layer here."""
    t = inputs.resnet_table(depth, seed=3 + depth, image_hw=hw, classes=10, width=8, mixed=mixed, int32_stream=wide)
    img = inputs.random_images(3, 2, hw)
    outs = run_network(t, img)
    want = hand_walk(t, img)
    seen = set()
    for i, (l, y, w) in enumerate(zip(t["layers"], outs, want)):
        assert np.array_equal(logical(y, l).reshape(w.shape), w), (i, l["op"])
        seen.add(l["op"])
        if l["op"] == "conv" and l["in1"] >= 0:
            seen.add("residual")
            if l["in1"] != i - 1:
                seen.add("residual from further back")
            if t["layers"][l["in1"]]["out_signed"] != t["layers"][l["in0"]]["out_signed"]:
                seen.add("operands of different sign")
    need = {"conv", "linear", "maxpool", "avgpool", "residual", "residual from further back", "operands of different sign"}
    if wide:              # Fig. 2 as drawn: INT32 stream, element-wise adds, one requantization per block input
        need = {"conv", "linear", "maxpool", "avgpool", "add", "requant"}
        assert sum(1 for l, y in zip(t["layers"], outs) if l["op"] == "add" and y.dtype == np.int32) == {18: 8, 50: 16}[depth]
    if mixed:
        need.add("requant")
    assert need <= seen, need - seen
    # outputs are not degenerate: the logits differ between the two images and between classes
    assert len(np.unique(outs[-1])) > 5
    assert outs[-1].dtype == np.int32 and outs[-1].shape == (2, 1, 1, 10)
    for i, l in enumerate(t["layers"]):
        if l["op"] == "conv" and l["bits"] == 4:
            assert t["bits"][l["in0"]] == 4
        h, w, c = t["shapes"][i]
        assert outs[i].shape[1:3] == (h, w)


@pytest.mark.parametrize("conv_bits", [4, 8])
def test_inception_walk_equals_layers_applied_by_hand(conv_bits):
    """A reduced table of Inception modules wired as Appendix E draws them (one requantization of the module input
    for the three convolution branches, INT32 window sums of the module input itself as the pooling branch, one DN per
    branch channel, concatenation): every layer of the oracle's walk against the hand-applied layers."""
    t = inputs.inception_table(9, conv_bits=conv_bits, image_hw=23, classes=7, width=8, modules35=1, modules17=1)
    img = inputs.random_images(5, 2, 23)
    outs = run_network(t, img)
    want = hand_walk(t, img)
    ops = [l["op"] for l in t["layers"]]
    assert ops.count("concat") == 2 and ops.count("sumpool") == 2 and ("requant" in ops) == (conv_bits == 4)
    for i, (l, y, w) in enumerate(zip(t["layers"], outs, want)):
        assert np.array_equal(logical(y, l).reshape(w.shape), w), (i, l["op"])
    for i, l in enumerate(t["layers"]):
        if l["op"] == "sumpool":
            assert outs[i].dtype == np.int32
        if l["op"] == "concat":
            pool = l["ins"][-1]
            assert t["layers"][pool]["op"] == "sumpool"                       # the pooling branch enters as INT32 sums
            src = t["layers"][pool]["in0"]
            assert t["layers"][src]["out_bits"] == 8                          # ... of the module input, not of the 4-bit copy
            mid = (outs[i] > 0) & (outs[i] < 255)
            assert mid.mean() > 0.05, "concatenation degenerate: everything saturates"


def test_maxpool_on_int32_matches_padded_numpy_max():
    g = np.random.default_rng(12)
    x = g.integers(-(1 << 30), 1 << 30, size=(2, 9, 10, 3)).astype(np.int32)
    y = hqref.maxpool(x, 3, 2, 1)
    xp = np.pad(x.astype(np.int64), ((0, 0), (1, 1), (1, 1), (0, 0)), constant_values=-(1 << 40))
    for oh in range(y.shape[1]):
        for ow in range(y.shape[2]):
            assert np.array_equal(y[:, oh, ow], xp[:, 2 * oh:2 * oh + 3, 2 * ow:2 * ow + 3].max(axis=(1, 2)))


def _tiny_network():
    import importlib.util
    spec = importlib.util.spec_from_file_location(
        "make_network_walk_golden", os.path.join(os.path.dirname(__file__), "golden", "make_network_walk_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_tiny_network_matches_stored_values_and_hand_walk(golden_dir):
    """A six-layer table typed in by hand (residual operand = layer 0, two layers back; a signed tensor feeding a
    conv and an add; average pool; INT32 logits): the oracle's walk equals the stored per-layer values AND the
    hand-applied layers."""
    mod = _tiny_network()
    table, img = mod.tiny_table(), mod.tiny_images()
    outs = run_network(table, img)
    stored = {}
    for line in open(os.path.join(golden_dir, "network_walk_tiny.txt")):
        if line.startswith("layer"):
            head, vals = line.split(":")
            stored[int(head.split()[1])] = np.array([int(v) for v in vals.split()], np.int64)
    want = hand_walk(table, img)
    assert len(stored) == len(outs) == 6
    for i, y in enumerate(outs):
        assert np.array_equal(y.astype(np.int64).ravel(), stored[i]), i
        assert np.array_equal(y.astype(np.int64).ravel(), want[i].ravel()), i
    # the residual really comes from layer 0: feeding layer 1 (the previous layer) instead changes layer 2
    wrong = mod.tiny_table()
    wrong["layers"][2]["in1"] = 1
    assert not np.array_equal(run_network(wrong, img)[2], outs[2])
    # first value of layer 2 by hand: acc = 2*(-9) - 16 + 0 + 3*14 = 8; (8 + 5) * 0.046875 = 0.61 -> 1; 0.7 * 22 = 15.4 -> 15
    assert int(outs[1].ravel()[0]) == -9 and int(outs[0].ravel()[0]) == 22 and int(outs[2].ravel()[0]) == 16
