"""The offline float -> integer parameter tool (Section 3.2 / Appendix D batch-norm fold, Appendix A quantizers,
INT32 bias at S_h S_w, DN for every edge): checked against the closed forms of the paper, against error bounds,
and end to end -- a small float network with batch norm and a residual block, quantized by the tool and run by the
integer-only oracle, tracks its own float evaluation."""
from __future__ import annotations

from fractions import Fraction

import numpy as np

from oracle.network import run_network
from paper_2011_10680_b200 import inputs, offline


def float_conv(x, w, stride, pad):
    """NHWC float convolution, one output element at a time (independent of the tool's own patch-matrix form)."""
    n, h, wd, ci = x.shape
    co, kh, kw, _ = w.shape
    ho, wo = (h + 2 * pad - kh) // stride + 1, (wd + 2 * pad - kw) // stride + 1
    out = np.zeros((n, ho, wo, co))
    for oh in range(ho):
        for ow in range(wo):
            for r in range(kh):
                for s in range(kw):
                    ih, iw = oh * stride + r - pad, ow * stride + s - pad
                    if 0 <= ih < h and 0 <= iw < wd:
                        out[:, oh, ow, :] += x[:, ih, iw, :] @ w[:, r, s, :].T
    return out


def test_bn_fold_is_the_closed_form_of_appendix_d():
    g = np.random.default_rng(1)
    x = g.normal(size=(2, 6, 7, 5))
    w = g.normal(size=(4, 3, 3, 5))
    beta, gamma = g.uniform(0.5, 2.0, 4), g.normal(size=4)          # the paper's symbols: beta scales, gamma shifts
    mu, sigma = g.normal(size=4), g.uniform(0.5, 2.0, 4)
    want = beta * (float_conv(x, w, 1, 1) - mu) / sigma + gamma      # conv followed by BN
    w_bar, b_bar = offline.fold_bn(w, beta, gamma, mu, sigma)
    got = float_conv(x, w_bar, 1, 1) + b_bar
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)
    # W_bar = beta W / sigma, b_bar = gamma - beta mu / sigma, element by element
    assert np.allclose(w_bar[2], beta[2] * w[2] / sigma[2]) and np.isclose(b_bar[1], gamma[1] - beta[1] * mu[1] / sigma[1])


def test_weight_quantizer_is_symmetric_channelwise_with_half_step_error():
    g = np.random.default_rng(2)
    w = g.normal(size=(6, 3, 3, 8)) * g.uniform(0.01, 3.0, size=(6, 1, 1, 1))
    for bits in (8, 4):
        q, s_w = offline.quantize_weights(w, bits)
        wmax = (1 << (bits - 1)) - 1
        assert q.min() >= -wmax and q.max() <= wmax
        assert np.all(np.abs(q).reshape(6, -1).max(axis=1) == wmax)              # every channel uses its full range
        assert np.allclose(s_w, np.abs(w).reshape(6, -1).max(axis=1) / wmax)     # S = max|r| / (2^(k-1) - 1), Z = 0
        assert np.all(np.abs(w - q * s_w[:, None, None, None]) <= s_w[:, None, None, None] / 2 + 1e-15)
    z, s = offline.quantize_weights(np.zeros((2, 1, 1, 4)), 8)                    # an all-zero channel stays zero
    assert not z.any() and np.all(s > 0)


def test_bias_is_int32_at_the_accumulators_scale():
    g = np.random.default_rng(3)
    b_bar, s_w, s_h = g.normal(size=16), g.uniform(1e-3, 1e-2, 16), 0.037
    qb = offline.quantize_bias(b_bar, s_h, s_w)
    assert qb.dtype == np.int32
    assert np.all(np.abs(b_bar - qb * s_h * s_w) <= s_h * s_w / 2 + 1e-15)        # S_b = S_h * S_w: adds to the accumulator


def test_layer_pairs_are_dn_of_the_scale_ratios():
    g = np.random.default_rng(4)
    w, b_bar = g.normal(size=(5, 1, 1, 8)), g.normal(size=5)
    pr = offline.conv_params(w, b_bar, s_in=0.05, s_out=0.11, bits=8, s_res=0.07)
    for oc in range(5):
        want = Fraction(float(pr["s_w"][oc])) * Fraction(0.05) / Fraction(0.11)
        err = abs(Fraction(int(pr["b"][oc]), 1 << int(pr["c"][oc])) - want)
        assert err <= Fraction(1, 1 << int(pr["c"][oc])), oc                     # DN(S_w S_h / S_a) within 2^-c
        assert 1 << 30 <= int(pr["b"][oc]) < 1 << 31
    err = abs(Fraction(int(pr["rb"][0]), 1 << int(pr["rc"][0])) - Fraction(0.07) / Fraction(0.11))
    assert err <= Fraction(1, 1 << int(pr["rc"][0]))                              # DN(S_r / S_a)
    assert inputs.dyadic_from_scale is offline.dyadic_from_scale                  # one DN for generators and tool


def small_float_network(seed=5, n=4, hw=12, c0=3, c1=8, classes=10):
    """conv + BN + ReLU, a residual block of two convs (the add takes the block input), average pool, classifier."""
    g = np.random.default_rng(seed)
    img_q = g.integers(0, 256, size=(n, hw, hw, c0)).astype(np.uint8)

    def bn(ch):
        return (g.uniform(0.8, 1.2, ch), g.normal(0, 0.1, ch), g.normal(0, 0.1, ch), g.uniform(0.8, 1.2, ch))

    layers = [
        dict(op="conv", in0=-1, in1=-1, w=g.normal(size=(c1, 3, 3, c0)) * 0.4, bn=bn(c1), stride=1, pad=1, bits=8, relu=True),
        dict(op="conv", in0=0, in1=-1, w=g.normal(size=(c1, 3, 3, c1)) * 0.15, bn=bn(c1), stride=1, pad=1, bits=8, relu=True),
        dict(op="conv", in0=1, in1=0, w=g.normal(size=(c1, 3, 3, c1)) * 0.15, bn=bn(c1), stride=1, pad=1, bits=8, relu=True),
        dict(op="avgpool", in0=2, hw=hw * hw, channels=c1),
        dict(op="linear", in0=3, in1=-1, w=g.normal(size=(classes, 1, 1, c1)) * 0.3, bn=None, bias=np.full(classes, 0.25),
             bits=8, relu=False, s_out=None),
    ]
    return layers, img_q


def test_quantized_network_tracks_its_float_evaluation():
    """Float network -> calibrate -> quantize_network -> the oracle's integer-only walk.  Activation scales come from
    a static calibration on the float activations, as in the paper; the de-quantized integer activations must stay
    close to the float ones at every layer (8 bit), and the classifier must pick the same classes."""
    layers, img_q = small_float_network()
    n = img_q.shape[0]
    s_img = 1.0 / 255.0
    floats = offline.float_forward(layers, img_q * s_img)
    net = offline.quantize_network(offline.calibrate(layers, img_q * s_img), s_img, image_hw=img_q.shape[1])
    outs = run_network(net, img_q)
    for i in range(4):
        deq = outs[i].astype(np.float64) * net["scales"][i]
        rel = np.linalg.norm(deq - floats[i]) / np.linalg.norm(floats[i])
        assert rel < 0.03, (i, rel)                                               # 8-bit: a few per cent at most
    _, s_w4 = offline.quantize_weights(layers[4]["w"], 8)
    logits = outs[4].reshape(n, -1) * (net["scales"][3] * s_w4)                  # INT32 logits at scale S_h * S_w[oc]
    f4 = floats[4].reshape(n, -1)
    assert np.linalg.norm(logits - f4) / np.linalg.norm(f4) < 0.05
    assert np.array_equal(np.argmax(logits, axis=1), np.argmax(f4, axis=1))
    # the residual operand of layer 2 is the block input (layer 0), with its own DN(S_r / S_a)
    assert net["layers"][2]["in1"] == 0 and net["layers"][2]["rb"] is not None


def test_input_zero_point_folds_into_the_bias_exactly():
    """Eq. 2's zero point on the network input: conv(q_x - Z) with bias equals conv(q_x) with the folded bias,
    integer for integer (unpadded layer), checked through the oracle's convolution; a padded layer is refused."""
    import pytest
    from oracle import hqref
    g = np.random.default_rng(7)
    n, hw, cin, cout, k, z = 2, 9, 3, 6, 3, 117
    qx = g.integers(0, 256, size=(n, hw, hw, cin)).astype(np.uint8)
    qw = g.integers(-127, 128, size=(cout, k, k, cin)).astype(np.int8)
    qb = g.integers(-(1 << 15), 1 << 15, size=cout).astype(np.int32)
    folded = offline.fold_input_zero_point(qb, qw, z)
    got = hqref.conv2d(qx, cin, 8, 0, qw, cout, k, k, 1, 0, folded, None, None, out_bits=32, out_signed=1,
                       qmin=-(1 << 31), qmax=(1 << 31) - 1)
    want = float_conv(qx.astype(np.float64) - z, qw.astype(np.float64), 1, 0) + qb         # exact in doubles at these sizes
    assert np.array_equal(got.astype(np.int64), want.astype(np.int64))
    with pytest.raises(ValueError):
        offline.fold_input_zero_point(qb, qw, z, pad=1)
    # Z = 128 on 8-bit data is the signed image: same real values, no fold needed
    signed = (qx.astype(np.int16) - 128).astype(np.int8)
    a = hqref.conv2d(signed, cin, 8, 1, qw, cout, k, k, 1, 1, qb, None, None, out_bits=32, out_signed=1,
                     qmin=-(1 << 31), qmax=(1 << 31) - 1)
    b = float_conv(qx.astype(np.float64) - 128, qw.astype(np.float64), 1, 1) + qb
    assert np.array_equal(a.astype(np.int64), b.astype(np.int64))
