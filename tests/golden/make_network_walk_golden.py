#!/usr/bin/env python
"""Writes tests/golden/network_walk_tiny.txt: every layer output of a six-layer hand-written table.

The table is small enough to read: a 1x1 conv on a 1x4x4x3 image, a signed 3x3 conv, a 1x1 conv whose
residual operand is layer 0 (NOT the layer before it: Fig. 2's shortcut skips the block body), an
element-wise add of two stored tensors (Section 3.3), the divisionless average pool (Appendix E) and a
linear layer with raw INT32 output.  All parameters are typed in below; nothing is drawn at random.

This script calls only the oracle (`oracle/`).  The stored values are a second pin beside the
hand-applied walk in tests/test_oracle_pins.py, which recomputes the same layers with exact integers.

    python tests/golden/make_network_walk_golden.py            # rewrites the file
"""
from __future__ import annotations

import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

OUT = os.path.join(HERE, "network_walk_tiny.txt")


def tiny_images() -> np.ndarray:
    """1 x 4 x 4 x 3 uint8: pixel (h, w), channel k holds (37 h + 11 w + 5 k + 3) * 3 mod 256."""
    h, w, k = np.meshgrid(np.arange(4), np.arange(4), np.arange(3), indexing="ij")
    return (((37 * h + 11 * w + 5 * k + 3) * 3) % 256).astype(np.uint8)[None]


def _pairs(num, shift):
    """Dyadic pairs b / 2^c given as (b, c) per channel, b in [2^30, 2^31)."""
    return np.array(num, np.int32), np.array(shift, np.int32)


def tiny_table() -> dict:
    i8 = np.int8
    # layer 0: 1x1 conv 3 -> 4, ReLU, uint8 out
    w0 = np.array([[1, -2, 3], [4, 0, -1], [-3, 2, 2], [0, 5, -4]], i8).reshape(4, 1, 1, 3)
    b0, c0 = _pairs([1 << 30, 1288490189, 1717986918, 1932735283], [32, 33, 33, 34])
    l0 = dict(op="conv", in0=-1, in1=-1, kh=1, kw=1, stride=1, pad=0, cin=3, cout=4, bits=8, wgt=w0,
              bias=np.array([10, -20, 300, 7], np.int32), b=b0, c=c0, rb=None, rc=None, relu=1, qmin=0, qmax=255,
              out_bits=8, out_signed=0)
    # layer 1: 3x3 conv 4 -> 4, pad 1, no ReLU, signed 8-bit out
    k = np.arange(4 * 3 * 3 * 4).reshape(4, 3, 3, 4)
    w1 = ((k * 7 + 3) % 11 - 5).astype(i8)
    b1, c1 = _pairs([1503238554, 1181116006, 2040109466, 1395864371], [35, 34, 36, 35])
    l1 = dict(op="conv", in0=0, in1=-1, kh=3, kw=3, stride=1, pad=1, cin=4, cout=4, bits=8, wgt=w1,
              bias=np.array([-400, 250, 0, 1000], np.int32), b=b1, c=c1, rb=None, rc=None, relu=0, qmin=-128,
              qmax=127, out_bits=8, out_signed=1)
    # layer 2: 1x1 conv 4 -> 4 on the SIGNED tensor 1, residual = tensor 0 (unsigned), ReLU
    w2 = np.array([[2, -1, 0, 3], [-2, 2, 1, 0], [1, 1, -3, 2], [0, -4, 2, 1]], i8).reshape(4, 1, 1, 4)
    b2, c2 = _pairs([1610612736, 1342177280, 1879048192, 1207959552], [35, 34, 36, 35])
    rb2, rc2 = _pairs([1503238554] * 4, [31] * 4)                  # 0.7 per channel
    l2 = dict(op="conv", in0=1, in1=0, kh=1, kw=1, stride=1, pad=0, cin=4, cout=4, bits=8, wgt=w2,
              bias=np.array([5, -5, 50, -50], np.int32), b=b2, c=c2, rb=rb2, rc=rc2, relu=1, qmin=0, qmax=255,
              out_bits=8, out_signed=0)
    # layer 3: stored tensors 2 (by 0.6) + 1 (signed, by 1.25), ReLU: the add of Section 3.3 on its own
    b3, c3 = _pairs([1288490189] * 4, [31] * 4)
    rb3, rc3 = _pairs([1342177280] * 4, [30] * 4)
    l3 = dict(op="add", in0=2, in1=1, cout=4, b=b3, c=c3, rb=rb3, rc=rc3, relu=1, qmin=0, qmax=255,
              out_bits=8, out_signed=0)
    # layer 4: average over the 16 pixels with 1/16 inside the pair (no division)
    b4, c4 = _pairs([1 << 30] * 4, [34] * 4)
    l4 = dict(op="avgpool", in0=3, in1=-1, cout=4, b=b4, c=c4, rb=None, rc=None, relu=0, qmin=0, qmax=255,
              out_bits=8, out_signed=0)
    # layer 5: linear 4 -> 3, raw INT32
    w5 = np.array([[3, -1, 2, 0], [-2, 4, 0, 1], [1, 1, 1, -5]], i8).reshape(3, 1, 1, 4)
    l5 = dict(op="linear", in0=4, in1=-1, kh=1, kw=1, stride=1, pad=0, cin=4, cout=3, bits=8, wgt=w5,
              bias=np.array([100, -100, 0], np.int32), b=None, c=None, rb=None, rc=None, relu=0,
              qmin=-(1 << 31), qmax=(1 << 31) - 1, out_bits=32, out_signed=1)
    return dict(layers=[l0, l1, l2, l3, l4, l5], image_hw=4, classes=3)


def main() -> None:
    from oracle.network import run_network
    outs = run_network(tiny_table(), tiny_images())
    with open(OUT, "w") as f:
        f.write("# Outputs of every layer of the six-layer table in make_network_walk_golden.py, image tiny_images().\n")
        f.write("# Written by that script, which calls only the oracle; row = `layer i: values in NHWC order`.\n")
        f.write("# Dataflow after Fig. 2 (fused form), Section 3.3 (two roundings, then add), Appendix E (pooling).\n")
        for i, y in enumerate(outs):
            f.write(f"layer {i}: " + " ".join(str(int(v)) for v in y.ravel()) + "\n")
    print("wrote", OUT)


if __name__ == "__main__":
    main()
