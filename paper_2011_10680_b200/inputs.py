"""Seeded synthetic workloads for the integer-only inference path of HAWQ-V3.

This module only *draws inputs*: tensors, weights, INT32 biases, dyadic pairs and the layer
tables of ResNet-shaped networks.  It contains none of the inference arithmetic (no convolution,
no requantization, no pooling), and it imports neither the CUDA binding nor the CPU oracle; both
consume what it produces, so generator details can never create a parity difference.

Value ranges follow the paper's quantizers (Section 3 "Uniform Quantization", Appendix A/B):
weights symmetric in [-(2^(k-1)-1), 2^(k-1)-1] per output channel, post-ReLU activations unsigned in
[0, 2^k-1] with zero point 0, bias in INT32 at scale S_h*S_w (Appendix D), every rescaling a
dyadic number b/2^c (Eq. 4 and the DN(.) definition).  Real-valued scales appear only here,
offline, exactly as in the paper, where DN(.) is evaluated once from statically known scales
(Section 3.3); the integer pipeline itself never sees them.
"""
from __future__ import annotations

import numpy as np

from .offline import dyadic_from_scale, quantize_weights   # DN(.) and the weight quantizer belong to the offline tool

__all__ = [
    "rng", "dyadic_from_scale", "pack4", "unpack4", "conv_case", "config1_case",
    "resnet_table", "inception_table", "table_cost", "out_hw", "SWEEP_LAYERS",
]


def rng(seed: int, *stream: int) -> np.random.Generator:
    """Counter-based generator keyed by (seed, stream ids): the same key gives the same numbers."""
    return np.random.Generator(np.random.Philox(key=np.random.SeedSequence([seed, *stream]).generate_state(2, np.uint64)))


# --------------------------------------------------------------------------------------------
# 4-bit packing (two per byte along the channel axis, even element in the low nibble)
# --------------------------------------------------------------------------------------------
def pack4(a: np.ndarray) -> np.ndarray:
    """Pack integers in [-8, 15] (last axis even) into bytes, element 2j -> bits 3:0 of byte j."""
    a = np.asarray(a)
    if a.shape[-1] % 2:
        raise ValueError("last axis must be even to pack 4-bit values")
    u = (a.astype(np.int16) & 0xF).astype(np.uint8)
    return (u[..., 0::2] | (u[..., 1::2] << 4)).astype(np.uint8)


def unpack4(p: np.ndarray, signed: bool) -> np.ndarray:
    """Inverse of pack4, returning int8 (signed) or uint8 values."""
    p = np.asarray(p, dtype=np.uint8)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), dtype=np.int16)
    out[..., 0::2] = p & 0xF
    out[..., 1::2] = p >> 4
    if signed:
        out = np.where(out >= 8, out - 16, out)
        return out.astype(np.int8)
    return out.astype(np.uint8)


def out_hw(h: int, w: int, k: int, stride: int, pad: int) -> tuple[int, int]:
    return (h + 2 * pad - k) // stride + 1, (w + 2 * pad - k) // stride + 1


# --------------------------------------------------------------------------------------------
# Single-layer cases (configs 1 and 5)
# --------------------------------------------------------------------------------------------
def conv_case(seed: int, n: int, h: int, w: int, cin: int, cout: int, k: int, stride: int = 1,
              pad: int = 0, bits: int = 8, out_bits: int = 8, residual: bool = False,
              res_bits: int = 8, relu: bool = True, in_signed: bool = False,
              c_range: tuple[int, int] = (36, 44), out_signed: bool | None = None) -> dict:
    """One fused conv layer with the value distributions of the single-layer benchmark config.

    Activations uniform over the full unsigned (or signed) range, weights uniform symmetric,
    bias uniform in [-2^15, 2^15], b uniform in [2^30, 2^31), c uniform in c_range, residual rescale
    (when asked for) with c in [28, 34] so that both roundings and both signs of `c - 32` occur.
    4-bit tensors are returned packed (last axis halved); `*_bits` say how to read them.
    """
    g = rng(seed, n, h, w, cin, cout, k, stride, pad, bits)
    amax = (1 << bits) - 1
    if in_signed:
        x = g.integers(-(1 << (bits - 1)), 1 << (bits - 1), size=(n, h, w, cin), dtype=np.int64)
    else:
        x = g.integers(0, amax + 1, size=(n, h, w, cin), dtype=np.int64)
    wmax = (1 << (bits - 1)) - 1
    wt = g.integers(-wmax, wmax + 1, size=(cout, k, k, cin), dtype=np.int64)
    bias = g.integers(-(1 << 15), (1 << 15) + 1, size=cout, dtype=np.int64).astype(np.int32)
    b = g.integers(1 << 30, 1 << 31, size=cout, dtype=np.int64).astype(np.int32)
    if bits == 4:
        # 4-bit accumulators are ~2^9 times smaller; keep a comparable spread of outputs
        c_lo, c_hi = c_range[0] - 8, c_range[1] - 8
    else:
        c_lo, c_hi = c_range
    c = g.integers(c_lo, c_hi + 1, size=cout, dtype=np.int64).astype(np.int32)
    ho, wo = out_hw(h, w, k, stride, pad)
    if out_signed is None:
        out_signed = not relu
    if out_bits == 32:
        qmin, qmax, out_signed = -(1 << 31), (1 << 31) - 1, True
    elif out_signed:
        qmin, qmax = -(1 << (out_bits - 1)), (1 << (out_bits - 1)) - 1
    else:
        qmin, qmax = 0, (1 << out_bits) - 1
    case = dict(
        n=n, h=h, w=w, cin=cin, cout=cout, kh=k, kw=k, stride=stride, pad=pad, bits=bits,
        in_signed=int(in_signed), ho=ho, wo=wo,
        x=(pack4(x) if bits == 4 else x.astype(np.int8 if in_signed else np.uint8)),
        wgt=(pack4(wt) if bits == 4 else wt.astype(np.int8)),
        bias=bias, b=b, c=c, relu=int(relu), qmin=qmin, qmax=qmax,
        out_bits=out_bits, out_signed=int(out_signed),
        res=None, res_bits=0, res_signed=0, rb=None, rc=None,
    )
    if residual:
        if res_bits == 32:
            r = g.integers(-(1 << 20), 1 << 20, size=(n, ho, wo, cout), dtype=np.int64).astype(np.int32)
            rc = g.integers(40, 47, size=cout, dtype=np.int64).astype(np.int32)
            case["res_signed"] = 1
        else:
            r = g.integers(0, 256, size=(n, ho, wo, cout), dtype=np.int64).astype(np.uint8)
            rc = g.integers(28, 35, size=cout, dtype=np.int64).astype(np.int32)
        case.update(res=r, res_bits=res_bits,
                    rb=g.integers(1 << 30, 1 << 31, size=cout, dtype=np.int64).astype(np.int32), rc=rc)
    return case


def config1_case() -> dict:
    """Benchmark config 1: batch 1, 56x56x64 -> 64, 3x3, stride 1, pad 1, seed 0, c in [36, 44]."""
    return conv_case(0, 1, 56, 56, 64, 64, 3, stride=1, pad=1, bits=8, relu=True)


# ResNet-50 layer shapes used by the conv/GEMM sweep (H=W, Cin, Cout, k, stride, has residual)
SWEEP_LAYERS = [
    (56, 64, 64, 1, 1, False), (56, 64, 64, 3, 1, False), (56, 64, 256, 1, 1, True),
    (56, 256, 64, 1, 1, False), (28, 128, 128, 3, 1, False), (28, 128, 512, 1, 1, True),
    (28, 512, 128, 1, 1, False), (14, 256, 256, 3, 1, False), (14, 256, 1024, 1, 1, True),
    (14, 1024, 256, 1, 1, False), (7, 512, 512, 3, 1, False), (7, 512, 2048, 1, 1, True),
    (7, 2048, 512, 1, 1, False),
]


# --------------------------------------------------------------------------------------------
# Network tables (configs 2-4)
# --------------------------------------------------------------------------------------------
def _draw_scale(g: np.random.Generator) -> float:
    """Activation scale, log-uniform in [2^-6, 2^-2): octave uniform in {-6..-3}, mantissa in [1,2)."""
    e = int(g.integers(-6, -2))
    return float(2.0 ** e * (1.0 + g.random()))


def _draw_weights(g: np.random.Generator, cout: int, k: int, cin: int, bits: int):
    """Real weights N(0, sqrt(2/fan_in)) quantized symmetrically per output channel (Appendix A)."""
    fan_in = k * k * cin
    wr = g.standard_normal(size=(cout, k, k, cin)) * np.sqrt(2.0 / fan_in)
    return quantize_weights(wr, bits)


class _Builder:
    def __init__(self, seed: int):
        self.g = rng(seed, 7)
        self.layers: list[dict] = []
        self.scale: dict[int, float] = {}
        self.chscale: dict[int, np.ndarray] = {}           # raw INT32 conv outputs: scale per channel, S_h * S_w[oc]
        self.shape: dict[int, tuple[int, int, int]] = {}   # h, w, c of each tensor id
        self.bits: dict[int, int] = {}

    def _emit(self, layer: dict, scale: float, hwc, bits: int) -> int:
        self.layers.append(layer)
        tid = len(self.layers) - 1
        self.scale[tid], self.shape[tid], self.bits[tid] = scale, hwc, bits
        return tid

    def conv(self, src: int, cout: int, k: int, stride: int, pad: int, bits: int, *, relu: bool,
             out_bits: int, out_signed: bool = False, res: int = -1, op: str = "conv", unit: int = -1) -> int:
        g = self.g
        h, w, cin = self.shape[src]
        assert self.bits[src] == bits, "conv input must already have the conv's bit-width"
        q, s_w = _draw_weights(g, cout, k, cin, bits)
        bias = g.integers(-(1 << 15), (1 << 15) + 1, size=cout, dtype=np.int64).astype(np.int32)
        ho, wo = out_hw(h, w, k, stride, pad)
        s_in = self.scale[src]
        layer = dict(op=op, in0=src, in1=res, kh=k, kw=k, stride=stride, pad=pad, cin=cin, cout=cout,
                     bits=bits, wgt=(pack4(q) if bits == 4 else q.astype(np.int8)), bias=bias,
                     relu=int(relu), out_bits=out_bits, out_signed=int(out_signed),
                     b=None, c=None, rb=None, rc=None, qmin=0, qmax=0,
                     macs=ho * wo * cout * k * k * cin, params=cout * k * k * cin, unit=unit)
        if out_bits == 32:                      # raw INT32 accumulator + bias (logits; main branch of an INT32 add)
            layer.update(qmin=-(1 << 31), qmax=(1 << 31) - 1, out_signed=1)
            tid = self._emit(layer, s_in * float(s_w.mean()), (ho, wo, cout), 32)
            self.chscale[tid] = s_in * s_w
            return tid
        s_out = _draw_scale(g)
        layer["b"], layer["c"] = dyadic_from_scale(s_w * s_in / s_out)
        if res >= 0:
            rb, rc = dyadic_from_scale(self.scale[res] / s_out)
            layer["rb"] = np.full(cout, rb[0], np.int32)
            layer["rc"] = np.full(cout, rc[0], np.int32)
        if out_signed:
            layer.update(qmin=-(1 << (out_bits - 1)), qmax=(1 << (out_bits - 1)) - 1)
        else:
            layer.update(qmin=0, qmax=(1 << out_bits) - 1)
        return self._emit(layer, s_out, (ho, wo, cout), out_bits)

    def add32(self, main: int, res: int, s_out: float, unit: int = -1) -> int:
        """The residual add of Section 3.3 / Fig. 2 on stored tensors with an INT32 result: both branches rescaled by
        their own dyadic pairs to s_out (per channel where a branch is a raw accumulator), rounded, added, ReLU."""
        h, w, c = self.shape[main]
        sm = self.chscale.get(main, np.full(c, self.scale[main]))
        sr = self.chscale.get(res, np.full(c, self.scale[res]))
        b, cc = dyadic_from_scale(sm / s_out)
        rb, rc = dyadic_from_scale(sr / s_out)
        layer = dict(op="add", in0=main, in1=res, cout=c, b=b, c=cc, rb=rb, rc=rc, relu=1, qmin=0, qmax=(1 << 31) - 1,
                     out_bits=32, out_signed=1, macs=0, params=0, unit=unit)
        return self._emit(layer, s_out, (h, w, c), 32)

    def requant(self, src: int, out_bits: int, unit: int = -1) -> int:
        """Unsigned stream tensor -> lower-bit unsigned copy (Fig. 2: quantize the input once)."""
        h, w, c = self.shape[src]
        s_out = _draw_scale(self.g) * (255.0 / 15.0 if out_bits == 4 else 1.0)
        b, cc = dyadic_from_scale(self.scale[src] / s_out)
        layer = dict(op="requant", in0=src, in1=-1, cout=c, b=np.full(c, b[0], np.int32),
                     c=np.full(c, cc[0], np.int32), rb=None, rc=None, relu=0, qmin=0,
                     qmax=(1 << out_bits) - 1, out_bits=out_bits, out_signed=0, macs=0, params=0, unit=unit)
        return self._emit(layer, s_out, (h, w, c), out_bits)

    def maxpool(self, src: int, k: int, stride: int, pad: int) -> int:
        h, w, c = self.shape[src]
        ho, wo = out_hw(h, w, k, stride, pad)
        layer = dict(op="maxpool", in0=src, in1=-1, pool_k=k, pool_stride=stride, pool_pad=pad, cout=c,
                     out_bits=8, out_signed=0, relu=0, qmin=0, qmax=255, macs=0, params=0)
        return self._emit(layer, self.scale[src], (ho, wo, c), 8)

    def sumpool(self, src: int, k: int, stride: int, pad: int) -> int:
        """k x k window sums in INT32 (Appendix E pools on the wide feature map); the tensor's scale carries the 1 / k^2 of
        the average, so that the consumer's dyadic pair turns the sum into the mean without a division."""
        h, w, c = self.shape[src]
        ho, wo = out_hw(h, w, k, stride, pad)
        layer = dict(op="sumpool", in0=src, in1=-1, pool_k=k, pool_stride=stride, pool_pad=pad, cout=c, out_bits=32,
                     out_signed=1, relu=0, qmin=-(1 << 31), qmax=(1 << 31) - 1, macs=0, params=0)
        return self._emit(layer, self.scale[src] / (k * k), (ho, wo, c), 32)

    def concat(self, srcs: list[int], out_bits: int = 8) -> int:
        """Concatenation along the channels with one dyadic pair per branch channel, DN(S_i / S_a) (Appendix E)."""
        h, w, _ = self.shape[srcs[0]]
        s_out = _draw_scale(self.g) * (255.0 / 15.0 if out_bits == 4 else 1.0)
        bs, cs = [], []
        for t in srcs:
            c = self.shape[t][2]
            b, cc = dyadic_from_scale(self.chscale.get(t, np.full(c, self.scale[t])) / s_out)
            bs.append(b); cs.append(cc)
        total = sum(self.shape[t][2] for t in srcs)
        layer = dict(op="concat", in0=srcs[0], in1=-1, ins=list(srcs), bs=bs, cs=cs, cout=total, relu=1, qmin=0,
                     qmax=(1 << out_bits) - 1, out_bits=out_bits, out_signed=0, macs=0, params=0)
        return self._emit(layer, s_out, (h, w, total), out_bits)

    def avgpool(self, src: int) -> int:
        h, w, c = self.shape[src]
        s_out = _draw_scale(self.g)
        b, cc = dyadic_from_scale(self.scale[src] / (h * w * s_out))   # 1/(h*w) folded in: no division
        layer = dict(op="avgpool", in0=src, in1=-1, cout=c, b=np.full(c, b[0], np.int32),
                     c=np.full(c, cc[0], np.int32), out_bits=8, out_signed=0, relu=0, qmin=0, qmax=255,
                     macs=0, params=0)
        return self._emit(layer, s_out, (1, 1, c), 8)


def resnet_choice_units(depth: int) -> int:
    """Number of per-layer bit-width choices of a ResNet table: the convs of the residual blocks, a
    down-sampling shortcut conv being tied to the block's first conv (they share one quantized input)."""
    return {18: 16, 50: 48}[depth]


def resnet_table(depth: int, seed: int, *, mixed: bool = False, stride_on_3x3: bool = False,
                 image_hw: int = 224, classes: int = 1000, width: int = 64,
                 conv_bits: list[int] | None = None, int32_stream: bool = False) -> dict:
    """Layer table of an ImageNet-shaped ResNet-18 or ResNet-50 with integer parameters.

    Tensor id -1 is the uint8 input image (n, image_hw, image_hw, 3); layer i produces tensor i.
    Dataflow (Fig. 2, fused form): every block output is stored as a uint8 stream tensor; the last
    conv of a block carries the residual add in its epilogue (both branches dyadically rescaled,
    each rounded, then added); a down-sampling shortcut is a 1x1 conv whose signed 8-bit output
    is the residual operand.  With mixed=True the convs of the last two stages run at 4 bit: the
    block input is requantized once to uint4 and shared by conv1 and the shortcut conv, and
    convs inside the block write uint4 directly.  First conv and classifier stay 8-bit
    (Appendix H).  ResNet-50 puts the stride on the first 1x1 of a down-sampling bottleneck unless
    stride_on_3x3 is set; only that placement reproduces the paper's BOPS column (Table 1b).
    conv_bits gives the bit-width (4 or 8) of every block conv in network order instead
    (resnet_choice_units(depth) entries, e.g. the answer of the bit-width ILP of Section 3.4): a conv
    writes its output at the bit-width of the conv that reads it, and a block whose first conv is
    4-bit requantizes the stream tensor once for that conv and the shortcut conv.
    int32_stream=True lays the table out as the paper draws Fig. 2: the residual stream between blocks is an INT32
    tensor (at 1/256 of an 8-bit activation scale), every block requantizes it once to the bit-width of its first
    conv, the block's last conv and a down-sampling shortcut conv return their raw INT32 accumulators, and an
    element-wise add rescales both branches with their own dyadic pairs, adds them in INT32 and applies the ReLU.
    """
    if depth not in (18, 50):
        raise ValueError("depth must be 18 or 50")
    bd = _Builder(seed)
    bd.scale[-1], bd.shape[-1], bd.bits[-1] = _draw_scale(bd.g), (image_hw, image_hw, 3), 8
    x = bd.conv(-1, width, 7, 2, 3, 8, relu=True, out_bits=8)
    x = bd.maxpool(x, 3, 2, 1)
    blocks = [2, 2, 2, 2] if depth == 18 else [3, 4, 6, 3]
    expansion = 1 if depth == 18 else 4
    per_block = 2 if depth == 18 else 3
    if conv_bits is None:
        conv_bits = [4 if (mixed and stage >= 2) else 8 for stage, nblk in enumerate(blocks)
                     for _ in range(nblk * per_block)]
    if len(conv_bits) != sum(blocks) * per_block or any(b not in (4, 8) for b in conv_bits):
        raise ValueError("conv_bits needs one entry (4 or 8) per block conv")
    unit = 0
    for stage, nblk in enumerate(blocks):
        planes = width << stage
        for blk in range(nblk):
            stride = 2 if (blk == 0 and stage > 0) else 1
            cin = bd.shape[x][2]
            need_ds = stride != 1 or cin != planes * expansion
            wb = conv_bits[unit:unit + per_block]
            u0 = unit                             # layers carry the index of the choice they belong to
            unit += per_block
            if int32_stream:
                # Fig. 2 as drawn: wide stream, one requantization per block input, raw accumulators into an INT32 add
                xin = bd.requant(x, wb[0], unit=u0) if (bd.bits[x] == 32 or wb[0] == 4) else x
                if depth == 18:
                    y = bd.conv(xin, planes, 3, stride, 1, wb[0], relu=True, out_bits=wb[1], unit=u0)
                    main = bd.conv(y, planes, 3, 1, 1, wb[1], relu=False, out_bits=32, unit=u0 + 1)
                    shortcut = bd.conv(xin, planes, 1, stride, 0, wb[0], relu=False, out_bits=32, unit=u0) if need_ds else x
                else:
                    s1, s2 = (1, stride) if stride_on_3x3 else (stride, 1)
                    y = bd.conv(xin, planes, 1, s1, 0, wb[0], relu=True, out_bits=wb[1], unit=u0)
                    y = bd.conv(y, planes, 3, s2, 1, wb[1], relu=True, out_bits=wb[2], unit=u0 + 1)
                    main = bd.conv(y, planes * 4, 1, 1, 0, wb[2], relu=False, out_bits=32, unit=u0 + 2)
                    shortcut = bd.conv(xin, planes * 4, 1, stride, 0, wb[0], relu=False, out_bits=32, unit=u0) if need_ds else x
                x = bd.add32(main, shortcut, _draw_scale(bd.g) / 256.0, unit=u0 + per_block - 1)
                continue
            xin = bd.requant(x, 4, unit=u0) if wb[0] == 4 else x
            if depth == 18:
                y = bd.conv(xin, planes, 3, stride, 1, wb[0], relu=True, out_bits=wb[1], unit=u0)
                shortcut = bd.conv(xin, planes, 1, stride, 0, wb[0], relu=False, out_bits=8,
                                   out_signed=True, unit=u0) if need_ds else x
                x = bd.conv(y, planes, 3, 1, 1, wb[1], relu=True, out_bits=8, res=shortcut, unit=u0 + 1)
            else:
                s1, s2 = (1, stride) if stride_on_3x3 else (stride, 1)
                y = bd.conv(xin, planes, 1, s1, 0, wb[0], relu=True, out_bits=wb[1], unit=u0)
                y = bd.conv(y, planes, 3, s2, 1, wb[1], relu=True, out_bits=wb[2], unit=u0 + 1)
                shortcut = bd.conv(xin, planes * 4, 1, stride, 0, wb[0], relu=False, out_bits=8,
                                   out_signed=True, unit=u0) if need_ds else x
                x = bd.conv(y, planes * 4, 1, 1, 0, wb[2], relu=True, out_bits=8, res=shortcut, unit=u0 + 2)
    x = bd.avgpool(x)
    x = bd.conv(x, classes, 1, 1, 0, 8, relu=False, out_bits=32, op="linear")
    return dict(layers=bd.layers, image_hw=image_hw, classes=classes, depth=depth, conv_bits=list(conv_bits),
                shapes=[bd.shape[i] for i in range(len(bd.layers))],
                bits=[bd.bits[i] for i in range(len(bd.layers))])


def inception_table(seed: int, *, conv_bits: int = 4, image_hw: int = 71, classes: int = 1000, width: int = 64,
                    modules35: int = 2, modules17: int = 2) -> dict:
    """Layer table shaped like InceptionV3's 35x35 and 17x17 modules, wired as the paper's Appendix E draws an
    Inception module: the module input is requantized once (to conv_bits, 4 in the figure) for the three convolution
    branches -- 1x1; 1x1 -> 5x5 (3x3 in the 17x17 modules); 1x1 -> 3x3 -> 3x3 -- while the pooling branch works on the
    module input itself in INT32 (3x3 window sums, the 1/9 of the average inside its dyadic pair); every branch is
    rescaled by its own DN(S_i / S_a) and the four are joined along the channels.  Channel counts per module (width 64):
    64 + 64 + 96 + the input's channels at 35x35 (InceptionV3: 64, 64, 96), 192 + 192 + 192 + the input's at 17x17.
    A 3x3 / stride 2 stem takes the image to 35x35 (image_hw 71), a 3x3 / stride 2 max pool takes 35x35 to 17x17;
    global average pool and an 8-bit classifier close the table.  First and last layer stay 8-bit (Appendix H)."""
    if conv_bits not in (4, 8):
        raise ValueError("conv_bits must be 4 or 8")
    bd = _Builder(seed)
    bd.scale[-1], bd.shape[-1], bd.bits[-1] = _draw_scale(bd.g), (image_hw, image_hw, 3), 8
    x = bd.conv(-1, width, 3, 2, 0, 8, relu=True, out_bits=8)

    def module(x, c1, c2a, c2b, k2, c3a, c3b):
        xin = bd.requant(x, conv_bits) if conv_bits == 4 else x
        cb = conv_bits
        m = bd.conv(xin, c1, 1, 1, 0, cb, relu=True, out_bits=8)
        n = bd.conv(xin, c2a, 1, 1, 0, cb, relu=True, out_bits=cb)
        n = bd.conv(n, c2b, k2, 1, k2 // 2, cb, relu=True, out_bits=8)
        l = bd.conv(xin, c3a, 1, 1, 0, cb, relu=True, out_bits=cb)
        l = bd.conv(l, c3b, 3, 1, 1, cb, relu=True, out_bits=cb)
        l = bd.conv(l, c3b, 3, 1, 1, cb, relu=True, out_bits=8)
        p = bd.sumpool(x, 3, 1, 1)
        return bd.concat([m, n, l, p])

    for _ in range(modules35):
        x = module(x, width, (width * 3) // 4, width, 5, width, (width * 3) // 2)
    x = bd.maxpool(x, 3, 2, 0)
    for _ in range(modules17):
        x = module(x, 3 * width, 2 * width, 3 * width, 3, 2 * width, 3 * width)
    x = bd.avgpool(x)
    x = bd.conv(x, classes, 1, 1, 0, 8, relu=False, out_bits=32, op="linear")
    return dict(layers=bd.layers, image_hw=image_hw, classes=classes, depth=0, conv_bits=[conv_bits],
                shapes=[bd.shape[i] for i in range(len(bd.layers))], bits=[bd.bits[i] for i in range(len(bd.layers))])


def table_cost(table: dict, force_bits: int | None = None) -> dict:
    """MACs, parameters, BOPS (= b_w * b_a * MACs, Section 3.4) and weight bytes of a table.

    force_bits=4 evaluates the uniform 4-bit variant with first and last layer kept at 8 bit.
    """
    convs = [l for l in table["layers"] if l["op"] in ("conv", "linear")]
    macs = params = bops = size_bits = 0
    for i, l in enumerate(convs):
        bits = l["bits"]
        if force_bits is not None:
            bits = 8 if (i == 0 or i == len(convs) - 1) else force_bits
        macs += l["macs"]
        params += l["params"]
        bops += bits * bits * l["macs"]
        size_bits += bits * l["params"]
    return dict(macs=macs, params=params, bops=bops, weight_bytes=size_bits // 8)


def synthetic_sensitivity(table: dict, seed: int) -> np.ndarray:
    """Synthetic stand-in for the Hessian-based perturbation Omega_i^(b) of Section 3.4, [units, 2] int64 for
    b = 4 and 8.  There are no trained weights here, so the average Hessian trace of a layer is drawn
    log-normally around a value that falls by three decades from the first block to the last (early layers
    are the sensitive ones in the paper's figures), and the squared quantization error of a layer is taken as
    params * 4^-b (uniform quantization noise).  Only the ILP's input, never part of the integer pipeline.
    """
    units = len(table["conv_bits"])
    g = rng(seed, 31, units)
    params = np.zeros(units)
    for l in table["layers"]:
        if l["op"] == "conv" and l.get("unit", -1) >= 0:
            params[l["unit"]] += l["params"]
    trace = 10.0 ** (3.0 - 3.0 * np.arange(units) / max(units - 1, 1)) * np.exp(g.normal(0.0, 0.5, size=units))
    om = np.stack([trace * params * 4.0 ** -4, trace * params * 4.0 ** -8], axis=1)
    return np.maximum(np.rint(om / om.max() * 2.0 ** 36), 1).astype(np.int64)


def concat_case(seed: int, n: int, hw: int, branches, out_bits: int = 8, out_signed: int = 0, relu: int = 1) -> dict:
    """Inputs of one Inception-style concatenation (Appendix E): `branches` lists (channels, bits, signed) per
    branch, e.g. the 35x35 module of InceptionV3: three convolution branches (stored 8-bit tensors) and the pooling
    branch kept in INT32.  Values: 8-/4-bit tensors uniform over their type's range, INT32 tensors uniform in
    [-2^22, 2^22); per-channel pairs DN(S_i / S_a) with log-uniform scale ratios chosen so that outputs use the
    output range (8-bit: ratio in [2^-1, 2); 32-bit: ratio in [2^-16, 2^-14))."""
    g = rng(seed, 77, n, hw)
    out = []
    for ch, bits, signed in branches:
        if bits == 32:
            x = g.integers(-(1 << 22), 1 << 22, size=(n, hw, hw, ch), dtype=np.int64).astype(np.int32)
            ratio = np.exp2(g.uniform(-16.0, -14.0, size=ch))
        elif bits == 8:
            x = g.integers(-128 if signed else 0, 128 if signed else 256, size=(n, hw, hw, ch), dtype=np.int64)
            x = x.astype(np.int8 if signed else np.uint8)
            ratio = np.exp2(g.uniform(-1.0, 1.0, size=ch)) * (1.0 if out_bits == 8 else 1.0 / 16)
        else:
            x = pack4(g.integers(-8 if signed else 0, 8 if signed else 16, size=(n, hw, hw, ch), dtype=np.int64))
            ratio = np.exp2(g.uniform(-1.0, 1.0, size=ch)) * (16.0 if out_bits == 8 else 1.0)
        b, c = dyadic_from_scale(ratio)
        out.append({"x": x, "bits": bits, "signed": signed, "ch": ch, "b": b, "c": c})
    lo = -(1 << (out_bits - 1)) if out_signed else 0
    hi = (1 << (out_bits - 1)) - 1 if out_signed else (1 << out_bits) - 1
    return {"branches": out, "relu": relu, "qmin": lo, "qmax": hi, "out_bits": out_bits, "out_signed": out_signed,
            "n": n, "hw": hw, "out_ch": sum(b[0] for b in branches)}


def random_images(seed: int, n: int, hw: int = 224) -> np.ndarray:
    """uint8 images uniform in [0, 255], NHWC with 3 channels."""
    return rng(seed, 99, n, hw).integers(0, 256, size=(n, hw, hw, 3), dtype=np.int64).astype(np.uint8)
