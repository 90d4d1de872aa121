"""Offline tool: float parameters -> the integer parameter set the inference kernels consume.

Everything here runs once, before inference, on the host, in double precision -- the paper's deployment
flow up to the point where the integer-only pipeline takes over (Section 3.2 and Appendix D for the
batch-norm fold, Appendix A for the quantizers, the DN(.) definition after Eq. 4 for the dyadic pairs).
Nothing in this module is called while a layer runs.

    fold_bn            conv weights + batch-norm statistics -> folded weights and bias          (Appendix D)
    quantize_weights   symmetric, per output channel, k bits                                    (Appendix A)
    quantize_bias      INT32 at scale S_h * S_w[oc], so that it adds to the accumulator         (Section 3.2)
    dyadic_from_scale  DN(.): real scale -> (b, c) with b / 2^c ~= scale                        (Section 3.1)
    conv_params        one layer: the arrays of an hq_conv_desc / a table row
    quantize_network   a list of float layers with static activation scales -> a layer table for hq_run_network
    float_forward      the float network evaluated in numpy (what the scales are calibrated on)
    calibrate          static activation scales from float activations (Appendix B: static quantization)
    fold_input_zero_point   an input tensor with a non-zero zero point Z (Eq. 2): Z leaves the tensor, its effect
                            goes into the first layer's INT32 bias
"""
from __future__ import annotations

import numpy as np

__all__ = ["dyadic_from_scale", "fold_bn", "quantize_weights", "quantize_bias", "conv_params", "quantize_network",
           "float_forward", "calibrate", "fold_input_zero_point"]


# --------------------------------------------------------------------------------------------
# DN(.): real scale -> dyadic pair (Section 3.1, equation after Eq. 4)
# --------------------------------------------------------------------------------------------
def dyadic_from_scale(s):
    """Return int32 arrays (b, c) with b / 2^c ~= s, 2^30 <= b < 2^31 and 1 <= c <= 62.

    The paper defines DN only by its result.  Reading used here: normalise s = m * 2^e with
    m in [0.5, 1), take b = round_half_up(m * 2^31), c = 31 - e (and renormalise if b hits 2^31).
    The error is at most 2^-(c+1).  Scales so small that c would pass 62 keep c = 62 and a
    smaller b; scales of 2^30 and above are rejected.
    """
    s = np.atleast_1d(np.asarray(s, dtype=np.float64))
    if np.any(~np.isfinite(s)) or np.any(s <= 0):
        raise ValueError("scale must be finite and positive")
    m, e = np.frexp(s)                       # s = m * 2^e, m in [0.5, 1): exact
    b = np.floor(np.ldexp(m, 31) + 0.5).astype(np.int64)
    c = 31 - e.astype(np.int64)
    hit = b == (1 << 31)
    b[hit] >>= 1
    c[hit] -= 1
    if np.any(c < 1):
        raise ValueError("scale too large for a dyadic pair with c >= 1")
    deep = c > 62
    if np.any(deep):
        b[deep] = np.floor(np.ldexp(s[deep], 62) + 0.5).astype(np.int64)
        c[deep] = 62
    return b.astype(np.int32), c.astype(np.int32)


# --------------------------------------------------------------------------------------------
# Batch-norm folding (Section 3.2, Appendix D).  The paper writes BN(a) = beta * (a - mu) / sigma + gamma:
# beta is the SCALE and gamma the SHIFT (the reverse of the common naming); sigma is the standard deviation.
# --------------------------------------------------------------------------------------------
def fold_bn(w: np.ndarray, beta: np.ndarray, gamma: np.ndarray, mu: np.ndarray, sigma: np.ndarray):
    """conv with weights w [cout][kh][kw][cin] followed by BN -> conv with folded weights and a bias:
    W_bar = beta * W / sigma,  b_bar = gamma - beta * mu / sigma  (per output channel)."""
    w = np.asarray(w, np.float64)
    k = np.asarray(beta, np.float64) / np.asarray(sigma, np.float64)
    return w * k[:, None, None, None], np.asarray(gamma, np.float64) - k * np.asarray(mu, np.float64)


# --------------------------------------------------------------------------------------------
# Quantizers (Appendix A; first and last layer and the input image stay 8-bit, Appendix H)
# --------------------------------------------------------------------------------------------
def quantize_weights(w: np.ndarray, bits: int):
    """Symmetric channel-wise quantization: S_w[oc] = max|w[oc]| / (2^(k-1) - 1), q = Int(w / S_w) in
    [-(2^(k-1)-1), 2^(k-1)-1].  Returns (q int64 [cout][kh][kw][cin], S_w float64 [cout])."""
    w = np.asarray(w, np.float64)
    cout = w.shape[0]
    wmax = (1 << (bits - 1)) - 1
    s_w = np.abs(w).reshape(cout, -1).max(axis=1) / wmax
    s_w = np.where(s_w > 0, s_w, 1.0)                 # an all-zero channel: any scale represents it
    q = np.floor(w / s_w[:, None, None, None] + 0.5)
    return np.clip(q, -wmax, wmax).astype(np.int64), s_w


def quantize_bias(b_bar: np.ndarray, s_h: float, s_w: np.ndarray) -> np.ndarray:
    """The folded bias as INT32 at scale S_h * S_w[oc]: it then adds directly to the INT32 accumulator."""
    q = np.floor(np.asarray(b_bar, np.float64) / (s_h * np.asarray(s_w, np.float64)) + 0.5)
    if np.any(np.abs(q) >= 2.0 ** 31):
        raise ValueError("bias does not fit INT32 at the accumulator's scale")
    return q.astype(np.int64).astype(np.int32)


def conv_params(w_bar: np.ndarray, b_bar: np.ndarray | None, s_in: float, s_out: float | None, bits: int,
                s_res: float | None = None) -> dict:
    """Integer parameters of one folded conv / linear layer: weights, INT32 bias, the requantization pairs
    DN(S_w[oc] S_in / S_out) and, with a residual operand at scale s_res, DN(s_res / s_out) for it.
    s_out None: the layer returns the raw INT32 accumulator (the logits)."""
    q, s_w = quantize_weights(w_bar, bits)
    cout = q.shape[0]
    out = {"q_w": q, "s_w": s_w, "bias": quantize_bias(b_bar, s_in, s_w) if b_bar is not None else np.zeros(cout, np.int32),
           "b": None, "c": None, "rb": None, "rc": None}
    if s_out is not None:
        out["b"], out["c"] = dyadic_from_scale(s_w * s_in / s_out)
        if s_res is not None:
            rb, rc = dyadic_from_scale(s_res / s_out)
            out["rb"], out["rc"] = np.full(cout, rb[0], np.int32), np.full(cout, rc[0], np.int32)
    return out


def _pack4(a: np.ndarray) -> np.ndarray:
    u = (np.asarray(a).astype(np.int16) & 0xF).astype(np.uint8)
    return (u[..., 0::2] | (u[..., 1::2] << 4)).astype(np.uint8)


def _float_conv(x, w, stride, pad):
    n, h, wd, ci = x.shape
    co, kh, kw, _ = w.shape
    xp = np.zeros((n, h + 2 * pad, wd + 2 * pad, ci))
    xp[:, pad:pad + h, pad:pad + wd] = x
    ho, wo = (h + 2 * pad - kh) // stride + 1, (wd + 2 * pad - kw) // stride + 1
    cols = np.empty((n, ho, wo, kh, kw, ci))
    for r in range(kh):
        for s in range(kw):
            cols[:, :, :, r, s] = xp[:, r:r + stride * ho:stride, s:s + stride * wo:stride]
    return (cols.reshape(n * ho * wo, -1) @ np.asarray(w, np.float64).reshape(co, -1).T).reshape(n, ho, wo, co)


def float_forward(layers: list[dict], x: np.ndarray) -> list[np.ndarray]:
    """Float activations of every layer of a float network description (see quantize_network) on the real-valued
    NHWC input x: convolution, batch norm (the paper's beta (a - mu) / sigma + gamma), bias, residual add, ReLU,
    pooling.  Offline only: this is what static activation ranges are measured on."""
    acts = {-1: np.asarray(x, np.float64)}
    for i, l in enumerate(layers):
        a = acts[l["in0"]]
        if l["op"] in ("conv", "linear"):
            if l["op"] == "linear":
                a = a.reshape(a.shape[0], 1, 1, -1)
            y = _float_conv(a, l["w"], l.get("stride", 1), l.get("pad", 0))
            if l.get("bias") is not None:
                y = y + np.asarray(l["bias"], np.float64)
            if l.get("bn") is not None:
                beta, gamma, mu, sigma = (np.asarray(v, np.float64) for v in l["bn"])
                y = beta * (y - mu) / sigma + gamma
            if l.get("in1", -1) >= 0:
                y = y + acts[l["in1"]]
            if l.get("relu", True):
                y = np.maximum(y, 0)
        elif l["op"] == "maxpool":
            k, st, pad = l["k"], l["stride"], l["pad"]
            ap = np.pad(a, ((0, 0), (pad, pad), (pad, pad), (0, 0)), constant_values=-np.inf)
            ho, wo = (a.shape[1] + 2 * pad - k) // st + 1, (a.shape[2] + 2 * pad - k) // st + 1
            y = np.stack([np.stack([ap[:, oh * st:oh * st + k, ow * st:ow * st + k].max(axis=(1, 2)) for ow in range(wo)], axis=1)
                          for oh in range(ho)], axis=1)
        elif l["op"] == "avgpool":
            y = a.mean(axis=(1, 2), keepdims=True)
        else:
            raise ValueError(l["op"])
        acts[i] = y
    return [acts[i] for i in range(len(layers))]


def calibrate(layers: list[dict], x: np.ndarray) -> list[dict]:
    """Copy of `layers` with the static output scale of every quantized tensor filled in from the float activations
    on the calibration batch x: S = r_max / (2^k - 1) after a ReLU (r_min = 0, zero point 0), S = max|r| / (2^(k-1) - 1)
    for signed tensors.  Layers whose "s_out" is None on purpose (raw INT32 logits) keep it."""
    acts = float_forward(layers, x)
    out = []
    for l, a in zip(layers, acts):
        l = dict(l)
        if l["op"] == "avgpool":
            l.setdefault("hw", None)
            l["s_out"] = float(a.max()) / 255.0
        elif l["op"] in ("conv", "linear") and "s_out" not in l:
            bits = l.get("out_bits", 8)
            if l.get("relu", True):
                l["s_out"] = float(a.max()) / ((1 << bits) - 1)
            else:
                l["s_out"] = float(np.abs(a).max()) / ((1 << (bits - 1)) - 1)
        out.append(l)
    return out


def quantize_network(layers: list[dict], s_image: float, image_hw: int | None = None) -> dict:
    """Float network -> layer table for hq_run_network / the oracle's walk.

    `layers` is a list of dicts, layer i producing tensor i (tensor -1 is the uint8 image at scale s_image):
      {"op": "conv", "in0", "in1" (residual tensor or -1), "w" [cout][kh][kw][cin] float, "bn": (beta, gamma, mu,
       sigma) or None, "bias" float or None, "stride", "pad", "bits", "relu", "s_out" (static activation scale of the
       output, from calibration), "out_bits", "out_signed"}
      {"op": "linear", ...} the same on a flattened input, s_out None -> INT32 logits
      {"op": "maxpool", "in0", "k", "stride", "pad"},  {"op": "avgpool", "in0", "s_out"}
    Scales follow the tensors: a conv's input scale is its producer's output scale; the average pool carries
    1 / (h w) inside its dyadic pair (no division at run time).
    """
    scale = {-1: float(s_image)}
    shape = {}
    table = []
    for i, l in enumerate(layers):
        op = l["op"]
        if op in ("conv", "linear"):
            w = np.asarray(l["w"], np.float64)
            b = None if l.get("bias") is None else np.asarray(l["bias"], np.float64)
            if l.get("bn") is not None:
                w, b_bn = fold_bn(w, *l["bn"])
                b = b_bn if b is None else b_bn + np.asarray(l["bn"][0], np.float64) / np.asarray(l["bn"][3], np.float64) * b
            s_in = scale[l["in0"]]
            s_res = scale[l["in1"]] if l.get("in1", -1) >= 0 else None
            pr = conv_params(w, b, s_in, l.get("s_out"), l["bits"], s_res)
            cout, kh, kw, cin = pr["q_w"].shape
            out_bits = 32 if l.get("s_out") is None else l.get("out_bits", 8)
            out_signed = 1 if out_bits == 32 else int(l.get("out_signed", not l.get("relu", True)))
            qmin = -(1 << (out_bits - 1)) if out_signed else 0
            qmax = (1 << (out_bits - 1)) - 1 if out_signed else (1 << out_bits) - 1
            table.append(dict(op=op, in0=l["in0"], in1=l.get("in1", -1), kh=kh, kw=kw, stride=l.get("stride", 1),
                              pad=l.get("pad", 0), cin=cin, cout=cout, bits=l["bits"],
                              wgt=_pack4(pr["q_w"]) if l["bits"] == 4 else pr["q_w"].astype(np.int8), bias=pr["bias"],
                              b=pr["b"], c=pr["c"], rb=pr["rb"], rc=pr["rc"], relu=int(l.get("relu", True)), qmin=qmin,
                              qmax=qmax, out_bits=out_bits, out_signed=out_signed))
            scale[i] = l["s_out"] if l.get("s_out") is not None else s_in * float(pr["s_w"].mean())
        elif op == "maxpool":
            table.append(dict(op="maxpool", in0=l["in0"], in1=-1, pool_k=l["k"], pool_stride=l["stride"], pool_pad=l["pad"],
                              cout=None, out_bits=8, out_signed=0, relu=0, qmin=0, qmax=255))
            scale[i] = scale[l["in0"]]
        elif op == "avgpool":
            hw = l["hw"]
            b, c = dyadic_from_scale(scale[l["in0"]] / (hw * l["s_out"]))
            ch = l["channels"]
            table.append(dict(op="avgpool", in0=l["in0"], in1=-1, cout=ch, b=np.full(ch, b[0], np.int32),
                              c=np.full(ch, c[0], np.int32), out_bits=8, out_signed=0, relu=0, qmin=0, qmax=255))
            scale[i] = l["s_out"]
        else:
            raise ValueError(f"unknown op {op!r}")
    classes = table[-1]["cout"] if table and table[-1]["op"] == "linear" else None
    return {"layers": table, "scales": [scale[i] for i in range(len(layers))], "image_hw": image_hw, "classes": classes}



# --------------------------------------------------------------------------------------------
# Non-zero zero point of the network input (Eq. 2 carries a zero point, Eq. 3-4 do not)
# --------------------------------------------------------------------------------------------
def fold_input_zero_point(q_bias: np.ndarray, q_w: np.ndarray, z: int, pad: int = 0) -> np.ndarray:
    """The kernels compute sum_k q_x[k] q_w[k] on stored values with zero point 0.  For an input whose
    real value is S (q_x - Z), sum_k (q_x[k] - Z) q_w[oc, k] = sum_k q_x[k] q_w[oc, k] - Z sum_k q_w[oc, k]:
    the correction is a per-channel constant and moves into the INT32 bias, exactly.  That holds where every
    tap of the window reads a stored value, i.e. for an unpadded layer (padding writes the integer 0, which
    stands for the real value -S Z, not 0); a padded first layer needs the input re-centred instead, which for
    Z = 128 on 8-bit data is the signed image the kernels accept as it is.

    q_bias: INT32 bias at S_h S_w (quantize_bias); q_w: integer weights [cout, kh, kw, cin]."""
    if pad != 0:
        raise ValueError("the fold is exact for unpadded layers only: re-centre the input (Z = 128: signed image) instead")
    corr = np.asarray(q_w, np.int64).reshape(q_w.shape[0], -1).sum(axis=1) * int(z)
    out = np.asarray(q_bias, np.int64) - corr
    if np.any(out < -(1 << 31)) or np.any(out >= (1 << 31)):
        raise ValueError("the folded bias leaves the INT32 range")
    return out.astype(np.int32)
