"""Oracle network walk: apply the layer functions over a table, in table order, keeping every output.

Follows the dataflow of the paper's Fig. 2 in its fused form: a conv layer may carry the residual
operand (tensor id in1); 'requant' quantizes a stream tensor once for all its consumers; 'add' is the
element-wise add of Section 3.3 on stored tensors; 'sumpool' and 'concat' are the pooling branch and
the concatenation of an Inception module (Appendix E).
"""
from __future__ import annotations

import numpy as np

from . import hqref


def run_network(table: dict, images: np.ndarray) -> list[np.ndarray]:
    """Return the list of every layer's output (the last one is the INT32 logits)."""
    outs: list[np.ndarray] = []
    meta = {-1: (8, 0)}                      # tensor id -> (bits, signed)

    def t(i):
        return images if i == -1 else outs[i]

    for li, l in enumerate(table["layers"]):
        op = l["op"]
        if op in ("conv", "linear"):
            in_bits, in_signed = meta[l["in0"]]
            res = rb = rc = None
            res_bits = res_signed = 0
            if l["in1"] >= 0:
                res = t(l["in1"])
                res_bits, res_signed = meta[l["in1"]]
                rb, rc = l["rb"], l["rc"]
            x = t(l["in0"])
            if op == "linear":
                y = hqref.linear(x.reshape(x.shape[0], -1), l["cin"], in_bits, in_signed, l["wgt"], l["cout"],
                                 l["bias"], l["b"], l["c"], l["relu"], l["qmin"], l["qmax"],
                                 l["out_bits"], l["out_signed"])
            else:
                y = hqref.conv2d(x, l["cin"], in_bits, in_signed, l["wgt"], l["cout"], l["kh"], l["kw"],
                                 l["stride"], l["pad"], l["bias"], l["b"], l["c"], res, res_bits, res_signed,
                                 rb, rc, l["relu"], l["qmin"], l["qmax"], l["out_bits"], l["out_signed"])
        elif op == "maxpool":
            y = hqref.maxpool(t(l["in0"]), l["pool_k"], l["pool_stride"], l["pool_pad"], meta[l["in0"]][1])
        elif op == "avgpool":
            in_bits, in_signed = meta[l["in0"]]
            y = hqref.avgpool_requant(t(l["in0"]), l["cout"], in_bits, in_signed, l["b"], l["c"],
                                      l["qmin"], l["qmax"], l["out_bits"], l["out_signed"])
        elif op in ("requant", "add"):
            in_bits, in_signed = meta[l["in0"]]
            res = rb = rc = None
            res_bits = res_signed = 0
            if l["in1"] >= 0:
                res = t(l["in1"])
                res_bits, res_signed = meta[l["in1"]]
                rb, rc = l["rb"], l["rc"]
            y = hqref.residual_add(t(l["in0"]), in_bits, in_signed, l["b"], l["c"], res, res_bits, res_signed,
                                   rb, rc, l["cout"], l["relu"], l["qmin"], l["qmax"],
                                   l["out_bits"], l["out_signed"])
        elif op == "sumpool":
            # the pooling branch of an Inception module works on the wide feature map: INT32 window sums (Appendix E)
            in_bits, in_signed = meta[l["in0"]]
            y = hqref.sumpool(t(l["in0"]), l["cout"], in_bits, in_signed, l["pool_k"], l["pool_stride"], l["pool_pad"])
        elif op == "concat":
            # every branch rescaled by its own dyadic pairs, then joined along the channels (Appendix E)
            branches = [{"x": t(i), "bits": meta[i][0], "signed": meta[i][1], "ch": int(len(b)), "b": b, "c": c}
                        for i, b, c in zip(l["ins"], l["bs"], l["cs"])]
            y = hqref.concat_requant(branches, l["relu"], l["qmin"], l["qmax"], l["out_bits"], l["out_signed"])
        else:
            raise ValueError(f"unknown op {op!r} in layer {li}")
        outs.append(y)
        meta[li] = (l["out_bits"], l["out_signed"])
    return outs
