"""Test oracle (not part of the product): the bit-width ILP of Section 3.4 (Eq. 5) solved by plain
enumeration.

Every layer takes one of two precisions; among all 2^L assignments that keep the summed model size,
BOPS and latency within their limits, the smallest summed perturbation Omega is the answer.  Nothing
is pruned, bounded or reordered: this is the definition written out, usable up to about 20 layers.
All quantities are integers, so the sums are exact.

Pinned (tests/test_oracle_pins.py) by a three-layer example worked by hand, by the unconstrained case
(every layer takes its smaller Omega), by single-limit cases that reduce to a textbook 0/1 knapsack
solved with the classic dynamic programme, and by G_i = b_w b_a MAC_i against the BOPS column the
paper prints for uniform ResNets (Table 1).
"""
from __future__ import annotations

import numpy as np


def solve_bruteforce(omega, size, bops, latency, size_limit: int = -1, bops_limit: int = -1,
                     latency_limit: int = -1):
    """Returns (objective, choices) of a minimal assignment, or (None, None) when none is feasible.

    omega, size, bops, latency: integer arrays [n_layers, 2]; a negative limit means no limit.
    Among several minimal assignments the one with the smallest binary code (layer 0 = lowest bit)
    is returned; callers should compare objectives, not assignments.
    """
    tabs = [np.asarray(t, dtype=np.int64) for t in (omega, size, bops, latency)]
    n = tabs[0].shape[0]
    if n > 22:
        raise ValueError("enumeration is meant for small instances")
    codes = np.arange(1 << n, dtype=np.int64)
    bits = (codes[:, None] >> np.arange(n, dtype=np.int64)[None, :]) & 1           # [2^n, n]
    sums = []
    for t in tabs:
        sums.append((t[None, :, 0] * (1 - bits) + t[None, :, 1] * bits).sum(axis=1) if n else np.zeros(1, np.int64))
    ok = np.ones(len(codes), dtype=bool)
    for s, lim in zip(sums[1:], (size_limit, bops_limit, latency_limit)):
        if lim >= 0:
            ok &= s <= lim
    if not ok.any():
        return None, None
    obj = np.where(ok, sums[0], np.iinfo(np.int64).max)
    k = int(np.argmin(obj))
    return int(obj[k]), bits[k].astype(np.int32)
