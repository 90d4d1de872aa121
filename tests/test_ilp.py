"""Bit-width ILP (Section 3.4, Eq. 5): the enumeration oracle against what the mathematics fixes, and the
library's exact solver (host code, runs without a GPU) against the oracle."""
import os

import numpy as np
import pytest

from oracle import ilp as oracle_ilp
from paper_2011_10680_b200 import binding, inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "ilp_three_layers.txt")


def read_golden():
    rows, cases = [], []
    for line in open(GOLDEN):
        line = line.strip()
        if line.startswith("layer"):
            rows.append([int(v) for v in line.split()[1:]])
        elif line.startswith("case"):
            lims, want = line[4:].split("->")
            cases.append(([int(v) for v in lims.split()], want.split()))
    t = np.array(rows, dtype=np.int64)
    return (t[:, 0:2], t[:, 2:4], t[:, 4:6], t[:, 6:8]), cases


def knapsack_min_omega(omega, res, limit):
    """Textbook dynamic programme over the capacity: minimal summed omega with summed res <= limit."""
    inf = np.iinfo(np.int64).max // 4
    best = np.full(limit + 1, inf, dtype=np.int64)
    best[0] = 0
    for i in range(len(omega)):
        nxt = np.full(limit + 1, inf, dtype=np.int64)
        for c in range(2):
            w, v = int(res[i, c]), int(omega[i, c])
            if w <= limit:
                cand = best[:limit + 1 - w] + v
                nxt[w:] = np.minimum(nxt[w:], cand)
        best = np.minimum(nxt, inf)
    m = int(best.min())
    return None if m >= inf else m


# ---- the oracle against hand-worked values, closed forms and a different algorithm ----------------------------

def test_oracle_matches_the_hand_worked_example():
    tabs, cases = read_golden()
    for lims, want in cases:
        obj, ch = oracle_ilp.solve_bruteforce(*tabs, *lims)
        if want[0] == "infeasible":
            assert obj is None
        else:
            assert obj == int(want[0])
            assert "".join(str(int(b)) for b in ch) == want[1]


def test_oracle_without_limits_takes_every_layers_smaller_omega():
    g = np.random.default_rng(5)
    for n in (1, 4, 9):
        tabs = [g.integers(0, 1000, size=(n, 2)) for _ in range(4)]
        obj, ch = oracle_ilp.solve_bruteforce(*tabs)
        assert obj == int(tabs[0].min(axis=1).sum())
        assert all(tabs[0][i, ch[i]] == tabs[0][i].min() for i in range(n))


@pytest.mark.parametrize("which", [0, 1, 2])
def test_oracle_single_limit_is_a_knapsack(which):
    g = np.random.default_rng(11 + which)
    for _ in range(20):
        n = int(g.integers(2, 11))
        tabs = [g.integers(0, 60, size=(n, 2)) for _ in range(4)]
        limit = int(g.integers(0, 40 * n))
        lims = [-1, -1, -1]
        lims[which] = limit
        obj, ch = oracle_ilp.solve_bruteforce(*tabs, *lims)
        want = knapsack_min_omega(tabs[0], tabs[1 + which], limit)
        assert obj == want
        if obj is not None:
            assert sum(int(tabs[1 + which][i, ch[i]]) for i in range(n)) <= limit


def test_oracle_tight_limits_force_the_cheapest_assignment():
    # limits equal to the cheapest possible sums leave exactly the all-cheapest assignment (strictly cheaper choice 0)
    g = np.random.default_rng(3)
    n = 7
    om = g.integers(0, 100, size=(n, 2))
    res = np.stack([g.integers(0, 50, size=n), g.integers(51, 100, size=n)], axis=1)
    obj, ch = oracle_ilp.solve_bruteforce(om, res, res, res, int(res[:, 0].sum()), -1, -1)
    assert obj == int(om[:, 0].sum()) and not ch.any()


# ---- the library's solver against the oracle --------------------------------------------------------------------

def test_solver_matches_the_hand_worked_example():
    tabs, cases = read_golden()
    for lims, want in cases:
        st, ch, obj = binding.ilp_solve(*tabs, *lims)
        if want[0] == "infeasible":
            assert st == binding.HQ_ERR_INFEASIBLE
        else:
            assert st == binding.HQ_OK and obj == int(want[0])


@pytest.mark.parametrize("seed", range(6))
def test_solver_equals_enumeration_on_random_instances(seed):
    g = np.random.default_rng(100 + seed)
    for _ in range(120):
        n = int(g.integers(0, 13))
        hi = int(g.choice([2, 50, 10 ** 6]))          # many ties, ordinary, wide ranges
        tabs = [g.integers(0, hi, size=(n, 2)) for _ in range(4)]
        lims = [int(g.integers(0, max(1, hi * n * 3 // 4))) if g.random() < 0.6 else -1 for _ in range(3)]
        st, ch, obj = binding.ilp_solve(*tabs, *lims)
        want, _ = oracle_ilp.solve_bruteforce(*tabs, *lims)
        if want is None:
            assert st == binding.HQ_ERR_INFEASIBLE
            continue
        assert st == binding.HQ_OK and obj == want
        # the assignment it reports is feasible and has that objective
        assert sum(int(tabs[0][i, ch[i]]) for i in range(n)) == obj
        for t, lim in zip(tabs[1:], lims):
            assert lim < 0 or sum(int(t[i, ch[i]]) for i in range(n)) <= lim


def test_solver_full_size_single_limits_equal_the_knapsack_programme():
    """48 layers (the block convs of ResNet-50) are beyond enumeration; with one limit the answer is a knapsack."""
    g = np.random.default_rng(77)
    n = inputs.resnet_choice_units(50)
    om = np.stack([g.integers(100, 5000, size=n), g.integers(0, 100, size=n)], axis=1)     # INT4 perturbs more
    res = np.stack([g.integers(10, 200, size=n), g.integers(150, 900, size=n)], axis=1)
    for frac in (0.0, 0.1, 0.35, 0.7, 1.0):
        lo, hi = int(res.min(axis=1).sum()), int(res.max(axis=1).sum())
        limit = lo + int(frac * (hi - lo))
        for which in range(3):
            lims = [-1, -1, -1]
            lims[which] = limit
            tabs = [om, res, res, res]
            st, ch, obj = binding.ilp_solve(*tabs, *lims)
            assert st == binding.HQ_OK
            assert obj == knapsack_min_omega(om, res, limit)
    st, _, _ = binding.ilp_solve(om, res, res, res, int(res.min(axis=1).sum()) - 1, -1, -1)
    assert st == binding.HQ_ERR_INFEASIBLE


def test_solver_three_limits_at_full_size_is_feasible_and_no_worse_than_greedy():
    g = np.random.default_rng(78)
    n = 48
    om = np.stack([g.integers(100, 5000, size=n), g.integers(0, 100, size=n)], axis=1)
    tabs = [om] + [np.stack([g.integers(10, 200, size=n), g.integers(150, 900, size=n)], axis=1) for _ in range(3)]
    lims = [int(t.min(axis=1).sum() * 1.8) for t in tabs[1:]]
    st, ch, obj = binding.ilp_solve(*tabs, *lims)
    assert st == binding.HQ_OK
    for t, lim in zip(tabs[1:], lims):
        assert sum(int(t[i, ch[i]]) for i in range(n)) <= lim
    # a greedy feasible assignment (upgrade by omega saved while everything still fits) is an upper bound
    cur = np.zeros(n, dtype=int)
    used = [int(t[:, 0].sum()) for t in tabs[1:]]
    for i in np.argsort(-(om[:, 0] - om[:, 1])):
        d = [int(t[i, 1] - t[i, 0]) for t in tabs[1:]]
        if all(u + x <= lim for u, x, lim in zip(used, d, lims)):
            cur[i] = 1
            used = [u + x for u, x in zip(used, d)]
    assert obj <= sum(int(om[i, cur[i]]) for i in range(n))
    # flipping any single layer of the reported optimum is infeasible or no better
    for i in range(n):
        alt = ch.copy()
        alt[i] ^= 1
        feasible = all(sum(int(t[j, alt[j]]) for j in range(n)) <= lim for t, lim in zip(tabs[1:], lims))
        assert not feasible or sum(int(om[j, alt[j]]) for j in range(n)) >= obj


def test_solver_rejects_bad_arguments():
    t = np.zeros((2, 2), dtype=np.int64)
    neg = t.copy()
    neg[1, 0] = -1
    assert binding.ilp_solve(neg, t, t, t)[0] == binding.HQ_ERR_INVALID_ARG
    big = t.copy()
    big[0, 1] = (1 << 40) + 1
    assert binding.ilp_solve(t, t, big, t)[0] == binding.HQ_ERR_INVALID_ARG
    assert binding.ilp_solve(np.zeros((0, 2), np.int64), np.zeros((0, 2), np.int64), np.zeros((0, 2), np.int64),
                             np.zeros((0, 2), np.int64))[0] == binding.HQ_OK
