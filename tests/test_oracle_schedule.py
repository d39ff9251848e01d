"""Pins of the oracle's depth rule and batch schedule (no GPU)."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle as O

CONFIG_RULES = [(4, 1.0), (4, 0.98), (4, 0.95), (32, 1.0), (32, 0.999), (32, 0.995), (32, 0.997),
                (40, 1.0), (40, 0.998), (80, 1.0), (80, 0.998), (32, 0.9), (32, 0.9999), (80, 0.8)]


def exact_depth(L, alpha, i):
    """floor(L * alpha^i) in exact rational arithmetic on the double's value."""
    return math.floor(L * Fraction(alpha) ** i)


@pytest.mark.parametrize("L,alpha", CONFIG_RULES)
def test_depth_is_the_closed_form(L, alpha):
    # Abstract / Sec. 3.4: floor(L * alpha^i) layers retained for token T_i
    for i in list(range(0, 300)) + [511, 767, 1023, 1229, 4000]:
        want = exact_depth(L, alpha, i)
        assert O.depth(L, alpha, i) == want, (L, alpha, i)
        assert O.depth_pow(L, alpha, i) == want, (L, alpha, i)


def test_depth_special_cases():
    for L in (1, 4, 32, 40, 80):
        assert O.depth(L, 1.0, 10 ** 6) == L          # alpha = 1 is the full model
        for a in (0.5, 0.9, 0.9999):
            assert O.depth(L, a, 0) == L              # the first generated token runs every layer
    assert O.depth(32, 0.9, 1) == 28 and O.depth(32, 0.9, 2) == 25 and O.depth(32, 0.9, 3) == 23
    assert O.depth(80, 0.5, 1) == 40 and O.depth(80, 0.5, 7) == 0
    for bad in (0.0, -0.5, 1.0001, float("nan")):
        assert O.depth(32, bad, 3) == -1
    assert O.depth(32, 0.9, -1) == -1


def test_printed_average_layers(golden_dir):
    rows = [l.split() for l in open(os.path.join(golden_dir, "avg_layers.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 6
    for _, L, alpha, N, s, printed in rows:
        L, alpha, N, s, printed = int(L), float(alpha), int(N), int(s), float(printed)
        tot = 0
        for i in range(N):
            n, lo, hi = O.window(L, alpha, i, s, O.ANCHOR_START)
            assert hi - lo == L - n and lo == s
            tot += n
        assert abs(tot / N - printed) <= 0.0055, (L, alpha, tot / N, printed)


def test_average_layers_reject_the_other_readings():
    # a drop set one layer short, a first generated token at i = 1, or no floor
    # at start_id each miss the printed 19.17 of the 7B BBH row
    L, a, N, s = 32, 0.9, 200, 19
    base = [max(O.depth(L, a, i), s) for i in range(N)]
    assert abs(sum(base) / N - 19.17) <= 0.0055
    shifted = [max(O.depth(L, a, i + 1), s) for i in range(N)]
    assert abs(sum(shifted) / N - 19.17) > 0.02
    unclamped = [O.depth(L, a, i) for i in range(N)]
    assert abs(sum(unclamped) / N - 19.17) > 1.0
    one_short = [min(L, n + 1) for n in (O.depth(32, 0.9999, i) for i in range(1024))]
    assert abs(sum(one_short) / 1024 - 29.90) > 0.5


@pytest.mark.parametrize("anchor", [O.ANCHOR_START, O.ANCHOR_TAIL])
@pytest.mark.parametrize("L,alpha,s", [(32, 0.995, 6), (32, 0.9, 19), (4, 0.95, 0), (80, 0.998, 16),
                                       (40, 0.9, 20), (8, 0.7, 8), (8, 0.7, 3)])
def test_depth_never_grows_and_windows_nest(L, alpha, s, anchor):
    prev = None
    for i in range(0, 400):
        n, lo, hi = O.window(L, alpha, i, s, anchor)
        assert 0 <= lo <= hi <= L and hi - lo == L - n
        if anchor == O.ANCHOR_START:
            assert n == max(O.depth(L, alpha, i), s) and lo == s
        else:
            assert n == O.depth(L, alpha, i) and hi == L
        if prev is not None:
            pn, plo, phi = prev
            assert n <= pn and lo <= plo and hi >= phi      # window_i-1 inside window_i
        prev = (n, lo, hi)


def test_window_rejects_bad_start():
    assert O.window(8, 0.9, 1, 9)[0] == -1
    assert O.window(8, 0.9, 1, -1)[0] == -1


@pytest.mark.parametrize("anchor", [O.ANCHOR_START, O.ANCHOR_TAIL])
def test_batch_schedule_against_brute_force(anchor):
    rng = np.random.default_rng(5)
    for L, alpha, s in [(32, 0.997, 6), (4, 0.95, 0), (40, 0.998, 8), (80, 0.99, 16), (32, 0.9, 19)]:
        for B in (1, 2, 7, 32):
            gi = rng.integers(1, 400, size=B).astype(np.int32)
            gi[B // 2] = gi[0]                                  # a tie
            sch = O.schedule(L, alpha, s, anchor, gi)
            n = [O.window(L, alpha, int(i), s, anchor)[0] for i in gi]
            assert list(sch["n"]) == n
            want_perm = sorted(range(B), key=lambda b: (-n[b], b))
            assert list(sch["perm"]) == want_perm               # stable, deepest first
            m = [sum(1 for b in range(B) if not (sch["lo"][b] <= l < sch["hi"][b]))
                 for l in range(L)]
            assert list(sch["m_per_layer"]) == m
            assert sch["rows_layers"] == sum(n) == sum(m)       # counting identity
            assert sch["layers_touched"] == sum(1 for v in m if v > 0)
            # the rows that run layer l are a prefix of the sorted order
            for l in range(L):
                act = {b for b in range(B) if not (sch["lo"][b] <= l < sch["hi"][b])}
                assert act == set(want_perm[:m[l]])


# ---------------------------------------------------- linear decay between two bounds

@pytest.mark.parametrize("upper,lower,span", [(32, 8, 255), (40, 14, 512), (80, 48, 100), (4, 0, 3),
                                              (7, 7, 10), (32, 31, 1000)])
def test_linear_depth_end_points_monotonicity_and_floor_sum(upper, lower, span):
    # Sec. 3.4 / Sec. 4.1: linear decay between an upper and a lower bound of executed layers.
    ns = [O.depth_linear(upper, lower, span, i) for i in range(span + 20)]
    assert ns[0] == upper and ns[span] == lower and all(n == lower for n in ns[span:])
    assert all(a >= b for a, b in zip(ns, ns[1:]))                     # never grows
    assert all(0 <= a - b <= max(1, -(-(upper - lower) // span)) for a, b in zip(ns, ns[1:]))
    # layers dropped over i = 0 .. span-1: the classical floor-sum identity
    #   sum_{i<n} floor(a i / n) = ((a - 1)(n - 1) + gcd(a, n) - 1) / 2      (a, n >= 1)
    a, n = upper - lower, span
    dropped = sum(upper - v for v in ns[:span])
    want = 0 if a == 0 else ((a - 1) * (n - 1) + math.gcd(a, n) - 1) // 2
    assert dropped == want
    # hence the mean retained count, the figure a target speed-up fixes
    assert Fraction(sum(ns[:span]), span) == upper - Fraction(want, span)


def test_linear_depth_rejects_bad_arguments():
    for args in [(-1, 0, 5, 0), (4, 5, 5, 0), (4, -1, 5, 0), (4, 0, 0, 0), (4, 0, 5, -1)]:
        assert O.depth_linear(*args) == -1


def test_window_of_a_given_depth_is_the_window_of_the_rule():
    L = 32
    for alpha in (0.9, 0.99, 0.999):
        for s, anchor in ((0, O.ANCHOR_START), (6, O.ANCHOR_START), (0, O.ANCHOR_TAIL)):
            for i in (0, 1, 7, 50, 300, 4000):
                assert O.window_of_depth(L, O.depth(L, alpha, i), s, anchor) == O.window(L, alpha, i, s, anchor)
    assert O.window_of_depth(L, L + 1, 0)[0] == -1 and O.window_of_depth(L, -1, 0)[0] == -1
