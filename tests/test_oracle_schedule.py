"""Pins for the oracle's schedule: what the paper prints and what arithmetic fixes."""
import os
import math
from fractions import Fraction

import pytest

from oracle import skipdecode_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_figure3_printed_points():
    # Figure 3: prompt 20, max_len 100 (closed interval => 81 generated positions).
    P, last, L, mx, mn = 20, 100, 12, 8, 2
    n, top = O.schedule(mx, mn, 0, last - P + 1, L)
    for x, val in ((int(a), int(b)) for a, b in _rows("fig3_schedule.txt")):
        got = L if x < P else n[x - P]
        assert got == val, (x, got, val)
    # never further than half a layer from the plotted line
    for g, v in enumerate(n):
        line = Fraction(mx) - Fraction(mx - mn) * Fraction(g, last - P)
        assert abs(v - line) <= Fraction(1, 2)


@pytest.mark.parametrize("row", _rows("table2_budgets.txt"))
def test_table2_mean_budget(row):
    L, _speed, avg, w, mn, mx = int(row[0]), int(row[1]), float(row[2]), int(row[3]), int(row[4]), int(row[5])
    for G in (2, 101, 160 - 60, 1024 - 512, 2048 - 1024):
        n, top = O.schedule(mx, mn, w, G, L)
        assert n[0] == mx and n[-1] == mn
        mean = Fraction(sum(n), G)
        # halves round up, so the mean sits at the midpoint or at most 1/2 layer-step above it
        assert 0 <= mean - Fraction(mn + mx, 2) <= Fraction(1, 2)
        if G % 2 == 0 and (mx - mn) % 2 == 1 and G == 2:
            assert mean == Fraction(mn + mx, 2)
    midpoint = (mn + mx) / 2
    if (L, mn, mx) == (32, 11, 22):
        assert midpoint == 16.5 and avg == 16          # the table's own inconsistency
    else:
        assert midpoint == avg
    # warm-up is inside the budget: w bottom layers + (n - w) top layers
    n, top = O.schedule(mx, mn, w, 64, L)
    for g in range(64):
        layers = O.active_layers(L, n[g], w)
        assert len(layers) == n[g] and layers[:w] == list(range(w))
        assert layers[w:] == list(range(top[g], L)) and top[g] == L - (n[g] - w)


CONFIG_SCHEDULES = [  # (L, max, min, G, expected sum = G (max+min)/2)
    (4, 4, 2, 32, 96), (12, 12, 4, 128, 1024), (24, 24, 8, 256, 4096),
    (32, 32, 8, 512, 10240), (32, 32, 4, 1024, 18432),
]


@pytest.mark.parametrize("L,mx,mn,G,total", CONFIG_SCHEDULES)
def test_budget_sum_and_invariants(L, mx, mn, G, total):
    n, top = O.schedule(mx, mn, 0, G, L)
    assert sum(n) == total == G * (mx + mn) // 2
    assert n[0] == mx and n[-1] == mn
    assert all(a >= b for a, b in zip(n, n[1:]))              # monotone non-increasing
    assert all(mn <= v <= mx for v in n)
    assert all(a <= b for a, b in zip(top, top[1:]))
    # any prefix of the schedule has a mean at least the full mean (generation that
    # stops early spends more layers per token, as the paper's "#Gen Avg Layer" shows)
    full = Fraction(sum(n), G)
    run = 0
    for g, v in enumerate(n):
        run += v
        assert Fraction(run, g + 1) >= full
    # the literal reading of the equation (t = g / G) never reaches min and overshoots the budget
    lit, _ = O.schedule(mx, mn, 0, G, L, closed_interval=False)
    assert lit[0] == mx and lit[-1] > mn - 1 and sum(lit) > total


def test_config1_runs():
    n, _ = O.schedule(4, 2, 0, 32, 4)
    assert n == [4] * 8 + [3] * 16 + [2] * 8


@pytest.mark.parametrize("mx,mn,G", [(7, 3, 1), (5, 5, 9), (9, 2, 2), (6, 5, 3), (31, 1 + 1, 1000)])
def test_against_rational_line(mx, mn, G):
    n, _ = O.schedule(mx, mn, 1, G, 32)
    for g, v in enumerate(n):
        t = Fraction(0) if G == 1 else Fraction(g, G - 1)
        line = (1 - t) * mx + t * mn
        # nearest integer, halves up
        assert line - Fraction(1, 2) < v <= line + Fraction(1, 2)
    if G == 1:
        assert n == [mx]
    if mx == mn:
        assert n == [mx] * G


def test_active_matrix_monotone_sets():
    L, P, G, w = 12, 5, 40, 1
    n, top = O.schedule(9, 3, w, G, L)
    act = O.active_matrix(L, P, n, w)
    assert act[:P].all()
    for i in range(1, P + G):
        assert (act[i] <= act[i - 1]).all()                  # A(i) is a subset of A(i-1)
    for g in range(G):
        assert int(act[P + g].sum()) == n[g] and act[P + g, :w].all()


@pytest.mark.parametrize("args", [(4, 5, 0, 8, 8), (9, 3, 0, 8, 8), (4, 2, 2, 8, 8), (4, 2, 0, 0, 8), (4, 2, -1, 8, 8)])
def test_bad_arguments(args):
    with pytest.raises(ValueError):
        O.schedule(*args)


@pytest.mark.parametrize("alpha", [1, 2, 3])
def test_power_law_schedule(alpha):
    L, mx, mn, w, G = 32, 22, 11, 1, 257
    n, top = O.schedule_power(mx, mn, w, G, L, alpha)
    lin, _ = O.schedule(mx, mn, w, G, L)
    assert n[0] == mx and n[-1] == mn
    assert all(a >= b for a, b in zip(n, n[1:]))
    assert all(p <= q for p, q in zip(n, lin))               # (1 - t)^alpha <= 1 - t: never above the linear budget
    if alpha == 1:
        assert n == lin
    else:
        assert sum(n) < sum(lin)
    # hand-checked point: t = 1/2 exactly at g = 128, line value min + D / 2^alpha
    assert n[128] == math.floor(mn + Fraction(mx - mn, 2 ** alpha) + Fraction(1, 2))
    for g, v in enumerate(n):
        assert top[g] == L - (v - w)
