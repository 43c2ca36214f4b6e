"""Pins for the oracle's budget schedule (Section 4.2.1, Eq. 1)."""
import os
from fractions import Fraction

import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

CASES = [
    (2, 64, 8, 20.0), (32, 128, 32, 20.0), (32, 512, 32, 20.0), (80, 128, 32, 20.0),
    (32, 64, 32, 20.0), (32, 2048, 32, 20.0), (32, 256, 32, 20.0), (32, 128, 8, 20.0),
    (32, 64, 8, 14.0), (32, 64, 8, 16.0), (32, 64, 8, 18.0), (48, 96, 16, 20.0),
    (7, 33, 5, 3.5), (3, 1000, 48, 1.0), (1, 77, 8, 20.0), (5, 8, 8, 20.0),
]


def eq1_real(m, B, alpha, beta):
    """Eq. 1 taken literally, in rationals: top layer, bottom layer, arithmetic sequence."""
    beta = Fraction(round(beta * 1024), 1024)
    k_total = Fraction(m * (B - alpha))
    if m == 1:
        return [k_total]
    k_top = k_total / (beta * m)
    k_bot = 2 * k_total / m - k_top
    return [k_bot - (k_bot - k_top) * l / (m - 1) for l in range(m)]


@pytest.mark.parametrize("m,B,alpha,beta", CASES)
def test_sum_is_total_and_shape_is_pyramid(m, B, alpha, beta):
    k = oracle.layer_budgets(m, B, alpha, beta)
    assert len(k) == m
    assert sum(k) == m * (B - alpha)                       # budgets sum to the total
    assert sum(x + alpha for x in k) == m * B              # capacities sum to m * B
    assert all(a >= b for a, b in zip(k, k[1:]))           # non-increasing with depth
    assert all(x >= 0 for x in k)


@pytest.mark.parametrize("m,B,alpha,beta", CASES)
def test_within_one_of_eq1(m, B, alpha, beta):
    k = oracle.layer_budgets(m, B, alpha, beta)
    real = eq1_real(m, B, alpha, beta)
    for got, want in zip(k, real):
        assert abs(Fraction(got) - want) <= 1
    # endpoints: k^{m-1} ~ k_total/(beta m); k^0 + k^{m-1} ~ 2 k_total / m
    if m > 1:
        assert abs(Fraction(k[0] + k[-1]) - Fraction(2 * m * (B - alpha), m)) < 2


@pytest.mark.parametrize("m,B,alpha,beta", CASES)
def test_floor_then_leftover_to_lowest_layers(m, B, alpha, beta):
    k = oracle.layer_budgets(m, B, alpha, beta)
    floors = [int(x // 1) for x in eq1_real(m, B, alpha, beta)]
    left = m * (B - alpha) - sum(floors)
    assert 0 <= left < max(m, 2)
    want = [f + (1 if l < left else 0) for l, f in enumerate(floors)]
    assert k == want


@pytest.mark.parametrize("m,B,alpha,beta", [c for c in CASES if c[0] >= 3])
def test_arithmetic_sequence_second_differences(m, B, alpha, beta):
    k = oracle.layer_budgets(m, B, alpha, beta)
    d1 = [a - b for a, b in zip(k, k[1:])]
    d2 = [a - b for a, b in zip(d1, d1[1:])]
    assert all(abs(x) <= 2 for x in d2)
    assert max(d1) - min(d1) <= 2


def test_hand_computed_rows():
    # m=2, B=64, alpha=8, beta=20: k_total=112, top=112/40=2.8, bottom=112-2.8=109.2 -> 109,2 (+1) = 110,2
    assert oracle.layer_budgets(2, 64, 8, 20.0) == [110, 2]
    # m=32, B=128, alpha=32: k_total=3072, top=4.8, bottom=187.2, step=182.4/31
    k = oracle.layer_budgets(32, 128, 32, 20.0)
    assert k[:3] == [188, 182, 176] and k[-2:] == [10, 4]
    # m=80, same B: top=4.8, bottom=187.2, step=182.4/79
    k = oracle.layer_budgets(80, 128, 32, 20.0)
    assert k[:3] == [188, 185, 183] and k[-2:] == [7, 4]
    # m=32, B=128, alpha=8: k_total=3840, top=6, bottom=234
    k = oracle.layer_budgets(32, 128, 8, 20.0)
    assert k[0] in (234, 235) and k[-1] == 6


def test_beta_one_is_uniform():
    for m, B, alpha in [(32, 128, 32), (5, 100, 8), (80, 64, 8)]:
        assert oracle.layer_budgets(m, B, alpha, 1.0) == [B - alpha] * m


def test_rejects_undefined_arguments():
    for args in [(0, 64, 8, 20.0), (4, 7, 8, 20.0), (4, 64, 0, 20.0), (4, 64, 8, 0.5),
                 (4, 64, 8, float("nan"))]:
        with pytest.raises(ValueError):
            oracle.layer_budgets(*args)


def test_table2_memory_is_linear_in_average_size():
    """Table 2: memory 428/856/1712/6848 MB for average sizes 512/1024/2048/8192 (full)."""
    rows = []
    with open(os.path.join(GOLDEN, "table2_memory.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                size, mb = line.split()
                rows.append((int(size), int(mb)))
    m, alpha, n = 32, 8, 8192
    full_size, full_mb = rows[-1]
    assert full_size == n
    for size, mb in rows:
        k = oracle.layer_budgets(m, size, alpha, 20.0)
        kept = sum(oracle.kept_count(size, alpha, kl, n) for kl in k)
        # kept rows over all layers, relative to the full cache, equals the table's memory ratio
        assert Fraction(kept, m * n) == Fraction(mb, full_mb)


def test_kept_count_rules():
    assert oracle.kept_count(128, 32, 100, 4096) == 132
    assert oracle.kept_count(128, 32, 100, 128) == 128      # context fits the budget: keep all
    assert oracle.kept_count(128, 32, 100, 100) == 100
    assert oracle.kept_count(128, 32, 188, 140) == 140      # budget exceeds the prefix
    assert oracle.kept_count(128, 32, 4, 140) == 36


# --------------------------------------------------------------------------------------------------
# Geometric decay (appendix "Allocation Strategies"): constant ratio between consecutive layers, the
# same two end constraints as Eq. 1 (top layer k_total / (beta m), budgets sum to k_total).

GEO_CASES = [c for c in CASES] + [(32, 64, 8, 20.0), (32, 64, 8, 2.0), (80, 2048, 32, 20.0), (16, 300, 16, 5.25)]


def geo_ratio(m, beta):
    """Root rho >= 1 of 1 + rho + ... + rho^(m-1) = beta m in rationals (bisection to 2^-60), then snapped to
    a multiple of 2^-20 as the reading says."""
    beta = Fraction(round(beta * 1024), 1024)
    if m == 1 or beta == 1:
        return Fraction(1)
    lo, hi = Fraction(1), beta * m
    while hi - lo > Fraction(1, 2 ** 60):
        mid = (lo + hi) / 2
        if sum(mid ** j for j in range(m)) < beta * m:
            lo = mid
        else:
            hi = mid
    return Fraction(round(lo * 2 ** 20), 2 ** 20)


def geo_real(m, B, alpha, beta):
    rho = geo_ratio(m, beta)
    total = sum(rho ** j for j in range(m))
    return [Fraction(m * (B - alpha)) * rho ** (m - 1 - l) / total for l in range(m)]


@pytest.mark.parametrize("m,B,alpha,beta", GEO_CASES)
def test_geometric_sum_shape_and_exact_floors(m, B, alpha, beta):
    k = oracle.layer_budgets(m, B, alpha, beta, schedule="geometric")
    assert sum(k) == m * (B - alpha)
    assert all(a >= b for a, b in zip(k, k[1:])) and all(x >= 0 for x in k)
    real = geo_real(m, B, alpha, beta)
    floors = [int(x // 1) for x in real]
    left = m * (B - alpha) - sum(floors)
    assert 0 <= left < max(m, 2)
    assert k == [f + (1 if l < left else 0) for l, f in enumerate(floors)]


@pytest.mark.parametrize("m,B,alpha,beta", [c for c in GEO_CASES if c[0] >= 2])
def test_geometric_end_constraints_and_constant_ratio(m, B, alpha, beta):
    k = oracle.layer_budgets(m, B, alpha, beta, schedule="geometric")
    bq = Fraction(round(beta * 1024), 1024)
    k_total = m * (B - alpha)
    # top layer: k_total / (beta m), up to the floor, a leftover unit and the 2^-20 snap of the ratio
    assert abs(Fraction(k[-1]) - Fraction(k_total) / (bq * m)) <= Fraction(3, 2)
    rho = geo_ratio(m, beta)
    for a, b in zip(k, k[1:]):                             # consecutive budgets: a ~ rho * b, both within 1 of real
        assert abs(Fraction(a) - rho * b) <= 1 + rho
    # the ratio solves the geometric-sum equation (to the snap)
    if bq > 1:
        assert abs(sum(rho ** j for j in range(m)) - bq * m) <= bq * m * m * Fraction(1, 2 ** 20)


def test_geometric_special_cases():
    # beta = 1: no decay at all
    for m, B, alpha in [(32, 128, 32), (5, 100, 8), (80, 64, 8)]:
        assert oracle.layer_budgets(m, B, alpha, 1.0, schedule="geometric") == [B - alpha] * m
    # two layers: both end constraints fix both budgets, so every decay shape gives Eq. 1's split
    for B, alpha, beta in [(64, 8, 20.0), (1000, 48, 3.5), (77, 8, 1.25), (2048, 32, 14.0)]:
        assert oracle.layer_budgets(2, B, alpha, beta, schedule="geometric") == oracle.layer_budgets(2, B, alpha, beta)
    # three layers: 1 + rho + rho^2 = 3 beta has the closed form rho = (sqrt(12 beta - 3) - 1) / 2;
    # beta = 7: rho = 4, shares 16 : 4 : 1 of k_total = 3 * 70 = 210 -> 160, 40, 10
    assert oracle.layer_budgets(3, 78, 8, 7.0, schedule="geometric") == [160, 40, 10]
    # beta = 13/3 is not on the 1/1024 grid; beta = 1 + 2 + 4 = 7 over m = 3 was; try m = 4, rho = 2: beta m = 15
    assert oracle.layer_budgets(4, 23, 8, 3.75, schedule="geometric") == [32, 16, 8, 4]
    assert oracle.layer_budgets(1, 77, 8, 20.0, schedule="geometric") == [69]


@pytest.mark.parametrize("m,B,alpha,beta", [c for c in GEO_CASES if c[0] >= 3 and c[3] > 1.0])
def test_geometric_is_front_loaded_against_linear(m, B, alpha, beta):
    """Same top layer and same sum, but convex: the lowest layer gets more than under Eq. 1 and the layers
    just below the top get less."""
    geo = oracle.layer_budgets(m, B, alpha, beta, schedule="geometric")
    lin = oracle.layer_budgets(m, B, alpha, beta)
    assert geo[0] >= lin[0]
    assert geo[-2] <= lin[-2] + 1
