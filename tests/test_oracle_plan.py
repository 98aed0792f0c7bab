"""Pins for the checker's budget planner (Section 3.3, Eq. (5)(6)(7)) against what the
paper and exact arithmetic fix."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import spindlekv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _table3():
    vals = {}
    with open(os.path.join(GOLDEN, "table3_hyperparameters.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, v = line.split()
            vals[k] = float(v)
    return vals


def test_alpha_matches_table3():
    t = _table3()
    # alpha = (1 + beta) / 2 and the paper prints alpha = 0.525 for beta = 0.05
    r0, r1 = O.pyramid_endpoints(t["alpha"], t["beta"])
    assert r0 == pytest.approx(1.0, abs=1e-15)
    assert r1 == pytest.approx(t["beta"], abs=1e-15)
    # just above alpha the other branch must give the same end points
    r0b, r1b = O.pyramid_endpoints(t["alpha"] + 1e-12, t["beta"])
    assert r0b == 1.0
    assert r1b == pytest.approx(t["beta"], abs=1e-11)


@pytest.mark.parametrize("beta", [0.05, 0.1, 0.2])
@pytest.mark.parametrize("m", [2, 3, 16, 32, 40])
def test_mean_over_layers_is_rc_and_range(beta, m):
    for r_c in np.linspace(beta + 1e-3, 1.0, 23):
        r0, r1 = O.pyramid_endpoints(float(r_c), beta)
        rs = [O.layer_ratio(r0, r1, m, lam, float(r_c)) for lam in range(m)]
        assert np.mean(rs) == pytest.approx(r_c, rel=1e-12)
        assert all(beta - 1e-12 <= r <= 1.0 + 1e-12 for r in rs)
        assert all(rs[i] >= rs[i + 1] - 1e-15 for i in range(m - 1))  # pyramid: non-increasing with depth
        assert rs[0] == r0 and rs[-1] == pytest.approx(r1, rel=1e-12)


def test_budget_errors():
    with pytest.raises(O.BudgetError):
        O.pyramid_endpoints(0.05, 0.05)  # r_c <= beta: undefined
    with pytest.raises(O.BudgetError):
        O.pyramid_endpoints(1.0001, 0.05)
    with pytest.raises(O.BudgetError):
        O.plan_layers(2, 1, [32], 32, 0.05, budget_tokens=16)  # l == l_w


def test_single_evicting_layer_is_flat():
    assert O.layer_ratio(0.3, 0.05, 1, 0, 0.2) == 0.2


def _exact_plan(n_deep, l, l_w, budget, beta):
    """Eq. (5)(6)(7) in exact rational arithmetic."""
    l_c = l - l_w
    r_c = (Fraction(budget) - l_w) / l_c
    beta = Fraction(beta)
    alpha = (1 + beta) / 2
    if beta < r_c <= alpha:
        r0, r1 = 2 * r_c - beta, beta
    else:
        assert alpha < r_c <= 1
        r0, r1 = Fraction(1), 2 * r_c - 1
    out = []
    for lam in range(n_deep):
        r = r_c if n_deep == 1 else r0 + (r1 - r0) / (n_deep - 1) * lam
        out.append(r * l_c)
    return out


def test_topk_sizes_against_exact_rationals():
    rng = np.random.default_rng(7)
    checked = 0
    for _ in range(300):
        l = int(rng.integers(200, 40000))
        l_w = int(rng.choice([16, 32, 64]))
        m = int(rng.integers(1, 41))
        l_c = l - l_w
        budget = int(rng.integers(int(0.06 * l_c) + l_w + 1, l))
        beta = Fraction(1, 20)
        exact = _exact_plan(m, l, l_w, budget, beta)
        _, ratio, k = O.plan_layers(m, 0, [l], l_w, 0.05, budget_tokens=budget)
        for lam, x in enumerate(exact):
            if abs(x - round(x)) < Fraction(1, 10 ** 6):
                continue  # a product that is an integer in exact arithmetic: floor of the double may go either way
            assert k[lam, 0] == min(l_c, int(x.__floor__())), (l, l_w, m, budget, lam)
            checked += 1
        tot = sum(exact)
        assert tot - m < int(k.sum()) <= tot + 1e-6
    assert checked > 1000


def test_named_configurations():
    # tiny case: one evicting layer, 128 kept per head with a 32-token window -> 96 context tokens
    mode, ratio, k = O.plan_layers(2, 1, [512], 32, 0.05, budget_tokens=128)
    assert list(mode) == [O.MODE_CODEBOOK, O.MODE_EVICT]
    assert k[0, 0] == 480 and k[1, 0] == 96
    # 8B shape, 16 evicting layers (hand arithmetic: r_c = 480/4064, 992/16352)
    _, _, k = O.plan_layers(32, 16, [4096], 32, 0.05, budget_tokens=512)
    assert k[16, 0] == 756 and k[31, 0] == 203
    _, _, k = O.plan_layers(32, 16, [16384], 32, 0.05, budget_tokens=1024)
    assert k[16, 0] == 1166 and k[31, 0] == 817
    _, _, k = O.plan_layers(80, 40, [32768], 32, 0.05, budget_tokens=2048)
    assert k[40, 0] == 2395 and k[79, 0] == 1636


def test_reserve_ratio_and_token_budget_agree():
    a = O.plan_layers(8, 2, [1000, 3000], 32, 0.05, reserve_ratio=0.25)
    for s, l in enumerate([1000, 3000]):
        b = O.plan_layers(8, 2, [l], 32, 0.05, budget_tokens=0.25 * l)
        assert np.array_equal(a[2][:, s], b[2][:, 0])
