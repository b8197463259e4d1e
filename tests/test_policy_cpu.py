"""Pins for the policy oracle (Eq. 1-3 and the measured-cost replay) against the paper's printed tables."""
import math

import numpy as np
import pytest

from kvr_synth import paper_wait_family, poisson_arrivals
from oracle import policy

B2, B3, C2, WREF = 0.02, 1.91, 425, 1800.0
LCRIT = C2 / WREF


def draws(family, mult, seed, n=4000):
    return poisson_arrivals(n, mult * LCRIT, seed), paper_wait_family(family, n, seed)


def test_cost_line_and_break_evens(golden):
    a1, b2, b3 = golden["price_vector_h100"]
    t1, tstar = policy.break_evens(a1, b2, b3)
    # at the break-even the two cost lines meet: alpha_1 t = beta_j (HBM has beta_1 = 0)
    assert policy.cost_line(a1, 0.0, t1) == pytest.approx(policy.cost_line(0.0, b2, t1))
    assert policy.cost_line(a1, 0.0, tstar) == pytest.approx(policy.cost_line(0.0, b3, tstar))
    assert abs(t1 - golden["t1_tstar_h100_printed"][0]) < 0.01 and round(tstar) == golden["t1_tstar_h100_printed"][1]


def test_congestion_price_and_timer():
    assert policy.alpha2(0.9 * LCRIT, C2, WREF, B3) == 0.0 and policy.t2(LCRIT, C2, WREF, B2, B3) == math.inf
    # at 2 lambda_crit the price is beta_3 / W_ref, so the timer is (beta_3 - beta_2) / beta_3 of W_ref
    assert policy.alpha2(2 * LCRIT, C2, WREF, B3) == pytest.approx(B3 / WREF)
    assert policy.t2(2 * LCRIT, C2, WREF, B2, B3) == pytest.approx((B3 - B2) / B3 * WREF)
    assert policy.t2(3 * LCRIT, C2, WREF, B2, B3) == pytest.approx(0.5 * (B3 - B2) / B3 * WREF)
    # host-retain at the timer costs as much as discarding: alpha_2 t_2 + beta_2 = beta_3
    lam = 2.4 * LCRIT
    assert policy.cost_line(policy.alpha2(lam, C2, WREF, B3), B2, policy.t2(lam, C2, WREF, B2, B3)) == pytest.approx(B3)


def test_wait_families_have_the_reference_mean():
    for fam in ("lognormal", "exponential", "mixture"):
        w = paper_wait_family(fam, 400000, 5)
        assert abs(w.mean() / WREF - 1) < 0.02, fam


@pytest.mark.parametrize("family", ["lognormal", "exponential", "mixture"])
def test_half_critical_load_costs_exactly_beta2(family, golden):
    arr, w = draws(family, 0.5, 1)
    cost, frac = policy.replay(arr, w, C2, math.inf, B2, B3)
    ttl_cost, _ = policy.replay(arr, w, C2, policy.t2(0.5 * LCRIT, C2, WREF, B2, B3), B2, B3)
    assert cost == pytest.approx(golden["sweep_half_load_cost"][0]) and ttl_cost == pytest.approx(cost) and frac == 1.0


# load-sweep table, fixed-timer columns at half the critical load (host not binding): lognormal 10/30/60 min,
# exponential, mixture
FIXED = {"lognormal": "sweep_fixed_lognormal", "exponential": "sweep_fixed_exponential", "mixture": "sweep_fixed_mixture"}


@pytest.mark.parametrize("family", sorted(FIXED))
def test_fixed_timers_uncongested_match_closed_form_and_table(family, golden):
    arr, w = draws(family, 0.5, 2)
    for minutes, printed in zip((10, 30, 60), golden[FIXED[family]]):
        T = 60.0 * minutes
        cost, frac = policy.replay(arr, w, C2, T, B2, B3)
        p = float(np.mean(w <= T))
        assert cost == pytest.approx(B2 * p + B3 * (1 - p)) and frac == pytest.approx(p)
        assert abs(cost - printed) < 0.04, (family, minutes, cost, printed)      # 4,000-sample noise


def test_congested_rows_and_branch_selection(golden):
    # host-retain column at 1, 2, 3 x lambda_crit (sample-dependent: loose), and the selected branches
    for family, key in (("lognormal", "sweep_retain_lognormal"), ("exponential", "sweep_retain_exponential"),
                        ("mixture", "sweep_retain_mixture")):
        for mult, printed in zip((1, 2, 3), golden[key]):
            costs = [policy.replay(*draws(family, mult, s), C2, math.inf, B2, B3)[0] for s in range(3, 8)]
            tol = 0.08 if mult == 1 else 0.06           # the critical point is the noisiest
            assert abs(float(np.mean(costs)) - printed) < tol, (family, mult, np.mean(costs), printed)
    votes = {}
    for family in ("lognormal", "exponential", "mixture"):
        picks = [policy.select_branch(*draws(family, 3, s), 3 * LCRIT, C2, WREF, B2, B3)[0] for s in range(10, 15)]
        votes[family] = max(set(picks), key=picks.count)
    assert votes == {"lognormal": "retain", "exponential": "retain", "mixture": "ttl"}


def test_replay_small_case_by_hand():
    # two slots; waits and a 10 s timer chosen so every rule fires once
    arr = [0.0, 1.0, 2.0, 12.0, 12.5]
    w = [5.0, 20.0, 3.0, 1.0, 1.0]
    # r0 admitted, resumes at 5 (beta_2); r1 admitted, timer fires at 11 before its resume at 21 (beta_3);
    # r2 arrives at 2 with both slots taken: not admitted (beta_3); r3 at 12: r0 left at 5, r1 at 11 -> admitted (beta_2);
    # r4 at 12.5: one slot free -> admitted (beta_2)
    cost, frac = policy.replay(arr, w, 2, 10.0, 1.0, 100.0)
    assert cost == pytest.approx((1 + 100 + 100 + 1 + 1) / 5) and frac == pytest.approx(3 / 5)
    # host-retain: r1 stays until 21, so r3 finds one slot (r0's) and r4 finds none
    cost, frac = policy.replay(arr, w, 2, math.inf, 1.0, 100.0)
    assert cost == pytest.approx((1 + 1 + 100 + 1 + 100) / 5) and frac == pytest.approx(3 / 5)


def test_replay_ties_by_hand():
    # one slot, a 10 s timer.  The two ties the paper leaves open, each worked by hand:
    #  * r0 (arrives 0, waits 4) leaves at 4.0; r1 arrives at exactly 4.0 -> the slot is free for it: admitted;
    #  * r1 waits exactly 10.0 = the timer -> it resumes in time: beta_2, and holds the slot until 14.0;
    #  * r2 arrives at 13.0 while r1 still holds the slot -> not admitted: beta_3;
    #  * r3 arrives at exactly 14.0 = r1's departure -> admitted; it waits 10.5 > timer -> expired at 24: beta_3;
    #  * r4 arrives at 24.0 = the instant r3's timer fired -> admitted, waits 1: beta_2.
    arr = [0.0, 4.0, 13.0, 14.0, 24.0]
    w = [4.0, 10.0, 1.0, 10.5, 1.0]
    cost, frac = policy.replay(arr, w, 1, 10.0, 1.0, 100.0)
    assert cost == pytest.approx((1 + 1 + 100 + 100 + 1) / 5) and frac == pytest.approx(3 / 5)
    # the same arrivals one tick earlier find the slot still taken
    eps = 1e-9
    cost, frac = policy.replay([0.0, 4.0 - eps, 13.0, 14.0, 24.0], w, 1, 10.0, 1.0, 100.0)
    # r1 rejected (beta_3); r2 at 13 finds the slot free (r0 left at 4): beta_2, leaves at 14 -> r3 admitted as before
    assert cost == pytest.approx((1 + 100 + 1 + 100 + 1) / 5) and frac == pytest.approx(3 / 5)


def test_replay_capacity_zero_and_empty_tier():
    # no host slots: everything recomputes; unlimited slots and no timer: everything resumes from host
    arr, w = [0.0, 1.0, 2.0], [5.0, 5.0, 5.0]
    assert policy.replay(arr, w, 0, math.inf, 1.0, 100.0) == (100.0, 0.0)
    assert policy.replay(arr, w, 3, math.inf, 1.0, 100.0) == (1.0, 1.0)


# ---- the library's policy functions against the oracle ---------------------------------------

def test_library_policy_matches_oracle():
    from paper_2608_30830_b200 import kvr
    prices = (0.0176, B2, B3)
    assert kvr.policy_break_evens(*prices) == policy.break_evens(*prices)
    for mult in (0.5, 1.0, 1.3, 2.0, 3.0):
        lam = mult * LCRIT
        a2, ttl = kvr.policy_host_ttl(prices, lam, C2, WREF)
        assert a2 == policy.alpha2(lam, C2, WREF, B3) and ttl == policy.t2(lam, C2, WREF, B2, B3)
    for family in ("lognormal", "exponential", "mixture"):
        for mult in (0.5, 2, 3):
            arr, w = draws(family, mult, 31)
            for ttl in (math.inf, 600.0, policy.t2(3 * LCRIT, C2, WREF, B2, B3)):
                want = policy.replay(arr, w, C2, ttl, B2, B3)
                got = kvr.policy_replay(prices, arr, w, C2, ttl)
                assert got[1] == want[1] and got[0] == pytest.approx(want[0], rel=1e-12)
            branch, cr, ct, t2v = kvr.policy_select(prices, arr, w, mult * LCRIT, C2, WREF)
            ob, ocr, oct_, ot2 = policy.select_branch(arr, w, mult * LCRIT, C2, WREF, B2, B3)
            assert (branch, t2v) == (ob, ot2) and cr == pytest.approx(ocr, rel=1e-12) and ct == pytest.approx(oct_, rel=1e-12)
    # the tie readings (departure exactly at an arrival; wait exactly equal to the timer)
    arr, w = [0.0, 4.0, 13.0, 14.0, 24.0], [4.0, 10.0, 1.0, 10.5, 1.0]
    assert kvr.policy_replay((1.0, 1.0, 100.0), arr, w, 1, 10.0) == pytest.approx(policy.replay(arr, w, 1, 10.0, 1.0, 100.0), rel=1e-12)
    with pytest.raises(kvr.KvrError):
        kvr.policy_break_evens(0.0, B2, B3)
    with pytest.raises(kvr.KvrError):
        kvr.policy_replay(prices, [2.0, 1.0], [1.0, 1.0], 4, math.inf)        # arrivals out of order
