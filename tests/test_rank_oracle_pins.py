"""Pins of the rank-selector oracle (Algorithm 2) to things other than itself: hand-worked cases, closed forms and
invariants that follow from Eq. 15-17, each chosen so that a plausible slip (wrong divisor, budget not carried over,
constraint against the wrong quantity, arg-max instead of arg-min) fails one of them."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import stief_rank_oracle as R
from paper_2601_21686_b200 import inputs as I

CAND = (32, 48, 64, 96, 128)


def _static(tables):
    return lambda l, chosen: tables[l]


def test_hand_worked_two_layers_carry_the_unspent_budget_forward():
    # L=2, candidates {64,128}, rho=0.75.  B_1 = 1.5, tau_1 = 0.75: (128,128) (cost 1) does not fit; of the other three
    # the table makes (64,64) (cost 0.5) the best.  B_2 = 1.0, tau_2 = 1.0: everything fits and (128,128) has error 0.
    t0 = [[0.10, 0.30], [0.20, 0.0]]
    t1 = [[0.90, 0.50], [0.40, 0.0]]
    ranks, spent = R.select_ranks(2, (64, 128), (64, 128), 0.75, _static([t0, t1]))
    assert ranks == [(64, 64), (128, 128)] and spent == Fraction(3, 2)


def test_hand_worked_three_layers():
    # L=3, rho=0.5, candidates {32,64,128}: B_1=1.5, tau_1=0.5 -> feasible costs <= 0.5: (32,32) .25, (32,64)/(64,32) .375,
    # (64,64) .5.  Layer 1 prefers (32,64).  B_2=1.125, tau_2=.5625: (32,128)/(128,32) cost .625 still out; layer 2 takes (64,64).
    # B_3=.625, tau_3=.625: now (32,128) fits and is layer 3's best.
    ck = cv = (32, 64, 128)
    def tab(best):
        t = [[1.0 + 0.01 * (i * 3 + j) for j in range(3)] for i in range(3)]
        t[2][2] = 0.0
        t[best[0]][best[1]] = 0.5
        return t
    tabs = [tab((0, 1)), tab((1, 1)), tab((0, 2))]
    ranks, spent = R.select_ranks(3, ck, cv, 0.5, _static(tabs))
    assert ranks == [(32, 64), (64, 64), (32, 128)]
    assert spent == Fraction(96 + 128 + 160, 256) == Fraction(3, 2)


def test_divisor_is_the_number_of_layers_left():
    # With the divisor printed in Eq. 15 the last-but-one layer would divide by zero and the first layer of an L=2 model
    # would see tau = B_1 / (2 - 2); with an off-by-one the first layer could spend more than its share: here tau_1 must be
    # exactly rho, so the full-rank pair (error 0, cost 1) must NOT be taken at rho = 0.75 although it has the least error.
    t = [[0.3, 0.2], [0.1, 0.0]]
    ranks, _ = R.select_ranks(2, (64, 128), (64, 128), 0.75, _static([t, t]))
    assert ranks[0] == (128, 64)            # least error among cost <= 0.75
    assert ranks[1] == (128, 64)            # B_2 = 0.75, tau_2 = 0.75


def test_identical_monotone_layers_give_the_uniform_allocation():
    # error strictly decreasing in both ranks, same table everywhere, rho equal to the cost of the pair (r, r): the
    # cheapest-error feasible pair costs exactly tau every time, nothing is carried over and every layer gets the same
    # pair with total cost L rho.  (64,64) vs (32,96) vs (96,32) all cost 0.5: the table makes (64,64) the best of them.
    tab = [[(2.0 - rk / 128) ** 2 + (2.0 - rv / 128) ** 2 + 3.0 * abs(rk - rv) / 128 for rv in CAND] for rk in CAND]
    tab[4][4] = 0.0
    ranks, spent = R.select_ranks(7, CAND, CAND, 0.5, _static([tab] * 7))
    assert ranks == [(64, 64)] * 7 and spent == Fraction(7, 2)


def test_rho_one_keeps_everything_full_rank_and_rho_below_the_cheapest_pair_is_infeasible():
    tabs = I.error_surfaces(5, 6)
    ranks, spent = R.select_ranks(6, CAND, CAND, 1.0, _static(tabs))
    assert ranks == [(128, 128)] * 6 and spent == 6
    with pytest.raises(R.Infeasible) as e:
        R.select_ranks(6, CAND, CAND, 0.2499, _static(tabs))
    assert e.value.layer == 0
    R.select_ranks(6, CAND, CAND, 0.25, _static(tabs))      # exactly the cheapest pair's cost: feasible to the end


@pytest.mark.parametrize("rho", [0.25, 0.3, 0.4375, 0.5, 0.61, 0.75, 0.9])
def test_invariants_on_synthetic_surfaces(rho):
    L = 32
    tabs = I.error_surfaces(11, L)
    ranks, spent = R.select_ranks(L, CAND, CAND, rho, _static(tabs))
    costs = [Fraction(rk + rv, 256) for rk, rv in ranks]
    assert sum(costs) == spent <= L * Fraction(rho)                     # the budget is never exceeded
    left = L * Fraction(rho)
    for l, (rk, rv) in enumerate(ranks):
        tau = left / (L - l)
        assert costs[l] <= tau
        chosen = tabs[l][CAND.index(rk)][CAND.index(rv)]
        for i, a in enumerate(CAND):                                      # nothing feasible is strictly better
            for j, b in enumerate(CAND):
                if Fraction(a + b, 256) <= tau:
                    assert tabs[l][i][j] >= chosen
        left -= costs[l]
    # what is left at the end is less than the step to the next costlier pair could use: no layer is starved while
    # budget for an upgrade of the LAST layer remains
    last_tau = left + costs[-1]
    better = [tabs[-1][i][j] for i, a in enumerate(CAND) for j, b in enumerate(CAND) if Fraction(a + b, 256) <= last_tau]
    assert min(better) == tabs[-1][CAND.index(ranks[-1][0])][CAND.index(ranks[-1][1])]


def test_surface_is_asked_for_after_the_prefix_is_chosen():
    seen = []
    tabs = I.error_surfaces(3, 4)
    def surface(l, chosen):
        seen.append((l, tuple(chosen)))
        return tabs[l] * (1.0 + 0.1 * len(chosen))
    ranks, _ = R.select_ranks(4, CAND, CAND, 0.5, surface)
    assert [s[0] for s in seen] == [0, 1, 2, 3]
    for l, prefix in seen:
        assert list(prefix) == ranks[:l]


def test_ties_take_the_cheaper_pair_then_the_smaller_key_rank():
    flat = [[0.0] * 3 for _ in range(3)]
    ranks, _ = R.select_ranks(2, (32, 64, 128), (32, 64, 128), 0.5, _static([flat, flat]))
    assert ranks[0] == (32, 32)
    t = [[1.0, 0.2, 1.0], [0.2, 1.0, 1.0], [1.0, 1.0, 1.0]]             # (32,64) and (64,32): same error, same cost
    ranks, _ = R.select_ranks(1, (32, 64, 128), (32, 64, 128), 0.5, _static([t]))
    assert ranks[0] == (32, 64)


def test_synthetic_profile_has_the_reported_shape():
    # the generator is built to mimic the measured surfaces; the selector on it should then reproduce the trends the
    # paper describes for its profiles (appendix on selected ranks): values keep more rank than keys on average, and the
    # first and last layers keep more than the middle.
    L = 32
    ranks, _ = R.select_ranks(L, CAND, CAND, 0.5, _static(I.error_surfaces(0, L)))
    rk = np.array([r[0] for r in ranks]); rv = np.array([r[1] for r in ranks])
    assert rv.mean() > rk.mean()
    tot = rk + rv
    assert tot[:4].mean() > tot[12:20].mean() and tot[-4:].mean() > tot[12:20].mean()
