"""The library's host-side rank selector against the exact-rational oracle: identical selections (integer results,
so the bar is equality), error behaviour, the callback form.  No GPU is needed: the function makes no CUDA call."""
import numpy as np
import pytest

import paper_2601_21686_b200 as S
from oracle import stief_rank_oracle as R
from paper_2601_21686_b200 import build as B
from paper_2601_21686_b200 import inputs as I

CAND = (32, 48, 64, 96, 128)


@pytest.fixture(scope="module", autouse=True)
def _built():
    B.build()


@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("rho", [0.25, 0.3, 1 / 3, 0.4375, 0.5, 0.5000000000000001, 0.61, 0.75, 0.9, 1.0])
def test_selection_equals_the_oracle(seed, rho):
    L = 32
    tabs = I.error_surfaces(seed, L)
    want, spent = R.select_ranks(L, CAND, CAND, rho, lambda l, chosen: tabs[l])
    got, got_spent = S.stief_select_ranks(L, CAND, CAND, rho, surfaces=tabs)
    assert got == want and got_spent == float(spent)


def test_boundary_budgets_are_decided_exactly():
    # a pair whose cost equals tau must be accepted; one ulp below, refused.  L = 3 makes tau = B / 3 inexact in floating
    # point: rho = 0.375 -> tau_1 = 0.375 = cost of (32,64)
    ck = cv = (32, 64, 128)
    tab = np.ones((3, 3, 3)); tab[:, 0, 1] = 0.1; tab[:, 0, 0] = 0.5
    for rho, first in ((0.375, (32, 64)), (np.nextafter(0.375, 0.0), (32, 32))):
        want, _ = R.select_ranks(3, ck, cv, float(rho), lambda l, c: tab[l])
        got, _ = S.stief_select_ranks(3, ck, cv, float(rho), surfaces=tab)
        assert got == want and got[0] == first


def test_random_small_problems_equal_the_oracle():
    rng = np.random.default_rng(7)
    for _ in range(200):
        L = int(rng.integers(1, 9))
        ck = sorted(set(rng.choice([8, 16, 24, 32, 48, 64, 96, 128], size=int(rng.integers(1, 5))).tolist()) | {128})
        cv = sorted(set(rng.choice([8, 16, 24, 32, 48, 64, 96, 128], size=int(rng.integers(1, 5))).tolist()) | {128})
        tab = np.round(rng.random((L, len(ck), len(cv))), 1)            # coarse values: ties are common
        rho = float(rng.choice([0.25, 0.3, 0.5, 0.7, 1.0, rng.random() * 0.9 + 0.1]))
        try:
            want = R.select_ranks(L, ck, cv, rho, lambda l, c: tab[l])[0]
        except R.Infeasible as e:
            with pytest.raises(S.StiefError) as err:
                S.stief_select_ranks(L, ck, cv, rho, surfaces=tab)
            assert err.value.code == S.STIEF_ERR_INFEASIBLE and f"layer {e.layer}" in str(err.value)
            continue
        assert S.stief_select_ranks(L, ck, cv, rho, surfaces=tab)[0] == want


def test_callback_sees_the_chosen_prefix_and_matches_the_oracle():
    L = 12
    tabs = I.error_surfaces(4, L)
    def surface(l, chosen):
        # error grows with how much the earlier layers were compressed (propagated error)
        lost = sum(2.0 - (rk + rv) / 128.0 for rk, rv in chosen)
        return tabs[l] * (1.0 + 0.05 * lost)
    want, _ = R.select_ranks(L, CAND, CAND, 0.5, surface)
    seen = []
    def spy(l, chosen):
        seen.append((l, list(chosen)))
        return surface(l, chosen)
    got, _ = S.stief_select_ranks(L, CAND, CAND, 0.5, surface=spy)
    assert got == want
    assert [l for l, _ in seen] == list(range(L)) and all(c == want[:l] for l, c in seen)


def test_argument_errors():
    tabs = I.error_surfaces(0, 4)
    for kw in (dict(rho=0.0), dict(rho=1.5), dict(rho=float("nan"))):
        with pytest.raises(S.StiefError) as e:
            S.stief_select_ranks(4, CAND, CAND, kw["rho"], surfaces=tabs)
        assert e.value.code == S.STIEF_ERR_INVALID_ARG
    with pytest.raises(S.StiefError):
        S.stief_select_ranks(4, CAND, CAND, 0.5)                                   # no table source
    with pytest.raises(S.StiefError):
        S.stief_select_ranks(4, (32, 256), CAND, 0.5, surfaces=I.error_surfaces(0, 4, (32, 256), CAND))   # rank above d_h
    bad = tabs.copy(); bad[2, 1, 1] = np.nan
    with pytest.raises(S.StiefError) as e:
        S.stief_select_ranks(4, CAND, CAND, 0.5, surfaces=bad)
    assert "layer 2" in str(e.value)
    with pytest.raises(ZeroDivisionError):
        S.stief_select_ranks(4, CAND, CAND, 0.5, surface=lambda l, c: 1 / 0)     # the callback's exception surfaces
    with pytest.raises(S.StiefError) as e:
        S.stief_select_ranks(4, CAND, CAND, 0.2, surfaces=tabs)
    assert e.value.code == S.STIEF_ERR_INFEASIBLE


def test_selected_profile_is_usable_by_the_library():
    ranks, spent = S.stief_select_ranks(32, CAND, CAND, 0.5, surfaces=I.error_surfaces(0, 32))
    assert all(rk in CAND and rv in CAND for rk, rv in ranks) and spent <= 16.0
    # cache bytes per token follow from the profile (Eq. 3 summed over layers): ratio to the uncompressed cache = spent / L
    assert abs(sum(rk + rv for rk, rv in ranks) / (32 * 256) - spent / 32) < 1e-15
