"""Pins for the oracle's budget rules (Eq. 9-15): hand-derived examples and invariants.  CPU only."""
import numpy as np
import pytest

from oracle import maskkv_oracle as O
from golden_io import head_budget_cases, layer_budget_cases


@pytest.mark.parametrize("case", layer_budget_cases(), ids=lambda c: f"kp{c['k_p']}_b{c['beta']}")
def test_layer_budgets_golden(case):
    assert O.layer_budgets(case["k_p"], case["beta"], case["importance"], case["is_boundary"]) == case["expected"]


def test_layer_budgets_default_boundary_is_first_and_last():
    c = layer_budget_cases()[0]
    assert O.layer_budgets(c["k_p"], c["beta"], c["importance"]) == c["expected"]


def test_layer_budgets_invariants():
    rng = np.random.default_rng(0)
    for _ in range(300):
        L = int(rng.integers(3, 48))
        k_p = int(rng.integers(L, 40000))
        beta = float(rng.uniform(0, 1))
        imp = rng.uniform(0.01, 1.0, L)
        k = O.layer_budgets(k_p, beta, imp)
        # only floors lose budget: the base remainder is carried in k_imp, each group loses < its size
        assert k_p - L < sum(k) <= k_p
        assert min(k) >= int(np.floor(beta * k_p / L + 1e-6))
        assert k[0] == k[-1] and len(set(k[1:-1])) == 1
        # more important group (per layer) never gets less
        if imp[[0, -1]].mean() >= imp[1:-1].mean():
            assert k[0] >= k[1]


def test_layer_budgets_equal_importance_is_uniform_up_to_floor():
    k = O.layer_budgets(32 * 256, 0.4, [1.0] * 32)
    assert set(k) == {256}


@pytest.mark.parametrize("case", head_budget_cases(), ids=lambda c: f"kl{c['k_l']}_a{c['alpha']}_n{c['n']}")
def test_head_budgets_golden(case):
    mp = np.array([case["mass_p"]], np.float64)
    mm = np.array([case["mass_m"]], np.float64)
    b, off = O.head_budgets(mp, mm, case["k_l"], case["alpha"], [case["n"]])
    assert b[0].tolist() == case["expected"]
    assert off.tolist() == np.concatenate([[0], np.cumsum(case["expected"])]).tolist()


def test_head_budgets_invariants_and_uniform_cases():
    rng = np.random.default_rng(1)
    for _ in range(300):
        Hkv = int(rng.choice([4, 8, 32]))
        R = int(rng.integers(1, 4))
        k_l = int(rng.integers(1, 2000))
        alpha = float(rng.uniform(0, 1))
        mp = rng.uniform(1, 200, (R, Hkv)).astype(np.float32)
        mm = rng.uniform(1, 200, (R, Hkv)).astype(np.float32)
        b, off = O.head_budgets(mp, mm, k_l, alpha, [10 ** 9] * R)
        tot = b.sum(1)
        assert ((Hkv * k_l - Hkv < tot) & (tot <= Hkv * k_l)).all()
        assert off[-1] == b.sum() and (np.diff(off) == b.reshape(-1)).all()
        # monotone in the prompt preference
        p = mp.astype(np.float64) / (mp.astype(np.float64) + mm)
        for r in range(R):
            order = np.argsort(p[r])
            assert (np.diff(b[r][order]) >= 0).all()
        # alpha = 1 and uniform preference both give k_l everywhere (the guarded floor case)
        b1, _ = O.head_budgets(mp, mm, k_l, 1.0, [10 ** 9] * R)
        assert (b1 == k_l).all()
        bu, _ = O.head_budgets(np.full((R, Hkv), 7.0, np.float32), np.full((R, Hkv), 3.0, np.float32), k_l, alpha, [10 ** 9] * R)
        assert (bu == k_l).all()


def test_head_budgets_per_request_k_and_clamp_and_capacity():
    mp = np.array([[3, 1], [1, 1], [2, 2]], np.float32)
    mm = np.array([[1, 3], [1, 1], [2, 2]], np.float32)
    b, off = O.head_budgets(mp, mm, [100, 50, 10], 0.0, [1000, 40, 1000])
    # request 0: P = .75/.25 -> 2*100*[.75,.25]; request 1: 50 each clamped to 40; request 2: 10 each
    assert b.tolist() == [[150, 50], [40, 40], [10, 10]]
    assert off.tolist() == [0, 150, 200, 240, 280, 290, 300]
    b, off = O.head_budgets(mp, mm, [100, 50, 10], 0.0, [1000, 40, 1000], capacity=215)
    assert b.tolist() == [[150, 50], [15, 0], [0, 0]] and off[-1] == 215
