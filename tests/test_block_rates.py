"""Block-rate selection ("Heterogeneous Block-Rate Optimization"): pins of the brute-force oracle,
then the library's solver against it.  No GPU is involved anywhere in this file."""
import json
import os

import numpy as np
import pytest

from oracle import block_rates as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "block_rates_hand_worked.json")


def _random_problem(rng, n_blocks, n_rates, integer_costs):
    """Costs fall and errors grow with the rate index, as for real hybrid rates; some noise on both."""
    base_c = np.sort(rng.uniform(1.0, 10.0, n_rates))[::-1]
    cost = base_c[None, :] * rng.uniform(0.9, 1.1, (n_blocks, n_rates))
    if integer_costs:
        cost = np.round(cost)
    err = np.cumsum(rng.uniform(0.0, 2.0, (n_blocks, n_rates)), axis=1) * rng.uniform(0.2, 3.0, (n_blocks, 1))
    err[:, 0] = 0.0
    return cost, err


# ------------------------------------------------------------------ oracle pins
def test_oracle_hand_worked_instance():
    g = json.load(open(GOLDEN))
    best_err, best = O.select_block_rates_bruteforce(g["cost"], g["err"], g["budget"])
    assert best_err == g["best_err"]
    assert best == [tuple(g["best_choice"])]
    assert O.total(g["cost"], best[0]) == g["best_cost"]


def test_oracle_unbounded_budget_takes_the_smallest_error_per_block():
    rng = np.random.default_rng(1)
    cost, err = _random_problem(rng, 5, 4, False)
    err = err + rng.uniform(0, 1, err.shape)          # no ties, minimum not always at index 0
    best_err, best = O.select_block_rates_bruteforce(cost, err, 1e9)
    assert best == [tuple(int(i) for i in err.argmin(axis=1))]
    assert best_err == pytest.approx(err.min(axis=1).sum(), rel=1e-14)


def test_oracle_tightest_budget_takes_the_cheapest_rate_per_block_and_less_is_infeasible():
    rng = np.random.default_rng(2)
    cost, err = _random_problem(rng, 5, 4, False)
    cheapest = tuple(int(i) for i in cost.argmin(axis=1))
    beta = O.total(cost, cheapest)
    best_err, best = O.select_block_rates_bruteforce(cost, err, beta)
    assert best == [cheapest]
    assert O.select_block_rates_bruteforce(cost, err, np.nextafter(beta, 0.0)) is None


def test_oracle_single_rate_is_the_homogeneous_selection():
    cost = [[3.0], [4.0], [5.0]]
    err = [[1.0], [2.0], [3.0]]
    assert O.select_block_rates_bruteforce(cost, err, 12.0) == (6.0, [(0, 0, 0)])
    assert O.select_block_rates_bruteforce(cost, err, 11.9) is None


def test_oracle_error_is_monotone_in_the_budget_and_scale_invariant():
    rng = np.random.default_rng(3)
    cost, err = _random_problem(rng, 6, 3, True)
    lo, hi = cost.min(axis=1).sum(), cost.max(axis=1).sum()
    prev = None
    for beta in np.linspace(lo, hi, 9):
        res = O.select_block_rates_bruteforce(cost, err, beta)
        assert res is not None
        if prev is not None:
            assert res[0] <= prev
        prev = res[0]
        # costs and budget times a power of two: the same assignments, bit for bit
        assert O.select_block_rates_bruteforce(cost * 4.0, err, beta * 4.0) == res


def test_oracle_reports_every_optimal_assignment_on_ties():
    cost = [[2.0, 1.0], [2.0, 1.0]]
    err = [[0.0, 1.0], [0.0, 1.0]]
    assert O.select_block_rates_bruteforce(cost, err, 3.0) == (1.0, [(0, 1), (1, 0)])
