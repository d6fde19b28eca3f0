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


# ------------------------------------------------------------------ the library's solver
@pytest.fixture(scope="module")
def solver():
    from paper_2509_24899_b200 import binding
    binding.lib()                       # raises when the library has not been built
    return binding


def _check_against_oracle(solver, cost, err, budget):
    ref = O.select_block_rates_bruteforce(cost, err, budget)
    if ref is None:
        with pytest.raises(solver.AsError) as ei:
            solver.as_select_block_rates(cost, err, budget)
        assert ei.value.status == solver.AS_ERR_INFEASIBLE
        return None
    choice, tc, te = solver.as_select_block_rates(cost, err, budget)
    # the minimal error is unique; the assignment only has to be one of those reaching it
    assert tuple(choice) in ref[1]
    assert te == O.total(err, choice) == ref[0]
    assert tc == O.total(cost, choice) and tc <= budget
    return choice


def test_solver_hand_worked_instance(solver):
    g = json.load(open(GOLDEN))
    choice, tc, te = solver.as_select_block_rates(g["cost"], g["err"], g["budget"])
    assert (choice, tc, te) == (g["best_choice"], g["best_cost"], g["best_err"])


@pytest.mark.parametrize("seed", range(12))
def test_solver_matches_bruteforce_on_small_problems(solver, seed):
    rng = np.random.default_rng(100 + seed)
    n_blocks, n_rates = int(rng.integers(1, 8)), int(rng.integers(1, 5))
    cost, err = _random_problem(rng, n_blocks, n_rates, integer_costs=bool(seed % 2))
    lo, hi = cost.min(axis=1).sum(), cost.max(axis=1).sum()
    for beta in [lo * 0.99, lo, lo + 0.3 * (hi - lo), lo + 0.7 * (hi - lo), hi, hi * 2]:
        _check_against_oracle(solver, cost.tolist(), err.tolist(), float(beta))


def test_solver_budget_met_exactly_and_ties(solver):
    cost = [[2.0, 1.0], [2.0, 1.0]]
    err = [[0.0, 1.0], [0.0, 1.0]]
    assert _check_against_oracle(solver, cost, err, 3.0) in ([0, 1], [1, 0])
    assert _check_against_oracle(solver, cost, err, 4.0) == [0, 0]
    assert _check_against_oracle(solver, cost, err, 2.0) == [1, 1]
    _check_against_oracle(solver, cost, err, 1.5)            # infeasible


def test_solver_stack_sized_problem_has_the_properties_of_an_optimum(solver):
    """30 blocks, 5 rates (the block-rate stack): too large to enumerate, so check what must hold at any
    size - feasibility, no single-block or two-block exchange that improves it, monotonicity in beta."""
    rng = np.random.default_rng(7)
    per_rate_ms = np.array([5.36, 1.45, 0.79, 0.48, 0.12])       # cost of a layer at rate 1, 1/4, 1/8, 1/16, 0
    cost = np.tile(per_rate_ms, (30, 1))
    err = np.cumsum(rng.uniform(0.0, 1.0, (30, 5)), axis=1) * rng.uniform(0.1, 4.0, (30, 1))
    err[:, 0] = 0.0
    prev = None
    for beta in [10.0, 30.0, 58.0, 100.0, 161.0]:
        choice, tc, te = solver.as_select_block_rates(cost.tolist(), err.tolist(), beta)
        assert tc <= beta and tc == O.total(cost, choice) and te == O.total(err, choice)
        if prev is not None:
            assert te <= prev
        prev = te
        c = np.array(choice)
        for i in range(30):
            for r in range(5):
                d_cost = cost[i, r] - cost[i, c[i]]
                d_err = err[i, r] - err[i, c[i]]
                if tc + d_cost <= beta:
                    assert d_err >= -1e-12                         # no single change improves it
                for k in range(i + 1, 30):
                    for q in range(5):
                        if tc + d_cost + cost[k, q] - cost[k, c[k]] <= beta:
                            assert d_err + err[k, q] - err[k, c[k]] >= -1e-12
    assert prev == 0.0                                             # budget for all-softmax: no error left


def test_solver_rejects_bad_arguments(solver):
    for bad in ([[float("nan")]], [[-1.0]], [[float("inf")]]):
        with pytest.raises(solver.AsError) as ei:
            solver.as_select_block_rates(bad, [[0.0]], 1.0)
        assert ei.value.status == solver.AS_ERR_INVALID_ARG
    with pytest.raises(solver.AsError):
        solver.as_select_block_rates([[1.0, 2.0]], [[1.0]], 1.0)
