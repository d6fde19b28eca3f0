"""Brute-force oracle for the block-rate selection problem (test infrastructure).

This module is TEST INFRASTRUCTURE: it is imported only by the tests.  It shares no
code with the library's solver and never imports it.

What it follows (paper: "Attention Surgery", arXiv 2509.24899, paragraph
"Heterogeneous Block-Rate Optimization"): with blocks i = 1..B, candidate rates r in R,
a cost c_ir and an error e_ir per block and rate, choose exactly one rate per block so
that the summed error is minimal while the summed cost stays within the budget beta
(a multiple-choice knapsack problem).  The oracle is that definition written out: it
enumerates all |R|^B assignments, so it is meant for small B only.

Readings taken where the paper is silent:

* The budget constraint is "sum of costs <= beta" with the sums taken in block order
  in float64 (the library adds in the same order, so both see the same rounded sums).
* Among assignments of equal minimal error the problem has no preference; the oracle
  reports the minimal error and ALL assignments that reach it, and a solver is correct
  when its assignment is feasible and reaches that error.
* A problem whose cheapest assignment already exceeds beta is infeasible: None.
"""
from __future__ import annotations

import itertools
from typing import List, Optional, Sequence, Tuple


def total(values: Sequence[Sequence[float]], choice: Sequence[int]) -> float:
    """Sum over blocks, in block order, of the chosen rate's value."""
    s = 0.0
    for i, r in enumerate(choice):
        s = s + float(values[i][r])
    return s


def select_block_rates_bruteforce(cost: Sequence[Sequence[float]], err: Sequence[Sequence[float]],
                                  budget: float) -> Optional[Tuple[float, List[Tuple[int, ...]]]]:
    """Minimal summed error under the budget and every assignment reaching it, or None when no
    assignment fits the budget.  cost, err: [B][R]; an assignment is a tuple of rate indices."""
    n_blocks = len(cost)
    n_rates = len(cost[0])
    best_err = None
    best: List[Tuple[int, ...]] = []
    for choice in itertools.product(range(n_rates), repeat=n_blocks):
        if total(cost, choice) > budget:
            continue
        e = total(err, choice)
        if best_err is None or e < best_err:
            best_err, best = e, [choice]
        elif e == best_err:
            best.append(choice)
    if best_err is None:
        return None
    return best_err, best
