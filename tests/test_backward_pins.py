"""Pins of the float64 gradient oracle (value-distillation loss w.r.t. the feature-map weights).

Nothing here touches the CUDA library.  The gradient oracle is pinned to something other than itself:
a case worked by hand from the equations, central finite differences of the FORWARD oracle's loss (a
different piece of code, itself pinned in test_oracle_pins.py), and the special cases where the
gradient must vanish.  Planted mistakes in copies of the oracle must be noticed.
"""
import json
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import hybrid_attention as O
from oracle import hybrid_backward as G

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_worked.json")


def _frac(x):
    return float(Fraction(x)) if isinstance(x, str) else float(x)


def _cases():
    with open(GOLDEN) as f:
        return json.load(f)["backward_cases"]


@pytest.mark.parametrize("case", _cases(), ids=lambda c: c["name"])
def test_hand_worked_gradient(case, oracle=G):
    arr = lambda k: np.array([[_frac(e) for e in row] for row in case[k]], dtype=np.float64)
    mask = np.array(case["is_softmax"], dtype=bool)
    for mode in (O.STAB_PAPER, O.STAB_EXACT):          # c_i = 0 in this case: both modes coincide
        loss, dwq, dwk = oracle.phi_weight_gradients_head(arr("q"), arr("k"), arr("v"), arr("wq"), arr("wk"), mask,
                                                          arr("y_teacher"), case["scale"], mode, case["degree"])
        assert abs(loss - _frac(case["loss"])) < 1e-13
        np.testing.assert_allclose(dwq, arr("dwq"), rtol=1e-12)
        np.testing.assert_allclose(dwk, arr("dwk"), rtol=1e-12)


def _rand(rng, N, d, F, R):
    q, k, v, y = (rng.standard_normal((N, d)) for _ in range(4))
    wq, wk = rng.uniform(-0.7, 0.7, (F, d)), rng.uniform(-0.7, 0.7, (F, d))
    mask = O.softmax_token_mask((1, 1, N), (1, 1, N), R)
    return q, k, v, y, wq, wk, mask


def _loss(q, k, v, y, wq, wk, mask, mode, degree):
    y_hat, _ = O.hybrid_attention_head(q, k, v, wq, wk, mask, None, mode, degree)
    return np.abs(y - y_hat).sum()


def _finite_differences(q, k, v, y, wq, wk, mask, mode, degree, h=1e-6):
    dq, dk = np.zeros_like(wq), np.zeros_like(wk)
    for W, dW in ((wq, dq), (wk, dk)):
        for idx in np.ndindex(W.shape):
            old = W[idx]
            W[idx] = old + h
            lp = _loss(q, k, v, y, wq, wk, mask, mode, degree)
            W[idx] = old - h
            lm = _loss(q, k, v, y, wq, wk, mask, mode, degree)
            W[idx] = old
            dW[idx] = (lp - lm) / (2 * h)
    return dq, dk


@pytest.mark.parametrize("mode", [O.STAB_PAPER, O.STAB_EXACT])
@pytest.mark.parametrize("R,degree,F", [(0, 2, 6), (2, 1, 4), (3, 2, 6), (4, 3, 6), (2, 4, 8)])
def test_gradient_equals_central_finite_differences_of_the_forward_loss(mode, R, degree, F, oracle=G):
    rng = np.random.default_rng(100 + 7 * R + degree)
    q, k, v, y, wq, wk, mask = _rand(rng, N=14, d=3, F=F, R=R)
    loss, dwq, dwk = oracle.phi_weight_gradients_head(q, k, v, wq, wk, mask, y, None, mode, degree)
    assert abs(loss - _loss(q, k, v, y, wq, wk, mask, mode, degree)) < 1e-12
    fq, fk = _finite_differences(q, k, v, y, wq, wk, mask, mode, degree)
    scale = max(np.abs(fq).max(), np.abs(fk).max())
    assert scale > 1e-3                               # the case does exercise the gradient
    np.testing.assert_allclose(dwq, fq, atol=2e-6 * scale, rtol=2e-6)
    np.testing.assert_allclose(dwk, fk, atol=2e-6 * scale, rtol=2e-6)


def test_gradient_vanishes_without_linear_tokens_and_at_the_teacher():
    rng = np.random.default_rng(5)
    q, k, v, y, wq, wk, mask = _rand(rng, N=12, d=3, F=4, R=3)
    _, dq, dk = G.phi_weight_gradients_head(q, k, v, wq, wk, np.ones(12, bool), y)       # rate 1: phi is not used
    assert not dq.any() and not dk.any()
    y_hat, _ = O.hybrid_attention_head(q, k, v, wq, wk, mask)
    loss, dq, dk = G.phi_weight_gradients_head(q, k, v, wq, wk, mask, y_hat)             # student == teacher
    assert loss == 0.0 and not dq.any() and not dk.any()


def test_batched_gradient_sums_over_the_batch():
    rng = np.random.default_rng(6)
    B, H, N, d, F = 2, 2, 10, 3, 4
    q, k, v, y = (rng.standard_normal((B, H, N, d)) for _ in range(4))
    wq, wk = rng.uniform(-0.7, 0.7, (H, F, d)), rng.uniform(-0.7, 0.7, (H, F, d))
    mask = O.softmax_token_mask((1, 1, N), (1, 1, N), 3)
    loss, dq, dk = G.phi_weight_gradients(q, k, v, wq, wk, mask, y)
    parts = [[G.phi_weight_gradients_head(q[b, h], k[b, h], v[b, h], wq[h], wk[h], mask, y[b, h]) for h in range(H)] for b in range(B)]
    assert abs(loss - sum(parts[b][h][0] for b in range(B) for h in range(H))) < 1e-12
    for h in range(H):
        np.testing.assert_allclose(dq[h], parts[0][h][1] + parts[1][h][1], rtol=1e-13)
        np.testing.assert_allclose(dk[h], parts[0][h][2] + parts[1][h][2], rtol=1e-13)


def _mutants():
    import inspect
    src = inspect.getsource(G)
    edits = {
        "sign_of_the_loss_derivative": ("G = np.sign(y_hat - y)", "G = np.sign(y - y_hat)"),
        "denominator_derivative_sign": ("s = -(G * y_hat).sum(axis=1) / den", "s = (G * y_hat).sum(axis=1) / den"),
        "lambda_missing_on_the_query_side": ("d_phi_q = lam[:, None] * (g @ S.T + s[:, None] * z[None, :])",
                                             "d_phi_q = (g @ S.T + s[:, None] * z[None, :])"),
        "z_term_missing": ("d_phi_k = v[lin] @ dS.T + dz[None, :]", "d_phi_k = v[lin] @ dS.T"),
        "power_factor_missing": ("slope_q = np.where(a_q > 0.0, p * r_q ** (p - 1.0), 0.0)",
                                 "slope_q = np.where(a_q > 0.0, r_q ** (p - 1.0), 0.0)"),
        "relu_gate_missing": ("slope_k = np.where(a_k > 0.0, p * r_k ** (p - 1.0), 0.0)",
                              "slope_k = p * np.abs(a_k) ** (p - 1.0)"),
        "key_side_gradient_doubled": ("dWk = (d_phi_k * slope_k).T @ k[lin]", "dWk = (d_phi_k * slope_k).T @ k[lin] * 2.0"),
        "dS_transposed": ("dS = (lam[:, None] * phi_q).T @ g", "dS = ((lam[:, None] * phi_q).T @ g).T"),
    }
    for name, (old, new) in edits.items():
        assert src.count(old) == 1, name
        ns = {"__name__": "oracle_backward_mutant_" + name}
        exec(compile(src.replace(old, new), "<mutant:%s>" % name, "exec"), ns)
        yield name, type("M", (), {k: staticmethod(v) if callable(v) else v for k, v in ns.items() if not k.startswith("__")})


@pytest.mark.parametrize("name,mutant", list(_mutants()), ids=lambda x: x if isinstance(x, str) else "")
def test_planted_mistakes_in_the_gradient_are_caught(name, mutant):
    failures = 0
    for case in _cases():
        try:
            test_hand_worked_gradient(case, oracle=mutant)
        except (AssertionError, ValueError):
            failures += 1
    for mode in (O.STAB_PAPER, O.STAB_EXACT):
        for R, degree, F in [(3, 2, 6), (4, 3, 6)]:
            try:
                test_gradient_equals_central_finite_differences_of_the_forward_loss(mode, R, degree, F, oracle=mutant)
            except (AssertionError, ValueError):
                failures += 1
    assert failures > 0, "no pin noticed the planted mistake '%s'" % name
