"""Pins of the float64 oracle against what the paper and the mathematics fix.

Nothing here touches the CUDA library.  The pins are chosen so that a plausible
mistake in the oracle (a dropped term, a wrong sign or index, a transposed operand, a
swapped power) fails at least one of them; `test_planted_mistakes_are_caught` plants
such mistakes in copies of the oracle and checks that the pins notice.
"""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import hybrid_attention as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_worked.json")


def _num(x):
    if isinstance(x, str):
        return eval(x, {"__builtins__": {}}, {"ln2": math.log(2.0), "exp": math.exp})
    return float(x)


def _arr(x):
    return np.array([[_num(e) for e in row] for row in x], dtype=np.float64)


def _rand_case(rng, N=24, d=6, F=8, R=3):
    q = rng.standard_normal((N, d))
    k = rng.standard_normal((N, d))
    v = rng.standard_normal((N, d))
    wq = rng.uniform(-0.7, 0.7, (F, d))
    wk = rng.uniform(-0.7, 0.7, (F, d))
    mask = O.softmax_token_mask((1, 1, N), (1, 1, N), R)
    return q, k, v, wq, wk, mask


# ---------------------------------------------------------------- hand-worked values
def _golden_cases():
    with open(GOLDEN) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _golden_cases(), ids=lambda c: c["name"])
@pytest.mark.parametrize("impl", ["factorised", "bruteforce"])
def test_hand_worked_values(case, impl, oracle=O):
    q, k, v = _arr(case["q"]), _arr(case["k"]), _arr(case["v"])
    wq, wk = _arr(case["wq"]), _arr(case["wk"])
    mask = np.array(case["is_softmax"], dtype=bool)
    scale = case["scale"]
    expected = {"paper": _arr(case["paper"]),
                "exact": _arr(case["exact_expr"] if "exact_expr" in case else case["exact"])}
    for mode, stab in (("paper", oracle.STAB_PAPER), ("exact", oracle.STAB_EXACT)):
        if impl == "factorised":
            y, aux = oracle.hybrid_attention_head(q, k, v, wq, wk, mask, scale, stab)
            if mode == "paper":
                np.testing.assert_allclose(aux[:, 0], [_num(x) for x in case["aux_c"]], atol=1e-13)
                np.testing.assert_allclose(aux[:, 1], [_num(x) for x in case["aux_den_s"]], rtol=1e-13)
                np.testing.assert_allclose(aux[:, 2], [_num(x) for x in case["aux_den_l"]], rtol=1e-13)
        else:
            y, _ = oracle.hybrid_attention_bruteforce(q, k, v, wq, wk, mask, scale, stab)
        np.testing.assert_allclose(y, expected[mode], rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- token rule
def test_token_rule_matches_paper_example_rate3():
    with open(GOLDEN) as f:
        g = json.load(f)["token_rule"]
    mask = O.softmax_token_mask((1, 1, 9), (1, 1, 9), 3)
    assert (np.flatnonzero(mask) + 1).tolist() == g["rate3_n9_one_indexed"]


@pytest.mark.parametrize("R", [2, 3, 4, 8, 16])
def test_whole_grid_block_is_the_1d_stride(R):
    T, Hg, Wg = 3, 5, 7
    mask = O.softmax_token_mask((T, Hg, Wg), (T, Hg, Wg), R)
    one_indexed = np.arange(1, T * Hg * Wg + 1)
    assert np.array_equal(mask, one_indexed % R == 1)


def test_token_rule_counts_on_benchmark_grids():
    # counts obtained by hand: a full 6x8 block holds ceil(48/R) softmax tokens, a clipped 6x4
    # block ceil(24/R); a 30x52 frame has 5 x 6 full and 5 x 1 clipped blocks.
    per_frame = {4: 5 * (6 * 12 + 6), 8: 5 * (6 * 6 + 3), 16: 5 * (6 * 3 + 2)}
    assert per_frame == {4: 390, 8: 195, 16: 100}
    for frames in (5, 21, 41):
        for R, pf in per_frame.items():
            m = O.softmax_token_mask((frames, 30, 52), (1, 6, 8), R)
            assert m.sum() == frames * pf
            assert m.reshape(frames, -1).sum(1).tolist() == [pf] * frames
    m = O.softmax_token_mask((4, 16, 16), (2, 4, 4), 32)   # one token per 2x4x4 block
    assert m.sum() == 32
    g = m.reshape(4, 16, 16)
    assert g[::2, ::4, ::4].all() and g.sum() == g[::2, ::4, ::4].sum()
    assert O.softmax_token_mask((2, 3, 4), (1, 2, 2), 1).all()
    assert not O.softmax_token_mask((2, 3, 4), (1, 2, 2), 0).any()


# ---------------------------------------------------------------- special cases -> library routines
@pytest.mark.parametrize("mode", [O.STAB_PAPER, O.STAB_EXACT])
def test_all_softmax_reduces_to_library_softmax_attention(mode):
    rng = np.random.default_rng(1)
    q, k, v, wq, wk, _ = _rand_case(rng, N=40, d=8)
    mask = np.ones(40, dtype=bool)
    y, aux = O.hybrid_attention_head(q, k, v, wq, wk, mask, None, mode)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(k)[None], torch.from_numpy(v)[None])[0].numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-12, atol=1e-12)
    lse = torch.logsumexp(torch.from_numpy(q @ k.T / math.sqrt(8)), dim=1).numpy()
    np.testing.assert_allclose(aux[:, 0] + np.log(aux[:, 1]), lse, rtol=1e-12)


def test_no_softmax_tokens_is_normalised_kernel_attention_with_identity_phi():
    # degree 1, W = I and non-negative inputs make phi the identity, so the output must be the
    # textbook kernel smoother  sum_j (q_i.k_j) v_j / sum_j (q_i.k_j)  built from library matmuls.
    rng = np.random.default_rng(2)
    N, d = 30, 5
    q, k = rng.uniform(0.1, 1, (N, d)), rng.uniform(0.1, 1, (N, d))
    v = rng.standard_normal((N, d))
    eye = np.eye(d)
    y, aux = O.hybrid_attention_head(q, k, v, eye, eye, np.zeros(N, bool), None, O.STAB_PAPER, degree=1)
    a = torch.from_numpy(q) @ torch.from_numpy(k).T
    ref = ((a / a.sum(1, keepdim=True)) @ torch.from_numpy(v)).numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-12)
    np.testing.assert_allclose(aux[:, 2], a.sum(1).numpy(), rtol=1e-12)


# ---------------------------------------------------------------- invariants
@pytest.mark.parametrize("mode", [O.STAB_PAPER, O.STAB_EXACT])
@pytest.mark.parametrize("R", [0, 1, 2, 3, 5])
def test_factorised_equals_bruteforce_and_weights_are_convex(mode, R):
    rng = np.random.default_rng(10 + R)
    q, k, v, wq, wk, mask = _rand_case(rng, N=20, d=4, F=6, R=R)
    y, _ = O.hybrid_attention_head(q, k, v, wq, wk, mask, None, mode)
    yb, w = O.hybrid_attention_bruteforce(q, k, v, wq, wk, mask, None, mode)
    np.testing.assert_allclose(y, yb, rtol=1e-10, atol=1e-12)
    # a query whose features are all zero at rate 0 has a zero denominator: both report NaN
    ok = np.isfinite(w).all(1)
    assert ok.sum() >= 15 and np.array_equal(ok, np.isfinite(y).all(1))
    w = w[ok]
    assert (w >= 0).all()
    np.testing.assert_allclose(w.sum(1), 1.0, rtol=1e-12)
    if R not in (0, 1):
        # both branches must carry weight in this test, or it would pin only one of them
        soft = w[:, mask].sum(1)
        assert 0.02 < np.median(soft) < 0.98


@pytest.mark.parametrize("mode", [O.STAB_PAPER, O.STAB_EXACT])
def test_key_permutation_invariance_and_query_equivariance(mode):
    rng = np.random.default_rng(3)
    q, k, v, wq, wk, mask = _rand_case(rng, N=32, d=6, F=8, R=4)
    y, _ = O.hybrid_attention_head(q, k, v, wq, wk, mask, None, mode)
    p = rng.permutation(32)
    y2, _ = O.hybrid_attention_head(q, k[p], v[p], wq, wk, mask[p], None, mode)
    np.testing.assert_allclose(y2, y, rtol=1e-10, atol=1e-12)
    y3, _ = O.hybrid_attention_head(q[p], k, v, wq, wk, mask, None, mode)
    np.testing.assert_allclose(y3, y[p], rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("mode", [O.STAB_PAPER, O.STAB_EXACT])
def test_constant_values_are_reproduced(mode):
    rng = np.random.default_rng(4)
    q, k, v, wq, wk, mask = _rand_case(rng, N=16, d=4, F=4, R=2)
    v[:] = np.array([1.5, -2.0, 0.25, 7.0])
    y, _ = O.hybrid_attention_head(q, k, v, wq, wk, mask, None, mode)
    np.testing.assert_allclose(y, v, rtol=1e-12)


def test_equal_keys_all_softmax_gives_mean_of_values():
    rng = np.random.default_rng(5)
    q, k, v, wq, wk, _ = _rand_case(rng, N=16, d=4, F=4)
    k[:] = k[0]
    y, _ = O.hybrid_attention_head(q, k, v, wq, wk, np.ones(16, bool))
    np.testing.assert_allclose(y, np.broadcast_to(v.mean(0), y.shape), rtol=1e-12)


def test_exact_mode_is_the_unstabilised_ratio_and_paper_mode_depends_on_c():
    rng = np.random.default_rng(6)
    q, k, v, wq, wk, mask = _rand_case(rng, N=24, d=6, F=8, R=3)
    ye, aux = O.hybrid_attention_head(q, k, v, wq, wk, mask, None, O.STAB_EXACT)
    yp, _ = O.hybrid_attention_head(q, k, v, wq, wk, mask, None, O.STAB_PAPER)
    # unstabilised ratio with torch ops, no c_i anywhere
    tq, tk, tv = (torch.from_numpy(a) for a in (q, k, v))
    e = torch.exp(tq @ tk[mask].T / math.sqrt(6))
    fq = torch.from_numpy(O.phi_features(q, wq))
    fk = torch.from_numpy(O.phi_features(k[~mask], wk))
    a = fq @ fk.T
    ref = (e @ tv[mask] + a @ tv[~mask]) / (e.sum(1) + a.sum(1))[:, None]
    np.testing.assert_allclose(ye, ref.numpy(), rtol=1e-11)
    # paper mode = exact mode evaluated with phi_q scaled by exp(+c_i) ... i.e. they differ
    assert np.abs(yp - ye).max() > 1e-3
    # and paper mode equals exact mode after folding exp(c_i) into the query features:
    # y_paper_i uses lambda=1, y_exact_i uses lambda=exp(-c_i); scaling W_q row-wise is not
    # possible, so check through the brute-force weights instead.
    _, wp = O.hybrid_attention_bruteforce(q, k, v, wq, wk, mask, None, O.STAB_PAPER)
    _, we = O.hybrid_attention_bruteforce(q, k, v, wq, wk, mask, None, O.STAB_EXACT)
    ratio_p = wp[:, ~mask].sum(1) / wp[:, mask].sum(1)
    ratio_e = we[:, ~mask].sum(1) / we[:, mask].sum(1)
    np.testing.assert_allclose(ratio_p, ratio_e * np.exp(aux[:, 0]), rtol=1e-10)


def _phi_cases():
    with open(GOLDEN) as f:
        return json.load(f)["phi_cases"]


def _layers(case):
    return [(np.array(l["W"], float), np.array(l["b"], float)) if "b" in l else np.array(l["W"], float)
            for l in case["layers"]]


@pytest.mark.parametrize("case", _phi_cases(), ids=lambda c: c["name"])
def test_feature_map_hand_worked_values(case, oracle=O):
    """Multi-layer embedding network, bias placement and power order against values worked by hand."""
    f = oracle.phi_features(np.array(case["x"], float), _layers(case), degree=case["degree"])
    np.testing.assert_allclose(f, np.array(case["phi"], float), rtol=1e-14, atol=1e-14)


def test_phi_is_nonnegative_and_shapes():
    rng = np.random.default_rng(7)
    x = rng.standard_normal((5, 4))
    w1, w2 = rng.standard_normal((8, 4)), rng.standard_normal((6, 8))
    f = O.phi_features(x, [w1, (w2, rng.standard_normal(6))], degree=3)
    assert f.shape == (5, 6) and (f >= 0).all()


@pytest.mark.parametrize("mode", [O.STAB_PAPER, O.STAB_EXACT])
def test_two_layer_operator_reduces_to_one_layer_when_the_second_is_the_identity(mode):
    # ReLU is idempotent, so [W, I] must give exactly what [W] gives, through the whole operator.
    rng = np.random.default_rng(17)
    q, k, v, wq, wk, mask = _rand_case(rng, N=24, d=6, F=8, R=3)
    eye = np.eye(8)
    y1, aux1 = O.hybrid_attention_head(q, k, v, wq, wk, mask, None, mode)
    y2, aux2 = O.hybrid_attention_head(q, k, v, [wq, eye], [wk, eye], mask, None, mode)
    np.testing.assert_allclose(y2, y1, rtol=1e-13)
    np.testing.assert_allclose(aux2, aux1, rtol=1e-13)
    S1, z1 = O.linear_state(k, v, wk, mask)
    S2, z2 = O.linear_state(k, v, [(wk, np.zeros(8)), eye], mask)
    np.testing.assert_allclose(S2, S1, rtol=1e-13)
    np.testing.assert_allclose(z2, z1, rtol=1e-13)


def test_rows_argument_selects_rows():
    rng = np.random.default_rng(8)
    q, k, v, wq, wk, mask = _rand_case(rng, N=24, d=6, F=8, R=3)
    y, aux = O.hybrid_attention_head(q, k, v, wq, wk, mask)
    rows = np.array([5, 0, 23])
    ys, auxs = O.hybrid_attention_head(q, k, v, wq, wk, mask, rows=rows, row_block=2)
    np.testing.assert_allclose(ys, y[rows], rtol=1e-13)
    np.testing.assert_allclose(auxs, aux[rows], rtol=1e-13)


def test_batched_wrapper_matches_per_head():
    rng = np.random.default_rng(9)
    B, H, N, d, F = 2, 3, 12, 4, 4
    q, k, v = (rng.standard_normal((B, H, N, d)) for _ in range(3))
    wq, wk = rng.standard_normal((H, F, d)), rng.standard_normal((H, F, d))
    mask = O.softmax_token_mask((1, 3, 4), (1, 2, 2), 2)
    y, aux = O.hybrid_attention(q, k, v, wq, wk, mask)
    y12, aux12 = O.hybrid_attention_head(q[1, 2], k[1, 2], v[1, 2], wq[2], wk[2], mask)
    np.testing.assert_array_equal(y[1, 2], y12)
    np.testing.assert_array_equal(aux[1, 2], aux12)


# ---------------------------------------------------------------- planted mistakes
def _mutants():
    """Copies of the oracle's source with one plausible mistake each."""
    import inspect
    src = inspect.getsource(O)
    edits = {
        "dropped_z_term": ("den += lam * den_l", "den += 0.0 * den_l"),
        "wrong_sign_on_c": ("e = np.exp(s - c[:, None])", "e = np.exp(s + c[:, None])"),
        "min_instead_of_max": ("c = s.max(axis=1)", "c = s.min(axis=1)"),
        "state_over_softmax_tokens": ("lin = ~np.asarray(is_softmax, dtype=bool)",
                                      "lin = np.asarray(is_softmax, dtype=bool)"),
        "powers_swapped": ("** (p + 1)", "** (P - p)"),
        "no_relu": ("a = np.maximum(a, 0.0)", "a = a"),
        "rule_off_by_one": ("return (ell % R == 0).reshape(n)", "return (ell % R == 1).reshape(n)"),
        "scale_missing": ("s = (qb @ k_s.T) * scale ", "s = (qb @ k_s.T) "),
        "lambda_inverted": ("lam = np.exp(-c)", "lam = np.exp(c)"),
        "S_transposed_use": ("num += lam[:, None] * (fq @ S)", "num += lam[:, None] * (fq @ S.T)"),
        "layers_in_reverse_order": ("for l, layer in enumerate(weights):", "for l, layer in enumerate(list(weights)[::-1]):"),
        "inner_relu_missing": ("a = np.maximum(a, 0.0)", "a = np.maximum(a, 0.0) if l == len(weights) - 1 else a"),
        "bias_dropped": ("a = a + np.asarray(b, dtype=np.float64)", "a = a"),
        "bias_after_relu": ("a = a + np.asarray(b, dtype=np.float64)\n        a = np.maximum(a, 0.0)",
                            "a = np.maximum(a, 0.0)\n            a = a + np.asarray(b, dtype=np.float64)\n"
                            "        a = a if b is not None else np.maximum(a, 0.0)"),
    }
    for name, (old, new) in edits.items():
        assert src.count(old) == 1, name
        ns = {"__name__": "oracle_mutant_" + name}
        exec(compile(src.replace(old, new), "<mutant:%s>" % name, "exec"), ns)
        yield name, type("M", (), {k: staticmethod(v) if callable(v) else v for k, v in ns.items()
                                   if not k.startswith("__")})


@pytest.mark.parametrize("name,mutant", list(_mutants()), ids=lambda x: x if isinstance(x, str) else "")
def test_planted_mistakes_are_caught(name, mutant):
    failures = 0
    for case in _golden_cases():
        try:
            test_hand_worked_values(case, "factorised", oracle=mutant)
        except (AssertionError, ValueError):
            failures += 1
    for case in _phi_cases():
        try:
            test_feature_map_hand_worked_values(case, oracle=mutant)
        except (AssertionError, ValueError):
            failures += 1
    try:
        with open(GOLDEN) as f:
            g = json.load(f)["token_rule"]
        mask = mutant.softmax_token_mask((1, 1, 9), (1, 1, 9), 3)
        assert (np.flatnonzero(mask) + 1).tolist() == g["rate3_n9_one_indexed"]
    except AssertionError:
        failures += 1
    assert failures > 0, "no pin noticed the planted mistake '%s'" % name
