"""Pins of the oracle's behaviour at the edges the paper does not cover: a residual of mass
zero (Algorithm 1 / 2, the line p := norm(max(0, p - q)) when the sum is 0), distributions
without mass (all -inf, NaN or +inf logits) and uniforms that are not inside (0, 1).  Every
expected value below is worked out by hand from the readings listed in the oracle's header."""
import math

import numpy as np
import pytest
import scipy.special

import oracle

DEGENERATE, BAD_TOKEN, NO_MASS = oracle.STATUS_DEGENERATE, oracle.STATUS_BAD_TOKEN, oracle.STATUS_NO_MASS


# ------------------------------------------------------------------ zero residual mass
@pytest.mark.parametrize("mode", [0, 1])
def test_zero_residual_mass_keeps_p_and_later_candidates_see_it(mode):
    """p == q and a candidate that is not a token: the rejection is forced, max(0, p - q) sums
    to 0, so p stays what it was and the next candidate is tested against it: ratio 1, accepted
    by every r < 1."""
    p = np.array([0.5, 0.25, 0.25])
    r = oracle.mcss(p, p.copy(), [3, 1], [0.5, 0.999], mode)
    assert r.status == (DEGENERATE | BAD_TOKEN)
    assert r.ratio[0] == -1.0 and r.S[0] == 0.0
    assert r.ratio[1] == 1.0 and r.accepted == 1
    assert np.array_equal(r.p, p)               # unchanged, bit for bit
    assert math.isnan(r.S[1])                   # no second rejection happened


@pytest.mark.parametrize("mode", [0, 1])
def test_zero_residual_mass_after_a_candidate_of_probability_zero(mode):
    """A candidate with q(x) = 0 where p(x) = 0 too (a token outside both supports) while p == q
    elsewhere: rejected without a ratio, residual mass 0, p kept; no BAD_TOKEN this time."""
    p = np.array([0.5, 0.5, 0.0])
    r = oracle.mcss(p, p.copy(), [2, 0], [0.3, 0.7], mode)
    assert r.status == DEGENERATE
    assert r.ratio[0] == -1.0 and r.S[0] == 0.0 and r.ratio[1] == 1.0 and r.accepted == 1
    assert np.array_equal(r.p, p) and np.array_equal(r.q, p)


@pytest.mark.parametrize("mode", [0, 1])
def test_all_candidates_rejected_on_zero_mass_draws_from_the_kept_p(mode):
    """Through the whole step: one node with two children that carry no token, target row equal
    to the draft row.  Nothing is accepted and the endpoint token is the inverse-CDF image of the
    second uniform under the untouched p = softmax(row)."""
    row = np.log(np.array([0.125, 0.5, 0.25, 0.125], dtype=np.float64)).astype(np.float32)   # exact probabilities
    parent = np.array([-1, 0, 0], dtype=np.int32)
    for u_end, want in ((0.05, 0), (0.125, 1), (0.62, 1), (0.63, 2), (0.9, 3)):
        unif = np.array([[[0.5, u_end], [0.5, 0.5], [0.5, 0.5]]], dtype=np.float32)
        res = oracle.verify(row[None, None].repeat(3, 1), row[None, None], parent,
                            np.array([[-1, 4, -7]], dtype=np.int32), unif, 1.0, mode)
        assert int(res.status[0]) == (DEGENERATE | BAD_TOKEN)
        assert int(res.accept_len[0]) == 0 and res.tokens[0].tolist() == [want, -1]
        assert np.allclose(res.residual[0], [0.125, 0.5, 0.25, 0.125], rtol=1e-7)


@pytest.mark.parametrize("mode", [0, 1])
def test_zero_residual_mass_on_a_long_row_whose_sum_is_not_exactly_one(mode):
    """The same with a softmax over 4000 logits, whose float64 sum is 1 only up to rounding: two
    candidates that are not tokens leave p and q bit for bit as they were (Algorithm 2 removes
    nothing from q, so it does not renormalise it either)."""
    rng = np.random.default_rng(31)
    p = oracle.softmax((rng.standard_normal(4000) * 2.5).astype(np.float32), 1.0)
    r = oracle.mcss(p, p.copy(), [4000, -1], [0.5, 0.5], mode)
    assert r.accepted == -1 and r.status == (DEGENERATE | BAD_TOKEN)
    assert np.array_equal(r.p, p) and np.array_equal(r.q, p)
    assert r.S[0] == 0.0 and r.S[1] == 0.0


# ------------------------------------------------------------------ no mass
@pytest.mark.parametrize("bad", ["all_minus_inf", "nan", "plus_inf"])
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_target_row_without_mass_at_the_root(bad, mode):
    """No distribution can be formed from the root's target row: nothing is accepted, the endpoint
    token is -1 and NO_MASS is set (with Algorithm 1 / 2 the failed residual update also reports
    DEGENERATE; naive sampling performs no such update)."""
    rng = np.random.default_rng(5)
    V = 6
    target = rng.standard_normal((1, 3, V)).astype(np.float32)
    draft = rng.standard_normal((1, 1, V)).astype(np.float32)
    if bad == "all_minus_inf":
        target[0, 0, :] = -np.inf
    elif bad == "nan":
        target[0, 0, 2] = np.nan
    else:
        target[0, 0, 4] = np.inf
    parent = np.array([-1, 0, 0], dtype=np.int32)
    cand = np.array([[-1, 1, 3]], dtype=np.int32)
    unif = np.full((1, 3, 2), 0.4, dtype=np.float32)
    res = oracle.verify(target, draft, parent, cand, unif, 1.0, mode)
    assert int(res.accept_len[0]) == 0 and res.tokens[0].tolist() == [-1, -1]
    assert int(res.status[0]) == (NO_MASS if mode == 2 else NO_MASS | DEGENERATE)
    assert int(res.node_accept[0, 0]) == -1 and int(res.node_bonus[0, 0]) == -1


def test_leaf_without_mass_ends_the_walk_with_no_token():
    """The root accepts its only child (target row == draft row, ratio 1); the child is a leaf
    whose target row is all -inf: one accepted token, endpoint -1, NO_MASS."""
    row = np.array([0.3, -1.2, 2.0, 0.1], dtype=np.float32)
    target = np.stack([row, np.full(4, -np.inf, dtype=np.float32)])[None]
    res = oracle.verify(target, row[None, None], np.array([-1, 0], dtype=np.int32),
                        np.array([[-1, 2]], dtype=np.int32), np.full((1, 2, 2), 0.5, dtype=np.float32), 1.0, 0)
    assert int(res.accept_len[0]) == 1 and res.tokens[0].tolist() == [2, -1]
    assert int(res.status[0]) == NO_MASS


@pytest.mark.parametrize("mode", [0, 1])
def test_draft_row_without_mass_rejects_everything_and_draws_from_p(mode):
    """An all -inf draft row gives no q: every candidate is rejected without a ratio, the
    residual update finds no mass (DEGENERATE) and the endpoint comes from p = softmax(target),
    which a library softmax and a plain cumulative sum fix."""
    rng = np.random.default_rng(11)
    V = 9
    target = rng.standard_normal((1, 3, V)).astype(np.float32)
    draft = np.full((1, 1, V), -np.inf, dtype=np.float32)
    unif = np.array([[[0.5, 0.37], [0.2, 0.5], [0.9, 0.5]]], dtype=np.float32)
    res = oracle.verify(target, draft, np.array([-1, 0, 0], dtype=np.int32), np.array([[-1, 1, 3]], dtype=np.int32),
                        unif, 1.0, mode)
    p = scipy.special.softmax(target[0, 0].astype(np.float64))
    want = int(np.searchsorted(np.cumsum(p), float(np.float32(0.37)) * p.sum(), side="right"))
    assert int(res.status[0]) == DEGENERATE
    assert int(res.accept_len[0]) == 0 and int(res.tokens[0, 0]) == want
    assert res.node_ratio[0, 1] == -1.0 and res.node_ratio[0, 2] == -1.0
    assert np.allclose(res.residual[0], p, rtol=1e-12)


# ------------------------------------------------------------------ uniforms outside (0, 1)
def _one_node(p_logits, q_logits, cands, rs, mode, u_end=0.5):
    k = len(cands)
    parent = np.array([-1] + [0] * k, dtype=np.int32)
    target = np.tile(np.asarray(p_logits, dtype=np.float32), (1, k + 1, 1))
    draft = np.asarray(q_logits, dtype=np.float32)[None, None]
    unif = np.full((1, k + 1, 2), u_end, dtype=np.float32)
    unif[0, 1:, 0] = rs
    return oracle.verify(target, draft, parent, np.array([[-1, *cands]], dtype=np.int32), unif, 1.0, mode)


def test_uniform_not_below_one_counts_as_one():
    """Through the verification step: r >= 1 or NaN accepts exactly when p(x) >= q(x); r <= 0
    accepts whenever q(x) > 0."""
    pl, ql = np.log([0.6, 0.4]), np.log([0.5, 0.5])
    for r in (1.0, 1.1, 1.5, float("inf"), float("nan")):
        assert int(_one_node(pl, ql, [0], [r], 0).node_accept[0, 0]) == 1        # ratio 1.2
        assert int(_one_node(pl, ql, [1], [r], 0).node_accept[0, 0]) == -1       # ratio 0.8
    for r in (0.0, -0.3, -float("inf")):
        assert int(_one_node(pl, ql, [1], [r], 0).node_accept[0, 0]) == 1
        assert int(_one_node([0.0, -np.inf], [-np.inf, 0.0], [0], [r], 0).node_accept[0, 0]) == -1   # q(x) = 0


@pytest.mark.parametrize("mode", [0, 1])
def test_with_such_uniforms_the_outcome_is_the_closed_form_with_r_equal_to_one(mode):
    """With every r not below 1 the step is deterministic: it accepts the first candidate whose
    ratio is at least 1.  The ratios follow from the closed form of the residual written out here
    (c_0 = 0, c_{n+1} = c_n + S_n / W_n; unnormalised residual max(p - c_n q, 0)), which holds
    because only a candidate with p(x) < q(x) is ever rejected."""
    rng = np.random.default_rng(21)
    seen_acc = seen_rej = 0
    for _ in range(200):
        V = int(rng.integers(3, 9))
        pl, ql = rng.standard_normal(V) * 1.5, rng.standard_normal(V) * 1.5
        p, q = scipy.special.softmax(pl.astype(np.float32).astype(np.float64)), scipy.special.softmax(ql.astype(np.float32).astype(np.float64))
        k = int(rng.integers(1, 4))
        cand = rng.choice(V, size=k, replace=False) if mode == 1 else rng.integers(0, V, size=k)
        rs = rng.choice([1.0, 1.7, float("nan"), float("inf")], size=k)
        res = _one_node(pl, ql, cand, rs, mode)
        c, S, W, want, on_boundary = 0.0, 1.0, 1.0, -1, False
        for i, x in enumerate(cand):
            Pn = np.maximum(p - c * q, 0)
            dup = mode == 1 and x in cand[:i]
            if not dup and abs(Pn[x] / S - q[x] / W) < 1e-9:
                on_boundary = True     # ratio 1 up to rounding (all remaining mass on one token): either way is right
                break
            if not dup and Pn[x] / S > q[x] / W:
                want = i + 1
                break
            c = c + S / W
            if mode == 1 and not dup:
                W -= q[x]
            S = np.maximum(p - c * q, 0).sum()
        if on_boundary:
            continue
        assert int(res.node_accept[0, 0]) == want
        if want < 0:
            assert np.allclose(res.residual[0], np.maximum(p - c * q, 0) / S, atol=1e-12)
            seen_rej += 1
        else:
            seen_acc += 1
    assert seen_acc > 30 and seen_rej > 30
