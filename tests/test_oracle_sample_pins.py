"""Pins of the oracle's candidate sampler (Section 3.2, Eq. 1) against what the paper and
arithmetic fix: independent draws reproduce q, draws without replacement follow the
chain of Eq. 1, temperature 0 is top-k, and the tree-level routine is the per-node routine
applied to every node in child order."""
import itertools
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2401_06706_b200 import synth


def _grid(n):
    return (np.arange(n) + 0.5) / n


def test_hand_computed_draws_without_replacement():
    # q = (1/4, 1/4, 1/2).  u1 = 0.3 falls in token 1's interval [1/4, 1/2).  Token 1 is then
    # removed: weights (1/4, 0, 1/2), total 3/4.  u2 = 0.2 -> 0.15 < 1/4 -> token 0;
    # u2 = 0.5 -> 0.375 > 1/4 -> token 2.  A third draw can only give the one token left.
    q = [0.25, 0.25, 0.5]
    assert oracle.draw(q, [0.3, 0.2], 1).tolist() == [1, 0]
    assert oracle.draw(q, [0.3, 0.5], 1).tolist() == [1, 2]
    assert oracle.draw(q, [0.3, 0.5, 0.99], 1).tolist() == [1, 2, 0]
    assert oracle.draw(q, [0.3, 0.5, 0.01, 0.5], 1).tolist() == [1, 2, 0, -1]   # nothing left
    # with replacement every draw sees the same q
    assert oracle.draw(q, [0.3, 0.3, 0.2, 0.75], 0).tolist() == [1, 1, 0, 2]


def test_draws_with_replacement_reproduce_q():
    rng = np.random.default_rng(11)
    q = rng.dirichlet(np.ones(9))
    n = 1 << 14
    xs = oracle.draw(q, _grid(n), 0)
    freq = np.bincount(xs, minlength=9) / n
    assert np.abs(freq - q).max() <= 1.0 / n + 1e-12          # each interval is hit to grid resolution


def test_draws_without_replacement_follow_eq1():
    """Measure of the set of (u1, u2) that yields the ordered pair (a, b) is q(a) q(b) / (1 - q(a))."""
    rng = np.random.default_rng(5)
    V, n = 5, 400
    q = rng.dirichlet(np.ones(V) * 2)
    counts = np.zeros((V, V))
    g = _grid(n)
    for u1 in g:
        for u2 in g:
            a, b = oracle.draw(q, [u1, u2], 1)
            counts[a, b] += 1
    counts /= n * n
    want = np.array([[0.0 if a == b else q[a] * q[b] / (1 - q[a]) for b in range(V)] for a in range(V)])
    assert np.all(np.diag(counts) == 0)                          # never the same token twice
    assert np.abs(counts - want).max() < 3.0 / n                 # boundary cells of the grid


def test_exact_interval_boundaries_with_rationals():
    """With rational q the CDF boundaries are exact; uniforms just below / above them flip the token."""
    q = [Fraction(1, 8), Fraction(3, 8), Fraction(1, 2)]
    qf = [float(x) for x in q]
    eps = 2.0 ** -40
    assert oracle.draw(qf, [0.125 - eps], 0)[0] == 0 and oracle.draw(qf, [0.125 + eps], 0)[0] == 1
    assert oracle.draw(qf, [0.5 - eps], 0)[0] == 1 and oracle.draw(qf, [0.5 + eps], 0)[0] == 2
    # after removing token 2 the boundary between 0 and 1 moves to (1/8) / (1/2) = 1/4
    assert oracle.draw(qf, [0.9, 0.25 - eps], 1).tolist() == [2, 0]
    assert oracle.draw(qf, [0.9, 0.25 + eps], 1).tolist() == [2, 1]


def test_temperature_zero_is_top_k_with_lowest_index_on_ties():
    rng = np.random.default_rng(3)
    logits = np.round(rng.normal(size=200) * 2).astype(np.float32)      # many ties
    want = np.lexsort((np.arange(200), -logits))[:12]
    assert oracle.topk(logits, 12).tolist() == want.tolist()


@pytest.mark.parametrize("mode,T", [(0, 1.0), (1, 0.7), (0, 0.0)])
def test_tree_level_routine_is_the_node_routine_in_child_order(mode, T):
    rng = np.random.default_rng(17 + mode)
    parent = synth.tree_from_kconfig([3, 2, 1])
    st = synth.tree_stats(parent)
    first, count = synth.children_ranges(parent)
    B, V = 4, 50
    draft = rng.normal(size=(B, st["n_internal"], V)).astype(np.float32) * 2
    u = ((rng.integers(0, 1 << 23, size=(B, st["n_nodes"])) + 0.5) * 2.0 ** -23).astype(np.float32)
    cand = oracle.sample(draft, parent, u, T, mode)
    assert (cand[:, 0] == -1).all()
    for b, n in itertools.product(range(B), range(st["n_internal"])):
        ch = np.arange(first[n], first[n] + count[n])
        if T == 0.0:
            want = oracle.topk(draft[b, n], len(ch))
        else:
            want = oracle.draw(oracle.softmax(draft[b, n], T), u[b, ch].astype(np.float64), mode)
        assert cand[b, ch].tolist() == want.tolist()
    # a sub-range touches only the children of its nodes
    part = oracle.sample(draft, parent, u, T, mode, node_begin=1, node_end=3)
    touched = np.concatenate([np.arange(first[n], first[n] + count[n]) for n in (1, 2)])
    mask = np.zeros(st["n_nodes"], dtype=bool)
    mask[touched] = True
    assert (part[:, ~mask] == -1).all() and (part[:, mask] == cand[:, mask]).all()
