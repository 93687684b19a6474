"""Pins of the oracle's naive-sampling mode (mode 2; the baseline of Section 2 that Section 4.5
and Appendix C compare multi-candidate speculative sampling with): the emitted token is a draw
from p whatever the candidates are, it is accepted exactly when a candidate carries it, and
averaged over candidates drawn from q its rejection probability is sum_x p(x)(1-q(x))^k, which
Appendix C proves to be at least that of Algorithm 1."""
import itertools

import numpy as np

import oracle


def _grid(n):
    return ((np.arange(n) + 0.5) / n).astype(np.float32)


def _one_node(p_logits, cands, u_end):
    """verify() on a root with len(cands) children; returns (accept_len, first emitted token)."""
    k = len(cands)
    parent = np.array([-1] + [0] * k, dtype=np.int32)
    n = u_end.shape[0]
    target = np.broadcast_to(np.asarray(p_logits, dtype=np.float32), (n, k + 1, len(p_logits))).copy()
    cand = np.broadcast_to(np.array([-1] + list(cands), dtype=np.int32), (n, k + 1)).copy()
    unif = np.full((n, k + 1, 2), 0.5, dtype=np.float32)
    unif[:, 0, 1] = u_end
    res = oracle.verify(target, None, parent, cand, unif, 1.0, 2)
    return res.accept_len, res.tokens[:, 0]


def test_emitted_token_is_a_draw_from_p_and_accepted_iff_a_candidate_carries_it():
    rng = np.random.default_rng(2)
    logits = rng.normal(size=7) * 1.5
    p = oracle.softmax(logits.astype(np.float32), 1.0)
    n = 1 << 13
    u = _grid(n)
    for cands in ([3], [1, 5], [6, 6, 0], [2, 4, 1, 3]):
        alen, tok = _one_node(logits, cands, u)
        want = np.array([oracle.invcdf(p, float(x)) for x in u])
        assert np.array_equal(tok, want)                              # the draw itself, candidates or not
        assert np.array_equal(alen == 1, np.isin(tok, cands))         # accepted iff a candidate carries it
        assert abs((alen == 1).mean() - p[sorted(set(cands))].sum()) <= len(set(cands)) * 2.0 / n


def test_average_rejection_probability_and_appendix_c():
    rng = np.random.default_rng(8)
    V, k, n = 4, 2, 2048
    tl = rng.normal(size=V).astype(np.float32) * 1.2
    dl = (tl + rng.normal(size=V) * 1.0).astype(np.float32)
    p, q = oracle.softmax(tl, 1.0), oracle.softmax(dl, 1.0)
    u = _grid(n)
    rej_naive = 0.0
    rej_mcss = 0.0
    for cands in itertools.product(range(V), repeat=k):
        weight = np.prod(q[list(cands)])                              # candidates drawn with replacement
        alen, _ = _one_node(tl, cands, u)
        rej_naive += weight * (alen == 0).mean()
        # Algorithm 1 rejects all k with probability prod_i (1 - min(1, rho_i)) along its own trace
        trace = oracle.mcss(p, q, np.array(cands, dtype=np.int32), np.full(k, 1e30), 0)   # huge r: follow the all-reject branch
        ratio = np.where(trace.ratio < 0, 0.0, trace.ratio)
        rej_mcss += weight * np.prod(1.0 - np.minimum(1.0, ratio))
    closed = float((p * (1.0 - q) ** k).sum())
    assert abs(rej_naive - closed) < 4.0 / n                          # sum_x p(x) (1 - q(x))^k
    assert rej_mcss <= closed + 1e-12                                  # Appendix C: P_S <= P_N


def test_walk_over_levels_and_leaf_endpoint():
    # chain of two draft nodes: the walk continues exactly while the drawn token equals the candidate
    rng = np.random.default_rng(4)
    V = 6
    parent = np.array([-1, 0, 1], dtype=np.int32)
    target = (rng.normal(size=(1, 3, V)) * 2).astype(np.float32)
    ps = [oracle.softmax(target[0, i], 1.0) for i in range(3)]
    for u0, u1, u2 in itertools.product([0.1, 0.5, 0.9], repeat=3):
        x0, x1, x2 = (oracle.invcdf(ps[i], u) for i, u in enumerate((u0, u1, u2)))
        for c1, c2 in ((x0, x1), (x0, (x1 + 1) % V), ((x0 + 1) % V, x1)):
            cand = np.array([[-1, c1, c2]], dtype=np.int32)
            unif = np.zeros((1, 3, 2), dtype=np.float32)
            unif[0, :, 1] = (u0, u1, u2)
            res = oracle.verify(target, None, parent, cand, unif, 1.0, 2)
            if c1 != x0:
                want = [x0, -1, -1]
            elif c2 != x1:
                want = [x0, x1, -1]
            else:
                want = [x0, x1, x2]                                   # leaf: endpoint from its own target row
            assert res.tokens[0].tolist() == want
            assert np.allclose(res.residual[0], ps[res.accept_len[0]])
            seq = oracle.verify(target, None, parent, cand, unif, 1.0, 2, sequential=True)
            assert seq.tokens[0].tolist() == want
