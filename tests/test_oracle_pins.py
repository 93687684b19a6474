"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these compares the oracle with itself through the same formula: each one
uses a closed form, an invariant proved in the paper's appendices, a special case
that reduces to a textbook or library routine, or brute-force enumeration.
"""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest
import scipy.special

import oracle
from paper_2401_06706_b200 import synth


def _rand_dist(rng, V, conc=1.0):
    x = rng.gamma(conc, size=V) + 1e-9
    return x / x.sum()


# ---------------------------------------------------------------- softmax / argmax / invcdf
@pytest.mark.parametrize("T", [1.0, 0.7, 2.5])
def test_softmax_matches_library_routine(T):
    rng = np.random.default_rng(1)
    for V in (1, 7, 1000):
        l = (rng.standard_normal(V) * 4).astype(np.float32)
        ref = scipy.special.softmax(l.astype(np.float64) / T)
        got = oracle.softmax(l, T)
        assert np.allclose(got, ref, rtol=1e-13, atol=0)
        assert abs(got.sum() - 1) < 1e-13


def test_softmax_handles_minus_inf_and_large_logits():
    l = np.array([1000.0, -np.inf, 999.0, -1000.0], dtype=np.float32)
    got = oracle.softmax(l, 1.0)
    e = math.exp(-1.0)
    assert np.allclose(got, [1 / (1 + e), 0.0, e / (1 + e), 0.0], rtol=1e-14)


def test_argmax_lowest_index_on_ties():
    assert oracle.argmax(np.array([1, 5, 5, 2, 5], dtype=np.float32)) == 1
    assert oracle.argmax(np.array([3], dtype=np.float32)) == 0
    rng = np.random.default_rng(2)
    for _ in range(50):
        l = rng.integers(0, 5, size=40).astype(np.float32)
        assert oracle.argmax(l) == int(np.flatnonzero(l == l.max())[0])


def test_invcdf_brute_force_exact_fractions():
    # weights are small integers / 64: sums are exact in double, so the brute force with
    # Fractions fixes the answer including the strict inequality at interval borders
    rng = np.random.default_rng(3)
    for _ in range(200):
        V = int(rng.integers(1, 9))
        w = rng.integers(0, 6, size=V)
        if w.sum() == 0:
            w[rng.integers(0, V)] = 1
        P = w / 64.0
        for u_num in range(0, 64):
            u = Fraction(u_num, 64)
            target = u * Fraction(int(w.sum()), 64)
            cum, want = Fraction(0), None
            for x in range(V):
                cum += Fraction(int(w[x]), 64)
                if w[x] > 0 and cum > target:
                    want = x
                    break
            assert oracle.invcdf(P, float(u)) == want


def test_invcdf_never_returns_zero_mass_and_clamps():
    P = np.array([0.0, 0.25, 0.0, 0.75, 0.0])
    assert oracle.invcdf(P, 0.0) == 1
    assert oracle.invcdf(P, 0.25) == 3      # cum(1) = 0.25 is not > 0.25
    assert oracle.invcdf(P, 0.2499999) == 1
    assert oracle.invcdf(P, 1.0) == 3       # clamp to last positive-mass token
    assert oracle.invcdf(np.zeros(4), 0.5) == -1
    # law of the draw: on a midpoint grid of u the frequencies are the normalised weights
    rng = np.random.default_rng(4)
    P = _rand_dist(rng, 6) * 3.7
    G = 20000
    hits = np.bincount([oracle.invcdf(P, (i + 0.5) / G) for i in range(G)], minlength=6)
    assert np.abs(hits / G - P / P.sum()).max() < 2.0 / G


# ---------------------------------------------------------------- k = 1: speculative sampling
def test_k1_is_textbook_speculative_sampling():
    """Section 2: accept w.p. min(1, p/q); residual norm(max(0, p-q)); acceptance rate
    sum_x min(p, q).  Both algorithms must reduce to it for k = 1."""
    rng = np.random.default_rng(5)
    for mode in (0, 1):
        for _ in range(20):
            V = int(rng.integers(2, 12))
            p, q = _rand_dist(rng, V), _rand_dist(rng, V)
            G = 512
            acc_rate = 0.0
            for x in range(V):
                n_acc = 0
                for i in range(G):
                    u = (i + 0.5) / G
                    res = oracle.mcss(p, q, [x], [u], mode)
                    want_accept = u <= p[x] / q[x]
                    assert (res.accepted == 0) == want_accept
                    if res.accepted < 0:
                        ref = np.maximum(p - q, 0)
                        assert np.allclose(res.p, ref / ref.sum(), rtol=1e-13, atol=1e-300)
                    n_acc += res.accepted == 0
                assert abs(n_acc / G - min(1.0, p[x] / q[x])) <= 1.0 / G
                acc_rate += q[x] * n_acc / G
            assert abs(acc_rate - np.minimum(p, q).sum()) < 1.5 / G


# ---------------------------------------------------------------- exact enumeration (App. A, B)
def _tuple_weight(q, tup, mode):
    """Probability of drawing the candidate tuple: i.i.d. from q (mode 0) or sequentially
    without replacement, Eq. 1 (mode 1).  Written from Eq. 1, independent of the oracle."""
    w = 1.0
    removed = set()
    for x in tup:
        if mode == 0:
            w *= q[x]
        else:
            if x in removed:
                return 0.0
            denom = sum(q[y] for y in range(len(q)) if y not in removed)
            w *= q[x] / denom
            removed.add(x)
    return w


def _output_marginal(p, q, k, mode):
    V = len(p)
    out = np.zeros(V)
    for tup in itertools.product(range(V), repeat=k):
        w = _tuple_weight(q, tup, mode)
        if w == 0.0:
            continue
        tr = oracle.mcss(p, q, list(tup), [np.inf] * k, mode)   # all-reject path, full trace
        assert tr.accepted == -1
        surv = 1.0
        for i, x in enumerate(tup):
            a = min(1.0, tr.ratio[i]) if tr.ratio[i] >= 0 else 0.0
            out[x] += w * surv * a
            surv *= 1.0 - a
        out += w * surv * tr.p
    return out


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("V,k", [(2, 1), (3, 2), (4, 3), (5, 4), (8, 2), (8, 3), (6, 4)])
def test_output_token_is_distributed_as_p(V, k, mode):
    """Appendix A (Alg. 1) and B (Alg. 2): the returned token follows p exactly, for any p, q, k."""
    if mode == 1 and k > V:
        pytest.skip("cannot draw more distinct tokens than the vocabulary")
    rng = np.random.default_rng(100 * V + 10 * k + mode)
    for trial in range(3):
        p = _rand_dist(rng, V, 0.7)
        q = _rand_dist(rng, V, 0.7)
        if trial == 2:           # a token the target gives zero mass, and a peaked draft
            p[0] = 0.0
            p /= p.sum()
            q = q ** 3
            q /= q.sum()
        marg = _output_marginal(p, q, k, mode)
        assert np.abs(marg - p).max() < 1e-12, (marg, p)


def test_output_marginal_through_verify_on_uniform_grid():
    """Same property through the uniform-consuming batch entry point (tree = root + k
    leaves): first emitted token ~ p_root on a midpoint grid of all uniforms, and after an
    acceptance the second token ~ target distribution of the accepted leaf."""
    rng = np.random.default_rng(7)
    V, k, G = 4, 2, 40
    parent = synth.tree_from_kconfig([k])
    for mode in (0, 1):
        tl = (rng.standard_normal((k + 1, V)) * 1.5).astype(np.float32)
        dl = (rng.standard_normal((1, V)) * 1.5).astype(np.float32)
        T = 0.8
        p = scipy.special.softmax(tl.astype(np.float64) / T, axis=-1)
        q = scipy.special.softmax(dl[0].astype(np.float64) / T)
        grid = (np.arange(G) + 0.5) / G
        u1, u2, ue = np.meshgrid(grid, grid, grid, indexing="ij")
        n = u1.size
        marg0 = np.zeros(V)
        marg1 = np.zeros((k, V))
        wacc = np.zeros(k)
        for tup in itertools.product(range(V), repeat=k):
            w = _tuple_weight(q, tup, mode)
            if w == 0:
                continue
            cand = np.tile(np.array([-1, *tup], dtype=np.int32), (n, 1))
            unif = np.zeros((n, k + 1, 2), dtype=np.float32)
            unif[:, 1, 0] = u1.ravel()
            unif[:, 2, 0] = u2.ravel()
            unif[:, :, 1] = ue.ravel()[:, None]
            res = oracle.verify(np.tile(tl, (n, 1, 1)), np.tile(dl, (n, 1, 1)), parent, cand, unif,
                                T, mode, want_residual=False)
            assert (res.status == 0).all()
            marg0 += w * np.bincount(res.tokens[:, 0], minlength=V) / n
            for i in range(k):
                sel = res.accept_len == 1
                sel &= res.node_accept[:, 0] == i + 1
                wacc[i] += w * sel.sum() / n
                marg1[i] += w * np.bincount(res.tokens[sel, 1], minlength=V) / n
            assert ((res.accept_len == 0) | (res.accept_len == 1)).all()
        assert np.abs(marg0 - p[0]).max() < 3.0 / G, (marg0, p[0])
        for i in range(k):
            assert np.abs(marg1[i] / wacc[i] - p[i + 1]).max() < 3.0 / G


# ---------------------------------------------------------------- invariants (App. A, B, C)
@pytest.mark.parametrize("mode", [0, 1])
def test_rejection_probability_is_the_normaliser_and_rejected_tokens_stay_zero(mode):
    """App. A: P(reject x_n | R_{n-1}) = sum max(p^ - q, 0) = 1 - sum min(q, p^); Section 3.1:
    a rejected token has probability 0 in every later residual."""
    rng = np.random.default_rng(11 + mode)
    for _ in range(100):
        V = int(rng.integers(3, 40))
        k = int(rng.integers(1, min(V, 6)))
        p, q = _rand_dist(rng, V, 0.5), _rand_dist(rng, V, 0.5)
        cand = rng.choice(V, size=k, replace=(mode == 0), p=q)
        pc, qc = p.copy(), q.copy()
        for n in range(1, k + 1):
            # state before test n must match the definition of p^_{n-1}, q-bar_{n-1}
            tr = oracle.mcss(p, q, cand[:n], [np.inf] * n, mode)
            assert abs(tr.S[n - 1] - (1.0 - np.minimum(pc, qc).sum())) < 1e-12
            assert abs(tr.p.sum() - 1) < 1e-12 and (tr.p >= 0).all()
            for x in cand[:n]:
                if tr.ratio[list(cand[:n]).index(x)] <= 1.0:
                    assert tr.p[x] == 0.0
            pc = tr.p
            qc = tr.q
            if mode == 1:
                assert all(qc[x] == 0 for x in cand[:n])
                assert abs(qc.sum() - 1) < 1e-12
            else:
                assert np.array_equal(qc, q)


def test_all_reject_probability_below_naive_sampling_bound():
    """Appendix C: P_S(x, R_k) <= p(x)(1-q(x))^k, so prod_i S_i <= sum_x p(x)(1-q(x))^k
    (with replacement the S_i do not depend on the candidates)."""
    rng = np.random.default_rng(13)
    for _ in range(200):
        V = int(rng.integers(2, 30))
        k = int(rng.integers(1, 8))
        p, q = _rand_dist(rng, V, 0.6), _rand_dist(rng, V, 0.6)
        cand = rng.choice(V, size=k, p=q)
        tr = oracle.mcss(p, q, cand, [np.inf] * k, 0)
        joint = np.prod(tr.S) * tr.p                       # P_S(x, R_k)
        assert (joint <= p * (1 - q) ** k + 1e-13).all()
        tr2 = oracle.mcss(p, q, rng.choice(V, size=k, p=q), [np.inf] * k, 0)
        assert np.allclose(tr.S, tr2.S, rtol=1e-12)        # independent of the candidates


@pytest.mark.parametrize("mode", [0, 1])
def test_closed_form_of_the_residual(mode):
    """Independent restatement: after n rejections the unnormalised residual is
    max(p - c_n q, 0) with c_0 = 0, c_{n+1} = c_n + S_n / W_n, S_n its sum, W_n = 1 (with
    replacement) or 1 - sum of the original q over the rejected tokens (without)."""
    rng = np.random.default_rng(17 + mode)
    seen = 0
    for _ in range(300):
        V = int(rng.integers(3, 50))
        k = int(rng.integers(1, min(V - 1, 7)))
        p, q = _rand_dist(rng, V, 0.5), _rand_dist(rng, V, 0.5)
        cand = rng.choice(V, size=k, replace=(mode == 0), p=q)
        # r = 1 rejects exactly when p/q < 1, the only rejections that can occur with r in (0,1);
        # the closed form does not describe a (never occurring) rejection at p/q >= 1
        tr = oracle.mcss(p, q, cand, [1.0] * k, mode)
        c, S, W = 0.0, 1.0, 1.0
        n_rej = k if tr.accepted < 0 else tr.accepted
        for n in range(n_rej + (tr.accepted >= 0)):
            x = cand[n]
            Pn = np.maximum(p - c * q, 0)
            rho = (Pn[x] / S) / (q[x] / W)
            assert abs(tr.ratio[n] - rho) <= 1e-10 * max(1.0, rho)
            if n == tr.accepted:
                assert rho >= 1.0 - 1e-12
                break
            c = c + S / W
            if mode == 1:
                W -= q[x]
            Pn1 = np.maximum(p - c * q, 0)
            assert abs(tr.S[n] - Pn1.sum() / S) < 1e-10
            S = Pn1.sum()
        assert np.abs(tr.p - np.maximum(p - c * q, 0) / S).max() < 1e-10
        seen += n_rej
    assert seen > 200      # the rejection chain was really exercised


def test_forced_rejection_on_zero_draft_probability():
    p = np.array([0.5, 0.5, 0.0])
    q = np.array([0.0, 0.5, 0.5])
    tr = oracle.mcss(p, q, [0], [1e-9], 0)
    assert tr.accepted == -1 and tr.ratio[0] == -1.0
    # duplicate candidate without replacement: second copy has q-bar = 0
    p = np.array([0.1, 0.6, 0.3])
    q = np.array([0.7, 0.2, 0.1])
    tr = oracle.mcss(p, q, [0, 0], [0.9, 1e-9], 1)
    assert tr.accepted == -1 and tr.ratio[1] == -1.0 and tr.q[0] == 0.0
    tr = oracle.mcss(p, q, [7], [0.5], 0)
    assert tr.accepted == -1 and tr.status & oracle.STATUS_BAD_TOKEN


# ---------------------------------------------------------------- temperature 0
def test_temperature_zero_is_greedy_matching():
    """Section 4.5: at temperature 0 acceptance means 'candidate equals the target argmax';
    the endpoint is the target argmax of the stopping node; draft logits are unused."""
    rng = np.random.default_rng(19)
    ks = [3, 2, 1]
    parent = synth.tree_from_kconfig(ks)
    n_nodes = parent.shape[0]
    first, count = synth.children_ranges(parent)
    B, V = 64, 11
    target = rng.integers(-3, 4, size=(B, n_nodes, V)).astype(np.float32)   # many ties
    cand = rng.integers(0, V, size=(B, n_nodes)).astype(np.int32)
    unif = rng.random((B, n_nodes, 2)).astype(np.float32)
    for mode in (0, 1):
        res = oracle.verify(target, None, parent, cand, unif, 0.0, mode)
        for b in range(B):
            n, toks = 0, []
            while True:
                a = int(np.flatnonzero(target[b, n] == target[b, n].max())[0])
                nxt = next((c for c in range(first[n], first[n] + count[n]) if cand[b, c] == a), None)
                if nxt is None:
                    toks.append(a)
                    break
                toks.append(int(cand[b, nxt]))
                n = nxt
            assert res.accept_len[b] == len(toks) - 1
            assert list(res.tokens[b, :len(toks)]) == toks
            assert (res.tokens[b, len(toks):] == -1).all()
            onehot = np.zeros(V)
            onehot[toks[-1]] = 1
            assert np.array_equal(res.residual[b], onehot)


# ---------------------------------------------------------------- the walk
def _random_case(rng, ks, B, V, mode, T=1.0):
    parent = synth.tree_from_kconfig(ks)
    st = synth.tree_stats(parent)
    target = (rng.standard_normal((B, st["n_nodes"], V)) * 2).astype(np.float32)
    draft = (target[:, :st["n_internal"]] + rng.standard_normal((B, st["n_internal"], V))).astype(np.float32)
    first, count = synth.children_ranges(parent)
    cand = np.full((B, st["n_nodes"]), -1, dtype=np.int32)
    for b in range(B):
        for n in range(st["n_internal"]):
            q = scipy.special.softmax(draft[b, n].astype(np.float64) / T)
            cand[b, first[n]:first[n] + count[n]] = rng.choice(V, size=count[n], replace=(mode == 0), p=q)
    unif = ((rng.integers(0, 1 << 23, size=(B, st["n_nodes"], 2)) + 0.5) * 2.0 ** -23).astype(np.float32)
    return parent, st, target, draft, cand, unif


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("ks", [[1, 1, 1, 1], [2, 2], [4, 2, 2, 1], [3], []])
def test_all_node_form_equals_sequential_walk(ks, mode):
    """Section 3: the literal procedure visits one node per step; evaluating every node first
    and then following the accepted children gives the same result because each test owns
    its uniform."""
    rng = np.random.default_rng(23 + mode + 10 * len(ks))
    parent, st, target, draft, cand, unif = _random_case(rng, ks, 48, 33, mode)
    a = oracle.verify(target, draft if st["n_internal"] else None, parent, cand, unif, 1.0, mode)
    s = oracle.verify(target, draft if st["n_internal"] else None, parent, cand, unif, 1.0, mode,
                      sequential=True)
    assert np.array_equal(a.accept_len, s.accept_len)
    assert np.array_equal(a.tokens, s.tokens)
    assert np.array_equal(a.residual, s.residual)
    gamma = st["gamma"]
    assert ((a.accept_len >= 0) & (a.accept_len <= gamma)).all()       # 1..gamma+1 tokens out
    n_tok = (a.tokens >= 0).sum(axis=1)
    assert np.array_equal(n_tok, a.accept_len + 1)
    visited = s.node_accept != -2
    assert np.array_equal(a.node_accept[visited], s.node_accept[visited])
    assert np.array_equal(a.node_bonus[visited], s.node_bonus[visited])
    # path consistency: accepted tokens are the candidates along parent links
    for b in range(a.tokens.shape[0]):
        n = 0
        for i in range(a.accept_len[b]):
            c = a.node_accept[b, n]
            assert parent[c] == n and a.tokens[b, i] == cand[b, c]
            n = c
        assert a.node_accept[b, n] == -1 and a.tokens[b, a.accept_len[b]] == a.node_bonus[b, n]


def test_chain_tree_is_standard_speculative_decoding():
    """Section 2: with one candidate per step, verification accepts a prefix of the draft
    and stops at the first rejection."""
    rng = np.random.default_rng(29)
    parent, st, target, draft, cand, unif = _random_case(rng, [1, 1, 1, 1, 1], 200, 17, 0)
    res = oracle.verify(target, draft, parent, cand, unif, 1.0, 0)
    for b in range(200):
        n_acc = 0
        for n in range(5):
            p = scipy.special.softmax(target[b, n].astype(np.float64))
            q = scipy.special.softmax(draft[b, n].astype(np.float64))
            x = cand[b, n + 1]
            if float(unif[b, n + 1, 0]) <= p[x] / q[x]:
                n_acc += 1
            else:
                break
        assert res.accept_len[b] == n_acc
    assert 0 < (res.accept_len == 5).sum() < 200


def test_rejects_malformed_trees():
    t = np.zeros((1, 3, 4), dtype=np.float32)
    d = np.zeros((1, 1, 4), dtype=np.float32)
    c = np.zeros((1, 3), dtype=np.int32)
    u = np.full((1, 3, 2), 0.5, dtype=np.float32)
    oracle.verify(t, d, np.array([-1, 0, 0]), c, u, 1.0, 0)
    with pytest.raises(ValueError):
        oracle.verify(t, d, np.array([0, 0, 0]), c, u, 1.0, 0)
    # not in level order: the children of node 2 come before those of node 1
    t5 = np.zeros((1, 5, 4), dtype=np.float32)
    with pytest.raises(ValueError):
        oracle.verify(t5, np.zeros((1, 3, 4), dtype=np.float32), np.array([-1, 0, 0, 2, 1]),
                      np.zeros((1, 5), dtype=np.int32), np.full((1, 5, 2), 0.5, dtype=np.float32), 1.0, 0)
