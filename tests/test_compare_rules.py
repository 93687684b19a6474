"""The comparison rules (oracle/compare.py) judge every GPU parity test, so they are tested
themselves, on CPU: the oracle's own outputs must pass with nothing counted, and every kind of
deviation the rules name must be either rejected or counted exactly as the rule says.  The
"implementation under test" here is the oracle's output with one planted deviation."""
import numpy as np
import pytest
import torch

import oracle
from oracle import compare
from paper_2401_06706_b200 import synth


def _case(mode=0, kconfig="3x2", vocab=60, batch=24, seed=11, sigma=1.0):
    w = synth.Workload("rules", batch, vocab, kconfig, "fp32", "normal", 2.0, 1.0, sigma, 1.0, mode, seed)
    inp = synth.make_inputs(w, "cpu")
    t, d, c, u = inp.host_f32()
    ref = oracle.verify(t, d, inp.parent, c, u, w.temperature, w.mode)
    gamma = oracle.tree_gamma(inp.parent)
    return w, inp, (t, d, c, u), ref, oracle.path_nodes(ref, gamma)


def _run(w, inp, arrays, **outs):
    t, d, c, u = arrays
    return compare.compare(t, d, inp.parent, c, u, w.temperature, w.mode, w.dtype, **outs)


def _outs(ref, paths, **change):
    o = dict(accept_len=ref.accept_len.copy(), tokens=ref.tokens.copy(), residual=ref.residual.astype(np.float32),
             node_accept=ref.node_accept.copy(), node_bonus=ref.node_bonus.copy(), status=ref.status.copy(),
             path_nodes=paths.copy())
    o.update(change)
    return o


@pytest.mark.parametrize("mode", [0, 1])
def test_the_oracles_own_outputs_pass_with_nothing_counted(mode):
    w, inp, arrays, ref, paths = _case(mode)
    rep = _run(w, inp, arrays, **_outs(ref, paths))
    assert rep.ok, rep.failures
    assert rep.n_flipped == 0 and rep.n_excluded_sequences == 0 and rep.n_bonus_tolerated == 0
    assert rep.n_tests > 0 and rep.n_bonus_draws > 0 and rep.max_residual_err < 1e-6


def test_each_plain_deviation_is_rejected():
    w, inp, arrays, ref, paths = _case()
    b = int(np.argmax(ref.accept_len > 0))          # a sequence that accepted something
    L = int(ref.accept_len[b])

    o = _outs(ref, paths); o["accept_len"][b] = L - 1
    assert any("accepted length" in f for f in _run(w, inp, arrays, **o).failures)

    o = _outs(ref, paths); o["tokens"][b, 0] = (o["tokens"][b, 0] + 1) % w.vocab
    assert any("accepted tokens" in f for f in _run(w, inp, arrays, **{k: v for k, v in o.items() if k != "path_nodes"}).failures)

    o = _outs(ref, paths)
    if L + 1 < o["tokens"].shape[1]:
        o["tokens"][b, L + 1] = 5
        assert any("padding" in f for f in _run(w, inp, arrays, **o).failures)

    o = _outs(ref, paths); o["residual"][b, 3] += 5e-5          # five times the fp32 tolerance
    assert any("residual" in f for f in _run(w, inp, arrays, **o).failures)

    o = _outs(ref, paths); o["status"][b] ^= 1
    assert any("status" in f for f in _run(w, inp, arrays, **o).failures)

    # an endpoint token far from the uniform's place in the distribution
    o = _outs(ref, paths)
    P = ref.residual[b]
    far = int(np.argmin(np.where(P > 0, np.abs(np.cumsum(P) - ((arrays[3][b, :, 1].max() + 0.5) % 1.0)), np.inf)))
    if far == int(ref.tokens[b, L]):
        far = (far + 7) % w.vocab
    o["tokens"][b, L] = far
    o["node_bonus"] = None
    rep = _run(w, inp, arrays, **o)
    assert any("endpoint token" in f for f in rep.failures) or rep.n_bonus_tolerated == 1
    # ... and one without any probability is never tolerated
    t2 = arrays[0].copy(); t2[:, :, 9] = -np.inf
    ref2 = oracle.verify(t2, arrays[1], inp.parent, arrays[2], arrays[3], 1.0, 0)
    o = _outs(ref2, oracle.path_nodes(ref2, oracle.tree_gamma(inp.parent)))
    o["tokens"][0, int(ref2.accept_len[0])] = 9
    o["node_bonus"] = None
    rep = compare.compare(t2, arrays[1], inp.parent, arrays[2], arrays[3], 1.0, 0, "fp32", **o)
    assert any("seq 0: endpoint token 9" in f for f in rep.failures)


def test_a_decision_that_differs_away_from_a_tie_is_rejected_and_one_at_a_tie_is_counted():
    w, inp, arrays, ref, paths = _case(mode=0, batch=16)
    t, d, c, u = arrays
    first, count = compare._children(inp.parent)
    # a root test whose outcome is moved by the uniform: put the uniform right at the ratio
    b = int(np.argmax((ref.node_ratio[:, 1] > 0.05) & (ref.node_ratio[:, 1] < 0.95)))
    rho = float(ref.node_ratio[b, 1])
    u_tie = u.copy(); u_tie[b, 1, 0] = np.float32(rho + 4e-6)            # just above: the oracle rejects candidate 1
    ref_tie = oracle.verify(t, d, inp.parent, c, u_tie, 1.0, 0)
    assert ref_tie.node_accept[b, 0] != 1
    # the implementation under test accepted candidate 1 (the other side of the tie) and walked on from there
    other = oracle.verify(t, d, inp.parent, c, np.where(np.arange(u.shape[1])[None, :, None] == 1,
                                                     np.float32(rho - 4e-6), u_tie).astype(np.float32), 1.0, 0)
    mixed = _outs(ref_tie, oracle.path_nodes(ref_tie, oracle.tree_gamma(inp.parent)))
    po = oracle.path_nodes(other, oracle.tree_gamma(inp.parent))
    for k in ("accept_len", "tokens", "node_accept", "node_bonus", "status"):
        mixed[k][b] = getattr(other, k)[b]
    mixed["residual"][b] = other.residual[b]
    mixed["path_nodes"][b] = po[b]
    rep = compare.compare(t, d, inp.parent, c, u_tie, 1.0, 0, "fp32", **mixed)
    assert rep.ok, rep.failures
    assert rep.n_flipped >= 1 and b in rep.excluded                      # counted, and left out of the path comparison
    # the same difference with the uniform far from the ratio is an error
    u_far = u.copy(); u_far[b, 1, 0] = np.float32(min(rho + 0.04, 0.999))
    ref_far = oracle.verify(t, d, inp.parent, c, u_far, 1.0, 0)
    wrong = _outs(ref_far, oracle.path_nodes(ref_far, oracle.tree_gamma(inp.parent)))
    wrong["node_accept"][b, 0] = 1 if ref_far.node_accept[b, 0] != 1 else 2
    assert any(f"seq {b} node 0" in f for f in compare.compare(t, d, inp.parent, c, u_far, 1.0, 0, "fp32", **wrong).failures)
    # a sequence on the other side of a tie must still be a walk of the tree
    broken = {k: (v.copy() if v is not None else None) for k, v in mixed.items()}
    if broken["accept_len"][b] > 0:
        broken["path_nodes"][b, 0] = first[0] + count[0]                 # a node that is no child of the root
        rep = compare.compare(t, d, inp.parent, c, u_tie, 1.0, 0, "fp32", **broken)
        assert any("not a walk of the tree" in f for f in rep.failures)
    broken = {k: (v.copy() if v is not None else None) for k, v in mixed.items()}
    broken["accept_len"][b] = 99
    assert any("outside" in f for f in compare.compare(t, d, inp.parent, c, u_tie, 1.0, 0, "fp32", **broken).failures)


def test_endpoint_draws_at_a_boundary_are_tolerated_counted_and_bounded():
    w, inp, arrays, ref, paths = _case(mode=0, batch=12, kconfig="2")
    t, d, c, u = arrays
    B = t.shape[0]
    # put every endpoint uniform right below the upper boundary of the oracle's token: the next token
    # with mass is then within the tolerance, any other is not
    u2 = u.copy()
    first = oracle.verify(t, d, inp.parent, c, u2, 1.0, 0)
    stop = np.array([n if first.node_accept[b, 0] < 0 else int(first.node_accept[b, 0]) for b, n in enumerate(np.zeros(B, int))])
    for b in range(B):
        P = first.residual[b]
        cdf = np.cumsum(P) / P.sum()
        tok = int(first.tokens[b, int(first.accept_len[b])])
        u2[b, stop[b], 1] = np.float32(cdf[tok] - 2e-6) if cdf[tok] < 0.999 else u2[b, stop[b], 1]
    ref2 = oracle.verify(t, d, inp.parent, c, u2, 1.0, 0)
    base = _outs(ref2, oracle.path_nodes(ref2, oracle.tree_gamma(inp.parent)), node_bonus=None)
    moved = 0
    for b in range(B):
        L = int(ref2.accept_len[b]); P = ref2.residual[b]
        tok = int(ref2.tokens[b, L])
        nxt = tok + 1
        while nxt < w.vocab and not P[nxt] > 0:
            nxt += 1
        cdf = np.cumsum(P) / P.sum()
        if nxt < w.vocab and abs(float(u2[b, stop[b], 1]) - cdf[tok]) < 5e-6 and moved < 5:
            base["tokens"][b, L] = nxt
            moved += 1
            if moved == 2:
                rep = compare.compare(t, d, inp.parent, c, u2, 1.0, 0, "fp32", **{k: (v.copy() if v is not None else None) for k, v in base.items()})
                assert rep.ok and rep.n_bonus_tolerated == 2, (rep.failures, rep.n_bonus_tolerated)
    assert moved >= 4, "the construction needs at least four sequences with a next token"
    rep = compare.compare(t, d, inp.parent, c, u2, 1.0, 0, "fp32", **base)
    # more than the limit (3 events at this size): rejected although each single draw is inside the tolerance
    assert compare.boundary_draw_limit(w.vocab, B) == 3.0
    assert rep.n_bonus_tolerated == moved and any("float rounding explains" in f for f in rep.failures)
    # two tokens further is outside the tolerance
    far = _outs(ref2, oracle.path_nodes(ref2, oracle.tree_gamma(inp.parent)), node_bonus=None)
    L = int(ref2.accept_len[0])
    far["tokens"][0, L] = (int(ref2.tokens[0, L]) + 17) % w.vocab
    rep = compare.compare(t, d, inp.parent, c, u2, 1.0, 0, "fp32", **far)
    assert any("seq 0: endpoint token" in f for f in rep.failures)


@pytest.mark.parametrize("mode", [0, 1])
def test_sample_rule_passes_the_oracles_draws_and_rejects_a_wrong_one(mode):
    w, inp, arrays, ref, paths = _case(mode, batch=6)
    t, d, c, u = arrays
    gen = torch.Generator().manual_seed(5)
    ud = synth.open_uniforms((t.shape[0], t.shape[1]), gen, "cpu").numpy()
    cand = oracle.sample(d, inp.parent, ud, 1.0, mode)
    rep = compare.compare_samples(d, inp.parent, ud, 1.0, mode, cand)
    assert rep.ok and rep.n_tolerated == 0 and rep.n_draws == t.shape[0] * (t.shape[1] - 1)
    bad = cand.copy()
    q = oracle.softmax(d[0, 0], 1.0)
    bad[0, 1] = int(np.argmin(q))                      # the least likely token in place of the first draw of the root
    if bad[0, 1] == cand[0, 1]:
        bad[0, 1] = int(np.argmax(q))
    rep = compare.compare_samples(d, inp.parent, ud, 1.0, mode, bad)
    assert (not rep.ok and "seq 0 node 0 draw 0" in rep.failures[0]) or rep.n_tolerated == 1
