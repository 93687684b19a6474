"""Pins of the oracle's tree-attention layout (Section 3.3): the mask is the reflexive-transitive
closure of the parent relation (checked by boolean matrix powers), a hand-drawn tree, and the
position ids are root position + depth."""
import numpy as np

import oracle
from paper_2401_06706_b200 import synth


def test_hand_drawn_tree():
    #        0
    #      /   \
    #     1     2
    #    / \    |
    #   3   4   5
    parent = [-1, 0, 0, 1, 1, 2]
    mask, pos = oracle.tree_attention_layout(parent, 10)
    want = np.array([[1, 0, 0, 0, 0, 0],
                     [1, 1, 0, 0, 0, 0],
                     [1, 0, 1, 0, 0, 0],
                     [1, 1, 0, 1, 0, 0],
                     [1, 1, 0, 0, 1, 0],
                     [1, 0, 1, 0, 0, 1]], dtype=np.uint8)
    assert np.array_equal(mask, want)
    assert pos.tolist() == [10, 11, 11, 12, 12, 12]


def test_mask_is_the_closure_of_the_parent_relation():
    for ks in ([4, 2, 2, 1], [2, 2, 2, 2], [8, 1, 1], [1, 1, 1, 1, 1], []):
        parent = synth.tree_from_kconfig(ks)
        n = parent.shape[0]
        mask, pos = oracle.tree_attention_layout(parent, 7)
        step = np.eye(n, dtype=np.int64)
        for c in range(1, n):
            step[c, parent[c]] = 1                       # reflexive parent relation
        closure = np.linalg.matrix_power(step, max(n, 1)) > 0
        assert np.array_equal(mask.astype(bool), closure)
        assert np.array_equal(mask.sum(axis=1), pos - 7 + 1)          # a node sees itself and depth ancestors
        assert np.array_equal(np.triu(mask, 1), np.zeros_like(mask))  # level order: nobody sees a later node
        assert (mask[:, 0] == 1).all()                                # everybody sees the root


def test_kv_rows_of_the_accepted_path_hand_example():
    # prefix of 2 committed tokens, the tree of test_hand_drawn_tree at positions 2..7, the walk accepted
    # nodes 2 and 5: position 3 takes the row of position 4, position 4 the row of position 7
    cache = np.arange(2 * 1 * 9 * 3).reshape(2, 1, 9, 3)
    out = oracle.gather_accepted_kv(cache, [2], [[2, 5, -1]], [2])
    for s in range(2):
        rows = [r.tolist() for r in cache[s, 0]]
        want = [rows[0], rows[1], rows[2], rows[4], rows[7], rows[5], rows[6], rows[7], rows[8]]
        assert [r.tolist() for r in out[s, 0]] == want
    # nothing accepted: nothing moves; a chain accepted in full: every row is where it belongs already
    assert np.array_equal(oracle.gather_accepted_kv(cache, [2], [[-1, -1, -1]], [0]), cache)
    assert np.array_equal(oracle.gather_accepted_kv(cache, [4], [[1, 2, 3]], [3]), cache)


def test_kv_rows_follow_the_accepted_tokens_of_verify():
    """A cache whose row at the position of node n holds that node's token: after the gather the
    committed positions hold exactly the accepted tokens that verification returned."""
    rng = np.random.default_rng(5)
    parent = synth.tree_from_kconfig([3, 2, 2])
    n = parent.shape[0]
    B, V, prefix = 6, 50, np.array([0, 3, 1, 7, 2, 5])
    target = rng.normal(size=(B, n, V)).astype(np.float32)
    n_int = int((np.bincount(parent[1:], minlength=n) > 0).sum())
    draft = (target[:, :n_int] + 0.3 * rng.normal(size=(B, n_int, V))).astype(np.float32)
    cand = rng.integers(0, V, size=(B, n)).astype(np.int32)
    unif = rng.uniform(0.01, 0.99, size=(B, n, 2)).astype(np.float32)
    res = oracle.verify(target, draft, parent, cand, unif, 1.0, 0)
    gamma = oracle.tree_gamma(parent)
    nodes = oracle.path_nodes(res, gamma)
    L = int(prefix.max()) + n
    cache = np.full((1, B, L, 1), -7, dtype=np.int64)
    for b in range(B):
        cache[0, b, prefix[b] + np.arange(n), 0] = cand[b]
    out = oracle.gather_accepted_kv(cache, prefix, nodes, res.accept_len)
    assert res.accept_len.max() > 0
    for b in range(B):
        k = int(res.accept_len[b])
        assert out[0, b, prefix[b] + 1: prefix[b] + 1 + k, 0].tolist() == res.tokens[b, :k].tolist()
        assert out[0, b, :prefix[b] + 1, 0].tolist() == cache[0, b, :prefix[b] + 1, 0].tolist()
