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
