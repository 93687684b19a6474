"""Host logic of the seeded input generators."""
import numpy as np
import pytest
import torch

from paper_2401_06706_b200 import synth


def test_kconfig_trees_have_the_stated_sizes():
    # node counts quoted with the configurations: 4x2x2x1 -> 44 draft nodes, 2x2x2x2 -> 30
    for text, n_draft, n_int, gamma in [("2", 2, 1, 1), ("4x2x2x1", 44, 29, 4), ("8x2x1", 40, 25, 3),
                                        ("2x2x2x2", 30, 15, 4), ("4x4x2x2x1", 180, 117, 5),
                                        ("1x1x1x1", 4, 4, 4), ("8x1x1x1", 32, 25, 4)]:
        parent = synth.tree_from_kconfig(synth.parse_kconfig(text))
        st = synth.tree_stats(parent)
        assert (st["n_draft"], st["n_internal"], st["gamma"]) == (n_draft, n_int, gamma)
        assert parent[0] == -1 and (parent[1:] < np.arange(1, len(parent))).all()
        assert (np.diff(parent) >= 0).all()                       # level order, children contiguous
        first, count = synth.children_ranges(parent)
        assert (count[:n_int] > 0).all() and (count[n_int:] == 0).all()
    assert synth.tree_from_kconfig([]).tolist() == [-1]
    with pytest.raises(ValueError):
        synth.parse_kconfig("4x0")


def test_uniforms_are_open_interval_and_exact():
    g = torch.Generator().manual_seed(1)
    u = synth.open_uniforms((100000,), g, "cpu")
    assert u.dtype == torch.float32 and float(u.min()) > 0 and float(u.max()) < 1
    i = u.double() * 2 ** 23 - 0.5
    assert torch.equal(i, i.round())
    assert abs(float(u.mean()) - 0.5) < 0.01


def test_inputs_are_reproducible_and_shaped():
    w = synth.Workload("t", 3, 257, "3x2", "bf16", "normal", 2.5, 0.8, 1.5, 1.0, 1, 99)
    a, b = synth.make_inputs(w), synth.make_inputs(w)
    assert torch.equal(a.target, b.target) and torch.equal(a.cand, b.cand) and torch.equal(a.unif, b.unif)
    assert a.target.shape == (3, 10, 257) and a.draft.shape == (3, 4, 257) and a.target.dtype == torch.bfloat16
    assert a.cand.shape == (3, 10) and (a.cand[:, 0] == -1).all()
    assert ((a.cand[:, 1:] >= 0) & (a.cand[:, 1:] < 257)).all()
    # without replacement: siblings are distinct
    first, count = synth.children_ranges(a.parent)
    for n in range(4):
        sib = a.cand[:, first[n]:first[n] + count[n]]
        for row in sib.tolist():
            assert len(set(row)) == len(row)
    assert a.logit_bytes() == (3 * 10 * 257 + 3 * 4 * 257) * 2


def test_temperature_zero_candidates_are_top_k_of_the_draft():
    w = synth.Workload("g", 2, 101, "3x1", "fp16", "normal", 3.0, 1.0, 2.0, 0.0, 0, 5)
    inp = synth.make_inputs(w)
    top = torch.topk(inp.draft[:, 0].float(), 3, dim=-1).indices
    assert torch.equal(inp.cand[:, 1:4].long(), top)


def test_named_and_sweep_workloads():
    named = synth.named_workloads()
    assert named["cfg4_opt"].vocab == 50272 and named["cfg3_greedy"].temperature == 0.0
    sweep = synth.sweep_workloads()
    assert len(sweep) == 300 and len({w.seed for w in sweep}) == 300
    big = named["cfg5_largest"]
    st = synth.tree_stats(synth.tree_from_kconfig(big.ks))
    assert big.batch * (st["n_nodes"] + st["n_internal"]) * big.vocab * 4 == 19_529_728_000
