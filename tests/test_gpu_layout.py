"""mcsd_tree_attention_layout and the accepted-path node output against the oracle (bit-exact)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2401_06706_b200 import binding, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    binding.load_library()


@pytest.mark.parametrize("kconfig", ["", "1", "4x2x2x1", "2x2x2x2", "8x2x1", "32", "1x1x1x1x1x1x1x1", "4x4x2x2x1", "8x8x6"])
def test_mask_and_positions(kconfig):
    parent = synth.tree_from_kconfig(synth.parse_kconfig(kconfig))
    mask, pos = binding.mcsd_tree_attention_layout(parent, 123)
    torch.cuda.synchronize()
    want_mask, want_pos = oracle.tree_attention_layout(parent, 123)
    assert np.array_equal(mask.cpu().numpy(), want_mask)
    assert np.array_equal(pos.cpu().numpy(), want_pos)


@pytest.mark.parametrize("entry,mode,T", [("mcsd_verify", 0, 1.0), ("mcsd_verify", 1, 0.7), ("mcsd_verify_path", 1, 1.0),
                                          ("mcsd_verify", 2, 1.0), ("mcsd_verify", 0, 0.0)])
def test_accepted_path_nodes(entry, mode, T):
    w = synth.Workload("pathnodes", 48, 5000, "4x2x2x1", "fp32", "normal", 2.5, 1.0, 0.7, T, min(mode, 1), 77)
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, torch.float32, "cuda")
    out = getattr(v, entry)(inp.target, inp.draft if (T > 0 and mode != 2) else None, inp.cand, inp.unif, T, mode)
    torch.cuda.synchronize()
    t, d, c, u = inp.host_f32()
    ref = oracle.verify(t, d if (T > 0 and mode != 2) else None, inp.parent, c, u, T, mode)
    want = oracle.path_nodes(ref, inp.stats["gamma"])
    same = out.accept_len.cpu().numpy() == ref.accept_len        # (sequences with a near-tie flip would differ)
    assert same.mean() > 0.95
    assert np.array_equal(out.path_nodes.cpu().numpy()[same], want[same])
    # the tokens on the path are the tokens of those nodes
    pn = out.path_nodes.cpu().numpy()
    tok = out.tokens.cpu().numpy()
    for b in range(w.batch):
        L = int(out.accept_len[b])
        assert (pn[b, L:] == -1).all() and (c[b, pn[b, :L]] == tok[b, :L]).all()
