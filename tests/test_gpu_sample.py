"""mcsd_sample_candidates (Section 3.2, Eq. 1) against the oracle's sampler on the same seeded
inputs: tokens identical except within 1e-5 (CDF units) of an interval boundary; top-k exact."""
import numpy as np
import pytest
import torch

import oracle
from oracle import compare as cmp
from paper_2401_06706_b200 import binding, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    binding.load_library()


def _inputs(w, seed):
    inp = synth.make_inputs(w, "cuda")
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    u = synth.open_uniforms((w.batch, inp.stats["n_nodes"]), gen, "cuda")
    return inp, u


def _check(inp, u, cand, T, mode, node_begin=0, node_end=None):
    d = inp.draft.to(torch.float32).cpu().numpy()
    rep = cmp.compare_samples(d, inp.parent, u.cpu().numpy(), T, mode, cand.cpu().numpy(), node_begin, node_end)
    assert rep.ok, "\n".join(rep.failures[:10])
    # (rep.ok includes the bound on draws that differ inside the tolerance: compare.boundary_draw_limit)
    return rep


@pytest.mark.parametrize("dtype", ["fp32", "bf16", "fp16"])
@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("vocab,kconfig", [(7, "3x2"), (1000, "4x2"), (8200, "8x1"), (32000, "4x2x2x1"),
                                           (32001, "2x2"), (50272, "2x2x2x2"), (65536, "32"), (32000, "32"), (20000, "16x2")])
def test_draws_match_the_oracle(vocab, kconfig, mode, dtype):
    if mode == 1 and vocab < 16:
        kconfig = "3x2"
    w = synth.Workload("sample", 6, vocab, kconfig, dtype, "normal", 2.5, 1.0, 1.0, 1.0, mode, 700 + vocab)
    inp, u = _inputs(w, 1 + vocab)
    cand = binding.mcsd_sample_candidates(inp.draft, inp.parent, u, 1.0, mode)
    torch.cuda.synchronize()
    rep = _check(inp, u, cand, 1.0, mode)
    c = cand.cpu().numpy()
    assert (c[:, 0] == -1).all() and (c[:, 1:] >= 0).all() and (c[:, 1:] < vocab).all()
    if mode == 1:   # Eq. 1: the children of a node carry distinct tokens
        first, count = synth.children_ranges(inp.parent)
        for n in range(inp.stats["n_internal"]):
            ch = c[:, first[n]:first[n] + count[n]]
            assert all(len(set(row)) == len(row) for row in ch.tolist())


@pytest.mark.parametrize("T,mode", [(1.0, 0), (1.0, 1), (0.0, 0)])
@pytest.mark.parametrize("dtype,vocab", [("fp32", 5003), ("bf16", 5003), ("fp16", 32001), ("fp32", 3), ("bf16", 5)])
def test_aligned_rows_whose_vocabulary_ends_inside_a_vector(dtype, vocab, T, mode):
    """Padded, 16-byte aligned rows: the padding in the last vector is larger than every logit
    and must neither be drawn nor carry weight."""
    w = synth.Workload("sample_tail", 5, vocab, "4x2" if vocab > 16 else "2x2", dtype, "normal", 2.5, 1.0, 1.0, 1.0, mode, 300 + vocab)
    inp, u = _inputs(w, 5 + vocab)
    per16 = 16 // inp.draft.element_size()
    ld = (vocab + per16 - 1) // per16 * per16
    assert ld > vocab
    dpad = torch.full((5, inp.stats["n_internal"], ld), 50.0, dtype=inp.draft.dtype, device="cuda")
    dpad[:, :, :vocab] = inp.draft
    cand = binding.mcsd_sample_candidates(dpad[:, :, :vocab], inp.parent, u, T, mode)
    torch.cuda.synchronize()
    c = cand.cpu().numpy()
    assert (c[:, 1:] >= 0).all() and (c[:, 1:] < vocab).all()
    if T > 0:
        _check(inp, u, cand, T, mode)
    else:
        d = inp.draft.to(torch.float32).cpu().numpy()
        first, count = synth.children_ranges(inp.parent)
        for b in range(5):
            for n in range(inp.stats["n_internal"]):
                want = oracle.topk(d[b, n], int(count[n]))
                got = c[b, first[n]:first[n] + count[n]]
                assert (d[b, n][got] == d[b, n][want]).all()


@pytest.mark.parametrize("T", [0.3, 0.7, 1.7])
def test_temperatures_and_peaked_rows(T):
    w = synth.Workload("sample_T", 16, 6000, "8x2", "fp16", "gumbel", 3.0, 1.0, 1.0, T, 1, 31)
    inp, u = _inputs(w, 77)
    cand = binding.mcsd_sample_candidates(inp.draft, inp.parent, u, T, 1)
    torch.cuda.synchronize()
    _check(inp, u, cand, T, 1)


def test_top_k_at_temperature_zero_with_ties():
    w = synth.Workload("sample_t0", 8, 3000, "16x2", "fp16", "normal", 1.0, 1.0, 0.5, 0.0, 0, 5)   # coarse fp16: many ties
    inp, u = _inputs(w, 3)
    cand = binding.mcsd_sample_candidates(inp.draft, inp.parent, None, 0.0, 0)
    torch.cuda.synchronize()
    rep = _check(inp, u, cand, 0.0, 0)
    assert rep.n_tolerated == 0
    # the input generator's own top-k (torch.topk, tie order unspecified) picks the same logit values
    first, count = synth.children_ranges(inp.parent)
    for n in range(inp.stats["n_internal"]):
        sl = slice(first[n], first[n] + count[n])
        mine = torch.gather(inp.draft[:, n].float(), 1, cand[:, sl].long())
        theirs = torch.gather(inp.draft[:, n].float(), 1, inp.cand[:, sl].long())
        assert torch.equal(mine, theirs)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("vocab", [32000, 40000])
def test_top_k_when_one_thread_holds_many_of_the_largest(dtype, vocab):
    """The k largest logits sit, with ties, at indices a single thread of the kernel reads (the
    same 16-byte group position in every step of one warp's run), so that thread has to renew
    its best after every pick; others are spread out.  Exact indices against the oracle."""
    w = synth.Workload("sample_t0_one_thread", 3, vocab, "32", dtype, "normal", 1.0, 1.0, 0.5, 0.0, 0, 11)
    inp, u = _inputs(w, 13)
    per_group = 16 // inp.draft.element_size()
    draft = inp.draft.clone()
    step = 32 * per_group
    for b in range(3):
        hot = [s * step + e for s in range(6) for e in range(per_group)][:24]      # one lane's groups
        vals = torch.tensor([20.0 + (i // 3) for i in range(len(hot))], dtype=draft.dtype)   # runs of three equal values
        draft[b, 0, torch.tensor(hot) + 1000 * b * 0] = vals.to(draft.device)
        draft[b, 0, vocab - 1 - b] = 19.5
    cand = binding.mcsd_sample_candidates(draft, inp.parent, None, 0.0, 0)
    torch.cuda.synchronize()
    d = draft.to(torch.float32).cpu().numpy()
    c = cand.cpu().numpy()
    for b in range(3):
        assert (c[b, 1:33] == oracle.topk(d[b, 0], 32)).all(), b


def test_node_range_touches_only_its_children_and_levels_compose():
    w = synth.Workload("sample_levels", 5, 4096, "3x2x2", "bf16", "normal", 2.5, 1.0, 1.0, 1.0, 1, 9)
    inp, u = _inputs(w, 21)
    whole = binding.mcsd_sample_candidates(inp.draft, inp.parent, u, 1.0, 1)
    by_level = torch.full_like(whole, -1)
    for lo, hi in ((0, 1), (1, 4), (4, 10)):           # root, level 1, level 2
        before = by_level.clone()
        binding.mcsd_sample_candidates(inp.draft, inp.parent, u, 1.0, 1, node_begin=lo, node_end=hi, cand=by_level)
        torch.cuda.synchronize()
        first, count = synth.children_ranges(inp.parent)
        touched = torch.zeros(whole.shape[1], dtype=torch.bool)
        for n in range(lo, hi):
            touched[first[n]:first[n] + count[n]] = True
        assert torch.equal(by_level[:, ~touched], before[:, ~touched])
    assert torch.equal(by_level, whole)


def test_sampled_candidates_feed_verification():
    """End to end on the device: draw the candidates, verify them, compare with the oracle doing both."""
    import oracle
    from gpu_util import assert_parity
    w = synth.Workload("sample_verify", 8, 32000, "4x2x1", "fp32", "normal", 2.5, 1.0, 1.0, 1.0, 1, 123)
    inp, u = _inputs(w, 8)
    cand = binding.mcsd_sample_candidates(inp.draft, inp.parent, u, 1.0, 1)
    _check(inp, u, cand, 1.0, 1)
    inp.cand = cand
    v = binding.Verifier(w.batch, inp.parent, w.vocab, torch.float32, "cuda", node_outputs=True)
    out = v.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, 1.0, 1)
    torch.cuda.synchronize()
    assert_parity(inp, out)
