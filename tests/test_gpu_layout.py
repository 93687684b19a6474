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
    from oracle import compare as cmp
    w = synth.Workload("pathnodes", 48, 5000, "4x2x2x1", "fp32", "normal", 2.5, 1.0, 0.7, T, min(mode, 1), 77)
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, torch.float32, "cuda")
    out = getattr(v, entry)(inp.target, inp.draft if (T > 0 and mode != 2) else None, inp.cand, inp.unif, T, mode)
    torch.cuda.synchronize()
    t, d, c, u = inp.host_f32()
    ref = oracle.verify(t, d if (T > 0 and mode != 2) else None, inp.parent, c, u, T, mode)
    want = oracle.path_nodes(ref, inp.stats["gamma"])
    pn = out.path_nodes.cpu().numpy()
    tok = out.tokens.cpu().numpy()
    # the comparison rule: a walk may leave the oracle's only at a test inside the near-tie band
    # (naive sampling: at a draw inside the boundary tolerance); every other sequence is exact
    rep = cmp.compare(t, d, inp.parent, c, u, T, mode, "fp32", oracle_result=ref, accept_len=out.accept_len.cpu().numpy(),
                      tokens=tok, residual=out.residual.cpu().numpy(), status=out.status.cpu().numpy(), path_nodes=pn)
    assert rep.ok, rep.failures[:5]
    keep = np.ones(w.batch, dtype=bool)
    keep[rep.excluded] = False
    assert keep.sum() >= w.batch - 2
    assert np.array_equal(pn[keep], want[keep])
    # the tokens on the path are the tokens of those nodes
    for b in range(w.batch):
        L = int(out.accept_len[b])
        assert (pn[b, L:] == -1).all() and (c[b, pn[b, :L]] == tok[b, :L]).all()


@pytest.mark.parametrize("dtype,row_shape", [(torch.float16, (8, 64)), (torch.bfloat16, (3, 5)), (torch.float32, (7,)),
                                             (torch.uint8, (13,)), (torch.float16, (2, 36))])
@pytest.mark.parametrize("kconfig,sigma", [("4x2x2x1", 0.5), ("1x1x1x1x1x1", 0.3), ("8x2", 2.0)])
def test_kv_rows_of_the_accepted_path(dtype, row_shape, kconfig, sigma):
    """mcsd_gather_accepted_kv, in place, against the oracle's copy semantics (bit-exact): the path
    nodes and accepted lengths come from mcsd_verify on the same trees; every unit width of the
    copy (16 down to 1 byte) is reached through the row shapes."""
    w = synth.Workload("kv", 9, 500, kconfig, "fp32", "normal", 2.5, 1.0, sigma, 1.0, 0, 31)
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, torch.float32, "cuda")
    out = v.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, 1.0, 0)
    torch.cuda.synchronize()
    n = inp.stats["n_nodes"]
    gen = torch.Generator(device="cuda"); gen.manual_seed(7)
    prefix = torch.randint(0, 20, (w.batch,), generator=gen, device="cuda", dtype=torch.int32)
    L = 20 + n + 3
    S = 4
    raw = torch.randint(0, 255, (S, w.batch, L) + row_shape, generator=gen, device="cuda", dtype=torch.uint8)
    cache = raw.to(dtype) if dtype != torch.uint8 else raw
    before = cache.clone()
    binding.mcsd_gather_accepted_kv(cache, prefix, out.path_nodes, out.accept_len)
    torch.cuda.synchronize()
    as_bits = lambda t: t.contiguous().view(torch.uint8).cpu().numpy()
    want = oracle.gather_accepted_kv(as_bits(before).reshape(S, w.batch, L, -1), prefix.cpu().numpy(),
                                     out.path_nodes.cpu().numpy(), out.accept_len.cpu().numpy())
    assert np.array_equal(as_bits(cache).reshape(S, w.batch, L, -1), want)
    assert int(out.accept_len.max()) > 0


def test_kv_gather_on_a_strided_cache_and_degenerate_calls():
    # a cache with padded rows and sequences (views of a larger tensor), accepted lengths of zero, an empty batch
    w = synth.Workload("kv2", 5, 300, "3x2x1", "fp32", "normal", 2.5, 1.0, 0.5, 1.0, 0, 32)
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, torch.float32, "cuda")
    out = v.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, 1.0, 0)
    torch.cuda.synchronize()
    n = inp.stats["n_nodes"]
    gen = torch.Generator(device="cuda"); gen.manual_seed(8)
    big = torch.randn((2, w.batch + 1, n + 9, 2, 40), generator=gen, device="cuda", dtype=torch.float16)
    big_before = big.clone()
    cache = big[:, :w.batch, 2:, :, :]            # non-trivial slab, sequence and position strides
    before = cache.clone()
    prefix = torch.full((w.batch,), 4, dtype=torch.int32, device="cuda")
    binding.mcsd_gather_accepted_kv(cache, prefix, out.path_nodes, out.accept_len)
    torch.cuda.synchronize()
    want = oracle.gather_accepted_kv(before.cpu().numpy().reshape(2, w.batch, n + 7, -1), prefix.cpu().numpy(),
                                     out.path_nodes.cpu().numpy(), out.accept_len.cpu().numpy())
    assert np.array_equal(cache.cpu().numpy().reshape(2, w.batch, n + 7, -1), want)
    # what lies outside the view is not touched
    assert torch.equal(big[:, w.batch], big_before[:, w.batch]) and torch.equal(big[:, :w.batch, :2], big_before[:, :w.batch, :2])
    # nothing accepted: nothing moves
    again = cache.clone()
    binding.mcsd_gather_accepted_kv(again, prefix, out.path_nodes, torch.zeros_like(out.accept_len))
    torch.cuda.synchronize()
    assert torch.equal(again, cache)
    # an empty batch enqueues nothing
    lib = binding.load_library()
    assert lib.mcsd_gather_accepted_kv(None, 4, 0, 0, 0, 16, 16, 10, None, None, None, 3, None) == 0
    assert lib.mcsd_gather_accepted_kv(None, 4, 64, 2, 32, 8, 16, 10, None, None, None, 3, None) == -7   # position stride below the row
