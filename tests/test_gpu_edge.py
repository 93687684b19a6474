"""The edges of the method through the C ABI, outputs and status words equal to the oracle's:
zero residual mass (Algorithm 1 / 2, the line p := norm(max(0, p - q)) when the sum is 0: p is
kept), rows from which no distribution can be formed (all -inf, NaN, +inf), uniforms outside
(0, 1).  All of these are ordinary inputs built on the host; nothing here waits or traps."""
import numpy as np
import pytest
import torch

import oracle
from oracle import compare as cmp
from paper_2401_06706_b200 import binding, synth
from gpu_util import Guards, assert_parity, to_np

pytestmark = pytest.mark.gpu
DEG, BAD, NOM = binding.STATUS_DEGENERATE, binding.STATUS_BAD_TOKEN, binding.STATUS_NO_MASS


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    binding.load_library()


def _edge_inputs(dtype, mode, vocab=4000):
    """Tree 2x1 (root, two children with one child each, two leaves).  One sequence per case."""
    w = synth.Workload("edge", 12, vocab, "2x1", dtype, "normal", 2.5, 1.0, 1.0, 1.0, mode, 4711)
    inp = synth.make_inputs(w, "cuda")
    t, d, c, u = inp.target, inp.draft, inp.cand, inp.unif
    V = vocab
    # 0: p == q at the root, first child carries no token: forced rejection, zero residual mass,
    #    p kept; the second child then has ratio exactly 1 and is accepted
    d[0, 0] = t[0, 0]; c[0, 1] = V
    # 1: p == q at the root and neither child carries a token: everything rejected, endpoint from the kept p
    d[1, 0] = t[1, 0]; c[1, 1] = V + 7; c[1, 2] = -3
    # 2: the root accepts its first child (p == q); at that node (one child) p == q again and the child
    #    carries no token: the only rejection of the node leaves zero mass
    d[2, 0] = t[2, 0]; d[2, 1] = t[2, 1]; c[2, 3] = V
    # 3: target row of the root all -inf
    t[3, 0] = float("-inf")
    # 4: a NaN in the target row of the root
    t[4, 0, 17] = float("nan")
    # 5: a +inf in the draft row of the root: no q, every candidate rejected, endpoint from p
    d[5, 0, 5] = float("inf")
    # 6: the walk reaches a leaf whose target row has no mass
    d[6, 0] = t[6, 0]; d[6, 1] = t[6, 1]; t[6, 3] = float("-inf")
    # 7: p == q, and the first child's token has probability 0 under both
    d[7, 0] = t[7, 0]; tok = int(c[7, 1]); t[7, 0, tok] = float("-inf"); d[7, 0, tok] = float("-inf")
    # 8: acceptance uniforms outside (0, 1)
    u[8, 1, 0] = 1.5; u[8, 2, 0] = float("nan"); u[8, 3, 0] = -0.25; u[8, 4, 0] = 1.0
    # 9: endpoint uniforms outside (0, 1) at every node
    u[9, :, 1] = torch.tensor([1.0, 2.0, -1.0, float("nan"), 0.0], device=u.device)
    # 10: draft row all -inf at a node below the root, target row of its sibling NaN
    d[10, 1] = float("-inf"); t[10, 2, 3] = float("nan")
    # 11: untouched
    return inp


@pytest.mark.parametrize("entry,node_outputs", [("mcsd_verify", True), ("mcsd_verify", False), ("mcsd_verify_path", False)])
@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("dtype", ["fp32", "bf16", "fp16"])
def test_zero_mass_no_mass_and_odd_uniforms(dtype, mode, entry, node_outputs):
    inp = _edge_inputs(dtype, mode)
    w = inp.workload
    v = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[dtype], "cuda", node_outputs=node_outputs)
    guards = Guards(v)
    out = getattr(v, entry)(inp.target, inp.draft, inp.cand, inp.unif, 1.0, mode)
    guards.check()
    assert_parity(inp, out, sequential=(entry == "mcsd_verify_path"))
    st, ln, tok = to_np(out.status), to_np(out.accept_len), to_np(out.tokens)
    # the statuses the hand cases must give (the oracle agrees: assert_parity compared them)
    assert st[0] == (DEG | BAD) and ln[0] >= 1
    assert st[1] == (DEG | BAD) and ln[1] == 0 and tok[1, 0] >= 0
    assert st[2] == (DEG | BAD) and ln[2] == 1 and tok[2, 1] >= 0
    assert st[3] == (DEG | NOM) and ln[3] == 0 and tok[3, 0] == -1
    assert st[4] == (DEG | NOM) and ln[4] == 0 and tok[4, 0] == -1
    assert st[5] == DEG and ln[5] == 0 and tok[5, 0] >= 0
    assert st[6] == NOM and ln[6] == 2 and tok[6, 2] == -1
    assert st[7] == DEG and ln[7] >= 1
    assert st[8] == 0 and st[9] == 0 and st[11] == 0
    assert not (st & binding.STATUS_TIMEOUT).any()
    # calling again gives the same words (they are written, not accumulated)
    out = getattr(v, entry)(inp.target, inp.draft, inp.cand, inp.unif, 1.0, mode)
    torch.cuda.synchronize()
    assert np.array_equal(st, to_np(out.status))


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_naive_mode_on_rows_without_mass(dtype):
    w = synth.Workload("edge_naive", 5, 3000, "2x1", dtype, "normal", 2.5, 1.0, 1.0, 1.0, 0, 4712)
    inp = synth.make_inputs(w, "cuda")
    inp.target[0, 0] = float("-inf")
    inp.target[1, 0, 9] = float("nan")
    inp.target[2, 0, 9] = float("inf")
    inp.unif[3, :, 1] = torch.tensor([1.0, 2.0, -1.0, float("nan"), 0.0], device="cuda")
    for entry in ("mcsd_verify", "mcsd_verify_path"):
        v = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[dtype], "cuda")
        out = getattr(v, entry)(inp.target, None, inp.cand, inp.unif, 1.0, 2)
        torch.cuda.synchronize()
        t, _, c, u = inp.host_f32()
        ref = oracle.verify(t, None, inp.parent, c, u, 1.0, 2, sequential=True)
        rep = cmp.compare(t, None, inp.parent, c, u, 1.0, 2, dtype, oracle_result=ref, accept_len=to_np(out.accept_len),
                          tokens=to_np(out.tokens), residual=to_np(out.residual), status=to_np(out.status))
        assert rep.ok, rep.failures[:5]
        st = to_np(out.status)
        assert (st[:3] == NOM).all() and (st[3:] == 0).all()
        assert (to_np(out.tokens)[:3, 0] == -1).all() and (to_np(out.accept_len)[:3] == 0).all()


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("dtype", ["fp32", "fp16"])
def test_sampler_on_rows_without_mass(dtype, mode):
    w = synth.Workload("edge_sample", 5, 3000, "4x1", dtype, "normal", 2.5, 1.0, 1.0, 1.0, mode, 4713)
    inp = synth.make_inputs(w, "cuda")
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    u = synth.open_uniforms((w.batch, inp.stats["n_nodes"]), gen, "cuda")
    d = inp.draft
    d[0, 0] = float("-inf")                 # nothing to draw from
    d[1, 0, 100] = float("nan")
    d[2, 0] = float("-inf"); d[2, 0, 40] = 1.0; d[2, 0, 2000] = 0.5      # two tokens for four draws
    u[3, 1:5] = torch.tensor([1.0, 1.5, -0.5, float("nan")], device="cuda")
    status = torch.zeros(w.batch, dtype=torch.int32, device="cuda")
    cand = binding.mcsd_sample_candidates(d, inp.parent, u, 1.0, mode, status=status)
    torch.cuda.synchronize()
    rep = cmp.compare_samples(d.to(torch.float32).cpu().numpy(), inp.parent, u.cpu().numpy(), 1.0, mode, cand.cpu().numpy())
    assert rep.ok, rep.failures[:5]
    c, st = cand.cpu().numpy(), status.cpu().numpy()
    assert (c[0, 1:5] == -1).all() and (c[1, 1:5] == -1).all() and st[0] == NOM and st[1] == NOM
    if mode == 1:
        assert sorted(c[2, 1:3].tolist()) == [40, 2000] and (c[2, 3:5] == -1).all() and st[2] == NOM
    else:
        assert set(c[2, 1:5].tolist()) <= {40, 2000} and st[2] == 0
    assert st[3] == 0 and st[4] == 0
