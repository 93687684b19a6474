"""MCSD_MODE_NAIVE (multi-candidate naive sampling, the ablation baseline of Section 4.5) against
the oracle's mode 2 on the same seeded inputs: accepted lengths and tokens identical except where
the draw's uniform lies within 1e-5 (CDF units) of an interval boundary, residual within the
parity tolerance."""
import numpy as np
import pytest
import torch

import oracle
from oracle import compare as cmp
from paper_2401_06706_b200 import binding, synth

pytestmark = pytest.mark.gpu
MODE_NAIVE = 2


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    binding.load_library()


def _run(w, entry="mcsd_verify"):
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[w.dtype], "cuda")
    out = getattr(v, entry)(inp.target, None, inp.cand, inp.unif, w.temperature, MODE_NAIVE)
    torch.cuda.synchronize()
    return inp, out


def _check(inp, out):
    w = inp.workload
    t, _, c, u = inp.host_f32()
    ref = oracle.verify(t, None, inp.parent, c, u, w.temperature, MODE_NAIVE, sequential=True)
    rep = cmp.compare(t, None, inp.parent, c, u, w.temperature, MODE_NAIVE, w.dtype,
                      accept_len=out.accept_len.cpu().numpy(), tokens=out.tokens.cpu().numpy(),
                      residual=out.residual.cpu().numpy(), status=out.status.cpu().numpy(), oracle_result=ref)
    assert rep.ok, "\n".join(rep.failures[:10]) + f"\n{rep.summary()}"
    return rep


@pytest.mark.parametrize("dtype", ["fp32", "bf16", "fp16"])
@pytest.mark.parametrize("vocab,kconfig,sigma", [(7, "3x2", 1.0), (1000, "4x2", 0.5), (32000, "4x2x2x1", 0.5),
                                                  (32001, "2x2", 1.0), (50272, "2x2x2x2", 1.0), (65536, "8", 2.0),
                                                  (4096, "", 1.0)])
def test_naive_mode_matches_the_oracle(vocab, kconfig, sigma, dtype):
    w = synth.Workload("naive", 24, vocab, kconfig, dtype, "normal", 2.5, 1.0, sigma, 1.0, 0, 300 + vocab)
    inp, out = _run(w)
    _check(inp, out)


def test_path_entry_point_gives_the_same_and_temperature_zero_is_the_argmax_rule():
    w = synth.Workload("naive_path", 16, 6000, "4x2x1", "fp16", "gumbel", 2.0, 1.0, 1.0, 0.8, 0, 17)
    inp, a = _run(w)
    a_len, a_tok = a.accept_len.clone(), a.tokens.clone()
    _, b = _run(w, "mcsd_verify_path")
    assert torch.equal(a_len, b.accept_len) and torch.equal(a_tok, b.tokens)
    w0 = synth.Workload("naive_t0", 16, 6000, "4x2x1", "fp16", "normal", 3.0, 1.0, 2.0, 0.0, 0, 18)
    inp0 = synth.make_inputs(w0, "cuda")
    v = binding.Verifier(w0.batch, inp0.parent, w0.vocab, torch.float16, "cuda")
    x = v.mcsd_verify(inp0.target, None, inp0.cand, inp0.unif, 0.0, MODE_NAIVE)
    xl, xt = x.accept_len.clone(), x.tokens.clone()
    y = v.mcsd_verify(inp0.target, None, inp0.cand, inp0.unif, 0.0, 1)
    torch.cuda.synchronize()
    assert torch.equal(xl, y.accept_len) and torch.equal(xt, y.tokens)


def test_naive_accepts_less_often_than_algorithm_one():
    """Appendix C in action on synthetic inputs: the mean accepted length of naive sampling
    does not exceed that of multi-candidate speculative sampling on the same trees."""
    w = synth.Workload("naive_vs", 256, 32000, "4x2x2x1", "fp32", "normal", 2.5, 1.0, 1.0, 1.0, 0, 5)
    inp, out = _run(w)
    naive = float(out.accept_len.float().mean())
    v = binding.Verifier(w.batch, inp.parent, w.vocab, torch.float32, "cuda")
    mcss = float(v.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, 1.0, 0).accept_len.float().mean())
    assert naive < mcss


def test_staged_entry_points_refuse_the_naive_mode():
    w = synth.Workload("naive_staged", 2, 1000, "2", "fp32", "normal", 2.5, 1.0, 1.0, 1.0, 0, 5)
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, torch.float32, "cuda")
    with pytest.raises(binding.McsdError) as e:
        v.mcsd_verify_nodes(inp.target, inp.draft, inp.cand, inp.unif, 1.0, MODE_NAIVE)
    assert e.value.code == -4
