"""mcsd_verify_path: the level-by-level form that evaluates only the nodes a walk visits
(the procedure as Section 3 states it).  Its outputs must equal the oracle's sequential
form and the all-node entry point on the same inputs, under the same tolerances."""
import numpy as np
import pytest
import torch

import oracle
from oracle import compare as cmp
from paper_2401_06706_b200 import binding, synth

pytestmark = pytest.mark.gpu
NAMED = synth.named_workloads()


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    binding.load_library()


def _run(w, entry):
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[w.dtype], "cuda")
    out = getattr(v, entry)(inp.target, inp.draft if w.temperature > 0 else None, inp.cand, inp.unif,
                            w.temperature, w.mode)
    torch.cuda.synchronize()
    return inp, v, out


def _check(inp, out):
    w = inp.workload
    t, d, c, u = inp.host_f32()
    # the oracle's sequential form: only visited nodes are evaluated
    ref = oracle.verify(t, d if w.temperature > 0 else None, inp.parent, c, u, w.temperature, w.mode,
                        sequential=True)
    rep = cmp.compare(t, d, inp.parent, c, u, w.temperature, w.mode, w.dtype,
                      accept_len=out.accept_len.cpu().numpy(), tokens=out.tokens.cpu().numpy(),
                      residual=out.residual.cpu().numpy(), status=out.status.cpu().numpy(), oracle_result=ref)
    assert rep.ok, "\n".join(rep.failures[:10]) + f"\n{rep.summary()}"
    return rep


@pytest.mark.parametrize("name", ["cfg1_tiny", "cfg2_b8_with", "cfg2_b8_without", "cfg3_greedy", "cfg4_opt"])
def test_named_configurations(name):
    inp, _, out = _run(NAMED[name], "mcsd_verify_path")
    _check(inp, out)


@pytest.mark.parametrize("dtype,vocab,kconfig,mode,T", [
    ("fp32", 32000, "4x4x2x2x1", 0, 1.0), ("bf16", 32000, "8x1x1x1", 1, 1.0), ("fp16", 50272, "2x2x2x2", 1, 0.7),
    ("fp32", 1000, "3x2", 1, 1.3), ("fp32", 32001, "2x2", 0, 1.0), ("bf16", 7, "2x2", 0, 1.0), ("fp32", 4096, "", 0, 1.0),
    ("fp16", 8200, "1x1x1x1x1x1", 0, 1.0), ("fp32", 65536, "2", 1, 1.0), ("fp16", 3000, "4x2", 0, 0.0),
])
def test_path_form_equals_all_node_form(dtype, vocab, kconfig, mode, T):
    w = synth.Workload("path", 37, vocab, kconfig, dtype, "normal", 2.5, 1.0, 1.0, T, mode, 5150 + vocab)
    inp, _, a = _run(w, "mcsd_verify")
    a_len, a_tok, a_res, a_st = (x.clone() for x in (a.accept_len, a.tokens, a.residual, a.status))
    _, _, b = _run(w, "mcsd_verify_path")
    assert torch.equal(a_len, b.accept_len) and torch.equal(a_tok, b.tokens) and torch.equal(a_st, b.status)
    assert torch.equal(a_res, b.residual)     # same kernels on the same nodes: bit-identical
    _check(inp, b)


def test_low_acceptance_stops_early_and_launch_count():
    w = synth.Workload("path_low", 64, 32000, "2x2x2x1", "fp32", "normal", 2.5, 1.0, 3.0, 1.0, 1, 99)
    inp, v, out = _run(w, "mcsd_verify_path")
    _check(inp, out)
    assert binding.mcsd_last_launch_count() == 2   # one kernel walks every sequence, then the walk kernel
    assert float(out.accept_len.float().mean()) < 1.0
    # temperature 0: one argmax launch per level, then the walk
    w0 = synth.Workload("path_low_t0", 64, 32000, "2x2x2x1", "fp32", "normal", 2.5, 1.0, 3.0, 0.0, 0, 99)
    inp0, _, out0 = _run(w0, "mcsd_verify_path")
    _check(inp0, out0)
    assert binding.mcsd_last_launch_count() == inp0.stats["gamma"] + 1 + 1


def test_empty_batch_and_root_only():
    w = synth.Workload("root_only", 9, 4096, "", "fp32", "normal", 2.0, 1.0, 1.0, 1.0, 0, 5)
    inp, v, out = _run(w, "mcsd_verify_path")
    _check(inp, out)
    v0 = binding.Verifier(0, inp.parent, 4096, torch.float32, "cuda")
    v0.mcsd_verify_path(inp.target[:0], None, inp.cand[:0], inp.unif[:0], 1.0, 0)
    torch.cuda.synchronize()
