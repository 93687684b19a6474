"""mcsd_verify_static: the entry point for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is not an option: a serving loop that has
promised its memory pool a fixed footprint, a plugin whose host application owns every
allocation, a process whose device memory is already handed out.  They cannot supply the
scratch buffer that mcsd_verify expects in its descriptor, so mcsd_verify_static keeps that
scratch in an array compiled into the library.  This file checks, through the C ABI, that

  * the call gives exactly what mcsd_verify gives on the same inputs,
  * a second call right after it, on other inputs, is not disturbed by what the first one
    left in the shared array,
  * a job whose scratch need exceeds the built-in array is turned away with the dedicated
    error code and nothing is enqueued.

The file name sorts last on purpose: with `pytest -x` every other test has run before this one.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2401_06706_b200 import binding, synth

pytestmark = pytest.mark.gpu

STATIC_BYTES = 4 << 20
ERR_STATIC_LIMIT = -11


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    binding.load_library()


def _both_ways(w):
    inp = synth.make_inputs(w, "cuda")
    dt = synth.TORCH_DTYPES[w.dtype]
    draft = inp.draft if w.temperature > 0 else None
    ref = binding.Verifier(w.batch, inp.parent, w.vocab, dt, "cuda")
    a = ref.mcsd_verify(inp.target, draft, inp.cand, inp.unif, w.temperature, w.mode)
    torch.cuda.synchronize()
    # a verifier object is used only for its output buffers and descriptor; its own
    # workspace is ignored by the static entry point
    other = binding.Verifier(w.batch, inp.parent, w.vocab, dt, "cuda")
    other.desc.workspace = None
    other.desc.workspace_bytes = 0
    b = other.mcsd_verify_static(inp.target, draft, inp.cand, inp.unif, w.temperature, w.mode)
    torch.cuda.synchronize()
    return a, b


def _same(a, b, tol):
    assert torch.equal(a.accept_len, b.accept_len)
    assert torch.equal(a.tokens, b.tokens)
    assert torch.equal(a.status, b.status)
    err = float((a.residual - b.residual).abs().max())
    assert err <= tol, err


def test_static_scratch_matches_caller_scratch_on_two_calls_in_a_row():
    # residual tolerances of the parity tests: 1e-5 for fp32 logits, 2e-3 for 2-byte logits
    first = synth.Workload("static_a", 8, 32000, "4x2x2x1", "bf16", "normal", 2.5, 0.8, 1.5, 1.0, 1, 9001)
    second = synth.Workload("static_b", 5, 5000, "2x2", "fp32", "normal", 2.5, 1.0, 1.0, 0.8, 0, 9002)
    _same(*_both_ways(first), 2e-3)
    _same(*_both_ways(second), 1e-5)
    # and the first one again, now that the array holds the second job's leftovers
    _same(*_both_ways(first), 2e-3)


def test_static_scratch_at_temperature_zero():
    w = synth.Workload("static_t0", 6, 4096, "4x2", "fp16", "normal", 3.0, 1.0, 2.0, 0.0, 0, 9003)
    _same(*_both_ways(w), 0.0)


def test_job_beyond_the_built_in_array_is_rejected():
    lib = binding.load_library()
    parent = synth.tree_from_kconfig([4, 4, 2, 2, 1])
    st = synth.tree_stats(parent)
    d = binding.McsdDesc()
    d.batch, d.n_nodes, d.n_internal, d.vocab = 512, st["n_nodes"], st["n_internal"], 32000
    d.dtype, d.ld_target, d.ld_draft = 0, 32000, 32000
    assert lib.mcsd_workspace_bytes(ctypes.byref(d)) > STATIC_BYTES
    # validation comes before any pointer is touched, so dummy non-null pointers are enough
    one = torch.zeros(4, dtype=torch.int32, device="cuda")
    rc = lib.mcsd_verify_static(ctypes.byref(d), one.data_ptr(), one.data_ptr(), parent.ctypes.data,
                                one.data_ptr(), one.data_ptr(), 1.0, 0, one.data_ptr(), one.data_ptr(), None)
    assert rc == ERR_STATIC_LIMIT
    assert "mcsd_verify_static" in binding.status_string(rc)
    torch.cuda.synchronize()
