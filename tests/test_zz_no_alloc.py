"""mcsd_verify_static: the entry point for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is not an option: a serving loop that has
promised its memory pool a fixed footprint, a plugin whose host application owns every
allocation, a process whose device memory is already handed out.  They cannot supply the
scratch buffer that mcsd_verify expects in its descriptor, so mcsd_verify_static keeps that
scratch in an array compiled into the library.  This file checks, through the C ABI, that

  * the call gives bit for bit what mcsd_verify gives on the same inputs (both run the same
    kernels) and agrees with the CPU oracle,
  * a second call right after it, on other inputs, is not disturbed by what the first one
    left in the shared array,
  * the call really allocates nothing: the device's free memory is the same before and after,
  * it also works when the caller passes no status buffer (the status words then live in the
    built-in array),
  * a job whose scratch need exceeds the built-in array is turned away with the dedicated
    error code and nothing is enqueued.

The file name sorts last on purpose: with `pytest -x` every other test has run before this one.
"""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

from paper_2401_06706_b200 import binding, synth
from gpu_util import assert_parity

pytestmark = pytest.mark.gpu


def _header_constant(name):
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    text = open(os.path.join(root, "include", "mcsd.h")).read()
    m = re.search(r"#define\s+" + name + r"\s+\(?\(?(-?\d+)u?\s*(?:<<\s*(\d+))?\)?", text)
    return int(m.group(1)) << int(m.group(2) or 0)


STATIC_BYTES = _header_constant("MCSD_STATIC_WORKSPACE_BYTES")
ERR_STATIC_LIMIT = _header_constant("MCSD_ERR_STATIC_LIMIT")


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
    other.mcsd_verify_static(inp.target, draft, inp.cand, inp.unif, w.temperature, w.mode)   # first call on the device: address lookup
    torch.cuda.synchronize()
    # (free memory is a property of the whole device: a call that allocates shows it every time, another
    # process that happens to allocate in between does not, so a difference is checked again)
    unchanged = False
    for _ in range(3):
        free_before = torch.cuda.mem_get_info()[0]
        b = other.mcsd_verify_static(inp.target, draft, inp.cand, inp.unif, w.temperature, w.mode)
        torch.cuda.synchronize()
        if torch.cuda.mem_get_info()[0] == free_before:
            unchanged = True
            break
    assert unchanged, "mcsd_verify_static changed the device's free memory"
    return inp, a, b


def _same(inp, a, b):
    # the two entry points run the same kernels on the same inputs: every output bit agrees
    assert torch.equal(a.accept_len, b.accept_len)
    assert torch.equal(a.tokens, b.tokens)
    assert torch.equal(a.status, b.status)
    assert torch.equal(a.path_nodes, b.path_nodes)
    assert torch.equal(a.residual.view(torch.int32), b.residual.view(torch.int32))
    # ... and the new entry point agrees with the oracle directly, under the parity tolerances
    assert_parity(inp, b)


def test_static_scratch_matches_caller_scratch_on_two_calls_in_a_row():
    first = synth.Workload("static_a", 8, 32000, "4x2x2x1", "bf16", "normal", 2.5, 0.8, 1.5, 1.0, 1, 9001)
    second = synth.Workload("static_b", 5, 5000, "2x2", "fp32", "normal", 2.5, 1.0, 1.0, 0.8, 0, 9002)
    _same(*_both_ways(first))
    _same(*_both_ways(second))
    # and the first one again, now that the array holds the second job's leftovers
    _same(*_both_ways(first))


def test_static_scratch_at_temperature_zero():
    w = synth.Workload("static_t0", 6, 4096, "4x2", "fp16", "normal", 3.0, 1.0, 2.0, 0.0, 0, 9003)
    _same(*_both_ways(w))


def test_status_words_inside_the_built_in_array():
    """A caller that passes no status buffer: the status words live in the built-in array; the
    other outputs are what the call with a status buffer gives."""
    w = synth.Workload("static_nostatus", 7, 6000, "3x2", "fp32", "normal", 2.5, 1.0, 1.0, 1.0, 1, 9004)
    inp = synth.make_inputs(w, "cuda")
    a = binding.Verifier(w.batch, inp.parent, w.vocab, torch.float32, "cuda")
    ra = a.mcsd_verify_static(inp.target, inp.draft, inp.cand, inp.unif, 1.0, 1)
    torch.cuda.synchronize()
    b = binding.Verifier(w.batch, inp.parent, w.vocab, torch.float32, "cuda")
    b.desc.out_status = None
    b.desc.workspace = None
    b.desc.workspace_bytes = 0
    rb = b.mcsd_verify_static(inp.target, inp.draft, inp.cand, inp.unif, 1.0, 1)
    torch.cuda.synchronize()
    assert torch.equal(ra.accept_len, rb.accept_len) and torch.equal(ra.tokens, rb.tokens)
    assert torch.equal(ra.residual, rb.residual)


def test_job_beyond_the_built_in_array_is_rejected():
    """A tiny vocabulary with many nodes: the scratch need is beyond the array while every
    input and output buffer exists at full size, so even a call that was wrongly let through
    would stay inside its buffers."""
    lib = binding.load_library()
    w = synth.Workload("static_big", 2048, 8, "4x4x2x2x1", "fp32", "normal", 2.5, 1.0, 1.0, 1.0, 0, 9005)
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, torch.float32, "cuda")
    assert lib.mcsd_workspace_bytes(ctypes.byref(v.desc)) > STATIC_BYTES
    v.tokens.fill_(-77)
    with pytest.raises(binding.McsdError) as e:
        v.mcsd_verify_static(inp.target, inp.draft, inp.cand, inp.unif, 1.0, 0)
    assert e.value.code == ERR_STATIC_LIMIT
    assert "mcsd_verify_static" in binding.status_string(e.value.code)
    torch.cuda.synchronize()
    assert bool((v.tokens == -77).all())          # nothing was enqueued
    # the same job is fine with caller-owned scratch
    out = v.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, 1.0, 0)
    torch.cuda.synchronize()
    assert bool((out.tokens[:, 0] >= 0).all())
