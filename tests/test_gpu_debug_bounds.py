"""The checked build of the library (libmcsd_debug.so, -DMCSD_DEBUG_BOUNDS): every read of caller
memory by the kernels that read logits is checked against the extents the descriptor implies; a
read outside them is skipped and counted, never trapped.  Together with the guard words around every
output (gpu_util.Guards) and the run-twice comparisons it does what a memory checker would, without
a tool around the process.  Across awkward shapes (ragged vocabularies, padded
and unaligned rows, every entry point) the count must stay 0 and the results must be the oracle's."""
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import compare as cmp
from paper_2401_06706_b200 import binding, build, synth
from gpu_util import assert_parity, library_options, run_library, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def checked_library():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    normal = binding.load_library()
    assert binding.mcsd_debug_bounds_hits() == -1          # the normal build has no checks
    build.build(debug_bounds=True)                          # (a no-op when the library is up to date)
    binding._lib = binding.load_library(binding.DEBUG_LIB_PATH)
    assert binding.mcsd_debug_bounds_hits(reset=True) >= 0
    yield
    binding._lib = normal


@pytest.mark.parametrize("entry", ["mcsd_verify", "mcsd_verify_path"])
@pytest.mark.parametrize("dtype,vocab,kconfig,T,mode", [
    ("fp32", 32000, "4x2x2x1", 1.0, 0), ("bf16", 32008, "4x2", 1.0, 1), ("fp16", 50272, "2x2x2", 0.7, 1),
    ("fp32", 1001, "3x2", 1.0, 1), ("bf16", 7, "2x2", 1.0, 0), ("fp16", 65536, "2", 1.0, 0), ("bf16", 4099, "8x1", 1.3, 1),
    ("fp16", 3001, "4x2", 0.0, 0), ("fp32", 2049, "2x1x1", 1.0, 2), ("bf16", 32000, "2x2", 1.0, 2)])
def test_no_read_outside_the_tensors(dtype, vocab, kconfig, T, mode, entry):
    w = synth.Workload("checked", 5, vocab, kconfig, dtype, "normal", 2.5, 0.9, 1.2, T, min(mode, 1), 8800 + vocab)
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[dtype], "cuda", node_outputs=(entry == "mcsd_verify"))
    out = getattr(v, entry)(inp.target, inp.draft if (T > 0 and mode != 2) else None, inp.cand, inp.unif, T, mode)
    torch.cuda.synchronize()
    assert binding.mcsd_debug_bounds_hits(reset=True) == 0
    t, d, c, u = inp.host_f32()
    use_d = d if (T > 0 and mode != 2) else None
    ref = oracle.verify(t, use_d, inp.parent, c, u, T, mode, sequential=(entry == "mcsd_verify_path" or mode == 2))
    rep = cmp.compare(t, use_d, inp.parent, c, u, T, mode, dtype, oracle_result=ref, accept_len=to_np(out.accept_len),
                      tokens=to_np(out.tokens), residual=to_np(out.residual), status=to_np(out.status))
    assert rep.ok, rep.failures[:5]


def test_padded_rows_sampler_and_forced_shapes():
    # rows with a stride larger than the vocabulary (views of a wider tensor)
    w = synth.Workload("checked_pad", 4, 5003, "3x2", "bf16", "normal", 2.5, 1.0, 1.0, 1.0, 1, 8900)
    inp = synth.make_inputs(w, "cuda")
    st = inp.stats
    tp = torch.full((4, st["n_nodes"], 5008), 50.0, dtype=torch.bfloat16, device="cuda")
    dp = torch.full((4, st["n_internal"], 5008), 50.0, dtype=torch.bfloat16, device="cuda")
    tp[:, :, :5003] = inp.target
    dp[:, :, :5003] = inp.draft
    v = binding.Verifier(4, inp.parent, 5003, torch.bfloat16, "cuda", node_outputs=True)
    out = v.mcsd_verify(tp[:, :, :5003], dp[:, :, :5003], inp.cand, inp.unif, 1.0, 1)
    torch.cuda.synchronize()
    assert binding.mcsd_debug_bounds_hits(reset=True) == 0
    assert_parity(inp, out)
    # the sampler, and the other cluster shapes of the node kernel
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1)
    u = synth.open_uniforms((w.batch, st["n_nodes"]), gen, "cuda")
    for T, mode in ((1.0, 0), (1.0, 1), (0.0, 0)):
        binding.mcsd_sample_candidates(inp.draft, inp.parent, u, T, mode)
    for cluster, ept in ((8, 16), (2, 64), (4, 32)):
        with library_options(cluster=cluster, ept=ept):
            _, out = run_library(inp)
        assert_parity(inp, out)
    assert binding.mcsd_debug_bounds_hits(reset=True) == 0


def test_the_checker_reports_reads_beyond_a_registered_extent():
    """Nothing is read out of bounds here: the extents handed to the checker are cut short by 64 bytes,
    so that perfectly valid reads of the last bytes of the last rows are reported and skipped."""
    w = synth.Workload("checked_fire", 3, 4096, "2", "fp32", "normal", 2.5, 1.0, 1.0, 1.0, 0, 8901)
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, torch.float32, "cuda")
    with library_options(test_shrink_ranges=64):
        v.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, 1.0, 0)
        torch.cuda.synchronize()
    assert binding.mcsd_debug_bounds_hits(reset=True) > 0
    v.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, 1.0, 0)
    torch.cuda.synchronize()
    assert binding.mcsd_debug_bounds_hits(reset=True) == 0
