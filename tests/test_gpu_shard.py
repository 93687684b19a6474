"""Verification with the vocabulary split over several devices (the mcsd_shard_* stages), with
the shards emulated one after the other on ONE device and the collectives replaced by copies:
decisions (node_accept, accepted lengths and tokens, path nodes, status words) must equal those
of mcsd_verify on the full tensors bit for bit, the endpoint token and the residual distribution
the oracle's under the usual rules."""
import numpy as np
import pytest
import torch

from paper_2401_06706_b200 import binding, synth
from gpu_util import assert_parity, library_options, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    binding.load_library()


def _sharded(inp, n_shards):
    w = inp.workload
    dt = synth.TORCH_DTYPES[w.dtype]
    shards = [binding.ShardedVerifier(w.batch, inp.parent, w.vocab, dt, n_shards, s, "cuda") for s in range(n_shards)]
    targets = [inp.target[:, :, sh.col_begin:sh.col_begin + sh.n_cols].contiguous() for sh in shards]
    drafts = [inp.draft[:, :, sh.col_begin:sh.col_begin + sh.n_cols].contiguous() if inp.draft is not None else None
              for sh in shards]
    out = binding.sharded_verify(shards, targets, drafts, inp.cand, inp.unif, w.temperature, w.mode, binding.LocalComm())
    torch.cuda.synchronize()
    residual = torch.cat([sh.residual[:, :sh.n_cols] for sh in shards if sh.n_cols], dim=1)
    return shards, out, residual


def _check(inp, n_shards):
    w = inp.workload
    ref = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[w.dtype], "cuda", node_outputs=True)
    a = ref.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, w.temperature, w.mode)
    torch.cuda.synchronize()
    shards, b, residual = _sharded(inp, n_shards)
    n_int = inp.stats["n_internal"]
    assert torch.equal(a.node_accept[:, :n_int], b.node_accept[:, :n_int])      # every decision, bit for bit
    assert torch.equal(a.accept_len, b.accept_len) and torch.equal(a.path_nodes, b.path_nodes)
    assert torch.equal(a.status, b.status)
    L = a.accept_len.long()
    cols = torch.arange(a.tokens.shape[1], device="cuda")[None, :]
    keep = cols != L[:, None]                                                     # all but the endpoint token
    assert torch.equal(a.tokens[keep], b.tokens[keep])
    for sh in shards[1:]:                                                         # every shard reaches the same outputs
        assert torch.equal(sh.tokens, b.tokens) and torch.equal(sh.accept_len, b.accept_len)
        assert torch.equal(sh.status, b.status) and torch.equal(sh.node_accept[:, :n_int], b.node_accept[:, :n_int])
    # endpoint token and residual: against the oracle (the runs of the inverse-CDF search differ
    # from those of the walk kernel, so tokens may differ inside the boundary tolerance)
    out = binding.VerifyOutput(b.accept_len, b.tokens, residual, b.status, path_nodes=b.path_nodes)
    return assert_parity(inp, out)


@pytest.mark.parametrize("n_shards", [1, 2, 3, 4])
@pytest.mark.parametrize("dtype,vocab,kconfig,mode", [("bf16", 32000, "4x2x2x1", 1), ("fp32", 32000, "4x4x2", 0),
                                                       ("fp16", 50272, "2x2x2x2", 1), ("fp32", 1000, "3x2", 0),
                                                       ("bf16", 7, "2x2", 0), ("fp32", 4099, "8x1", 1),
                                                       ("fp16", 65536, "2", 0), ("fp32", 5000, "", 0)])
def test_sharded_equals_single_device(dtype, vocab, kconfig, mode, n_shards):
    w = synth.Workload("shard", 9, vocab, kconfig, dtype, "normal", 2.5, 1.0, 1.2, 0.9, mode, 8100 + vocab)
    inp = synth.make_inputs(w, "cuda")
    if vocab % 8:       # (rows of odd length: the single-device call takes its plain-load path; same arithmetic)
        pass
    _check(inp, n_shards)


@pytest.mark.parametrize("n_shards", [2, 4])
@pytest.mark.parametrize("mode", [0, 1])
def test_sharded_on_the_edge_cases(mode, n_shards):
    from test_gpu_edge import _edge_inputs
    inp = _edge_inputs("fp32", mode)
    rep = _check(inp, n_shards)
    assert rep.n_tests > 0


def test_sharded_with_forced_run_length():
    """Shorter runs (16 elements per thread): more entries, other shard boundaries."""
    w = synth.Workload("shard_ept", 6, 9000, "4x2x1", "bf16", "normal", 2.5, 1.0, 1.0, 1.0, 1, 8200)
    inp = synth.make_inputs(w, "cuda")
    with library_options(cluster=8, ept=16):
        _check(inp, 3)


def test_larger_batch_and_tree_two_shards():
    w = synth.Workload("shard_big", 64, 32000, "4x4x2x2x1", "bf16", "normal", 2.5, 1.0, 1.0, 1.0, 0, 8300)
    inp = synth.make_inputs(w, "cuda")
    rep = _check(inp, 2)
    assert rep.n_tests > 4000


def test_temperature_zero_is_refused():
    w = synth.Workload("shard_t0", 2, 1000, "2", "fp32", "normal", 2.5, 1.0, 1.0, 1.0, 0, 8400)
    inp = synth.make_inputs(w, "cuda")
    sh = binding.ShardedVerifier(w.batch, inp.parent, w.vocab, torch.float32, 1, 0, "cuda")
    with pytest.raises(binding.McsdError) as e:
        sh.mcsd_shard_partials(inp.target, inp.draft, inp.cand, 0.0, 0)
    assert e.value.code == -10
