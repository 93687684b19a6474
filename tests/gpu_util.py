"""Shared helpers of the GPU parity tests: run the CUDA library through its C ABI on seeded
inputs and judge the result against the CPU oracle.  Every output buffer and the workspace of
a run are placed between guard words that are checked afterwards (compute-sanitizer is not
available, so writes outside a buffer have to be caught by the tests themselves)."""
from __future__ import annotations

import contextlib

import numpy as np
import torch

import oracle
from oracle import compare as cmp
from paper_2401_06706_b200 import binding, synth

GUARD_BYTES = 256
GUARD_BYTE = 0xA5


class Guards:
    """Re-homes the output tensors and the workspace of a Verifier into buffers with GUARD_BYTES
    of a fixed pattern on both sides; check() fails if any guard byte changed."""

    def __init__(self, v: binding.Verifier):
        self.v, self.buffers = v, []
        for name, field in (("accept_len", None), ("tokens", None), ("residual", None), ("status", "out_status"),
                            ("path_nodes", "out_path_nodes"), ("node_accept", "node_accept"),
                            ("node_bonus", "node_bonus"), ("node_ratio", "node_ratio"),
                            ("node_residual", "node_residual")):
            t = getattr(v, name)
            if t is None:
                continue
            view = self._guarded(t.numel() * t.element_size(), 16).view(t.dtype).view(t.shape)
            view.copy_(t)
            setattr(v, name, view)
            if field is not None:
                setattr(v.desc, field, view.data_ptr())
        ws = self._guarded(int(v.desc.workspace_bytes), 256)
        v.workspace = ws
        v.desc.workspace = ws.data_ptr()

    def _guarded(self, nbytes: int, align: int) -> torch.Tensor:
        pad = (-nbytes) % 16
        raw = torch.full((GUARD_BYTES + nbytes + pad + GUARD_BYTES + align,), GUARD_BYTE, dtype=torch.uint8,
                         device=self.v.device)
        off = (-(raw.data_ptr() + GUARD_BYTES)) % align + GUARD_BYTES
        self.buffers.append((raw, off, nbytes))
        return raw[off:off + nbytes]

    def check(self):
        torch.cuda.synchronize()
        for raw, off, nbytes in self.buffers:
            assert bool((raw[:off] == GUARD_BYTE).all()), "bytes in front of a buffer were overwritten"
            assert bool((raw[off + nbytes:] == GUARD_BYTE).all()), "bytes behind a buffer were overwritten"


@contextlib.contextmanager
def library_options(**opts):
    """Sets MCSD_OPT_* overrides (cluster=, ept=, direct=, sample_ahead=, wait_polls=, test_extra_tx=, pdl=)
    (and split=) for the duration of a block and restores what was there before."""
    ids = {"cluster": binding.OPT_CLUSTER, "ept": binding.OPT_EPT, "direct": binding.OPT_DIRECT,
           "sample_ahead": binding.OPT_SAMPLE_AHEAD, "wait_polls": binding.OPT_WAIT_POLLS,
           "test_extra_tx": binding.OPT_TEST_EXTRA_TX, "pdl": binding.OPT_PDL,
           "test_shrink_ranges": binding.OPT_TEST_SHRINK_RANGES, "split": binding.OPT_SPLIT, "trace": binding.OPT_TRACE, "walk_cluster": binding.OPT_WALK_CLUSTER}
    before = {k: binding.mcsd_get_option(ids[k]) for k in opts}
    try:
        for k, val in opts.items():
            binding.mcsd_set_option(ids[k], val)
        yield
    finally:
        for k, val in before.items():
            binding.mcsd_set_option(ids[k], val)


def run_library(inp: synth.Inputs, *, node_outputs: bool = True, want_residual: bool = True, entry: str = "mcsd_verify"):
    w = inp.workload
    v = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[w.dtype], inp.target.device,
                         want_residual=want_residual, node_outputs=node_outputs)
    guards = Guards(v)
    needs_draft = w.temperature > 0 and w.mode != 2
    out = getattr(v, entry)(inp.target, inp.draft if needs_draft else None, inp.cand, inp.unif,
                            w.temperature, w.mode)
    guards.check()
    return v, out


def to_np(t):
    return None if t is None else t.detach().cpu().numpy()


def check_against_oracle(inp: synth.Inputs, out, b0: int = 0, b1=None, *, sequential: bool = False,
                         with_path_nodes: bool = True) -> cmp.ParityReport:
    """sequential: the outputs under test come from the path form, whose per-node outputs cover the
    visited nodes only; the oracle then runs its sequential form and node outputs are not compared."""
    w = inp.workload
    b1 = w.batch if b1 is None else b1
    t, d, c, u = inp.host_f32(b0, b1)
    sl = slice(b0, b1)
    ref = None
    if sequential:
        ref = oracle.verify(t, d if (w.temperature > 0 and w.mode != 2) else None, inp.parent, c, u, w.temperature,
                            w.mode, sequential=True)
    per_node = not sequential
    return cmp.compare(t, d, inp.parent, c, u, w.temperature, w.mode, w.dtype, oracle_result=ref,
                       accept_len=to_np(out.accept_len[sl]), tokens=to_np(out.tokens[sl]),
                       residual=to_np(out.residual[sl]) if out.residual is not None else None,
                       node_accept=to_np(out.node_accept[sl]) if (per_node and out.node_accept is not None) else None,
                       node_bonus=to_np(out.node_bonus[sl]) if (per_node and out.node_bonus is not None) else None,
                       path_nodes=to_np(out.path_nodes[sl]) if (with_path_nodes and out.path_nodes is not None) else None,
                       status=to_np(out.status[sl]))


def assert_parity(inp: synth.Inputs, out, b0: int = 0, b1=None, **kw) -> cmp.ParityReport:
    rep = check_against_oracle(inp, out, b0, b1, **kw)
    assert rep.ok, "\n".join(rep.failures[:10]) + f"\n{rep.summary()}"
    return rep
