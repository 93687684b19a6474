"""Shared helpers of the GPU parity tests: run the CUDA library through its C ABI on seeded
inputs and judge the result against the CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from oracle import compare as cmp
from paper_2401_06706_b200 import binding, synth


def run_library(inp: synth.Inputs, *, node_outputs: bool = True, want_residual: bool = True):
    w = inp.workload
    v = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[w.dtype], inp.target.device,
                         want_residual=want_residual, node_outputs=node_outputs)
    out = v.mcsd_verify(inp.target, inp.draft if w.temperature > 0 else None, inp.cand, inp.unif,
                        w.temperature, w.mode)
    torch.cuda.synchronize()
    return v, out


def to_np(t):
    return None if t is None else t.detach().cpu().numpy()


def check_against_oracle(inp: synth.Inputs, out, b0: int = 0, b1=None) -> cmp.ParityReport:
    w = inp.workload
    b1 = w.batch if b1 is None else b1
    t, d, c, u = inp.host_f32(b0, b1)
    sl = slice(b0, b1)
    return cmp.compare(t, d, inp.parent, c, u, w.temperature, w.mode, w.dtype,
                       accept_len=to_np(out.accept_len[sl]), tokens=to_np(out.tokens[sl]),
                       residual=to_np(out.residual[sl]) if out.residual is not None else None,
                       node_accept=to_np(out.node_accept[sl]) if out.node_accept is not None else None,
                       node_bonus=to_np(out.node_bonus[sl]) if out.node_bonus is not None else None,
                       status=to_np(out.status[sl]))


def assert_parity(inp: synth.Inputs, out, b0: int = 0, b1=None) -> cmp.ParityReport:
    rep = check_against_oracle(inp, out, b0, b1)
    assert rep.ok, "\n".join(rep.failures[:10]) + f"\n{rep.summary()}"
    return rep
