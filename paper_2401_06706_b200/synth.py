"""Seeded synthetic inputs for the verification step (shared by tests, bench and smoke).

This module holds input generation only: tree topologies from k-configs, logits
with the stated distributions, candidate tokens drawn by library routines
(``torch.multinomial`` / ``torch.topk``) and pre-drawn uniforms.  None of the
verification arithmetic (acceptance test, residual, walk) lives here, and it
imports neither the CUDA binding nor the CPU oracle, so both sides can be fed
the very same tensors.

The synthetic logits stand in for the paper's LLaMA/Vicuna/OPT outputs on
Alpaca / WMT prompts (Section 4.1), which need model weights and datasets that
are not available offline; only the shapes (vocabulary 32000 and 50272), the
half/float dtypes and the k-config trees (Section 4.3) are taken from there.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

BASE_SEED = 240106706

TORCH_DTYPES = {"fp32": torch.float32, "bf16": torch.bfloat16, "fp16": torch.float16}
DTYPE_CODES = {"fp32": 0, "bf16": 1, "fp16": 2}


def parse_kconfig(text) -> List[int]:
    """'4x2x2x1' -> [4, 2, 2, 1] (the paper's k-config notation, Section 4.3)."""
    if isinstance(text, (list, tuple)):
        ks = [int(k) for k in text]
    else:
        ks = [int(t) for t in str(text).lower().replace("*", "x").split("x") if t != ""]
    if any(k < 1 for k in ks):
        raise ValueError(f"bad k-config {text!r}")
    return ks


def tree_from_kconfig(ks: Sequence[int]) -> np.ndarray:
    """Parent array of the k-ary draft tree in generation (level) order.

    Node 0 is the root (the last committed token); level l holds prod(ks[:l])
    nodes, each node of level l-1 having ks[l-1] consecutive children.  With an
    empty k-config the tree is the root alone.
    """
    parent = [-1]
    level = [0]
    for k in ks:
        nxt = []
        for p in level:
            for _ in range(k):
                nxt.append(len(parent))
                parent.append(p)
        level = nxt
    return np.asarray(parent, dtype=np.int32)


def tree_stats(parent: np.ndarray) -> Dict[str, int]:
    n_nodes = int(parent.shape[0])
    has_child = np.zeros(n_nodes, dtype=bool)
    if n_nodes > 1:
        has_child[parent[1:]] = True
    depth = np.zeros(n_nodes, dtype=np.int64)
    for n in range(1, n_nodes):
        depth[n] = depth[parent[n]] + 1
    return {"n_nodes": n_nodes, "n_draft": n_nodes - 1, "n_internal": int(has_child.sum()),
            "gamma": int(depth.max()) if n_nodes else 0}


def children_ranges(parent: np.ndarray):
    """(first_child, n_children) per node for a level-ordered tree."""
    n_nodes = parent.shape[0]
    first = np.full(n_nodes, -1, dtype=np.int64)
    count = np.zeros(n_nodes, dtype=np.int64)
    for c in range(1, n_nodes):
        p = parent[c]
        if count[p] == 0:
            first[p] = c
        count[p] += 1
    return first, count


def open_uniforms(shape, generator: torch.Generator, device) -> torch.Tensor:
    """Uniforms on the open interval: (i + 0.5) * 2**-23, i in [0, 2**23), exact in float32,
    so neither 0 nor 1 can occur in an acceptance test."""
    i = torch.randint(0, 1 << 23, shape, generator=generator, device=device, dtype=torch.int32)
    return (i.to(torch.float32) + 0.5) * (2.0 ** -23)


@dataclass(frozen=True)
class Workload:
    """One synthetic verification workload."""
    name: str
    batch: int
    vocab: int
    kconfig: str
    dtype: str = "fp32"              # fp32 | bf16 | fp16
    target_dist: str = "normal"      # normal | gumbel
    target_scale: float = 2.5
    draft_gain: float = 1.0          # draft = draft_gain * target + N(0, draft_sigma^2)
    draft_sigma: float = 1.0
    temperature: float = 1.0
    mode: int = 0                    # 0 with replacement (Alg. 1), 1 without (Alg. 2)
    seed: int = BASE_SEED

    @property
    def ks(self) -> List[int]:
        return parse_kconfig(self.kconfig)


# The five named configurations; 5 is one point (the largest) of the sweep.
def named_workloads() -> Dict[str, Workload]:
    w = {}
    w["cfg1_tiny"] = Workload("cfg1_tiny", 1, 32000, "2", "fp32", "normal", 2.0, 1.0, 1.0, 1.0, 0,
                              BASE_SEED + 1)
    w["cfg2_b8_with"] = Workload("cfg2_b8_with", 8, 32000, "4x2x2x1", "bf16", "normal", 2.5, 0.8, 1.5,
                                 1.0, 0, BASE_SEED + 2)
    w["cfg2_b8_without"] = replace(w["cfg2_b8_with"], name="cfg2_b8_without", mode=1)
    w["cfg3_greedy"] = Workload("cfg3_greedy", 32, 32000, "8x2x1", "fp16", "normal", 3.0, 1.0, 2.0,
                                0.0, 0, BASE_SEED + 3)
    w["cfg4_opt"] = Workload("cfg4_opt", 64, 50272, "2x2x2x2", "fp16", "gumbel", 2.0, 1.0, 1.2, 0.7, 1,
                             BASE_SEED + 4)
    w["cfg5_largest"] = Workload("cfg5_largest", 512, 32000, "4x4x2x2x1", "fp32", "normal", 2.5, 1.0,
                                 1.0, 1.0, 0, BASE_SEED + 1000)
    return w


SWEEP_BATCHES = (1, 16, 64, 256, 512)
SWEEP_KCONFIGS = ("1x1x1x1", "2x2x2x1", "4x2x2x1", "4x4x2x2x1", "8x1x1x1")
SWEEP_SIGMAS = (0.5, 1.0, 2.0)
SWEEP_DTYPES = ("fp32", "bf16")


def sweep_workloads() -> List[Workload]:
    """The 300-point throughput sweep (dtype x batch x k-config x sigma x mode)."""
    out = []
    j = 0
    for dt in SWEEP_DTYPES:
        for b in SWEEP_BATCHES:
            for kc in SWEEP_KCONFIGS:
                for sg in SWEEP_SIGMAS:
                    for mode in (0, 1):
                        out.append(Workload(f"sweep_{dt}_b{b}_{kc}_s{sg}_m{mode}", b, 32000, kc, dt,
                                            "normal", 2.5, 1.0, sg, 1.0, mode, BASE_SEED + 1000 + j))
                        j += 1
    return out


@dataclass
class Inputs:
    workload: Workload
    parent: np.ndarray            # [n_nodes] int32, host
    target: torch.Tensor          # [B, n_nodes, V] workload dtype
    draft: Optional[torch.Tensor]  # [B, n_internal, V] workload dtype
    cand: torch.Tensor            # [B, n_nodes] int32 (entry 0 = -1, unused)
    unif: torch.Tensor            # [B, n_nodes, 2] float32
    stats: Dict[str, int] = field(default_factory=dict)

    def logit_bytes(self) -> int:
        """Bytes of logits the step has to read: every target row once, every draft row once
        (no draft rows at temperature 0)."""
        n = self.target.numel() * self.target.element_size()
        if self.workload.temperature > 0 and self.draft is not None:
            n += self.draft.numel() * self.draft.element_size()
        return n

    def host_f32(self, b0: int = 0, b1: Optional[int] = None):
        """float32 numpy copies (exact widening of the rounded logits) of sequences [b0, b1)."""
        b1 = self.target.shape[0] if b1 is None else b1
        t = self.target[b0:b1].to(torch.float32).cpu().numpy()
        d = None if self.draft is None else self.draft[b0:b1].to(torch.float32).cpu().numpy()
        return t, d, self.cand[b0:b1].cpu().numpy(), self.unif[b0:b1].cpu().numpy()


def _noise(shape, dist: str, gen: torch.Generator, device) -> torch.Tensor:
    if dist == "normal":
        return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if dist == "gumbel":
        u = torch.rand(shape, generator=gen, device=device, dtype=torch.float32)
        u = u.clamp_(min=2.0 ** -24, max=1.0 - 2.0 ** -24)
        return -torch.log(-torch.log(u))
    raise ValueError(dist)


def make_inputs(w: Workload, device="cpu", batch_chunk: int = 32) -> Inputs:
    """Generate the tensors of one workload, all from ``w.seed``.

    Target logits are scale * noise; the draft row of a node is the stated
    function of the target row of the same node; both are rounded to the workload
    dtype.  The children of a node carry k tokens drawn from softmax(draft / T)
    of that node with ``torch.multinomial`` (with replacement for mode 0, without
    for mode 1), or the top-k draft logits in descending order at temperature 0.
    """
    device = torch.device(device)
    gen = torch.Generator(device=device)
    gen.manual_seed(int(w.seed))
    parent = tree_from_kconfig(w.ks)
    st = tree_stats(parent)
    n_nodes, n_int = st["n_nodes"], st["n_internal"]
    first, count = children_ranges(parent)
    dt = TORCH_DTYPES[w.dtype]
    B, V = w.batch, w.vocab

    target = torch.empty((B, n_nodes, V), dtype=dt, device=device)
    draft = torch.empty((B, n_int, V), dtype=dt, device=device) if n_int > 0 else None
    cand = torch.full((B, n_nodes), -1, dtype=torch.int32, device=device)
    for b0 in range(0, B, batch_chunk):
        b1 = min(B, b0 + batch_chunk)
        t32 = _noise((b1 - b0, n_nodes, V), w.target_dist, gen, device) * w.target_scale
        target[b0:b1] = t32.to(dt)
        if n_int == 0:
            continue
        d32 = w.draft_gain * t32[:, :n_int] + w.draft_sigma * torch.randn(
            (b1 - b0, n_int, V), generator=gen, device=device, dtype=torch.float32)
        del t32
        draft[b0:b1] = d32.to(dt)
        del d32
        dq = draft[b0:b1].to(torch.float32)
        # nodes with the same number of children are sampled together
        for k in sorted(set(int(c) for c in count[:n_int])):
            nodes = [n for n in range(n_int) if count[n] == k]
            rows = dq[:, nodes].reshape(-1, V)
            if w.temperature > 0:
                probs = torch.softmax(rows / w.temperature, dim=-1)
                toks = torch.multinomial(probs, k, replacement=(w.mode == 0), generator=gen)
            else:
                toks = torch.topk(rows, k, dim=-1).indices
            toks = toks.reshape(b1 - b0, len(nodes), k).to(torch.int32)
            for j, n in enumerate(nodes):
                cand[b0:b1, first[n]:first[n] + k] = toks[:, j]
        del dq
    unif = open_uniforms((B, n_nodes, 2), gen, device)
    return Inputs(w, parent, target, draft, cand, unif, st)
