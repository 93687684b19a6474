"""Seeded random configurations (vocabulary, tree, dtype, temperature, mode, batch, row padding)
through all three verification entry points, each against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from oracle import compare as cmp
from paper_2401_06706_b200 import binding, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    binding.load_library()


def _random_case(seed):
    rng = np.random.default_rng(seed)
    vocab = int(rng.choice([5, 33, 257, 1000, 4099, 8192, 20000, 32000, 32003, 40000, 50272, 65536]))
    depth = int(rng.integers(0, 5))
    ks = [int(rng.choice([1, 2, 3, 4, 8])) for _ in range(depth)]
    while int(np.prod(ks)) > 64 and ks:
        ks[int(np.argmax(ks))] = 1
    mode = int(rng.integers(0, 3))
    if mode == 1 and ks and max(ks) >= vocab:
        mode = 0
    dtype = str(rng.choice(["fp32", "bf16", "fp16"]))
    T = float(rng.choice([0.0, 0.5, 1.0, 1.0, 1.6]))
    batch = int(rng.choice([1, 3, 17, 40]))
    sigma = float(rng.choice([0.3, 1.0, 2.5]))
    dist = str(rng.choice(["normal", "gumbel"]))
    pad = int(rng.choice([0, 0, 8, 24]))
    return dict(vocab=vocab, kconfig="x".join(map(str, ks)), mode=mode, dtype=dtype, T=T, batch=batch,
                sigma=sigma, dist=dist, pad=pad, seed=1000 + seed)


@pytest.mark.parametrize("seed", range(36))
def test_random_configuration(seed):
    c = _random_case(seed)
    w = synth.Workload(f"fuzz{seed}", c["batch"], c["vocab"], c["kconfig"], c["dtype"], c["dist"], 2.5, 1.0, c["sigma"],
                       c["T"], min(c["mode"], 1), c["seed"])
    inp = synth.make_inputs(w, "cuda")
    dt = synth.TORCH_DTYPES[w.dtype]
    target, draft = inp.target, inp.draft
    if c["pad"]:      # rows with a stride larger than the vocabulary, filled with large logits that must be ignored
        ld = w.vocab + c["pad"]
        tp = torch.full((w.batch, inp.stats["n_nodes"], ld), 40.0, dtype=dt, device="cuda")
        tp[:, :, :w.vocab] = target
        target = tp[:, :, :w.vocab]
        if draft is not None:
            dp = torch.full((w.batch, inp.stats["n_internal"], ld), 40.0, dtype=dt, device="cuda")
            dp[:, :, :w.vocab] = draft
            draft = dp[:, :, :w.vocab]
    mode, T = c["mode"], c["T"]
    use_draft = T > 0 and mode != 2
    t, d, cn, u = inp.host_f32()
    ref_all = oracle.verify(t, d if use_draft else None, inp.parent, cn, u, T, mode)
    for entry in ("mcsd_verify", "mcsd_verify_path"):
        v = binding.Verifier(w.batch, inp.parent, w.vocab, dt, "cuda")
        out = getattr(v, entry)(target, draft if use_draft else None, inp.cand, inp.unif, T, mode)
        torch.cuda.synchronize()
        ref = ref_all if entry == "mcsd_verify" and mode != 2 else \
            oracle.verify(t, d if use_draft else None, inp.parent, cn, u, T, mode, sequential=True)
        rep = cmp.compare(t, d if use_draft else None, inp.parent, cn, u, T, mode, w.dtype,
                          accept_len=out.accept_len.cpu().numpy(), tokens=out.tokens.cpu().numpy(),
                          residual=out.residual.cpu().numpy(), status=out.status.cpu().numpy(), oracle_result=ref)
        assert rep.ok, f"{c} {entry}\n" + "\n".join(rep.failures[:8])
