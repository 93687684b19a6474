"""The bounded wait of the node kernel's exchange really gives up, and the kernel still returns.

Nothing here hangs or faults a GPU: the exchange barrier of a single-CTA cluster is armed for
16 bytes more than are sent (MCSD_OPT_TEST_EXTRA_TX), so the wait of the CTA's leader warp is a
wait for a flag nothing sets; with a budget of a few polls (MCSD_OPT_WAIT_POLLS) it runs out
within microseconds.  The kernel then stops waiting, arming and sending, finishes its items
without results, meets the final cluster barrier and exits; the status words say TIMEOUT.  A
normal call right after it works again."""
import numpy as np
import pytest
import torch

from paper_2401_06706_b200 import binding, synth
from gpu_util import Guards, assert_parity, library_options, to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("entry", ["mcsd_verify", "mcsd_verify_path"])
def test_expired_exchange_wait_sets_timeout_and_returns(entry):
    assert torch.cuda.is_available(), "this test needs a CUDA device"
    w = synth.Workload("timeout", 3, 2000, "2", "fp32", "normal", 2.5, 1.0, 1.0, 1.0, 0, 606)
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, torch.float32, "cuda")
    guards = Guards(v)
    with library_options(cluster=1, wait_polls=4, test_extra_tx=16, pdl=0):
        out = getattr(v, entry)(inp.target, inp.draft, inp.cand, inp.unif, 1.0, 0)
        guards.check()                       # synchronises: the kernel has returned
    st = to_np(out.status)
    assert (st & binding.STATUS_TIMEOUT).all(), st
    # the library and the context are as usable as before
    out = getattr(v, entry)(inp.target, inp.draft, inp.cand, inp.unif, 1.0, 0)
    guards.check()
    assert not (to_np(out.status) & binding.STATUS_TIMEOUT).any()
    assert_parity(inp, out, sequential=(entry == "mcsd_verify_path"))
