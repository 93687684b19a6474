"""mcsd_verify and mcsd_verify_path neither allocate nor synchronise, so after one ordinary call
(which looks up per-device launch attributes) they can be captured in a CUDA graph; a replay must
give what the direct call gave."""
import pytest
import torch

from paper_2401_06706_b200 import binding, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    binding.load_library()


@pytest.mark.parametrize("form", ["mcsd_verify", "mcsd_verify_path"])
@pytest.mark.parametrize("dtype,T,mode", [("fp32", 1.0, 0), ("bf16", 0.8, 1), ("fp16", 0.0, 0)])
def test_replay_of_a_captured_call_equals_the_direct_call(form, dtype, T, mode):
    w = synth.Workload("graph", 6, 32000, "4x2x2x1", dtype, "normal", 2.5, 1.0, 1.0, T, mode, 77)
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[dtype], "cuda")
    draft = inp.draft if T > 0 else None
    call = getattr(v, form)
    out = call(inp.target, draft, inp.cand, inp.unif, T, mode)
    torch.cuda.synchronize()
    want = [t.clone() for t in (out.accept_len, out.tokens, out.residual, out.status, out.path_nodes)]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):        # warm-up on a side stream, as graph capture asks for
        call(inp.target, draft, inp.cand, inp.unif, T, mode)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call(inp.target, draft, inp.cand, inp.unif, T, mode)
    for _ in range(2):
        for t in (out.accept_len, out.tokens, out.path_nodes):
            t.fill_(-5)
        out.residual.fill_(-5.0)
        graph.replay()
        torch.cuda.synchronize()
        got = (out.accept_len, out.tokens, out.residual, out.status, out.path_nodes)
        assert all(torch.equal(a, b) for a, b in zip(got, want))
