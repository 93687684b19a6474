"""Parity of the CUDA library (called through its C ABI) with the CPU oracle on the same
seeded inputs.  Tolerances: accept decisions and tokens bit-exact except near-ties
|u - rho| < 1e-5 (counted, <= 0.01 % of decisions); residual max abs error <= 1e-5 for fp32
logits and <= 2e-3 for bf16/fp16 logits."""
import os

import numpy as np
import pytest
import torch

from paper_2401_06706_b200 import binding, synth
from gpu_util import assert_parity, library_options, run_library, to_np

pytestmark = pytest.mark.gpu

NAMED = synth.named_workloads()


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    binding.load_library()


@pytest.mark.parametrize("name", ["cfg1_tiny", "cfg2_b8_with", "cfg2_b8_without", "cfg3_greedy", "cfg4_opt"])
def test_named_configurations_full_parity(name):
    inp = synth.make_inputs(NAMED[name], "cuda")
    _, out = run_library(inp)
    rep = assert_parity(inp, out)
    assert rep.n_tests > 0 and rep.n_excluded_sequences == 0
    print(name, rep.summary())


@pytest.mark.parametrize("dtype", ["fp32", "bf16", "fp16"])
@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("vocab,kconfig", [
    (7, "2x2"), (8, "3"), (96, "1x1x1"), (1000, "4x2"), (2048, "2x2x2"), (2049, "2"),
    (8200, "8x1"), (32000, "2x2"), (32008, "4"), (50272, "2x2"), (65536, "2"),
])
def test_shapes_spanning_tiles_and_ragged_tails(vocab, kconfig, mode, dtype):
    if mode == 1 and vocab < 16 and max(synth.parse_kconfig(kconfig)) > 3:
        pytest.skip("not enough distinct tokens")
    w = synth.Workload(f"edge_{vocab}_{kconfig}", 5, vocab, kconfig, dtype, "normal", 2.5, 0.9, 1.2, 1.0,
                       mode, 1234 + vocab)
    inp = synth.make_inputs(w, "cuda")
    _, out = run_library(inp)
    assert_parity(inp, out)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("vocab", [1001, 32001, 50257])
def test_unaligned_rows_take_the_plain_load_path(vocab, dtype):
    """A contiguous tensor whose row length is not a multiple of 16 bytes."""
    w = synth.Workload("unaligned", 3, vocab, "3x2", dtype, "normal", 2.5, 1.0, 1.0, 0.9, 1, 77 + vocab)
    inp = synth.make_inputs(w, "cuda")
    assert (vocab * inp.target.element_size()) % 16 != 0
    _, out = run_library(inp)
    assert_parity(inp, out)


def test_padded_row_stride():
    w = synth.Workload("strided", 4, 5000, "2x2", "fp16", "normal", 2.5, 1.0, 1.0, 1.0, 0, 4242)
    inp = synth.make_inputs(w, "cuda")
    ld = 5120
    st = inp.stats
    tpad = torch.full((4, st["n_nodes"], ld), 30.0, dtype=torch.float16, device="cuda")
    dpad = torch.full((4, st["n_internal"], ld), 30.0, dtype=torch.float16, device="cuda")
    tpad[:, :, :5000] = inp.target
    dpad[:, :, :5000] = inp.draft
    v = binding.Verifier(4, inp.parent, 5000, torch.float16, "cuda", node_outputs=True)
    out = v.mcsd_verify(tpad[:, :, :5000], dpad[:, :, :5000], inp.cand, inp.unif, 1.0, 0)
    torch.cuda.synchronize()
    assert v.desc.ld_target == ld
    assert_parity(inp, out)


@pytest.mark.parametrize("T", [1.0, 0.0])
@pytest.mark.parametrize("dtype,vocab", [("fp32", 5003), ("bf16", 5003), ("fp16", 8197), ("fp32", 32002), ("bf16", 32001),
                                         ("fp32", 3), ("bf16", 5)])
def test_aligned_rows_whose_vocabulary_ends_inside_a_vector(dtype, vocab, T):
    """Rows padded to a 16-byte multiple take the vector path; the vector that holds the last
    elements also holds padding, here larger than every logit, which must not count."""
    w = synth.Workload("tail", 4, vocab, "3x2" if vocab > 16 else "2x2", dtype, "normal", 2.5, 1.0, 1.0, T, 1 if T > 0 else 0, 99 + vocab)
    inp = synth.make_inputs(w, "cuda")
    dt = synth.TORCH_DTYPES[dtype]
    per16 = 16 // inp.target.element_size()
    ld = (vocab + per16 - 1) // per16 * per16
    assert ld > vocab
    st = inp.stats
    tpad = torch.full((4, st["n_nodes"], ld), 50.0, dtype=dt, device="cuda")
    dpad = torch.full((4, st["n_internal"], ld), 50.0, dtype=dt, device="cuda")
    tpad[:, :, :vocab] = inp.target
    dpad[:, :, :vocab] = inp.draft
    v = binding.Verifier(4, inp.parent, vocab, dt, "cuda", node_outputs=True)
    out = v.mcsd_verify(tpad[:, :, :vocab], dpad[:, :, :vocab] if T > 0 else None, inp.cand, inp.unif, T, w.mode)
    torch.cuda.synchronize()
    assert v.desc.ld_target == ld and (ld * inp.target.element_size()) % 16 == 0
    assert_parity(inp, out)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("cluster,ept", [(1, 64), (2, 16), (4, 16), (8, 16), (8, 32), (2, 64), (4, 32), (3, 16), (7, 32)])
def test_forced_cluster_shapes(cluster, ept, dtype):
    """Every cluster size / per-thread share computes the same thing (128 threads per CTA; with the
    larger shapes some CTAs of the cluster own nothing but -inf)."""
    vocab = min(cluster * ept * 128 - 24, 9000)
    w = synth.Workload("forced", 6, vocab, "4x2x1", dtype, "normal", 2.5, 1.0, 1.0, 1.0, 1, 31 + cluster + ept)
    inp = synth.make_inputs(w, "cuda")
    with library_options(cluster=cluster, ept=ept):
        _, out = run_library(inp)
    assert_parity(inp, out)


@pytest.mark.parametrize("dtype,vocab,kconfig,mode", [("bf16", 32000, "4x2x2x1", 1), ("fp32", 32001, "2x1x1", 0),
                                                       ("fp16", 50272, "2x2x2x2", 1), ("fp32", 1000, "4x1", 0),
                                                       ("bf16", 9000, "1x1x1", 0), ("fp16", 5003, "3x2x1", 1)])
def test_split_launch_equals_single_launch(dtype, vocab, kconfig, mode):
    """Large launches give the cluster kernel only the nodes with two or more children and stream
    the rows of the others with a kernel of its own; the results must be those of the single
    launch bit for bit (same runs, same order of every sum), and the oracle's."""
    w = synth.Workload("split", 7, vocab, kconfig, dtype, "normal", 2.5, 0.9, 1.2, 0.9, mode, 4500 + vocab)
    inp = synth.make_inputs(w, "cuda")
    outs = []
    for split in (1, 2):                      # 1: never, 2: always
        with library_options(split=split):
            _, out = run_library(inp)
            outs.append([to_np(x).copy() for x in (out.accept_len, out.tokens, out.residual, out.node_accept,
                                                   out.node_bonus, out.status, out.node_ratio)])
            assert_parity(inp, out)
            assert binding.mcsd_last_launch_count() >= 1
    for a, b in zip(*outs):
        assert np.array_equal(a, b, equal_nan=True)


@pytest.mark.parametrize("dtype,vocab,kconfig,mode,T", [("bf16", 32000, "4x2x2x1", 1, 1.0), ("fp32", 32000, "2", 0, 0.7),
                                                       ("fp16", 50272, "2x2", 1, 1.3), ("fp32", 1000, "3x2x1", 0, 1.0),
                                                       ("bf16", 7, "2x2", 0, 1.0), ("fp32", 65536, "1x1", 0, 1.0),
                                                       ("fp16", 4099, "8x1", 1, 0.0)])
def test_clustered_walk_equals_single_cta_walk(dtype, vocab, kconfig, mode, T):
    """Small batches give every sequence a cluster of eight CTAs in the walk stage; its 32 warps own the
    runs the 32 warps of the one-CTA form of 1024 threads own and sum in the same order, so every output
    agrees bit for bit, and with the oracle.  (With per-node outputs the one-CTA form has 16 warps and
    other runs: there both are held against the oracle.)"""
    w = synth.Workload("cwalk", 5, vocab, kconfig, dtype, "normal", 2.5, 0.9, 1.2, T, mode, 5100 + vocab)
    inp = synth.make_inputs(w, "cuda")
    outs = []
    for wc in (1, 2):                         # 1: never, 2: always
        with library_options(walk_cluster=wc):
            _, out = run_library(inp, node_outputs=False)
            outs.append([to_np(x).copy() for x in (out.accept_len, out.tokens, out.residual, out.status, out.path_nodes)])
            assert_parity(inp, out)
            _, out = run_library(inp, node_outputs=True)
            assert_parity(inp, out)
    for a, b in zip(*outs):
        assert np.array_equal(a, b, equal_nan=True)


def test_traced_call_reports_its_layout_and_changes_nothing(capfd):
    """MCSD_OPT_TRACE 3: a line on stderr per call (with how the node stage was laid out) and an NVTX
    range around it; the outputs are those of the untraced call."""
    w = synth.Workload("traced", 5, 32000, "4x2x1", "bf16", "normal", 2.5, 0.9, 1.2, 1.0, 1, 4711)
    inp = synth.make_inputs(w, "cuda")
    with library_options(split=2):
        _, plain = run_library(inp, node_outputs=False)
        want = [to_np(x).copy() for x in (plain.accept_len, plain.tokens, plain.residual, plain.status)]
        capfd.readouterr()
        with library_options(trace=3):
            _, traced = run_library(inp, node_outputs=False)
        torch.cuda.synchronize()
    lines = [l for l in capfd.readouterr().err.splitlines() if l.startswith("[mcsd] mcsd_verify ")]
    assert len(lines) == 1
    for part in ("batch=5", "vocab=32000", "dtype=1", "mode=1", "rc=0", "launches=4", "cluster=4 x 128 threads",
                 "64 elements/thread", "split launch"):
        assert part in lines[0], (part, lines[0])
    for a, b in zip(want, (traced.accept_len, traced.tokens, traced.residual, traced.status)):
        assert np.array_equal(a, to_np(b), equal_nan=True)


def test_direct_path_matches_bulk_copy_path():
    w = synth.Workload("direct", 6, 32000, "4x2", "bf16", "normal", 2.5, 0.8, 1.5, 1.0, 0, 99)
    inp = synth.make_inputs(w, "cuda")
    _, a = run_library(inp)
    a_acc, a_bon, a_res = to_np(a.node_accept), to_np(a.node_bonus), to_np(a.residual)
    with library_options(direct=1):
        _, b = run_library(inp)
    assert np.array_equal(a_acc, to_np(b.node_accept)) and np.array_equal(a_bon, to_np(b.node_bonus))
    assert np.array_equal(a_res, to_np(b.residual))
    assert_parity(inp, b)


def test_root_only_tree_and_empty_batch():
    w = synth.Workload("root_only", 9, 4096, "", "fp32", "normal", 2.0, 1.0, 1.0, 1.0, 0, 5)
    inp = synth.make_inputs(w, "cuda")
    assert inp.stats["n_nodes"] == 1 and inp.draft is None
    _, out = run_library(inp)
    rep = assert_parity(inp, out)
    assert (to_np(out.accept_len) == 0).all()
    v = binding.Verifier(0, inp.parent, 4096, torch.float32, "cuda")
    out0 = v.mcsd_verify(inp.target[:0], None, inp.cand[:0], inp.unif[:0], 1.0, 0)
    torch.cuda.synchronize()
    assert out0.accept_len.numel() == 0


def test_wide_and_deep_trees():
    for kc, seed in (("32", 1), ("16x2", 2), ("1x1x1x1x1x1x1x1", 3), ("4x4x2x2x1", 4)):
        w = synth.Workload("tree_" + kc, 3, 3000, kc, "fp32", "normal", 2.5, 1.0, 2.0, 1.0, 1, 600 + seed)
        inp = synth.make_inputs(w, "cuda")
        _, out = run_library(inp)
        assert_parity(inp, out)


def test_temperatures():
    for T in (0.3, 0.7, 1.0, 1.7):
        w = synth.Workload("temp", 8, 6000, "3x2x1", "fp16", "gumbel", 2.0, 1.0, 1.2, T, 1, int(T * 100))
        inp = synth.make_inputs(w, "cuda")
        _, out = run_library(inp)
        assert_parity(inp, out)


def test_degenerate_inputs_set_status_and_never_hang():
    w = synth.Workload("degenerate", 6, 4000, "3x2", "fp32", "normal", 2.0, 1.0, 1.0, 1.0, 1, 808)
    inp = synth.make_inputs(w, "cuda")
    # sequence 0: an out-of-range candidate as first child of the root (forced rejection)
    inp.cand[0, 1] = 4000
    # sequence 1: duplicate siblings in the without-replacement mode
    inp.cand[1, 2] = inp.cand[1, 1]
    # sequence 2: -inf logits on half of the draft row of the root (probability 0 is legal)
    inp.draft[2, 0, ::2] = float("-inf")
    # sequence 3: target equals draft at the root: candidates are accepted unless u is ~1
    inp.draft[3, 0] = inp.target[3, 0]
    # sequence 4: a negative candidate
    inp.cand[4, 3] = -5
    _, out = run_library(inp)
    rep = assert_parity(inp, out)
    st = to_np(out.status)
    assert st[0] & binding.STATUS_BAD_TOKEN       # the root is on every walk
    assert not (st & binding.STATUS_TIMEOUT).any()


def test_argmax_ties_take_the_lowest_index():
    w = synth.Workload("ties", 16, 3001, "4x2", "fp16", "normal", 3.0, 1.0, 2.0, 0.0, 0, 321)
    inp = synth.make_inputs(w, "cuda")
    # quantise hard so that every row has many equal maxima
    inp.target.copy_((inp.target.float() / 4).round().clamp(-1, 1).to(torch.float16))
    first, count = synth.children_ranges(inp.parent)
    amax = inp.target.float().cpu().numpy().argmax(axis=-1)          # numpy returns the first maximum
    inp.cand[:, 1] = torch.from_numpy(amax[:, 0]).to(inp.cand)        # make the root accept child 1
    _, out = run_library(inp)
    assert_parity(inp, out)
    assert (to_np(out.accept_len) >= 1).all()


def test_staged_entry_points_equal_the_fused_call():
    w = NAMED["cfg2_b8_without"]
    inp = synth.make_inputs(w, "cuda")
    v, out = run_library(inp)
    ref = (to_np(out.accept_len).copy(), to_np(out.tokens).copy(), to_np(out.residual).copy())
    v2 = binding.Verifier(w.batch, inp.parent, w.vocab, torch.bfloat16, "cuda")
    v2.mcsd_verify_nodes(inp.target, inp.draft, inp.cand, inp.unif, w.temperature, w.mode)
    o2 = v2.mcsd_verify_walk(inp.target, inp.draft, inp.cand, inp.unif, w.temperature)
    torch.cuda.synchronize()
    assert np.array_equal(ref[0], to_np(o2.accept_len)) and np.array_equal(ref[1], to_np(o2.tokens))
    assert np.array_equal(ref[2], to_np(o2.residual))
    assert np.array_equal(to_np(out.status), to_np(o2.status))
    assert binding.mcsd_last_launch_count() == 1


def test_repeated_calls_are_bit_identical():
    inp = synth.make_inputs(NAMED["cfg4_opt"], "cuda")
    v, out = run_library(inp)
    first = [to_np(x).copy() for x in (out.accept_len, out.tokens, out.residual, out.node_accept, out.node_bonus)]
    for _ in range(3):
        out = v.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, 0.7, 1)
        torch.cuda.synchronize()
        again = [to_np(x) for x in (out.accept_len, out.tokens, out.residual, out.node_accept, out.node_bonus)]
        for a, b in zip(first, again):
            assert np.array_equal(a, b, equal_nan=True)


def test_host_buffer_entry_point():
    for name in ("cfg2_b8_with", "cfg3_greedy"):
        w = NAMED[name]
        inp = synth.make_inputs(w, "cuda")
        _, dev = run_library(inp, node_outputs=False)
        host = binding.mcsd_verify_host(inp.target.cpu().pin_memory(),
                                        None if inp.draft is None else inp.draft.cpu().pin_memory(),
                                        inp.parent, inp.cand.cpu().pin_memory(), inp.unif.cpu().pin_memory(),
                                        w.temperature, w.mode)
        assert np.array_equal(to_np(dev.accept_len), host.accept_len.numpy())
        assert np.array_equal(to_np(dev.tokens), host.tokens.numpy())
        assert np.array_equal(to_np(dev.residual), host.residual.numpy())


@pytest.mark.parametrize("idx", [0, 37, 95, 141, 150, 208, 262, 299])
def test_sweep_points_sampled(idx):
    """Points of the throughput sweep (both dtypes, small and large batches); parity on 16
    sequences of each, the library running the whole batch in the launch shape the bench times."""
    w = synth.sweep_workloads()[idx]
    if w.batch > 64:
        w = synth.Workload(w.name, 64, w.vocab, w.kconfig, w.dtype, w.target_dist, w.target_scale,
                           w.draft_gain, w.draft_sigma, w.temperature, w.mode, w.seed)
    inp = synth.make_inputs(w, "cuda")
    _, out = run_library(inp)
    assert_parity(inp, out, 0, min(16, w.batch))


def _parity_in_chunks(inp, out, chunk=64, **kw):
    """Oracle parity on every sequence, a chunk at a time (the float32 host copies of 512 sequences
    would be 19.5 GB at once); the near-tie share is judged on the totals."""
    from oracle import compare as cmp
    w = inp.workload
    tests = near = flipped = tolerated = draws = 0
    for b0 in range(0, w.batch, chunk):
        rep = assert_parity(inp, out, b0, min(w.batch, b0 + chunk), **kw)
        tests += rep.n_tests; near += rep.n_near_tie; flipped += rep.n_flipped
        tolerated += rep.n_bonus_tolerated; draws += rep.n_bonus_draws
    assert near <= max(cmp.NEAR_TIE_MIN_EVENTS, cmp.NEAR_TIE_SHARE * tests), (near, tests)
    assert tolerated <= cmp.boundary_draw_limit(w.vocab, draws), (tolerated, draws)
    return {"tests": tests, "near_ties": near, "flipped": flipped, "bonus_tolerated": tolerated, "bonus_draws": draws}


@pytest.mark.skipif(os.environ.get("MCSD_SKIP_LARGE") == "1", reason="large case disabled")
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_largest_configuration_full_parity_and_properties(dtype):
    """B = 512, 4x4x2x2x1, V = 32000 (19.5 GB of fp32 logits), in the launch shape the bench times:
    oracle parity on ALL 512 sequences, node by node, plus structural properties."""
    from dataclasses import replace
    w = replace(NAMED["cfg5_largest"], dtype=dtype)
    inp = synth.make_inputs(w, "cuda")
    _, out = run_library(inp)
    totals = _parity_in_chunks(inp, out)
    print(dtype, totals)
    assert totals["tests"] > 60000
    acc, bon = to_np(out.node_accept), to_np(out.node_bonus)
    tok, ln = to_np(out.tokens), to_np(out.accept_len)
    first, count = synth.children_ranges(inp.parent)
    parent = inp.parent
    cand = to_np(inp.cand)
    assert (to_np(out.status) == 0).all()
    for n in range(parent.shape[0]):
        a = acc[:, n]
        ok = (a == -1) | ((a >= first[n]) & (a < first[n] + count[n]))
        assert ok.all()
        assert ((bon[:, n] >= 0) == (a == -1)).all()
    assert ((bon >= -1) & (bon < w.vocab)).all()
    for b in range(w.batch):
        n = 0
        for i in range(ln[b]):
            n = acc[b, n]
            assert tok[b, i] == cand[b, n]
        assert acc[b, n] == -1 and tok[b, ln[b]] == bon[b, n] and (tok[b, ln[b] + 1:] == -1).all()
    res = out.residual
    s = res.sum(dim=1)
    assert float((s - 1).abs().max()) < 1e-4 and float(res.min()) >= 0.0
    end = torch.from_numpy(tok[np.arange(w.batch), ln]).to(res.device).long()
    assert bool((res.gather(1, end[:, None]) > 0).all())       # the endpoint token has positive mass
    assert 0.5 < ln.mean() < 4.5


@pytest.mark.parametrize("dtype,T,mode", [("fp32", 1.0, 0), ("fp32", 0.7, 1), ("bf16", 1.0, 1), ("fp16", 0.0, 0)])
def test_per_node_residual_output(dtype, T, mode):
    """node_residual: for every node that can end a walk, the distribution its endpoint token is
    drawn from (Algorithm 1 / 2 residual after k rejections, target distribution at a leaf,
    one-hot at temperature 0), against the oracle node by node; other rows stay untouched."""
    import oracle
    w = synth.Workload("node_res", 3, 3000, "3x2x1", dtype, "normal", 2.5, 1.0, 1.5, T, mode, 808)
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[dtype], "cuda", node_outputs=True,
                         node_residual=True)
    out = v.mcsd_verify(inp.target, inp.draft if T > 0 else None, inp.cand, inp.unif, T, mode)
    torch.cuda.synchronize()
    assert_parity(inp, out)
    t, d, c, u = inp.host_f32()
    acc = to_np(out.node_accept)
    res = to_np(out.node_residual)
    first, count = synth.children_ranges(inp.parent)
    tol = 1e-5 if dtype == "fp32" else 2e-3
    seen_stop = seen_skip = 0
    for b in range(w.batch):
        for n in range(inp.stats["n_nodes"]):
            if acc[b, n] >= 0:
                assert np.isnan(res[b, n]).all()      # a walk never stops here: row not written
                seen_skip += 1
                continue
            seen_stop += 1
            if T == 0:
                want = np.zeros(w.vocab)
                want[oracle.argmax(t[b, n])] = 1.0
            else:
                want = oracle.softmax(t[b, n], T)
                k = int(count[n])
                if k:
                    ch = np.arange(first[n], first[n] + k)
                    r = oracle.mcss(want, oracle.softmax(d[b, n], T), c[b, ch], u[b, ch, 0].astype(np.float64), mode)
                    assert r.accepted == -1
                    want = r.p
            assert np.abs(res[b, n] - want).max() <= tol, (b, n)
    assert seen_stop > 0 and seen_skip > 0


@pytest.mark.skipif(os.environ.get("MCSD_SKIP_LARGE") == "1", reason="large case disabled")
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_largest_configuration_path_form_and_sampler(dtype):
    """The same full-size inputs through the other entry points, in the launch shapes the bench
    times: the path form must reproduce the all-node form bit for bit on all 512 sequences (and the
    oracle on sampled ones); the sampler is compared with the oracle on sampled sequences and must
    draw valid, and without replacement distinct, tokens everywhere."""
    from dataclasses import replace
    from oracle import compare as cmp
    w = replace(NAMED["cfg5_largest"], dtype=dtype, mode=1)
    inp = synth.make_inputs(w, "cuda")
    v = binding.Verifier(w.batch, inp.parent, w.vocab, synth.TORCH_DTYPES[dtype], "cuda")
    a = v.mcsd_verify(inp.target, inp.draft, inp.cand, inp.unif, w.temperature, w.mode)
    torch.cuda.synchronize()
    a_len, a_tok, a_res, a_st = (x.clone() for x in (a.accept_len, a.tokens, a.residual, a.status))
    b = v.mcsd_verify_path(inp.target, inp.draft, inp.cand, inp.unif, w.temperature, w.mode)
    torch.cuda.synchronize()
    assert torch.equal(a_len, b.accept_len) and torch.equal(a_tok, b.tokens) and torch.equal(a_st, b.status)
    assert torch.equal(a_res, b.residual)
    for b0 in (0, 300, 506):
        assert_parity(inp, b, b0, b0 + 6, sequential=True)
    # sampler
    gen = torch.Generator(device="cuda")
    gen.manual_seed(99)
    u = synth.open_uniforms((w.batch, inp.stats["n_nodes"]), gen, "cuda")
    cand = binding.mcsd_sample_candidates(inp.draft, inp.parent, u, 1.0, 1)
    torch.cuda.synchronize()
    c = cand.cpu().numpy()
    assert (c[:, 0] == -1).all() and (c[:, 1:] >= 0).all() and (c[:, 1:] < w.vocab).all()
    first, count = synth.children_ranges(inp.parent)
    for n in range(inp.stats["n_internal"]):
        ch = np.sort(c[:, first[n]:first[n] + count[n]], axis=1)
        assert (np.diff(ch, axis=1) > 0).all()          # Eq. 1: the children of a node carry distinct tokens
    for b0 in (0, 400, 508):
        sl = slice(b0, b0 + 4)
        rep = cmp.compare_samples(inp.draft[sl].to(torch.float32).cpu().numpy(), inp.parent, u[sl].cpu().numpy(), 1.0, 1,
                                  c[sl], 0, None)
        assert rep.ok, rep.failures[:5]       # (includes the bound on draws that differ inside the tolerance)
