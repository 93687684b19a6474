"""The C-ABI library: it loads, exports every symbol the header declares, and its host-side
validation answers with the documented codes before touching a GPU."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2401_06706_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "mcsd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mcsd_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert set(names) == set(binding.EXPORTS)
    for name in names:
        assert getattr(lib, name) is not None
    assert lib.mcsd_version() == 102


def test_header_constants_match_binding():
    text = open(os.path.join(ROOT, "include", "mcsd.h")).read()
    consts = dict(re.findall(r"#define\s+(MCSD_[A-Z0-9_]+)\s+\(?(-?\d+)\)?", text))
    assert int(consts["MCSD_MAX_NODES"]) == binding.MAX_NODES
    assert int(consts["MCSD_MAX_CHILDREN"]) == binding.MAX_CHILDREN
    assert int(consts["MCSD_MAX_VOCAB"]) == binding.MAX_VOCAB
    assert int(consts["MCSD_STATUS_TIMEOUT"]) == binding.STATUS_TIMEOUT
    assert int(consts["MCSD_DTYPE_BF16"]) == 1 and int(consts["MCSD_DTYPE_F16"]) == 2
    for name in ("CLUSTER", "EPT", "DIRECT", "SAMPLE_AHEAD", "WAIT_POLLS", "TEST_EXTRA_TX", "PDL", "TEST_SHRINK_RANGES", "SPLIT", "TIME_KERNELS", "TRACE", "WALK_CLUSTER"):
        assert int(consts["MCSD_OPT_" + name]) == getattr(binding, "OPT_" + name)


def test_options_are_set_read_back_and_validated(lib):
    n = int(re.search(r"#define\s+MCSD_OPT_COUNT\s+(\d+)", open(os.path.join(ROOT, "include", "mcsd.h")).read()).group(1))
    before = [binding.mcsd_get_option(i) for i in range(n)]
    try:
        for i in range(n):
            binding.mcsd_set_option(i, 3)
            assert binding.mcsd_get_option(i) == 3
        for bad in (-1, n, 99):
            assert lib.mcsd_set_option(bad, 1) == -2 and lib.mcsd_get_option(bad) == -2
        assert lib.mcsd_set_option(0, -5) == -2
    finally:
        for i, val in enumerate(before):
            binding.mcsd_set_option(i, val)


def test_trace_option_reports_rejected_calls_on_stderr(lib, capfd):
    """MCSD_OPT_TRACE bit 0: one line per call with the shape, the temperature, the mode and the return
    code; here for calls the host checks reject (nothing is enqueued, the fake pointers are never used)."""
    d, parent = _desc(ws=(0x10000, 1 << 20))
    before = binding.mcsd_get_option(binding.OPT_TRACE)
    try:
        binding.mcsd_set_option(binding.OPT_TRACE, 1)
        assert lib.mcsd_verify(ctypes.byref(d), 0x1000, 0x1000, parent.ctypes.data, 0x1000, 0x1000, -0.5, 0,
                               0x1000, 0x1000, None) == -5
        assert lib.mcsd_verify_path(None, 0x1000, 0x1000, parent.ctypes.data, 0x1000, 0x1000, 1.0, 1,
                                    0x1000, 0x1000, None) == -1
        binding.mcsd_set_option(binding.OPT_TRACE, 0)
        assert lib.mcsd_verify(ctypes.byref(d), 0x1000, 0x1000, parent.ctypes.data, 0x1000, 0x1000, -0.5, 0,
                               0x1000, 0x1000, None) == -5
    finally:
        binding.mcsd_set_option(binding.OPT_TRACE, before)
    lines = [l for l in capfd.readouterr().err.splitlines() if l.startswith("[mcsd]")]
    assert len(lines) == 2                                       # nothing once the option is off again
    assert "mcsd_verify " in lines[0] and f"batch={d.batch}" in lines[0] and f"vocab={d.vocab}" in lines[0]
    assert "T=-0.5" in lines[0] and "rc=-5" in lines[0] and "launches=0" in lines[0]
    assert "mcsd_verify_path desc=NULL" in lines[1] and "rc=-1" in lines[1]


def test_tree_depth_and_contract(lib):
    for text, gamma in [("2", 1), ("4x2x2x1", 4), ("4x4x2x2x1", 5), ("1x1x1", 3)]:
        parent = synth.tree_from_kconfig(synth.parse_kconfig(text))
        assert binding.mcsd_tree_depth(parent) == gamma
    assert binding.mcsd_tree_depth(np.array([-1], dtype=np.int32)) == 0
    for bad in ([0, 0], [-1, 1], [-1, 0, 0, 2, 1], [-1, -1]):
        with pytest.raises(binding.McsdError) as e:
            binding.mcsd_tree_depth(np.array(bad, dtype=np.int32))
        assert e.value.code == -6
    with pytest.raises(binding.McsdError) as e:      # 33 children of one node
        binding.mcsd_tree_depth(np.array([-1] + [0] * 33, dtype=np.int32))
    assert e.value.code == -10


def _desc(batch=2, parent=None, vocab=64, dtype=0, ws=None):
    parent = synth.tree_from_kconfig([2, 1]) if parent is None else parent
    d = binding.McsdDesc()
    d.batch, d.n_nodes, d.vocab, d.dtype = batch, parent.shape[0], vocab, dtype
    d.n_internal = binding._n_internal(parent)
    d.ld_target = d.ld_draft = vocab
    if ws is not None:
        d.workspace, d.workspace_bytes = ws
    return d, parent


def test_workspace_bytes(lib):
    d, _ = _desc()
    n = lib.mcsd_workspace_bytes(ctypes.byref(d))
    assert n >= 2 * 5 * (4 + 4 + 32) and n % 256 == 0
    d.batch = 4
    assert lib.mcsd_workspace_bytes(ctypes.byref(d)) > n
    d.vocab = 0
    assert lib.mcsd_workspace_bytes(ctypes.byref(d)) == 0
    assert lib.mcsd_workspace_bytes(None) == 0


def test_host_validation_codes(lib):
    """Every rejected call returns before anything is enqueued; pointers are fakes that are
    never dereferenced on these paths (tree_parent is the only host array)."""
    fake = 0x1000
    ws = (0x10000, 1 << 20)

    def call(d, parent, *, target=fake, draft=fake, cand=fake, unif=fake, T=1.0, mode=0, out_len=fake,
             out_tok=fake):
        return lib.mcsd_verify(ctypes.byref(d) if d is not None else None, target, draft,
                               parent.ctypes.data if parent is not None else None, cand, unif, T, mode,
                               out_len, out_tok, None)

    d, parent = _desc(ws=ws)
    assert call(None, parent) == -1
    assert call(d, None) == -1
    assert call(d, parent, target=None) == -1
    assert call(d, parent, draft=None) == -1
    assert call(d, parent, unif=None) == -1
    assert call(d, parent, out_len=None) == -1
    assert call(d, parent, T=-0.5) == -5
    assert call(d, parent, T=float("nan")) == -5
    assert call(d, parent, T=float("inf")) == -5
    assert call(d, parent, mode=3) == -4
    d2, _ = _desc(ws=ws); d2.dtype = 7
    assert call(d2, parent) == -3
    d2, _ = _desc(ws=ws); d2.vocab = 0
    assert call(d2, parent) == -2
    d2, _ = _desc(ws=ws); d2.reserved = 1
    assert call(d2, parent) == -2
    d2, _ = _desc(ws=ws); d2.vocab = 70000; d2.ld_target = d2.ld_draft = 70000
    assert call(d2, parent) == -10
    d2, _ = _desc(ws=ws); d2.ld_target = 63
    assert call(d2, parent) == -7
    d2, _ = _desc(ws=ws); d2.ld_draft = 10
    assert call(d2, parent) == -7
    d2, _ = _desc(ws=ws); d2.n_internal = 1
    assert call(d2, parent) == -6
    assert call(d, np.array([-1, 0, 0, 2, 1], dtype=np.int32)) == -6
    d2, _ = _desc(); assert call(d2, parent) == -8                     # no workspace
    d2, _ = _desc(ws=(0x10000, 16)); assert call(d2, parent) == -8     # too small
    d2, _ = _desc(ws=(0x10010, 1 << 20)); assert call(d2, parent) == -8  # misaligned
    for code in range(-11, 1):
        assert len(binding.status_string(code)) > 0
    assert binding.status_string(-99) == "unknown code"


def test_binding_fails_loudly_without_library(tmp_path):
    with pytest.raises(RuntimeError, match="missing"):
        binding.load_library(str(tmp_path / "libmcsd.so"))


def test_the_build_entry_point_runs():
    """build() of the repository's entry file compiles the CUDA library and the oracle and checks
    the library against the header; it needs nvcc and gcc but no GPU."""
    import __graft_entry__
    __graft_entry__.build()
