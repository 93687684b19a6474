"""Thin Python binding of libmcsd.so: argument marshalling only.

Every step of the verification runs inside the CUDA library; this module turns
torch tensors into raw pointers, fills the descriptor and raises on a non-zero
return code.  It fails loudly when the library is missing: there is no CPU or
eager fallback.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmcsd.so")
DEBUG_LIB_PATH = os.path.join(_HERE, "libmcsd_debug.so")      # the checked build (see mcsd_debug_bounds_hits)

MCSD_DTYPE = {torch.float32: 0, torch.bfloat16: 1, torch.float16: 2}
STATUS_DEGENERATE, STATUS_BAD_TOKEN, STATUS_NO_MASS, STATUS_TIMEOUT = 1, 2, 4, 8
MAX_NODES, MAX_CHILDREN, MAX_VOCAB = 512, 32, 65536

EXPORTS = ("mcsd_verify", "mcsd_verify_nodes", "mcsd_verify_walk", "mcsd_verify_host", "mcsd_verify_static", "mcsd_verify_path", "mcsd_sample_candidates", "mcsd_tree_attention_layout",
           "mcsd_gather_accepted_kv",
           "mcsd_workspace_bytes", "mcsd_tree_depth", "mcsd_last_launch_count", "mcsd_status_string",
           "mcsd_version", "mcsd_set_option", "mcsd_get_option", "mcsd_release_host_staging",
           "mcsd_shard_columns", "mcsd_shard_workspace_bytes", "mcsd_shard_rounds", "mcsd_shard_partials",
           "mcsd_shard_decide", "mcsd_shard_endpoint", "mcsd_shard_finish", "mcsd_shard_commit", "mcsd_debug_bounds_hits", "mcsd_last_kernel_times")
OPT_CLUSTER, OPT_EPT, OPT_DIRECT, OPT_SAMPLE_AHEAD, OPT_WAIT_POLLS, OPT_TEST_EXTRA_TX, OPT_PDL, OPT_TEST_SHRINK_RANGES, OPT_SPLIT, OPT_TIME_KERNELS, OPT_TRACE, OPT_WALK_CLUSTER = range(12)


class McsdDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_nodes", ctypes.c_int32), ("n_internal", ctypes.c_int32),
                ("vocab", ctypes.c_int32), ("dtype", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("ld_target", ctypes.c_int64), ("ld_draft", ctypes.c_int64),
                ("stream", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
                ("workspace_bytes", ctypes.c_size_t),
                ("node_accept", ctypes.c_void_p), ("node_bonus", ctypes.c_void_p),
                ("node_ratio", ctypes.c_void_p), ("out_status", ctypes.c_void_p),
                ("out_path_nodes", ctypes.c_void_p), ("node_residual", ctypes.c_void_p)]


class McsdShardDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_nodes", ctypes.c_int32), ("n_internal", ctypes.c_int32),
                ("vocab", ctypes.c_int32), ("dtype", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("n_shards", ctypes.c_int32), ("shard", ctypes.c_int32),
                ("ld_target", ctypes.c_int64), ("ld_draft", ctypes.c_int64),
                ("stream", ctypes.c_void_p), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
                ("node_ratio", ctypes.c_void_p), ("node_accept", ctypes.c_void_p)]


class McsdError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"libmcsd error {code}: {text}")
        self.code = code


_lib = None


def load_library(path: Optional[str] = None):
    """dlopen libmcsd.so and declare its signatures.  Raises if it has not been built."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise RuntimeError(f"{p} is missing: build it with `python -m paper_2401_06706_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(p)
    vp, i32, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_float
    dp = ctypes.POINTER(McsdDesc)
    lib.mcsd_verify.argtypes = [dp, vp, vp, vp, vp, vp, f32, ctypes.c_int, vp, vp, vp]
    lib.mcsd_verify.restype = ctypes.c_int
    lib.mcsd_verify_path.argtypes = [dp, vp, vp, vp, vp, vp, f32, ctypes.c_int, vp, vp, vp]
    lib.mcsd_verify_path.restype = ctypes.c_int
    lib.mcsd_sample_candidates.argtypes = [dp, vp, vp, vp, f32, ctypes.c_int, i32, i32, vp]
    lib.mcsd_sample_candidates.restype = ctypes.c_int
    lib.mcsd_tree_attention_layout.argtypes = [vp, i32, i32, vp, vp, vp]
    lib.mcsd_tree_attention_layout.restype = ctypes.c_int
    i64 = ctypes.c_int64
    lib.mcsd_gather_accepted_kv.argtypes = [vp, i64, i64, i32, i64, i64, i64, i64, vp, vp, vp, i32, vp]
    lib.mcsd_gather_accepted_kv.restype = ctypes.c_int
    lib.mcsd_verify_static.argtypes = [dp, vp, vp, vp, vp, vp, f32, ctypes.c_int, vp, vp, vp]
    lib.mcsd_verify_static.restype = ctypes.c_int
    lib.mcsd_verify_nodes.argtypes = [dp, vp, vp, vp, vp, vp, f32, ctypes.c_int]
    lib.mcsd_verify_nodes.restype = ctypes.c_int
    lib.mcsd_verify_walk.argtypes = [dp, vp, vp, vp, vp, vp, f32, vp, vp, vp]
    lib.mcsd_verify_walk.restype = ctypes.c_int
    lib.mcsd_verify_host.argtypes = [dp, vp, vp, vp, vp, vp, f32, ctypes.c_int, vp, vp, vp, vp]
    lib.mcsd_verify_host.restype = ctypes.c_int
    lib.mcsd_workspace_bytes.argtypes = [dp]
    lib.mcsd_workspace_bytes.restype = ctypes.c_size_t
    lib.mcsd_tree_depth.argtypes = [vp, i32]
    lib.mcsd_tree_depth.restype = ctypes.c_int
    lib.mcsd_last_launch_count.argtypes = []
    lib.mcsd_last_launch_count.restype = ctypes.c_int
    lib.mcsd_status_string.argtypes = [ctypes.c_int]
    lib.mcsd_status_string.restype = ctypes.c_char_p
    lib.mcsd_version.argtypes = []
    lib.mcsd_version.restype = ctypes.c_int
    lib.mcsd_set_option.argtypes = [ctypes.c_int, ctypes.c_int]
    lib.mcsd_set_option.restype = ctypes.c_int
    lib.mcsd_get_option.argtypes = [ctypes.c_int]
    lib.mcsd_get_option.restype = ctypes.c_int
    lib.mcsd_release_host_staging.argtypes = []
    lib.mcsd_release_host_staging.restype = ctypes.c_int
    sp = ctypes.POINTER(McsdShardDesc)
    lib.mcsd_shard_columns.argtypes = [i32, i32, i32, i32, vp, vp, vp]
    lib.mcsd_shard_columns.restype = ctypes.c_int
    lib.mcsd_shard_workspace_bytes.argtypes = [sp]
    lib.mcsd_shard_workspace_bytes.restype = ctypes.c_size_t
    lib.mcsd_shard_rounds.argtypes = [vp, i32]
    lib.mcsd_shard_rounds.restype = ctypes.c_int
    lib.mcsd_shard_partials.argtypes = [sp, vp, vp, vp, vp, f32, i32, vp, vp]
    lib.mcsd_shard_partials.restype = ctypes.c_int
    lib.mcsd_shard_decide.argtypes = [sp, vp, vp, vp, f32, ctypes.c_int, i32, vp, vp]
    lib.mcsd_shard_decide.restype = ctypes.c_int
    lib.mcsd_shard_endpoint.argtypes = [sp, vp, vp, vp, f32, i32, vp, vp, vp]
    lib.mcsd_shard_endpoint.restype = ctypes.c_int
    lib.mcsd_shard_finish.argtypes = [sp, vp, vp, vp, vp, vp, f32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.mcsd_shard_finish.restype = ctypes.c_int
    lib.mcsd_shard_commit.argtypes = [sp, vp, vp, vp, vp]
    lib.mcsd_shard_commit.restype = ctypes.c_int
    lib.mcsd_last_kernel_times.argtypes = [vp, i32]
    lib.mcsd_last_kernel_times.restype = ctypes.c_int
    lib.mcsd_debug_bounds_hits.argtypes = [ctypes.c_int]
    lib.mcsd_debug_bounds_hits.restype = ctypes.c_longlong
    if path is None:
        _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().mcsd_status_string(int(code)).decode()


def _check(code: int):
    if code != 0:
        raise McsdError(code, status_string(code))


def mcsd_version() -> int:
    return int(load_library().mcsd_version())


def mcsd_tree_depth(parent) -> int:
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    rc = load_library().mcsd_tree_depth(parent.ctypes.data, parent.shape[0])
    _check(rc if rc < 0 else 0)
    return rc


def mcsd_last_launch_count() -> int:
    return int(load_library().mcsd_last_launch_count())


def mcsd_set_option(option: int, value: int) -> None:
    _check(load_library().mcsd_set_option(int(option), int(value)))


def mcsd_get_option(option: int) -> int:
    rc = load_library().mcsd_get_option(int(option))
    _check(rc if rc < 0 else 0)
    return rc


def mcsd_last_kernel_times():
    """[cluster / argmax / naive, streaming statistics, single test, walk] kernel milliseconds of the last call
    (needs MCSD_OPT_TIME_KERNELS); None where no such kernel ran."""
    ms = (ctypes.c_float * 4)()
    rc = load_library().mcsd_last_kernel_times(ctypes.addressof(ms), 4)
    _check(rc if rc < 0 else 0)
    return [None if x < 0 else float(x) for x in ms]


def mcsd_debug_bounds_hits(reset: bool = False) -> int:
    return int(load_library().mcsd_debug_bounds_hits(1 if reset else 0))


def mcsd_release_host_staging() -> None:
    _check(load_library().mcsd_release_host_staging())


def _n_internal(parent: np.ndarray) -> int:
    has = np.zeros(parent.shape[0], dtype=bool)
    if parent.shape[0] > 1:
        has[parent[1:][parent[1:] >= 0]] = True
    return int(has.sum())


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _row_stride(t: torch.Tensor) -> int:
    """Elements between consecutive rows of a [B, rows, V] tensor whose rows are contiguous and
    whose leading dimensions collapse to one stride."""
    assert t.dim() == 3 and (t.shape[2] == 1 or t.stride(2) == 1), "vocabulary axis must be contiguous"
    ld = t.stride(1) if t.shape[1] > 1 else max(t.shape[2], t.stride(1))
    if t.shape[0] > 1:
        assert t.stride(0) == ld * t.shape[1], "batch stride must equal rows * row stride"
    return int(ld)


@dataclass
class VerifyOutput:
    accept_len: torch.Tensor            # [B] int32
    tokens: torch.Tensor                # [B, gamma+1] int32
    residual: Optional[torch.Tensor]    # [B, V] float32
    status: torch.Tensor                # [B] int32
    node_accept: Optional[torch.Tensor] = None
    node_bonus: Optional[torch.Tensor] = None
    node_ratio: Optional[torch.Tensor] = None
    path_nodes: Optional[torch.Tensor] = None  # [B, gamma+1] tree nodes of the accepted tokens, -1 padded
    node_residual: Optional[torch.Tensor] = None  # [B, n_nodes, V] float32; rows of nodes that cannot end a walk are NaN


class Verifier:
    """Holds the descriptor and device buffers for one (batch, tree, vocab, dtype) shape so that
    repeated calls allocate nothing."""

    def __init__(self, batch: int, parent, vocab: int, dtype: torch.dtype, device="cuda", *,
                 want_residual: bool = True, node_outputs: bool = False, ld_target: Optional[int] = None,
                 ld_draft: Optional[int] = None, node_residual: bool = False):
        self.lib = load_library()
        self.parent = np.ascontiguousarray(parent, dtype=np.int32)
        self.device = torch.device(device)
        self.batch, self.vocab, self.dtype = int(batch), int(vocab), dtype
        self.n_nodes = int(self.parent.shape[0])
        self.n_internal = _n_internal(self.parent)
        gamma = self.lib.mcsd_tree_depth(self.parent.ctypes.data, self.n_nodes)
        _check(gamma if gamma < 0 else 0)
        self.gamma = gamma
        self.desc = McsdDesc()
        d = self.desc
        d.batch, d.n_nodes, d.n_internal, d.vocab = self.batch, self.n_nodes, self.n_internal, self.vocab
        d.dtype = MCSD_DTYPE[dtype]
        d.ld_target = int(ld_target if ld_target is not None else vocab)
        d.ld_draft = int(ld_draft if ld_draft is not None else vocab)
        ws = int(self.lib.mcsd_workspace_bytes(ctypes.byref(d)))
        if ws == 0:
            _check(-2)
        self.workspace = torch.empty(ws + 256, dtype=torch.uint8, device=self.device)
        base = self.workspace.data_ptr()
        d.workspace = (base + 255) // 256 * 256
        d.workspace_bytes = ws
        i32 = dict(dtype=torch.int32, device=self.device)
        self.accept_len = torch.empty(self.batch, **i32)
        self.tokens = torch.empty((self.batch, self.gamma + 1), **i32)
        self.residual = (torch.empty((self.batch, self.vocab), dtype=torch.float32, device=self.device)
                         if want_residual else None)
        self.status = torch.zeros(self.batch, **i32)
        d.out_status = self.status.data_ptr()
        self.path_nodes = torch.empty((self.batch, self.gamma + 1), **i32)
        d.out_path_nodes = self.path_nodes.data_ptr()
        self.node_accept = self.node_bonus = self.node_ratio = None
        if node_outputs:
            self.node_accept = torch.empty((self.batch, self.n_nodes), **i32)
            self.node_bonus = torch.empty((self.batch, self.n_nodes), **i32)
            self.node_ratio = torch.full((self.batch, self.n_nodes), float("nan"), dtype=torch.float32,
                                         device=self.device)
            d.node_accept = self.node_accept.data_ptr()
            d.node_bonus = self.node_bonus.data_ptr()
            d.node_ratio = self.node_ratio.data_ptr()
        self.node_residual = None
        if node_residual:   # a debugging output: B * n_nodes * V floats
            self.node_residual = torch.full((self.batch, self.n_nodes, self.vocab), float("nan"), dtype=torch.float32,
                                            device=self.device)
            d.node_residual = self.node_residual.data_ptr()

    def _bind(self, target, draft):
        assert target.dtype == self.dtype and target.shape == (self.batch, self.n_nodes, self.vocab)
        self.desc.ld_target = _row_stride(target)
        if draft is not None:
            assert draft.dtype == self.dtype and draft.shape == (self.batch, self.n_internal, self.vocab)
            self.desc.ld_draft = _row_stride(draft) if self.n_internal else self.vocab
        self.desc.stream = torch.cuda.current_stream(self.device).cuda_stream

    def _out(self) -> VerifyOutput:
        return VerifyOutput(self.accept_len, self.tokens, self.residual, self.status, self.node_accept,
                            self.node_bonus, self.node_ratio, self.path_nodes, self.node_residual)

    def mcsd_verify(self, target, draft, cand, unif, temperature: float, mode: int) -> VerifyOutput:
        self._bind(target, draft)
        if self.node_ratio is not None:
            self.node_ratio.fill_(float("nan"))
        _check(self.lib.mcsd_verify(ctypes.byref(self.desc), _ptr(target), _ptr(draft), self.parent.ctypes.data,
                                    _ptr(cand), _ptr(unif), float(temperature), int(mode),
                                    _ptr(self.accept_len), _ptr(self.tokens), _ptr(self.residual)))
        return self._out()

    def mcsd_verify_path(self, target, draft, cand, unif, temperature: float, mode: int) -> VerifyOutput:
        """Level-by-level form: only the nodes the walks visit are evaluated (see mcsd.h)."""
        self._bind(target, draft)
        if self.node_ratio is not None:
            self.node_ratio.fill_(float("nan"))
        _check(self.lib.mcsd_verify_path(ctypes.byref(self.desc), _ptr(target), _ptr(draft),
                                         self.parent.ctypes.data, _ptr(cand), _ptr(unif), float(temperature),
                                         int(mode), _ptr(self.accept_len), _ptr(self.tokens), _ptr(self.residual)))
        return self._out()

    def mcsd_verify_static(self, target, draft, cand, unif, temperature: float, mode: int) -> VerifyOutput:
        """The same call with the library's built-in scratch array instead of this object's
        workspace (for callers that may not allocate device memory); see mcsd.h for its limit."""
        self._bind(target, draft)
        if self.node_ratio is not None:
            self.node_ratio.fill_(float("nan"))
        _check(self.lib.mcsd_verify_static(ctypes.byref(self.desc), _ptr(target), _ptr(draft),
                                           self.parent.ctypes.data, _ptr(cand), _ptr(unif), float(temperature),
                                           int(mode), _ptr(self.accept_len), _ptr(self.tokens),
                                           _ptr(self.residual)))
        return self._out()

    def mcsd_verify_nodes(self, target, draft, cand, unif, temperature: float, mode: int) -> None:
        self._bind(target, draft)
        _check(self.lib.mcsd_verify_nodes(ctypes.byref(self.desc), _ptr(target), _ptr(draft),
                                          self.parent.ctypes.data, _ptr(cand), _ptr(unif), float(temperature),
                                          int(mode)))

    def mcsd_verify_walk(self, target, draft, cand, unif, temperature: float) -> VerifyOutput:
        self._bind(target, draft)
        _check(self.lib.mcsd_verify_walk(ctypes.byref(self.desc), _ptr(target), _ptr(draft),
                                         self.parent.ctypes.data, _ptr(cand), _ptr(unif), float(temperature),
                                         _ptr(self.accept_len), _ptr(self.tokens), _ptr(self.residual)))
        return self._out()


def mcsd_verify(target, draft, parent, cand, unif, temperature: float, mode: int, *,
                want_residual: bool = True, node_outputs: bool = False) -> VerifyOutput:
    """One-shot convenience wrapper: device tensors in, device tensors out."""
    B, _, V = target.shape
    v = Verifier(B, parent, V, target.dtype, target.device, want_residual=want_residual,
                 node_outputs=node_outputs)
    return v.mcsd_verify(target, draft, cand, unif, temperature, mode)


def mcsd_tree_attention_layout(parent, prefix_len: int, device="cuda"):
    """Ancestor-only attention mask [n, n] (uint8) and position ids [n] (int32) of the flattened tree."""
    lib = load_library()
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    n = int(parent.shape[0])
    mask = torch.empty((n, n), dtype=torch.uint8, device=device)
    pos = torch.empty(n, dtype=torch.int32, device=device)
    _check(lib.mcsd_tree_attention_layout(parent.ctypes.data, n, int(prefix_len), _ptr(mask), _ptr(pos),
                                          torch.cuda.current_stream(torch.device(device)).cuda_stream))
    return mask, pos


def mcsd_gather_accepted_kv(cache: torch.Tensor, prefix_len: torch.Tensor, path_nodes: torch.Tensor,
                            accept_len: torch.Tensor) -> torch.Tensor:
    """Moves, in place, the cache rows of the accepted path to their committed positions (see mcsd.h).
    cache: device tensor [slabs, batch, positions, ...] whose trailing dimensions form one contiguous row;
    prefix_len, accept_len: int32 [batch]; path_nodes: int32 [batch, gamma + 1].  Returns cache."""
    lib = load_library()
    assert cache.dim() >= 4 and cache.is_cuda
    S, B, L = cache.shape[:3]
    row = cache[0, 0, 0]
    assert row.is_contiguous(), "the trailing dimensions must form one contiguous row"
    es = cache.element_size()
    assert path_nodes.dtype == torch.int32 and path_nodes.is_contiguous() and path_nodes.shape[0] == B
    assert prefix_len.dtype == torch.int32 and accept_len.dtype == torch.int32
    gamma = int(path_nodes.shape[1]) - 1
    _check(lib.mcsd_gather_accepted_kv(cache.data_ptr(), S, cache.stride(0) * es, B, cache.stride(1) * es,
                                       cache.stride(2) * es, row.numel() * es, L, _ptr(prefix_len),
                                       _ptr(path_nodes), _ptr(accept_len), gamma,
                                       torch.cuda.current_stream(cache.device).cuda_stream))
    return cache


def mcsd_sample_candidates(draft, parent, unif_draw, temperature: float, mode: int, *, node_begin: int = 0,
                           node_end: Optional[int] = None, cand: Optional[torch.Tensor] = None,
                           status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Candidate tokens of the children of nodes [node_begin, node_end): device tensors in, the
    [B, n_nodes] int32 token tensor out (entries outside the range keep their value, -1 if new)."""
    lib = load_library()
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    B, n_internal, V = draft.shape
    n_nodes = int(parent.shape[0])
    d = McsdDesc()
    d.batch, d.n_nodes, d.n_internal, d.vocab = B, n_nodes, n_internal, V
    d.dtype = MCSD_DTYPE[draft.dtype]
    d.ld_target = V
    d.ld_draft = _row_stride(draft) if n_internal else V
    d.stream = torch.cuda.current_stream(draft.device).cuda_stream
    d.out_status = _ptr(status)
    if cand is None:
        cand = torch.full((B, n_nodes), -1, dtype=torch.int32, device=draft.device)
    _check(lib.mcsd_sample_candidates(ctypes.byref(d), _ptr(draft), parent.ctypes.data, _ptr(unif_draw),
                                      float(temperature), int(mode), int(node_begin),
                                      int(n_internal if node_end is None else node_end), _ptr(cand)))
    return cand


def mcsd_verify_host(target, draft, parent, cand, unif, temperature: float, mode: int, *,
                     want_residual: bool = True, out: Optional[dict] = None) -> VerifyOutput:
    """Host tensors (CPU, ideally pinned) in, host tensors out; all copies happen inside the library."""
    lib = load_library()
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    B, n_nodes, V = target.shape
    assert not target.is_cuda and target.is_contiguous()
    d = McsdDesc()
    d.batch, d.n_nodes, d.n_internal, d.vocab = B, n_nodes, _n_internal(parent), V
    d.dtype = MCSD_DTYPE[target.dtype]
    d.ld_target = V
    d.ld_draft = V
    gamma = lib.mcsd_tree_depth(parent.ctypes.data, n_nodes)
    _check(gamma if gamma < 0 else 0)
    if out is None:
        out = {}
    pin = torch.cuda.is_available()
    accept_len = out.get("accept_len", torch.empty(B, dtype=torch.int32, pin_memory=pin))
    tokens = out.get("tokens", torch.empty((B, gamma + 1), dtype=torch.int32, pin_memory=pin))
    residual = out.get("residual", torch.empty((B, V), dtype=torch.float32, pin_memory=pin)) if want_residual else None
    status = out.get("status", torch.zeros(B, dtype=torch.int32, pin_memory=pin))
    _check(lib.mcsd_verify_host(ctypes.byref(d), _ptr(target), _ptr(draft), parent.ctypes.data, _ptr(cand),
                                _ptr(unif), float(temperature), int(mode), _ptr(accept_len), _ptr(tokens),
                                _ptr(residual), _ptr(status)))
    return VerifyOutput(accept_len, tokens, residual, status)


# ---------------------------------------------------------------- vocabulary split over several devices
def mcsd_shard_columns(vocab: int, dtype: torch.dtype, n_shards: int, shard: int):
    """(col_begin, n_cols, entries_per_shard) of one shard; host only (see mcsd.h)."""
    a, b, c = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _check(load_library().mcsd_shard_columns(int(vocab), MCSD_DTYPE[dtype], int(n_shards), int(shard),
                                             ctypes.addressof(a), ctypes.addressof(b), ctypes.addressof(c)))
    return a.value, b.value, c.value


class ShardedVerifier:
    """One shard of the verification with the vocabulary split over several devices: holds the
    descriptor, the workspace and the exchange buffers of its device and exposes the stage calls of
    mcsd.h under their own names (argument marshalling only).  `sharded_verify` runs a step."""

    def __init__(self, batch: int, parent, vocab: int, dtype: torch.dtype, n_shards: int, shard: int, device="cuda"):
        self.lib = load_library()
        self.parent = np.ascontiguousarray(parent, dtype=np.int32)
        self.device = torch.device(device)
        self.batch, self.vocab, self.dtype = int(batch), int(vocab), dtype
        self.n_nodes, self.n_internal = int(self.parent.shape[0]), _n_internal(self.parent)
        self.n_shards, self.shard = int(n_shards), int(shard)
        self.col_begin, self.n_cols, self.eps = mcsd_shard_columns(vocab, dtype, n_shards, shard)
        self.gamma = mcsd_tree_depth(self.parent)
        rounds = self.lib.mcsd_shard_rounds(self.parent.ctypes.data, self.n_nodes)
        _check(rounds if rounds < 0 else 0)
        self.rounds = rounds
        d = self.desc = McsdShardDesc()
        d.batch, d.n_nodes, d.n_internal, d.vocab = self.batch, self.n_nodes, self.n_internal, self.vocab
        d.dtype, d.n_shards, d.shard = MCSD_DTYPE[dtype], self.n_shards, self.shard
        d.ld_target = d.ld_draft = max(self.n_cols, 1)
        ws = int(self.lib.mcsd_shard_workspace_bytes(ctypes.byref(d)))
        if ws == 0:
            _check(-2)
        self.workspace = torch.zeros(ws + 256, dtype=torch.uint8, device=self.device)
        d.workspace = (self.workspace.data_ptr() + 255) // 256 * 256
        d.workspace_bytes = ws
        n_items = self.batch * self.n_nodes
        f32 = dict(dtype=torch.float32, device=self.device)
        i32 = dict(dtype=torch.int32, device=self.device)
        # exchanged buffers: this shard's part, and what the collective gathers from all shards
        self.part = torch.zeros((n_items, self.eps, 4), **f32)
        self.cval = torch.zeros((n_items, 2), **f32)
        self.totals = torch.zeros((self.batch, self.eps), dtype=torch.float64, device=self.device)
        self.stats_all = torch.zeros((self.n_shards, n_items, self.eps, 4), **f32)
        self.part_all = torch.zeros((self.n_shards, n_items, self.eps, 4), **f32)
        self.cval_all = torch.zeros((self.n_shards, n_items, 2), **f32)
        self.totals_all = torch.zeros((self.n_shards, self.batch, self.eps), dtype=torch.float64, device=self.device)
        self.endpoint_part = torch.full((self.batch,), -1, **i32)
        self.accept_len = torch.empty(self.batch, **i32)
        self.tokens = torch.empty((self.batch, self.gamma + 1), **i32)
        self.status = torch.zeros(self.batch, **i32)
        self.path_nodes = torch.empty((self.batch, self.gamma + 1), **i32)
        self.residual = torch.zeros((self.batch, max(self.n_cols, 1)), **f32)
        self.node_accept = torch.full((self.batch, self.n_nodes), -1, **i32)
        d.node_accept = self.node_accept.data_ptr()

    def _bind(self, target, draft):
        if self.n_cols:
            assert target.dtype == self.dtype and target.shape == (self.batch, self.n_nodes, self.n_cols)
            self.desc.ld_target = _row_stride(target)
            if self.n_internal:
                assert draft.shape == (self.batch, self.n_internal, self.n_cols)
                self.desc.ld_draft = _row_stride(draft)
        self.desc.stream = torch.cuda.current_stream(self.device).cuda_stream

    def mcsd_shard_partials(self, target, draft, cand, temperature: float, rnd: int):
        self._bind(target, draft)
        _check(self.lib.mcsd_shard_partials(ctypes.byref(self.desc), _ptr(target), _ptr(draft), self.parent.ctypes.data,
                                            _ptr(cand), float(temperature), int(rnd), _ptr(self.part), _ptr(self.cval)))

    def mcsd_shard_decide(self, cand, unif, temperature: float, mode: int, rnd: int):
        self.desc.stream = torch.cuda.current_stream(self.device).cuda_stream
        gathered = self.stats_all if rnd == 0 else self.part_all
        _check(self.lib.mcsd_shard_decide(ctypes.byref(self.desc), self.parent.ctypes.data, _ptr(cand), _ptr(unif),
                                          float(temperature), int(mode), int(rnd), _ptr(gathered), _ptr(self.cval_all)))

    def mcsd_shard_endpoint(self, target, draft, temperature: float, attempt: int):
        self._bind(target, draft)
        _check(self.lib.mcsd_shard_endpoint(ctypes.byref(self.desc), _ptr(target), _ptr(draft), self.parent.ctypes.data,
                                            float(temperature), int(attempt), _ptr(self.stats_all), _ptr(self.totals),
                                            _ptr(self.residual)))

    def mcsd_shard_finish(self, target, draft, cand, unif, temperature: float, attempt: int):
        self._bind(target, draft)
        _check(self.lib.mcsd_shard_finish(ctypes.byref(self.desc), _ptr(target), _ptr(draft), self.parent.ctypes.data,
                                          _ptr(cand), _ptr(unif), float(temperature), int(attempt), _ptr(self.stats_all),
                                          _ptr(self.totals_all), _ptr(self.accept_len), _ptr(self.tokens),
                                          _ptr(self.status), _ptr(self.path_nodes), _ptr(self.endpoint_part),
                                          _ptr(self.residual)))


    def mcsd_shard_commit(self):
        self.desc.stream = torch.cuda.current_stream(self.device).cuda_stream
        _check(self.lib.mcsd_shard_commit(ctypes.byref(self.desc), self.parent.ctypes.data, _ptr(self.endpoint_part),
                                          _ptr(self.accept_len), _ptr(self.tokens)))


class DistComm:
    """The collectives of a step over torch.distributed (NCCL between GPUs): all-gathers of a few
    floats per node and one maximum of an int32 per sequence.  No logit crosses devices."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group

    def all_gather(self, shards, name_local: str, name_all: str):
        (sh,) = shards
        self.dist.all_gather_into_tensor(getattr(sh, name_all).view(-1), getattr(sh, name_local).contiguous().view(-1),
                                         group=self.group)

    def all_reduce_max(self, shards, name: str):
        (sh,) = shards
        self.dist.all_reduce(getattr(sh, name), op=self.dist.ReduceOp.MAX, group=self.group)


class LocalComm:
    """The same collectives between shard objects that live in one process (several shards on one
    device, for tests): plain copies."""

    def all_gather(self, shards, name_local: str, name_all: str):
        for dst in shards:
            for src in shards:
                getattr(dst, name_all)[src.shard].copy_(getattr(src, name_local))

    def all_reduce_max(self, shards, name: str):
        best = torch.stack([getattr(sh, name) for sh in shards]).max(dim=0).values
        for sh in shards:
            getattr(sh, name).copy_(best)


def sharded_verify(shards, targets, drafts, cand, unif, temperature: float, mode: int, comm) -> VerifyOutput:
    """One verification step over column-split logits, following the call sequence of mcsd.h.
    shards: the ShardedVerifier objects this process drives (one per rank under torch.distributed; all of
    them when several shards are emulated on one device), targets / drafts: their column slices, in the
    same order; cand, unif: replicated inputs.  Returns the outputs of the first shard; its `residual`
    holds that shard's columns of the distribution."""
    T = float(temperature)
    for sh, t, d in zip(shards, targets, drafts):
        sh.mcsd_shard_partials(t, d, cand, T, 0)
    comm.all_gather(shards, "part", "stats_all")
    comm.all_gather(shards, "cval", "cval_all")
    for sh in shards:
        sh.mcsd_shard_decide(cand, unif, T, mode, 0)
    for rnd in range(1, shards[0].rounds + 1):
        for sh, t, d in zip(shards, targets, drafts):
            sh.mcsd_shard_partials(t, d, cand, T, rnd)
        comm.all_gather(shards, "part", "part_all")
        for sh in shards:
            sh.mcsd_shard_decide(cand, unif, T, mode, rnd)
    for attempt in (0, 1):
        for sh, t, d in zip(shards, targets, drafts):
            sh.mcsd_shard_endpoint(t, d, T, attempt)
        comm.all_gather(shards, "totals", "totals_all")
        for sh, t, d in zip(shards, targets, drafts):
            sh.mcsd_shard_finish(t, d, cand, unif, T, attempt)
    comm.all_reduce_max(shards, "endpoint_part")
    for sh in shards:
        sh.mcsd_shard_commit()
    sh = shards[0]
    return VerifyOutput(sh.accept_len, sh.tokens, sh.residual, sh.status, node_accept=sh.node_accept,
                        path_nodes=sh.path_nodes)
