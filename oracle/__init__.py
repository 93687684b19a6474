"""ctypes front end of the CPU oracle (``mcsd_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the tests, the smoke check and the
CPU-baseline legs of the bench may import this package; the CUDA library and its
Python binding never do.  Nothing here imports the CUDA package either.

The C file is compiled with gcc on first use (or by :func:`build`) into
``libmcsd_oracle.so`` beside it.  Arrays are numpy; logits are float32 arrays that
hold the exact dtype-rounded values and are widened to double inside the C code.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mcsd_oracle.c")
_LIB = os.path.join(_HERE, "libmcsd_oracle.so")

STATUS_DEGENERATE = 1
STATUS_BAD_TOKEN = 2
STATUS_NO_MASS = 4

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over sequences). Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _bind(lib):
    """Declare the C signatures on a loaded library handle."""
    c_i32, c_dbl = ctypes.c_int32, ctypes.c_double
    P = ctypes.c_void_p
    lib.mcsd_oracle_num_threads.restype = c_i32
    lib.mcsd_oracle_softmax.argtypes = [P, c_i32, c_dbl, P]
    lib.mcsd_oracle_softmax.restype = None
    lib.mcsd_oracle_argmax.argtypes = [P, c_i32]
    lib.mcsd_oracle_argmax.restype = c_i32
    lib.mcsd_oracle_invcdf.argtypes = [P, c_i32, c_dbl]
    lib.mcsd_oracle_invcdf.restype = c_i32
    lib.mcsd_oracle_mcss.argtypes = [P, P, c_i32, P, P, c_i32, c_i32, P, P, P]
    lib.mcsd_oracle_mcss.restype = c_i32
    lib.mcsd_oracle_draw.argtypes = [P, c_i32, P, c_i32, c_i32, P]
    lib.mcsd_oracle_draw.restype = c_i32
    lib.mcsd_oracle_topk.argtypes = [P, c_i32, c_i32, P]
    lib.mcsd_oracle_topk.restype = None
    lib.mcsd_oracle_sample.argtypes = [c_i32, c_i32, c_i32, c_i32, P, P, P, c_dbl, c_i32, c_i32, c_i32, P]
    lib.mcsd_oracle_sample.restype = c_i32
    lib.mcsd_oracle_verify.argtypes = [c_i32, c_i32, c_i32, c_i32, P, P, P, P, P, c_dbl, c_i32,
                                       c_i32, P, P, P, P, P, P, P]
    lib.mcsd_oracle_verify.restype = c_i32
    return lib


def _load():
    global _lib
    if _lib is None:
        _lib = _bind(ctypes.CDLL(build()))
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(_load().mcsd_oracle_num_threads())


def softmax(logits, T: float) -> np.ndarray:
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    out = np.empty(logits.shape[0], dtype=np.float64)
    _load().mcsd_oracle_softmax(_ptr(logits), logits.shape[0], float(T), _ptr(out))
    return out


def argmax(logits) -> int:
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    return int(_load().mcsd_oracle_argmax(_ptr(logits), logits.shape[0]))


def invcdf(P, u: float) -> int:
    P = np.ascontiguousarray(P, dtype=np.float64)
    return int(_load().mcsd_oracle_invcdf(_ptr(P), P.shape[0], float(u)))


def draw(q, u, mode: int) -> np.ndarray:
    """k draws from q by inverse CDF with the uniforms u: with replacement (mode 0) or without,
    Eq. 1 (mode 1).  Returns the k tokens (-1 where no mass was left)."""
    q = np.array(q, dtype=np.float64, copy=True)
    u = np.ascontiguousarray(u, dtype=np.float64)
    x = np.empty(u.shape[0], dtype=np.int32)
    _load().mcsd_oracle_draw(_ptr(q), q.shape[0], _ptr(u), u.shape[0], int(mode), _ptr(x))
    return x


def topk(logits, k: int) -> np.ndarray:
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    x = np.empty(k, dtype=np.int32)
    _load().mcsd_oracle_topk(_ptr(logits), logits.shape[0], int(k), _ptr(x))
    return x


def sample(draft, parent, unif_draw, T: float, mode: int, node_begin: int = 0, node_end=None, cand=None) -> np.ndarray:
    """Candidate tokens of the children of the nodes [node_begin, node_end) of every tree; see
    ``mcsd_oracle_sample``.  Returns cand [B, n_nodes] (entries outside the range keep -1 / their input)."""
    draft = np.ascontiguousarray(draft, dtype=np.float32)
    B, n_internal, V = draft.shape
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    n_nodes = parent.shape[0]
    unif_draw = np.ascontiguousarray(unif_draw, dtype=np.float32)
    assert unif_draw.shape == (B, n_nodes)
    node_end = n_internal if node_end is None else node_end
    out = np.full((B, n_nodes), -1, dtype=np.int32) if cand is None else np.ascontiguousarray(cand, dtype=np.int32)
    rc = _load().mcsd_oracle_sample(B, n_nodes, n_internal, V, _ptr(draft), _ptr(parent), _ptr(unif_draw),
                                    float(T), int(mode), int(node_begin), int(node_end), _ptr(out))
    if rc != 0:
        raise ValueError(f"mcsd_oracle_sample rejected its arguments (code {rc})")
    return out


@dataclass
class McssResult:
    accepted: int          # index in [0, k) or -1
    p: np.ndarray          # p when the loop ended (final residual if accepted == -1)
    q: np.ndarray          # q when the loop ended
    ratio: np.ndarray      # p(x~)/q(x~) seen by each test; -1 forced reject; NaN not reached
    S: np.ndarray          # residual normaliser after each rejection; NaN not reached
    status: int


def mcss(p, q, cand, r, mode: int) -> McssResult:
    """Algorithm 1 (mode 0) / Algorithm 2 (mode 1) at one node, on copies of p and q."""
    p = np.array(p, dtype=np.float64, copy=True)
    q = np.array(q, dtype=np.float64, copy=True)
    cand = np.ascontiguousarray(cand, dtype=np.int32)
    r = np.ascontiguousarray(r, dtype=np.float64)
    k = cand.shape[0]
    assert r.shape[0] == k and p.shape == q.shape
    ratio = np.empty(k, dtype=np.float64)
    S = np.empty(k, dtype=np.float64)
    status = np.zeros(1, dtype=np.int32)
    acc = _load().mcsd_oracle_mcss(_ptr(p), _ptr(q), p.shape[0], _ptr(cand), _ptr(r), k, int(mode),
                                   _ptr(ratio), _ptr(S), _ptr(status))
    return McssResult(int(acc), p, q, ratio, S, int(status[0]))


@dataclass
class VerifyResult:
    accept_len: np.ndarray   # [B] int32
    tokens: np.ndarray       # [B, gamma+1] int32, -1 padded
    residual: np.ndarray     # [B, V] float64 (None if not requested)
    node_accept: np.ndarray  # [B, n_nodes] int32
    node_bonus: np.ndarray   # [B, n_nodes] int32
    node_ratio: np.ndarray   # [B, n_nodes] float64
    status: np.ndarray       # [B] int32


def tree_gamma(parent) -> int:
    parent = np.asarray(parent)
    depth = np.zeros(parent.shape[0], dtype=np.int64)
    for n in range(1, parent.shape[0]):
        depth[n] = depth[parent[n]] + 1
    return int(depth.max()) if parent.shape[0] else 0


def verify(target, draft, parent, cand, unif, T: float, mode: int, *, sequential: bool = False,
           want_residual: bool = True) -> VerifyResult:
    """Whole verification step; see ``mcsd_oracle_verify`` in the C file for the layout."""
    target = np.ascontiguousarray(target, dtype=np.float32)
    B, n_nodes, V = target.shape
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    assert parent.shape == (n_nodes,)
    has_child = np.zeros(n_nodes, dtype=bool)
    has_child[parent[1:]] = True
    n_internal = int(has_child.sum())
    if draft is not None:
        draft = np.ascontiguousarray(draft, dtype=np.float32)
        assert draft.shape == (B, n_internal, V), (draft.shape, (B, n_internal, V))
    cand = np.ascontiguousarray(cand, dtype=np.int32)
    unif = np.ascontiguousarray(unif, dtype=np.float32)
    assert cand.shape == (B, n_nodes) and unif.shape == (B, n_nodes, 2)
    gamma = tree_gamma(parent)
    accept_len = np.empty(B, dtype=np.int32)
    tokens = np.empty((B, gamma + 1), dtype=np.int32)
    residual = np.empty((B, V), dtype=np.float64) if want_residual else None
    node_accept = np.empty((B, n_nodes), dtype=np.int32)
    node_bonus = np.empty((B, n_nodes), dtype=np.int32)
    node_ratio = np.empty((B, n_nodes), dtype=np.float64)
    status = np.zeros(B, dtype=np.int32)
    rc = _load().mcsd_oracle_verify(B, n_nodes, n_internal, V, _ptr(target), _ptr(draft), _ptr(parent),
                                    _ptr(cand), _ptr(unif), float(T), int(mode), int(sequential),
                                    _ptr(accept_len), _ptr(tokens), _ptr(residual), _ptr(node_accept),
                                    _ptr(node_bonus), _ptr(node_ratio), _ptr(status))
    if rc != 0:
        raise ValueError(f"mcsd_oracle_verify rejected its arguments (code {rc})")
    return VerifyResult(accept_len, tokens, residual, node_accept, node_bonus, node_ratio, status)


def tree_attention_layout(parent, prefix_len: int):
    """Section 3.3 written out: mask[i][j] = 1 iff j is i or an ancestor of i (the reflexive and
    transitive closure of the parent relation, by following parents), position id = prefix_len +
    depth.  Returns (mask uint8 [n, n], position_ids int32 [n])."""
    parent = np.asarray(parent, dtype=np.int64)
    n = parent.shape[0]
    mask = np.zeros((n, n), dtype=np.uint8)
    pos = np.zeros(n, dtype=np.int32)
    for i in range(n):
        a, depth = i, 0
        while a >= 0:
            mask[i, a] = 1
            a = int(parent[a])
            if a >= 0:
                depth += 1
        pos[i] = prefix_len + depth
    return mask, pos


def path_nodes(result: "VerifyResult", gamma: int) -> np.ndarray:
    """Tree nodes of the accepted tokens of every sequence, -1 padded to gamma + 1 columns: the walk
    of Section 3 followed through node_accept."""
    B = result.accept_len.shape[0]
    out = np.full((B, gamma + 1), -1, dtype=np.int32)
    for b in range(B):
        n, i = 0, 0
        while result.node_accept[b, n] >= 0:
            n = int(result.node_accept[b, n])
            out[b, i] = n
            i += 1
    return out


def gather_accepted_kv(cache, prefix_len, path_nodes, accept_len) -> np.ndarray:
    """What stays of the target model's key/value cache after verification (Sections 3 and 3.3).
    The tree was fed as one flattened sequence, node n at position prefix_len[b] + n, so the cache
    holds one row per tree node; the i-th accepted token (node path_nodes[b][i], depth i + 1) belongs
    at position prefix_len[b] + 1 + i of the committed sequence.  cache: [S][B][L][R] (S independent
    slabs: layers, keys and values, heads).  Returns a copy with those rows moved there; every other
    row is as it was."""
    cache = np.asarray(cache)
    out = cache.copy()
    S, B = cache.shape[0], cache.shape[1]
    for s in range(S):
        for b in range(B):
            for i in range(int(accept_len[b])):
                out[s, b, int(prefix_len[b]) + 1 + i] = cache[s, b, int(prefix_len[b]) + int(path_nodes[b][i])]
    return out
