"""Comparison rules between the CPU oracle and another implementation's outputs.

TEST INFRASTRUCTURE (same standing as the oracle itself).  Works on numpy arrays
only; imports nothing from the CUDA package.

Rules
  * Acceptance decisions are compared node by node and must be identical, except
    that a node whose first differing test has |u - rho_oracle| < NEAR_TIE is
    counted as a flipped near-tie and the rest of that node is skipped.
  * Every test the oracle performed with |u - rho| < NEAR_TIE is counted as a
    near-tie decision; these must stay below NEAR_TIE_SHARE of all decisions (small
    samples: at most NEAR_TIE_MIN_EVENTS events).
  * A sequence whose oracle path crosses a flipped node is excluded from the path
    and residual comparison (and counted); its outputs must still be a valid walk of the
    tree.  All other sequences must have the same accepted length and accepted tokens.
  * Endpoint tokens are draws by inverse CDF; a different token is tolerated only
    if it has positive oracle probability and u lies within NEAR_TIE (in CDF
    units) of that token's oracle CDF interval.  Such cases are counted.
  * Residual distributions agree within `residual_tol` max abs error (not compared where the
    oracle reports NO_MASS: there is no distribution then, its entries are NaN).
  * Status words describe the walk: they are compared with those of the oracle's sequential
    form (the nodes the procedure of Section 3 evaluates), bit for bit.
  * Tolerated endpoint draws are bounded: their count may not exceed BOUNDARY_DRAW_LIMIT(V, draws)
    (three times the expected number of draws whose uniform falls within float rounding of one of
    the V interval boundaries, at least 3 events).
  * Naive sampling (mode 2): every emitted token is such a draw; the first differing token of a
    sequence is judged by the endpoint rule and the rest of that sequence is skipped.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

from . import verify as oracle_verify, softmax as oracle_softmax, mcss as oracle_mcss

NEAR_TIE = 1e-5
NEAR_TIE_SHARE = 1e-4
# The share is a rate: on a sample of a few hundred tests one single event already exceeds
# 0.01 %, which says nothing about the rate (uniforms on a 2^-23 grid put about 2e-5 of all
# tests inside the band by chance alone).  Up to this many events are always allowed.
NEAR_TIE_MIN_EVENTS = 3
RESIDUAL_TOL = {"fp32": 1e-5, "bf16": 2e-3, "fp16": 2e-3}
STATUS_NO_MASS = 4


def boundary_draw_limit(vocab: int, draws: int) -> float:
    """Most inverse-CDF draws that may land on the other side of an interval boundary.  A float32
    evaluation places each of the V boundaries within about 1e-7 (CDF units) of its exact position,
    so a draw differs with probability about 2e-7 * V; three times that expectation is allowed,
    and never fewer than 3 events."""
    return max(3.0, 3 * 2e-7 * vocab * draws)


@dataclass
class ParityReport:
    n_sequences: int = 0
    n_tests: int = 0                 # acceptance tests the oracle performed (all nodes)
    n_near_tie: int = 0              # of those, |u - rho| < NEAR_TIE
    n_flipped: int = 0               # nodes whose decision differs inside the near-tie band
    n_excluded_sequences: int = 0    # sequences whose oracle path crosses a flipped node
    n_bonus_tolerated: int = 0       # endpoint tokens that differ within the CDF tolerance
    n_bonus_draws: int = 0           # endpoint draws that were compared
    n_nodes_compared: int = 0
    excluded: List[int] = field(default_factory=list)   # sequences left out of the path comparison
    max_residual_err: float = 0.0
    failures: List[str] = field(default_factory=list)

    @property
    def ok(self) -> bool:
        return not self.failures

    def summary(self) -> dict:
        return {"sequences": self.n_sequences, "tests": self.n_tests, "near_ties": self.n_near_tie,
                "flipped": self.n_flipped, "excluded_sequences": self.n_excluded_sequences,
                "bonus_tolerated": self.n_bonus_tolerated, "bonus_draws": self.n_bonus_draws,
                "max_residual_err": self.max_residual_err,
                "failures": len(self.failures)}


def _children(parent):
    n = parent.shape[0]
    first = np.full(n, -1, dtype=np.int64)
    count = np.zeros(n, dtype=np.int64)
    for c in range(1, n):
        p = parent[c]
        if count[p] == 0:
            first[p] = c
        count[p] += 1
    return first, count


def _bonus_tolerated(P: np.ndarray, g: int, u: float) -> bool:
    if g < 0 or g >= P.shape[0] or not (P[g] > 0):
        return False
    cdf = np.cumsum(P) / P.sum()
    lo = cdf[g - 1] if g > 0 else 0.0
    return lo - NEAR_TIE <= u <= cdf[g] + NEAR_TIE


def _node_residual(target_b, draft_b, parent, cand_b, unif_b, n, first, count, T, mode):
    """Oracle residual of a single node (only used to judge a differing endpoint token)."""
    p = oracle_softmax(target_b[n], T)
    k = int(count[n])
    if k == 0:
        return p
    q = oracle_softmax(draft_b[n], T)
    ch = np.arange(first[n], first[n] + k)
    r = oracle_mcss(p, q, cand_b[ch], unif_b[ch, 0].astype(np.float64), mode)
    return r.p


def compare(target, draft, parent, cand, unif, T: float, mode: int, dtype_name: str, *,
            accept_len, tokens, residual=None, node_accept=None, node_bonus=None, status=None,
            path_nodes=None, oracle_result=None, max_failures: int = 20) -> ParityReport:
    """target/draft: float32 numpy (exact widening of the rounded logits); the keyword arrays are
    the outputs under test (numpy).  path_nodes (tree nodes of the accepted tokens, -1 padded), when
    given, is compared too and lets a diverging walk be traced to the test where it diverged."""
    parent = np.asarray(parent, dtype=np.int32)
    ref = oracle_result if oracle_result is not None else oracle_verify(
        target, draft if T > 0 else None, parent, cand, unif, T, mode)
    B, n_nodes = cand.shape
    V = target.shape[-1]
    first, count = _children(parent)
    rep = ParityReport(n_sequences=B)
    # the status words describe the walk: the oracle's sequential form evaluates exactly those nodes
    ref_status = None
    if status is not None:
        ref_status = oracle_verify(target, draft if T > 0 else None, parent, cand, unif, T, mode,
                                   sequential=True, want_residual=False).status
    tol = RESIDUAL_TOL[dtype_name]

    def fail(msg):
        if len(rep.failures) < max_failures:
            rep.failures.append(msg)

    # decisions the oracle made, and how many sat inside the near-tie band
    tested = ~np.isnan(ref.node_ratio)
    tested[:, 0] = False
    rep.n_tests = int(tested.sum())
    if T > 0:
        u0 = unif[:, :, 0].astype(np.float64)
        near = tested & (ref.node_ratio >= 0) & (np.abs(u0 - ref.node_ratio) < NEAR_TIE)
        rep.n_near_tie = int(near.sum())
        if rep.n_near_tie > max(NEAR_TIE_MIN_EVENTS, NEAR_TIE_SHARE * rep.n_tests):
            fail(f"{rep.n_near_tie} near-tie decisions out of {rep.n_tests} exceed the allowed share")

    flipped = np.zeros((B, n_nodes), dtype=bool)
    if node_accept is not None:
        diff = np.argwhere(node_accept != ref.node_accept)
        for b, n in diff:
            ao, ag = int(ref.node_accept[b, n]), int(node_accept[b, n])
            cands = [c for c in (ao, ag) if c >= 0]
            i_star = min(cands)
            in_range = first[n] <= i_star < first[n] + count[n]
            rho = ref.node_ratio[b, i_star] if in_range else np.nan
            u = float(unif[b, i_star, 0]) if in_range else np.nan
            if T > 0 and in_range and rho >= 0 and abs(u - rho) < NEAR_TIE:
                flipped[b, n] = True
            else:
                fail(f"seq {b} node {n}: accepted child {ag}, oracle {ao} (u={u}, rho={rho})")
        rep.n_flipped = int(flipped.sum())
        rep.n_nodes_compared = B * n_nodes

    if node_bonus is not None:
        both_stop = (ref.node_accept < 0) & ~flipped
        if node_accept is not None:
            both_stop &= node_accept < 0
        rep.n_bonus_draws += int(both_stop.sum()) if T > 0 else 0
        diff = np.argwhere(both_stop & (node_bonus != ref.node_bonus))
        for b, n in diff:
            g = int(node_bonus[b, n])
            okk = False
            if T > 0:
                P = _node_residual(target[b], None if draft is None else draft[b], parent, cand[b], unif[b], n,
                                   first, count, T, mode)
                okk = _bonus_tolerated(P, g, float(unif[b, n, 1]))
            if okk:
                rep.n_bonus_tolerated += 1
            else:
                fail(f"seq {b} node {n}: endpoint token {g}, oracle {int(ref.node_bonus[b, n])}")
        acc_nodes = (ref.node_accept >= 0) & ~flipped
        if node_accept is not None:
            acc_nodes &= node_accept >= 0
        bad = np.argwhere(acc_nodes & (node_bonus != -1))
        for b, n in bad[:max_failures]:
            fail(f"seq {b} node {n}: endpoint token set on a node that accepted a candidate")

    # sequence level
    for b in range(B):
        n, path_flipped = 0, bool(flipped[b, 0])
        while ref.node_accept[b, n] >= 0:
            n = int(ref.node_accept[b, n])
            path_flipped |= bool(flipped[b, n])
        if path_flipped:
            rep.n_excluded_sequences += 1
            rep.excluded.append(b)
            continue
        L = int(ref.accept_len[b])
        if path_nodes is not None and T > 0 and mode != 2:
            # where does the walk under test leave the oracle's?  At that node both evaluated the same
            # tests in the same order; the first test whose outcome differs decides
            po, nn = [], 0
            while ref.node_accept[b, nn] >= 0:
                nn = int(ref.node_accept[b, nn])
                po.append(nn)
            pg = [int(x) for x in path_nodes[b] if x >= 0]
            if po != pg:
                i = 0
                while i < min(len(po), len(pg)) and po[i] == pg[i]:
                    i += 1
                ends = [c for c in ((po[i] if i < len(po) else -1), (pg[i] if i < len(pg) else -1)) if c >= 0]
                i_star = min(ends)
                rho, u = ref.node_ratio[b, i_star], float(unif[b, i_star, 0])
                if rho >= 0 and abs(u - rho) < NEAR_TIE:
                    rep.n_flipped += 1
                    rep.n_excluded_sequences += 1
                    rep.excluded.append(b)
                else:
                    fail(f"seq {b}: path {pg}, oracle {po} (u={u}, rho={rho} at node {i_star})")
                continue
        if mode == 2 and T > 0 and not np.array_equal(tokens[b], ref.tokens[b]):
            # naive sampling: every emitted token is itself a draw by inverse CDF.  At the first
            # position where the token sequences differ, the other token passes under the same
            # rule as an endpoint token; what follows depends on it and is not compared.
            i = int(np.argmax(tokens[b] != ref.tokens[b]))
            node = 0
            for _ in range(i):
                node = int(ref.node_accept[b, node])
            if node >= 0 and _bonus_tolerated(oracle_softmax(target[b, node], T), int(tokens[b, i]),
                                              float(unif[b, node, 1])):
                rep.n_bonus_tolerated += 1
                rep.n_excluded_sequences += 1
                rep.excluded.append(b)
            else:
                fail(f"seq {b}: tokens {tokens[b].tolist()}, oracle {ref.tokens[b].tolist()}")
            continue
        if int(accept_len[b]) != L:
            fail(f"seq {b}: accepted length {int(accept_len[b])}, oracle {L}")
            continue
        if not np.array_equal(tokens[b, :L], ref.tokens[b, :L]):
            fail(f"seq {b}: accepted tokens {tokens[b, :L].tolist()}, oracle {ref.tokens[b, :L].tolist()}")
            continue
        if not (tokens[b, L + 1:] == -1).all():
            fail(f"seq {b}: padding after the endpoint token is not -1")
        g, o = int(tokens[b, L]), int(ref.tokens[b, L])
        if T > 0 and node_bonus is None:
            rep.n_bonus_draws += (L + 1) if mode == 2 else 1
        if g != o:
            if T > 0 and _bonus_tolerated(ref.residual[b], g, float(unif[b, n, 1])):
                if node_bonus is None:
                    rep.n_bonus_tolerated += 1
            else:
                fail(f"seq {b}: endpoint token {g}, oracle {o}")
        if residual is not None and not (int(ref.status[b]) & STATUS_NO_MASS):
            err = float(np.abs(residual[b].astype(np.float64) - ref.residual[b]).max())
            rep.max_residual_err = max(rep.max_residual_err, err)
            if not err <= tol:
                fail(f"seq {b}: residual max abs error {err:.3e} > {tol:.1e}")
        if status is not None and int(status[b]) != int(ref_status[b]):
            fail(f"seq {b}: status {int(status[b])}, oracle (sequential form) {int(ref_status[b])}")
    # A sequence left out above took the other branch of a near-tie: its outputs are not the oracle's,
    # but they still have to be a walk of this tree — a length within the depth, -1 padding, and, where
    # the nodes of the walk are reported, a chain of children from the root carrying the emitted tokens.
    gamma_p1 = tokens.shape[1]
    for b in rep.excluded:
        Lg = int(accept_len[b])
        if not 0 <= Lg < gamma_p1:
            fail(f"seq {b} (near-tie branch): accepted length {Lg} outside [0, {gamma_p1 - 1}]")
            continue
        if not (tokens[b, Lg + 1:] == -1).all():
            fail(f"seq {b} (near-tie branch): padding after the endpoint token is not -1")
        if path_nodes is not None:
            pg = [int(x) for x in path_nodes[b, :Lg]]
            prev = 0
            for i, node in enumerate(pg):
                if not (0 < node < n_nodes) or int(parent[node]) != prev or int(tokens[b, i]) != int(cand[b, node]):
                    fail(f"seq {b} (near-tie branch): accepted path {pg} is not a walk of the tree carrying its tokens")
                    break
                prev = node
    if rep.n_bonus_tolerated > boundary_draw_limit(V, max(rep.n_bonus_draws, 1)):
        fail(f"{rep.n_bonus_tolerated} of {rep.n_bonus_draws} endpoint draws differ inside the tolerance: "
             f"more than the {boundary_draw_limit(V, max(rep.n_bonus_draws, 1)):.1f} float rounding explains")
    return rep


@dataclass
class SampleReport:
    n_draws: int = 0
    n_tolerated: int = 0      # first differing draw of a node lies within NEAR_TIE of a CDF boundary
    failures: List[str] = field(default_factory=list)

    @property
    def ok(self) -> bool:
        return not self.failures


def compare_samples(draft, parent, unif_draw, T: float, mode: int, cand, node_begin: int = 0, node_end=None,
                    max_failures: int = 20) -> SampleReport:
    """Candidate tokens drawn by another implementation against the oracle's (Section 3.2, Eq. 1).
    Tokens must be identical, except that at the first differing draw of a node the other token is
    accepted if it has positive probability under the distribution of that draw and the uniform lies
    within NEAR_TIE (CDF units) of its interval; the later draws of that node (which depend on the
    earlier ones when drawing without replacement) are then not compared.  Temperature 0: exact."""
    from . import sample as oracle_sample
    parent = np.asarray(parent, dtype=np.int32)
    B, n_internal, V = draft.shape
    node_end = n_internal if node_end is None else node_end
    ref = oracle_sample(draft, parent, unif_draw, T, mode, node_begin, node_end)
    first, count = _children(parent)
    rep = SampleReport()
    for b in range(B):
        for n in range(node_begin, node_end):
            ch = np.arange(first[n], first[n] + count[n])
            rep.n_draws += len(ch)
            if np.array_equal(cand[b, ch], ref[b, ch]):
                continue
            i = int(np.argmax(cand[b, ch] != ref[b, ch]))
            g, okk = int(cand[b, ch[i]]), False
            if T > 0:
                q = oracle_softmax(draft[b, n], T)
                if mode == 1:
                    q[ref[b, ch[:i]]] = 0.0      # the tokens drawn before (identical on both sides)
                okk = _bonus_tolerated(q, g, float(unif_draw[b, ch[i]]))
            if okk:
                rep.n_tolerated += 1
            elif len(rep.failures) < max_failures:
                rep.failures.append(f"seq {b} node {n} draw {i}: token {g}, oracle {int(ref[b, ch[i]])}")
    if T > 0 and rep.n_tolerated > boundary_draw_limit(V, max(rep.n_draws, 1)):
        rep.failures.append(f"{rep.n_tolerated} of {rep.n_draws} draws differ inside the tolerance: more than the "
                            f"{boundary_draw_limit(V, max(rep.n_draws, 1)):.1f} float rounding explains")
    return rep
