"""TEST INFRASTRUCTURE — the CPU oracle of the PSD hot path.

Only ``tests/``, the smoke check and the benchmark's ``cpu_baseline`` / reference leg may
import this package.  It shares no code with the CUDA path and must never serve as a
fallback for it.  It is deliberately plain and slow: every function is the paper's
definition (or, where the paper is silent, the stated reading of it) written out in
fp64 / exact integers so that it can be checked against the paper by eye.

Contents
  confidence, logits        Sec. 3.1: x^_i = argmax_v p(v), c_i = max_v p(v)   (psd_oracle.c)
  select_unmask             Sec. 3.2 Stage 1, Eq. (1); threshold policy of App. B.2
  build_drafts              Sec. 3.2 Stage 2, Eq. (2); Algorithm 1 "Stage 2"
  verify_accept             Sec. 3.2 Stage 3; Algorithm 1 "Stage 3"
  build_drafts_dag, verify_accept_dag   the same two stages for a general multi-parent draft graph
  decode_block              Algorithm 1, the whole loop over one block
  decode_block_one_pass     the same loop with one model call per iteration (the verification
                            pass doubles as the next iteration's pass on the state)

Pins: every function above is pinned by ``tests/test_oracle_*.py`` to closed forms,
brute-force enumeration, library routines and the invariants the paper states.  The parts
that are readings of an open point of the paper rather than something it fixes
(how many positions each depth adds, the chain shape of the draft graph, the exact form
of the acceptance criterion A_pi, what the extra commit of Algorithm 1's last step
checks) are parameters here; they are "parity unpinned" in the sense that nothing in the
paper can confirm the reading, although each offered mode is pinned to its own definition.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "psd_oracle.c")
_LIB = os.path.join(_HERE, "libpsd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile psd_oracle.c into libpsd_oracle.so next to it (no-op when up to date)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i64, vp = ctypes.c_int64, ctypes.c_void_p
        lib.psd_oracle_threads.restype = ctypes.c_int
        lib.psd_oracle_logits.restype = ctypes.c_int
        lib.psd_oracle_logits.argtypes = [vp, vp, i64, i64, i64, vp]
        lib.psd_oracle_row_stats.restype = None
        lib.psd_oracle_row_stats.argtypes = [vp, i64, vp, vp, vp, vp]
        lib.psd_oracle_confidence.restype = ctypes.c_int
        lib.psd_oracle_confidence.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp, vp]
        _lib = lib
    return _lib


def threads() -> int:
    """Number of host threads the confidence oracle uses."""
    return int(_load().psd_oracle_threads())


def _u16(a, name):
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16 or a.ndim != 2:
        raise ValueError(f"{name} must be a 2-D uint16 array of bf16 bit patterns")
    return a


def logits(hidden_bits, w_bits) -> np.ndarray:
    """``l[r, v] = sum_j hidden[r, j] W[v, j]`` in fp64, summed in index order (Sec. 3.1)."""
    h, w = _u16(hidden_bits, "hidden"), _u16(w_bits, "W")
    if h.shape[1] != w.shape[1]:
        raise ValueError("hidden and W disagree on H")
    out = np.empty((h.shape[0], w.shape[0]), dtype=np.float64)
    if _load().psd_oracle_logits(h.ctypes.data, w.ctypes.data, h.shape[0], h.shape[1], w.shape[0],
                                 out.ctypes.data):
        raise MemoryError("psd_oracle_logits")
    return out


def row_stats(logit_row):
    """(token, conf, lse, gap) of one row of fp64 logits: the softmax-max definition of Sec. 3.1."""
    l = np.ascontiguousarray(logit_row, dtype=np.float64)
    tok = ctypes.c_int32()
    conf, lse, gap = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    _load().psd_oracle_row_stats(l.ctypes.data, l.shape[0], ctypes.byref(tok), ctypes.byref(conf),
                                 ctypes.byref(lse), ctypes.byref(gap))
    return tok.value, conf.value, lse.value, gap.value


def confidence(hidden_bits, w_bits):
    """Per row: (token int32, conf fp64, lse fp64, gap fp64).

    token = argmax_v p(v) (lowest index among equal maxima), conf = max_v p(v) with p the
    softmax of the LM-head logits (Sec. 3.1); lse = log sum_v exp(l_v); gap = top-1 logit minus
    the best logit at any other index (used by tests to set near-ties aside).
    """
    h, w = _u16(hidden_bits, "hidden"), _u16(w_bits, "W")
    if h.shape[1] != w.shape[1]:
        raise ValueError("hidden and W disagree on H")
    n = h.shape[0]
    tok = np.empty(n, dtype=np.int32)
    conf = np.empty(n, dtype=np.float64)
    lse = np.empty(n, dtype=np.float64)
    gap = np.empty(n, dtype=np.float64)
    if _load().psd_oracle_confidence(h.ctypes.data, w.ctypes.data, n, h.shape[1], w.shape[0],
                                     tok.ctypes.data, conf.ctypes.data, lse.ctypes.data, gap.ctypes.data):
        raise MemoryError("psd_oracle_confidence")
    return tok, conf, lse, gap


# --------------------------------------------------------------------------------------
# Policy, drafts, acceptance: exact integer logic on top of given confidences.
# --------------------------------------------------------------------------------------

ACCEPT_AGREE_AND_CONF = 0   # speculated token equals the parent's prediction and that prediction's conf > tau
ACCEPT_AGREE_ONLY = 1       # token agreement alone
ACCEPT_AGREE_AND_POLICY = 2 # agreement, and the policy run on the parent's node would have picked the slot


@dataclass(frozen=True)
class Policy:
    """Parameters of the transfer policy pi and of the draft chain.

    tau      commit / acceptance threshold, strict '>' ("exceeds", App. B.2)
    k_min    at least this many positions per step (progress of Algorithm 1's while loop)
    k_max    at most this many; 0 = no cap
    depth    D = number of chain nodes, root included (the paper's draft depth d is D-1)
    stride   positions each depth adds; 0 = k_min
    accept_mode  which form of the acceptance criterion A_pi is used (see constants above)
    mask_id  token id of [M]
    """
    tau: float = 0.9
    k_min: int = 1
    k_max: int = 0
    depth: int = 1
    stride: int = 0
    accept_mode: int = ACCEPT_AGREE_AND_CONF
    mask_id: int = -1

    def check(self):
        if self.k_min < 1 or (self.k_max != 0 and self.k_max < self.k_min) or self.depth < 1 \
                or self.stride < 0 or self.accept_mode not in (0, 1, 2) or math.isnan(self.tau):
            raise ValueError(f"bad policy {self}")

    @property
    def step(self) -> int:
        return self.stride if self.stride > 0 else self.k_min


def _rank_key(conf_row, i):
    """Descending confidence, then ascending slot; NaN ranks below every number."""
    c = float(conf_row[i])
    return (1, 0.0, i) if math.isnan(c) else (0, -c, i)


def policy_count(conf_row, slots, p: Policy) -> int:
    """|T| for the clamped threshold policy: all masked slots whose confidence exceeds tau
    (App. B.2), but at least k_min (so that the loop progresses) and at most k_max."""
    n_thr = sum(1 for i in slots if float(conf_row[i]) > p.tau)
    n = max(n_thr, p.k_min)
    if p.k_max > 0:
        n = min(n, p.k_max)
    return min(n, len(slots))


def policy_set(conf_row, mask_row, p: Policy):
    """T = pi(x, c): the policy_count highest-confidence masked slots, in rank order."""
    slots = [i for i in range(len(mask_row)) if mask_row[i] != 0]
    order = sorted(slots, key=lambda i: _rank_key(conf_row, i))
    return order[:policy_count(conf_row, slots, p)]


def select_unmask(conf, tok, tokens, mask, p: Policy):
    """Stage 1 (Sec. 3.2; Algorithm 1, "positions to commit" and the state update, Eq. (1)).

    conf, tok: [B, M] predictions of the node the step starts from; tokens, mask: [B, M] state.
    Returns new (tokens, mask) and sel[B, M] (0/1), n_sel[B], sel_pos[B, M] (slots in rank
    order, -1 padded).
    """
    p.check()
    conf = np.asarray(conf, dtype=np.float64)
    tok = np.asarray(tok)
    tokens = np.array(tokens, dtype=np.int32, copy=True)
    mask = np.array(mask, dtype=np.int32, copy=True)
    B, M = mask.shape
    sel = np.zeros((B, M), dtype=np.int32)
    n_sel = np.zeros(B, dtype=np.int32)
    sel_pos = np.full((B, M), -1, dtype=np.int32)
    for b in range(B):
        T = policy_set(conf[b], mask[b], p)
        n_sel[b] = len(T)
        for r, i in enumerate(T):
            sel[b, i] = 1
            sel_pos[b, r] = i
            tokens[b, i] = tok[b, i]      # Eq. (1): x_i <- x^_i for i in T
            mask[b, i] = 0
    return tokens, mask, sel, n_sel, sel_pos


def build_drafts(conf, tok, tokens, mask, p: Policy):
    """Stage 2 (Sec. 3.2; Algorithm 1 "Stage 2"; Eq. (2)) for a chain of D nodes.

    conf, tok: the cached step-t predictions [B, M]; tokens, mask: the state after Stage 1.
    sigma = still-masked slots by descending step-t confidence; node d fills
    S_d = {sigma_1 .. sigma_{n_d}}, n_d = min(m, d*stride); draft d is Eq. (2).
    Returns sigma[B, M] (-1 padded), n_fill[B, D], draft_tokens[B, D, M], draft_mask[B, D, M].
    """
    p.check()
    conf = np.asarray(conf, dtype=np.float64)
    tok = np.asarray(tok)
    tokens = np.asarray(tokens, dtype=np.int32)
    mask = np.asarray(mask, dtype=np.int32)
    B, M = mask.shape
    D = p.depth
    sigma = np.full((B, M), -1, dtype=np.int32)
    n_fill = np.zeros((B, D), dtype=np.int32)
    draft_tokens = np.empty((B, D, M), dtype=np.int32)
    draft_mask = np.empty((B, D, M), dtype=np.int32)
    for b in range(B):
        residual = [i for i in range(M) if mask[b, i] != 0]
        order = sorted(residual, key=lambda i: _rank_key(conf[b], i))
        m = len(order)
        sigma[b, :m] = order
        for d in range(D):
            n_d = min(m, d * p.step)
            n_fill[b, d] = n_d
            draft_tokens[b, d] = tokens[b]
            draft_mask[b, d] = mask[b]
            for i in order[:n_d]:             # Eq. (2): x~_{d,i} = x^_i for i in S_d
                draft_tokens[b, d, i] = tok[b, i]
                draft_mask[b, d, i] = 0
    return sigma, n_fill, draft_tokens, draft_mask


def verify_accept(tokV, confV, sigma, n_fill, draft_tokens, draft_mask, p: Policy):
    """Stage 3 (Sec. 3.2; Algorithm 1 "Stage 3") for the chain.

    tokV, confV: [B, D, M] verifier predictions for every draft.  The root is accepted; node d
    is accepted iff node d-1 is and every newly speculated slot i in S_d \\ S_{d-1} passes
    A_pi(x~_{d,i}, x^_{d-1,i}, c_{d-1,i}).  k* = the accepted node with the most filled slots
    (lowest index among equals).  The state becomes draft k*, and the verifier's predictions of
    node k* are committed too wherever a still-masked slot has confidence above tau.
    Returns tokens[B, M], mask[B, M], k_star[B], n_spec_accepted[B], n_committed[B], accepted[B, D].
    """
    p.check()
    tokV = np.asarray(tokV)
    confV = np.asarray(confV, dtype=np.float64)
    B, D, M = draft_tokens.shape
    tokens = np.empty((B, M), dtype=np.int32)
    mask = np.empty((B, M), dtype=np.int32)
    k_star = np.zeros(B, dtype=np.int32)
    n_spec = np.zeros(B, dtype=np.int32)
    n_comm = np.zeros(B, dtype=np.int32)
    accepted = np.zeros((B, D), dtype=np.int32)
    for b in range(B):
        accepted[b, 0] = 1
        for d in range(1, D):
            if not accepted[b, d - 1]:
                break
            parent = d - 1
            ok = True
            pol = None
            for j in range(int(n_fill[b, parent]), int(n_fill[b, d])):
                i = int(sigma[b, j])
                agree = int(tokV[b, parent, i]) == int(draft_tokens[b, d, i])
                if p.accept_mode == ACCEPT_AGREE_AND_CONF:
                    good = agree and float(confV[b, parent, i]) > p.tau
                elif p.accept_mode == ACCEPT_AGREE_ONLY:
                    good = agree
                else:
                    if pol is None:
                        pol = set(policy_set(confV[b, parent], draft_mask[b, parent], p))
                    good = agree and i in pol
                ok = ok and good
            accepted[b, d] = 1 if ok else 0
        best, best_n = 0, -1
        for d in range(D):
            if accepted[b, d] and int(n_fill[b, d]) > best_n:
                best, best_n = d, int(n_fill[b, d])
        k_star[b] = best
        n_spec[b] = best_n
        tokens[b] = draft_tokens[b, best]
        mask[b] = draft_mask[b, best]
        extra = 0
        for i in range(M):
            if mask[b, i] != 0 and float(confV[b, best, i]) > p.tau:
                tokens[b, i] = tokV[b, best, i]
                mask[b, i] = 0
                extra += 1
        n_comm[b] = best_n + extra
    return tokens, mask, k_star, n_spec, n_comm, accepted


def decode_block(model, M: int, p: Policy, max_steps: int | None = None, node_ranks=None, edges=None):
    """Algorithm 1 for one block.  With node_ranks (and optionally edges) the drafts form that graph
    instead of the chain of p.depth nodes.

    ``model(tokens[K, M], mask[K, M]) -> (tok[K, M], conf[K, M])`` stands for p_theta.
    Returns the final tokens, the number of model calls, and a per-iteration log of
    (|T|, k*, n_spec_accepted, n_committed).
    """
    p.check()
    tokens = np.full((1, M), p.mask_id, dtype=np.int32)
    mask = np.ones((1, M), dtype=np.int32)
    calls, log = 0, []
    limit = max_steps if max_steps is not None else 4 * M + 4
    while mask.any():
        if len(log) >= limit:
            raise RuntimeError("decode_block did not terminate")
        tok, conf = model(tokens, mask)
        calls += 1
        tokens, mask, _, n_sel, _ = select_unmask(conf, tok, tokens, mask, p)
        if not mask.any() or (p.depth == 1 if node_ranks is None else len(node_ranks) == 1):
            # the block is resolved (Algorithm 1's early break), or there is nothing to speculate:
            # a chain of the root alone is plain spatial decoding, one model call per iteration
            log.append((int(n_sel[0]), 0, 0, 0))
            continue
        if node_ranks is None:
            sigma, n_fill, dt, dm = build_drafts(conf, tok, tokens, mask, p)
        else:
            sigma, n_fill, dt, dm = build_drafts_dag(conf, tok, tokens, mask, p, node_ranks)
        tv, cv = model(dt[0], dm[0])
        calls += 1
        if node_ranks is None:
            tokens, mask, ks, ns, nc, _ = verify_accept(np.asarray(tv)[None], np.asarray(cv)[None],
                                                        sigma, n_fill, dt, dm, p)
        else:
            tokens, mask, ks, ns, nc, _ = verify_accept_dag(np.asarray(tv)[None], np.asarray(cv)[None],
                                                            sigma, dt, dm, p, node_ranks, edges)
        log.append((int(n_sel[0]), int(ks[0]), int(ns[0]), int(nc[0])))
    return tokens[0], calls, log


def decode_block_one_pass(model, M: int, p: Policy, max_steps: int | None = None, node_ranks=None, edges=None):
    """Algorithm 1 rearranged so that every iteration costs ONE model call.

    The batched pass on the D drafts also scores the root (the current state) and every accepted
    node, so its predictions for node k* are exactly what Stage 1 of the next iteration would
    compute on the state that acceptance leaves behind (node_ranks / edges: drafts form that graph
    instead of the chain).  An iteration is therefore:
    model(drafts) -> Stage 3 (acceptance and its extra commit) -> Stage 1 (policy on node k*'s
    predictions, Eq. (1)) -> Stage 2 (next drafts from the same predictions).  The first iteration
    verifies D copies of the initial state with nothing speculated.  This is an arrangement of the
    paper's three stages, not something the paper prints: after the extra commit nothing left exceeds
    tau, so Stage 1 then adds its k_min fallback positions.
    Returns the final tokens, the number of model calls, and a per-iteration log of
    (|T|, k*, n_spec_accepted, n_committed).
    """
    p.check()
    D = p.depth if node_ranks is None else len(node_ranks)
    tokens = np.full((1, M), p.mask_id, dtype=np.int32)
    mask = np.ones((1, M), dtype=np.int32)
    sigma = np.full((1, M), -1, dtype=np.int32)
    n_fill = np.zeros((1, D), dtype=np.int32)
    dt = np.repeat(tokens[:, None, :], D, axis=1)
    dm = np.repeat(mask[:, None, :], D, axis=1)
    calls, log = 0, []
    limit = max_steps if max_steps is not None else 4 * M + 4
    while mask.any():
        if len(log) >= limit:
            raise RuntimeError("decode_block_one_pass did not terminate")
        tv, cv = model(dt[0], dm[0])
        calls += 1
        tv, cv = np.asarray(tv)[None], np.asarray(cv, dtype=np.float64)[None]
        if node_ranks is None:
            tokens, mask, ks, ns, nc, _ = verify_accept(tv, cv, sigma, n_fill, dt, dm, p)
        else:
            tokens, mask, ks, ns, nc, _ = verify_accept_dag(tv, cv, sigma, dt, dm, p, node_ranks, edges)
        ck, tk = cv[:, int(ks[0])], tv[:, int(ks[0])]
        tokens, mask, _, n_sel, _ = select_unmask(ck, tk, tokens, mask, p)
        if node_ranks is None:
            sigma, n_fill, dt, dm = build_drafts(ck, tk, tokens, mask, p)
        else:
            sigma, n_fill, dt, dm = build_drafts_dag(ck, tk, tokens, mask, p, node_ranks)
        log.append((int(n_sel[0]), int(ks[0]), int(ns[0]), int(nc[0])))
    return tokens[0], calls, log


# --------------------------------------------------------------------------------------
# General draft graph (Sec. 3.2 Stage 2-3; Algorithm 1 with a DAG): nodes are sets of RANKS of
# the speculative ordering sigma; an edge (p, k) exists whenever S_p is a strict subset of S_k.
# --------------------------------------------------------------------------------------

def dag_edges(node_ranks):
    """All (p, k) with S_p a strict subset of S_k (Sec. 3.2: "an edge exists whenever S_p ⊂ S_k")."""
    sets = [frozenset(s) for s in node_ranks]
    return [(p, k) for k in range(len(sets)) for p in range(len(sets)) if sets[p] < sets[k]]


def build_drafts_dag(conf, tok, tokens, mask, p: Policy, node_ranks):
    """Stage 2 for a draft graph.  node_ranks[k] = the ranks j (0-based positions in sigma) that node k
    speculates; node 0 must be the root (empty).  With m residual slots only ranks < m exist:
    S_k = {sigma_j : j in node_ranks[k], j < m}; draft k is Eq. (2).
    Returns sigma[B, M], n_fill[B, K] (= |S_k|), draft_tokens[B, K, M], draft_mask[B, K, M]."""
    p.check()
    if len(node_ranks) < 1 or len(node_ranks[0]) != 0:
        raise ValueError("node 0 must be the root (no speculated ranks)")
    conf = np.asarray(conf, dtype=np.float64)
    tok = np.asarray(tok)
    tokens = np.asarray(tokens, dtype=np.int32)
    mask = np.asarray(mask, dtype=np.int32)
    B, M = mask.shape
    K = len(node_ranks)
    sigma = np.full((B, M), -1, dtype=np.int32)
    n_fill = np.zeros((B, K), dtype=np.int32)
    draft_tokens = np.empty((B, K, M), dtype=np.int32)
    draft_mask = np.empty((B, K, M), dtype=np.int32)
    for b in range(B):
        residual = [i for i in range(M) if mask[b, i] != 0]
        order = sorted(residual, key=lambda i: _rank_key(conf[b], i))
        m = len(order)
        sigma[b, :m] = order
        for k in range(K):
            S = [order[j] for j in sorted(node_ranks[k]) if j < m]
            n_fill[b, k] = len(S)
            draft_tokens[b, k] = tokens[b]
            draft_mask[b, k] = mask[b]
            for i in S:                              # Eq. (2)
                draft_tokens[b, k, i] = tok[b, i]
                draft_mask[b, k, i] = 0
    return sigma, n_fill, draft_tokens, draft_mask


def verify_accept_dag(tokV, confV, sigma, draft_tokens, draft_mask, p: Policy, node_ranks, edges=None):
    """Stage 3 for a draft graph (Algorithm 1 "Stage 3").  `edges` = list of (p, k) with S_p a strict
    subset of S_k; None means every such pair (the paper's definition of the edge set).

    The root is accepted.  Nodes are visited in topological order (fewer speculated ranks first, lower
    index first among equals); node k is accepted iff some ACCEPTED p with an edge (p, k) passes
    A_pi(x~_{k,i}, x^_{p,i}, c_{p,i}) on every i in S_k \\ S_p (an empty difference passes).
    k* = the accepted node with the largest |S_k|, lowest index among equals; then the state becomes
    draft k* and node k*'s own predictions above tau are committed as well.
    Returns tokens, mask, k_star[B], n_spec_accepted[B], n_committed[B], accepted[B, K]."""
    p.check()
    tokV = np.asarray(tokV)
    confV = np.asarray(confV, dtype=np.float64)
    B, K, M = draft_tokens.shape
    if edges is None:
        edges = dag_edges(node_ranks)
    for (q, k) in edges:
        if not frozenset(node_ranks[q]) < frozenset(node_ranks[k]):
            raise ValueError("an edge (p, k) needs S_p to be a strict subset of S_k")
    topo = sorted(range(K), key=lambda k: (len(node_ranks[k]), k))
    tokens = np.empty((B, M), dtype=np.int32)
    mask = np.empty((B, M), dtype=np.int32)
    k_star = np.zeros(B, dtype=np.int32)
    n_spec = np.zeros(B, dtype=np.int32)
    n_comm = np.zeros(B, dtype=np.int32)
    accepted = np.zeros((B, K), dtype=np.int32)
    for b in range(B):
        m = int((sigma[b] >= 0).sum())
        S = [set(int(sigma[b, j]) for j in node_ranks[k] if j < m) for k in range(K)]
        pol = {}
        accepted[b, 0] = 1
        for k in topo:
            if k == 0:
                continue
            for (q, kk) in edges:
                if kk != k or not accepted[b, q]:
                    continue
                ok = True
                for i in S[k] - S[q]:
                    agree = int(tokV[b, q, i]) == int(draft_tokens[b, k, i])
                    if p.accept_mode == ACCEPT_AGREE_AND_CONF:
                        good = agree and float(confV[b, q, i]) > p.tau
                    elif p.accept_mode == ACCEPT_AGREE_ONLY:
                        good = agree
                    else:
                        if q not in pol:
                            pol[q] = set(policy_set(confV[b, q], draft_mask[b, q], p))
                        good = agree and i in pol[q]
                    ok = ok and good
                if ok:
                    accepted[b, k] = 1
                    break
        best, best_n = 0, -1
        for k in range(K):
            if accepted[b, k] and len(S[k]) > best_n:
                best, best_n = k, len(S[k])
        k_star[b] = best
        n_spec[b] = best_n
        tokens[b] = draft_tokens[b, best]
        mask[b] = draft_mask[b, best]
        extra = 0
        for i in range(M):
            if mask[b, i] != 0 and float(confV[b, best, i]) > p.tau:
                tokens[b, i] = tokV[b, best, i]
                mask[b, i] = 0
                extra += 1
        n_comm[b] = best_n + extra
    return tokens, mask, k_star, n_spec, n_comm, accepted


def chain_as_dag(depth: int, step: int):
    """The chain of `depth` nodes (root included) adding `step` ranks per depth, as node rank sets."""
    return [set(range(d * step)) for d in range(depth)]
