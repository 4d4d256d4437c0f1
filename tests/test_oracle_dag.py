"""Pins of the oracle's draft-graph stages (Sec. 3.2 Stages 2-3 with a multi-parent DAG; Algorithm 1).

What fixes them: the chain functions (already pinned) as the special case of a path graph; a
brute-force reading of "accepted iff reachable from the root through edges whose checks pass";
hand-built cases for the multi-parent rule and for the deepest-node choice."""
import itertools

import numpy as np
import pytest

import oracle
from oracle import Policy

MASK = 999


def _case(rng, B, M, K_sets, p_masked=0.8):
    conf = rng.permutation(B * M).reshape(B, M) / (B * M + 1.0) * 0.98 + 0.01
    tok = rng.integers(0, 50, size=(B, M)).astype(np.int32)
    mask = (rng.random((B, M)) < p_masked).astype(np.int32)
    tokens = np.where(mask == 1, MASK, rng.integers(0, 50, size=(B, M))).astype(np.int32)
    return conf, tok, tokens, mask


@pytest.mark.parametrize("accept_mode", [0, 1, 2])
@pytest.mark.parametrize("D,step", [(1, 1), (4, 1), (3, 2), (5, 3)])
def test_path_graph_with_immediate_edges_equals_the_chain(D, step, accept_mode):
    # the chain's three acceptance modes are pinned on their own (per-depth enumeration, the mode-2 hand
    # case): on a path graph the graph's branch of every mode has to give the chain's result
    rng = np.random.default_rng(D * 10 + step)
    B, M = 6, 12
    p = Policy(tau=0.5, k_min=step, k_max=0, depth=D, stride=step, accept_mode=accept_mode, mask_id=MASK)
    conf, tok, tokens, mask = _case(rng, B, M, None)
    ranks = oracle.chain_as_dag(D, step)
    a = oracle.build_drafts(conf, tok, tokens, mask, p)
    b = oracle.build_drafts_dag(conf, tok, tokens, mask, p, ranks)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)
    sigma, n_fill, dt, dm = a
    tokV = np.where(rng.random((B, D, M)) < 0.7, tok[:, None, :], 77).astype(np.int32)
    confV = rng.random((B, D, M))
    chain = oracle.verify_accept(tokV, confV, sigma, n_fill, dt, dm, p)
    path = oracle.verify_accept_dag(tokV, confV, sigma, dt, dm, p, ranks, edges=[(d - 1, d) for d in range(1, D)])
    for x, y in zip(chain, path):
        assert np.array_equal(x, y)
    # with every subset edge the graph can only accept more
    full = oracle.verify_accept_dag(tokV, confV, sigma, dt, dm, p, ranks)
    assert (full[5] >= path[5]).all() and (full[3] >= path[3]).all()


def _policy_slots_by_sorting(conf_q, masked_q, p):
    """pi(parent's draft) restated with a numpy sort: among the slots still masked in the parent's draft,
    ordered by (confidence descending, slot ascending), the first n, with n the number above tau clamped
    to [k_min, k_max] and to the number of masked slots (Sec. 3.2 Stage 1; App. B.2)."""
    slots = np.nonzero(masked_q)[0]
    order = slots[np.lexsort((slots, -conf_q[slots]))]
    n = max(int((conf_q[slots] > p.tau).sum()), p.k_min)
    if p.k_max:
        n = min(n, p.k_max)
    return set(order[:min(n, len(order))].tolist())


def _reachable_by_brute_force(tokV, confV, sigma_b, tok_t, node_ranks, p, b, draft_mask):
    """Accepted set from the definition: k is accepted iff there is a sequence root = q0, q1, .., k of
    nodes, each a strict superset of the one before, every step passing its checks."""
    K = len(node_ranks)
    m = int((sigma_b >= 0).sum())
    S = [frozenset(int(sigma_b[j]) for j in node_ranks[k] if j < m) for k in range(K)]
    nominal = [frozenset(s) for s in node_ranks]

    def slot_ok(q, i):
        if int(tokV[b, q, i]) != int(tok_t[i]):
            return False
        if p.accept_mode == 0:
            return float(confV[b, q, i]) > p.tau
        if p.accept_mode == 1:
            return True
        return i in _policy_slots_by_sorting(confV[b, q], draft_mask[b, q], p)

    def step_ok(q, k):
        return all(slot_ok(q, i) for i in S[k] - S[q])

    acc = set()
    for k in range(K):
        others = [q for q in range(1, K) if q != k]
        found = k == 0
        for r in range(len(others) + 1):
            for mid in itertools.permutations(others, r):
                path = (0,) + mid + ((k,) if k != 0 else ())
                if all(nominal[path[t]] < nominal[path[t + 1]] and step_ok(path[t], path[t + 1])
                       for t in range(len(path) - 1)):
                    found = True
                    break
            if found:
                break
        if found:
            acc.add(k)
    return acc, S


@pytest.mark.parametrize("accept_mode,k_max", [(0, 0), (1, 0), (2, 0), (2, 2)])
def test_acceptance_equals_path_enumeration(accept_mode, k_max):
    rng = np.random.default_rng(5)
    node_ranks = [set(), {0}, {1}, {0, 1}, {0, 2}, {0, 1, 2}]
    B, M = 40, 6
    p = Policy(tau=0.5, k_min=1, k_max=k_max, depth=len(node_ranks), accept_mode=accept_mode, mask_id=MASK)
    conf, tok, tokens, mask = _case(rng, B, M, None, p_masked=0.9)
    sigma, n_fill, dt, dm = oracle.build_drafts_dag(conf, tok, tokens, mask, p, node_ranks)
    K = len(node_ranks)
    tokV = np.where(rng.random((B, K, M)) < 0.75, tok[:, None, :], 77).astype(np.int32)
    confV = rng.random((B, K, M)) * 0.5 + (0.45 if accept_mode == 0 else 0.25)
    tokens2, mask2, k_star, n_spec, n_comm, accepted = oracle.verify_accept_dag(tokV, confV, sigma, dt, dm, p,
                                                                                node_ranks)
    seen_multi = 0
    for b in range(B):
        acc, S = _reachable_by_brute_force(tokV, confV, sigma[b], tok[b], node_ranks, p, b, dm)
        assert set(np.nonzero(accepted[b])[0].tolist()) == acc
        best = max(sorted(acc), key=lambda k: len(S[k]))
        assert len(S[k_star[b]]) == len(S[best]) == n_spec[b] and k_star[b] in acc
        assert k_star[b] == min(k for k in acc if len(S[k]) == n_spec[b])
        seen_multi += int(3 in acc and not (1 in acc and 2 in acc))
    assert accepted[:, 0].all() and (accepted.sum(axis=1) > 1).any() and seen_multi > 0
    assert (accepted.sum(axis=1) < K).any()                    # and something was rejected


def test_a_second_parent_rescues_a_node():
    # Ranks 0 and 1.  Against the root, slot sigma_0 fails (low confidence) and sigma_1 passes: {0} is
    # rejected, {1} accepted.  {0,1} then has one accepted parent, {1}, whose own prediction of
    # sigma_0 passes: accepted through it, although the path through {0} is closed.
    node_ranks = [set(), {0}, {1}, {0, 1}]
    p = Policy(tau=0.5, k_min=1, depth=4, mask_id=MASK)
    conf = np.array([[0.9, 0.8, 0.1]])
    tok = np.array([[5, 6, 7]], dtype=np.int32)
    tokens = np.full((1, 3), MASK, dtype=np.int32)
    mask = np.ones((1, 3), dtype=np.int32)
    sigma, n_fill, dt, dm = oracle.build_drafts_dag(conf, tok, tokens, mask, p, node_ranks)
    assert sigma[0].tolist() == [0, 1, 2] and n_fill[0].tolist() == [0, 1, 1, 2]
    assert dt[0, 3].tolist() == [5, 6, MASK] and dm[0, 2].tolist() == [1, 0, 1]
    tokV = np.tile(tok[:, None, :], (1, 4, 1))
    confV = np.full((1, 4, 3), 0.9)
    confV[0, 0, 0] = 0.3                       # the root is unsure of sigma_0
    out = oracle.verify_accept_dag(tokV, confV, sigma, dt, dm, p, node_ranks)
    assert out[5][0].tolist() == [1, 0, 1, 1] and out[2][0] == 3 and out[3][0] == 2
    # with the edge ({1}, {0,1}) removed the node is lost
    out = oracle.verify_accept_dag(tokV, confV, sigma, dt, dm, p, node_ranks, edges=[(0, 1), (0, 2), (1, 3), (0, 3)])
    assert out[5][0].tolist() == [1, 0, 1, 0] and out[2][0] == 2 and out[3][0] == 1


def test_structure_and_truncation():
    rng = np.random.default_rng(9)
    node_ranks = [set(), {0, 1}, {0, 1, 2, 3}, {2}, {0, 1, 2, 3, 4, 5, 6, 7}]
    B, M = 8, 10
    p = Policy(tau=0.5, k_min=1, depth=5, mask_id=MASK)
    conf, tok, tokens, mask = _case(rng, B, M, None, p_masked=0.45)
    sigma, n_fill, dt, dm = oracle.build_drafts_dag(conf, tok, tokens, mask, p, node_ranks)
    for b in range(B):
        m = int(mask[b].sum())
        assert (sigma[b, :m] >= 0).all() and (sigma[b, m:] == -1).all()
        c = conf[b, sigma[b, :m]]
        assert (np.diff(c) <= 0).all()                               # sigma is by descending confidence
        for k, ranks in enumerate(node_ranks):
            S = {int(sigma[b, j]) for j in ranks if j < m}
            assert n_fill[b, k] == len(S)
            changed = set(np.nonzero(dt[b, k] != tokens[b])[0].tolist()) | set(np.nonzero(dm[b, k] != mask[b])[0].tolist())
            assert changed <= S and (dm[b, k][list(S)] == 0).all() and (dt[b, k][list(S)] == tok[b][list(S)]).all()
    with pytest.raises(ValueError):
        oracle.build_drafts_dag(conf, tok, tokens, mask, p, [{0}, {0, 1}])
    with pytest.raises(ValueError):
        oracle.verify_accept_dag(np.zeros((B, 5, M), int), np.zeros((B, 5, M)), sigma, dt, dm, p, node_ranks,
                                 edges=[(1, 3)])


class _Stable:
    """A model whose predictions never change: target tokens, confidence falling with the slot index."""

    def __init__(self, M):
        self.target = np.arange(100, 100 + M, dtype=np.int32)
        self.calls = []

    def __call__(self, tokens, mask):
        mask = np.atleast_2d(mask)
        self.calls.append(mask.shape[0])
        conf = np.tile(0.8 - 0.03 * np.arange(mask.shape[1]), (mask.shape[0], 1))
        return np.tile(self.target, (mask.shape[0], 1)), conf


@pytest.mark.parametrize("loop", [oracle.decode_block, oracle.decode_block_one_pass])
def test_loops_with_a_path_graph_equal_the_chain_loops(loop):
    M, D = 14, 4
    p = Policy(tau=1.0, k_min=1, k_max=1, depth=D, accept_mode=1, mask_id=MASK)
    chain = loop(_Stable(M), M, p)
    graph = loop(_Stable(M), M, p, node_ranks=oracle.chain_as_dag(D, 1), edges=[(d - 1, d) for d in range(1, D)])
    assert (chain[0] == graph[0]).all() and chain[1] == graph[1] and chain[2] == graph[2]


def test_loop_with_a_wider_graph_commits_every_slot_once():
    M = 20
    ranks = [set(), {0}, {1}, {0, 1}, {0, 1, 2}, {0, 2}]
    p = Policy(tau=0.5, k_min=1, k_max=3, depth=1, accept_mode=1, mask_id=MASK)
    for loop in (oracle.decode_block, oracle.decode_block_one_pass):
        m = _Stable(M)
        tokens, calls, log = loop(m, M, p, node_ranks=ranks)
        assert (tokens == m.target).all() and sum(n + nc for n, _, _, nc in log) == M
        assert max(ks for _, ks, _, _ in log) > 0 and set(m.calls) <= {1, len(ranks)}
