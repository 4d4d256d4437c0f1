"""Pins for the oracle's policy / draft / acceptance stages (Sec. 3.2, Eq. (1), Eq. (2), Algorithm 1).

Each test restates the property from the paper (or from the stated reading of an open point)
in a different form than the oracle uses: brute-force enumeration, numpy sorting routines,
or structural invariants.
"""
import itertools
import math

import numpy as np
import pytest

import oracle
from oracle import Policy

MASK = 999


def _rand_case(rng, B, M, D=1, p_masked=0.7, distinct=True):
    conf = rng.random((B, M))
    if not distinct:
        conf = np.round(conf * 4) / 4
    tok = rng.integers(0, 900, size=(B, M)).astype(np.int32)
    mask = (rng.random((B, M)) < p_masked).astype(np.int32)
    tokens = np.where(mask == 1, MASK, rng.integers(0, 900, size=(B, M))).astype(np.int32)
    return conf, tok, tokens, mask


# ------------------------------------------------------------------ Stage 1: select / Eq. (1)

def test_tau_one_selects_exactly_k_min():
    rng = np.random.default_rng(0)
    for k in (1, 2, 5):
        conf, tok, tokens, mask = _rand_case(rng, 6, 12)
        conf[0, :] = 1.0                                  # even conf == 1 does not "exceed" tau = 1
        _, _, sel, n_sel, _ = oracle.select_unmask(conf, tok, tokens, mask, Policy(tau=1.0, k_min=k))
        for b in range(6):
            assert n_sel[b] == min(k, mask[b].sum()) == sel[b].sum()


def test_negative_tau_selects_everything_up_to_k_max():
    rng = np.random.default_rng(1)
    conf, tok, tokens, mask = _rand_case(rng, 8, 10)
    for kmax in (0, 3, 7):
        _, m2, _, n_sel, _ = oracle.select_unmask(conf, tok, tokens, mask, Policy(tau=-1.0, k_min=1, k_max=kmax))
        for b in range(8):
            want = mask[b].sum() if kmax == 0 else min(mask[b].sum(), kmax)
            assert n_sel[b] == want
            assert m2[b].sum() == mask[b].sum() - want


def test_fixed_k_equals_sort_and_take_k():
    rng = np.random.default_rng(2)
    conf, tok, tokens, mask = _rand_case(rng, 10, 16, distinct=False)   # ties present
    for k in (1, 3, 4):
        _, _, sel, n_sel, sel_pos = oracle.select_unmask(conf, tok, tokens, mask,
                                                         Policy(tau=0.5, k_min=k, k_max=k))
        for b in range(10):
            slots = np.nonzero(mask[b])[0]
            # numpy: stable sort on (-conf) keeps lower slots first among equals
            order = slots[np.argsort(-conf[b, slots], kind="stable")]
            want = order[:k].tolist()
            assert sel_pos[b, :len(want)].tolist() == want
            assert (sel_pos[b, len(want):] == -1).all()
            assert sorted(np.nonzero(sel[b])[0].tolist()) == sorted(want)


def test_threshold_clamp_count_and_dominance():
    rng = np.random.default_rng(3)
    conf, tok, tokens, mask = _rand_case(rng, 40, 9)
    p = Policy(tau=0.6, k_min=2, k_max=4)
    t2, m2, sel, n_sel, sel_pos = oracle.select_unmask(conf, tok, tokens, mask, p)
    for b in range(40):
        masked = mask[b] == 1
        n_thr = int(((conf[b] > 0.6) & masked).sum())
        assert n_sel[b] == min(int(masked.sum()), 4, max(n_thr, 2))
        chosen = sel[b] == 1
        assert not (chosen & ~masked).any()               # T is a subset of M(x)
        if chosen.any() and (masked & ~chosen).any():
            assert conf[b, chosen].min() >= conf[b, masked & ~chosen].max()
        # Eq. (1): chosen slots take the prediction, all others keep their value
        assert (t2[b, chosen] == tok[b, chosen]).all()
        assert (t2[b, ~chosen] == tokens[b, ~chosen]).all()
        assert (m2[b] == (masked & ~chosen)).all()
        ranked = sel_pos[b, :n_sel[b]]
        assert (np.diff(conf[b, ranked]) <= 0).all()


def test_select_brute_force_over_subsets():
    # For M <= 6 enumerate every subset of the masked slots of the required size; the policy's
    # set is the one with the largest total confidence (unique: confidences are distinct).
    rng = np.random.default_rng(4)
    for _ in range(60):
        M = int(rng.integers(1, 7))
        conf, tok, tokens, mask = _rand_case(rng, 1, M)
        p = Policy(tau=float(rng.choice([0.3, 0.6, 0.95])), k_min=int(rng.integers(1, 3)),
                   k_max=int(rng.choice([0, 3, 5])))
        if p.k_max and p.k_max < p.k_min:
            continue
        _, _, sel, n_sel, _ = oracle.select_unmask(conf, tok, tokens, mask, p)
        slots = [i for i in range(M) if mask[0, i]]
        n_thr = sum(conf[0, i] > p.tau for i in slots)
        n = max(n_thr, p.k_min)
        n = min(n, p.k_max) if p.k_max else n
        n = min(n, len(slots))
        best = max(itertools.combinations(slots, n), key=lambda s: sum(conf[0, i] for i in s))
        assert n_sel[0] == n
        assert sorted(np.nonzero(sel[0])[0].tolist()) == sorted(best)


def test_ties_break_to_lower_slot_and_nan_ranks_last():
    conf = np.array([[0.5, 0.7, 0.7, float("nan"), 0.5, 0.2]])
    tok = np.arange(6, dtype=np.int32)[None]
    tokens = np.full((1, 6), MASK, dtype=np.int32)
    mask = np.ones((1, 6), dtype=np.int32)
    _, _, _, n_sel, sel_pos = oracle.select_unmask(conf, tok, tokens, mask, Policy(tau=-1.0, k_min=1))
    # NaN is never above tau: the threshold admits the five numbers, not the NaN slot
    assert n_sel[0] == 5 and sel_pos[0].tolist() == [1, 2, 0, 4, 5, -1]
    # the full ordering (the speculative ordering sigma uses the same ranking) puts NaN last
    sigma, _, _, _ = oracle.build_drafts(conf, tok, tokens, mask, Policy(tau=0.5, k_min=1, depth=2))
    assert sigma[0].tolist() == [1, 2, 0, 4, 5, 3]


# ------------------------------------------------------------------ Stage 2: drafts / Eq. (2)

@pytest.mark.parametrize("stride,k_min,D", [(0, 1, 4), (0, 3, 3), (2, 1, 6), (4, 4, 6), (1, 1, 1)])
def test_draft_structure(stride, k_min, D):
    rng = np.random.default_rng(10 + D)
    B, M = 12, 14
    conf, tok, tokens, mask = _rand_case(rng, B, M, distinct=False)
    mask[0] = 0
    tokens[0] = 5                                           # a fully decoded block: m = 0
    p = Policy(tau=0.9, k_min=k_min, k_max=max(k_min, 4), depth=D, stride=stride)
    sigma, n_fill, dt, dm = oracle.build_drafts(conf, tok, tokens, mask, p)
    s = stride if stride else k_min
    for b in range(B):
        m = int(mask[b].sum())
        sg = sigma[b, :m]
        assert sorted(sg.tolist()) == np.nonzero(mask[b])[0].tolist()      # sigma permutes the residual set
        assert (sigma[b, m:] == -1).all()
        assert (np.diff(conf[b, sg]) <= 0).all()                           # c_sigma1 >= c_sigma2 >= ...
        # root: S_r is empty, the draft is the current state
        assert (dt[b, 0] == tokens[b]).all() and (dm[b, 0] == mask[b]).all() and n_fill[b, 0] == 0
        prev = set()
        for d in range(D):
            assert n_fill[b, d] == min(m, d * s)
            S = set(sg[:n_fill[b, d]].tolist())
            assert prev <= S                                                # S_d contains S_{d-1}
            prev = S
            diff = set(np.nonzero(dt[b, d] != tokens[b])[0].tolist())
            filled = set(np.nonzero(dm[b, d] != mask[b])[0].tolist())
            assert filled == S                                              # mask drops exactly S_d
            assert diff <= S                                                # tokens differ only on S_d
            for i in S:
                assert dt[b, d, i] == tok[b, i]                             # Eq. (2): cached step-t prediction
            untouched = [i for i in range(M) if i not in S]
            assert (dt[b, d, untouched] == tokens[b, untouched]).all()      # committed tokens unchanged
    assert (n_fill[0] == 0).all() and (dm[0] == 0).all()


# ------------------------------------------------------------------ Stage 3: acceptance

def _accept_by_definition(tokV, confV, sigma, n_fill, tok_t, tau, mode):
    """accepted[d] straight from the definition, without the incremental recursion: node d is
    accepted iff every slot speculated by any node e <= d passes the check against node e-1."""
    D = n_fill.shape[0]
    out = []
    for d in range(D):
        ok = True
        for e in range(1, d + 1):
            js = np.arange(n_fill[e - 1], n_fill[e])
            slots = sigma[js]
            agree = (tokV[e - 1, slots] == tok_t[slots]).all()
            conf_ok = (confV[e - 1, slots] > tau).all()
            ok = ok and bool(agree) and (bool(conf_ok) or mode == 1)
        out.append(ok)
    return out


@pytest.mark.parametrize("mode", [0, 1])
def test_accept_matches_enumeration_over_depths(mode):
    rng = np.random.default_rng(20 + mode)
    B, M, D = 60, 10, 5
    conf, tok, tokens, mask = _rand_case(rng, B, M)
    p = Policy(tau=0.5, k_min=1, k_max=0, depth=D, stride=2, accept_mode=mode)
    sigma, n_fill, dt, dm = oracle.build_drafts(conf, tok, tokens, mask, p)
    # verifier: mostly agrees with the cached predictions, with random flips and confidences
    tokV = np.repeat(tok[:, None, :], D, axis=1).copy()
    flips = rng.random((B, D, M)) < 0.15
    tokV[flips] += 1
    confV = rng.random((B, D, M)) ** 0.3
    t2, m2, ks, nspec, ncomm, acc = oracle.verify_accept(tokV, confV, sigma, n_fill, dt, dm, p)
    seen = set()
    for b in range(B):
        want = _accept_by_definition(tokV[b], confV[b], sigma[b], n_fill[b], tok[b], p.tau, mode)
        assert acc[b].tolist() == [int(x) for x in want]
        assert acc[b, 0] == 1                                              # root always accepted
        assert (np.diff(acc[b]) <= 0).all()                                # accepted nodes form a prefix
        best_n = max(int(n_fill[b, d]) for d in range(D) if want[d])
        k = min(d for d in range(D) if want[d] and n_fill[b, d] == best_n)
        assert ks[b] == k and nspec[b] == best_n
        seen.add(int(ks[b]))
        # state = draft k*, plus verifier predictions of node k* above tau on still-masked slots
        extra = (dm[b, k] == 1) & (confV[b, k] > p.tau)
        assert (t2[b] == np.where(extra, tokV[b, k], dt[b, k])).all()
        assert (m2[b] == ((dm[b, k] == 1) & ~extra)).all()
        assert ncomm[b] == best_n + int(extra.sum())
        # tokens committed before this step never change
        was = mask[b] == 0
        assert (t2[b, was] == tokens[b, was]).all()
    assert len(seen) >= 3                                                  # the case mix reaches several depths


def test_accept_all_agree_with_full_confidence_reaches_deepest():
    rng = np.random.default_rng(30)
    B, M, D = 8, 12, 4
    conf, tok, tokens, mask = _rand_case(rng, B, M, p_masked=1.0)
    p = Policy(tau=0.9, k_min=1, depth=D, stride=3)
    sigma, n_fill, dt, dm = oracle.build_drafts(conf, tok, tokens, mask, p)
    tokV = np.repeat(tok[:, None, :], D, axis=1)
    confV = np.ones((B, D, M))
    _, m2, ks, nspec, ncomm, acc = oracle.verify_accept(tokV, confV, sigma, n_fill, dt, dm, p)
    assert (ks == D - 1).all() and (acc == 1).all()
    assert (nspec == n_fill[:, -1]).all()
    assert (m2 == 0).all() and (ncomm == M).all()          # conf 1 > tau: everything else commits too


def test_accept_all_disagree_stays_at_root():
    rng = np.random.default_rng(31)
    B, M, D = 8, 12, 4
    conf, tok, tokens, mask = _rand_case(rng, B, M, p_masked=1.0)
    p = Policy(tau=0.9, k_min=1, depth=D, stride=2)
    sigma, n_fill, dt, dm = oracle.build_drafts(conf, tok, tokens, mask, p)
    tokV = np.repeat(tok[:, None, :], D, axis=1) + 1
    confV = np.full((B, D, M), 0.5)
    t2, m2, ks, nspec, ncomm, acc = oracle.verify_accept(tokV, confV, sigma, n_fill, dt, dm, p)
    assert (ks == 0).all() and (nspec == 0).all() and (ncomm == 0).all()
    assert (acc[:, 0] == 1).all() and (acc[:, 1:] == 0).all()
    assert (t2 == tokens).all() and (m2 == mask).all()


def test_accept_strict_threshold_and_saturation():
    # conf exactly tau does not pass ("exceeds"); a saturated chain picks the lowest node index
    # among those that fill the same number of slots.
    conf = np.array([[0.9, 0.8, 0.7, 0.6]])
    tok = np.array([[10, 11, 12, 13]], dtype=np.int32)
    tokens = np.array([[MASK, MASK, 7, 8]], dtype=np.int32)
    mask = np.array([[1, 1, 0, 0]], dtype=np.int32)
    p = Policy(tau=0.75, k_min=1, depth=5, stride=1)
    sigma, n_fill, dt, dm = oracle.build_drafts(conf, tok, tokens, mask, p)
    assert n_fill.tolist() == [[0, 1, 2, 2, 2]]
    tokV = np.repeat(tok[:, None, :], 5, axis=1)
    confV = np.full((1, 5, 4), 0.99)
    _, _, ks, nspec, _, acc = oracle.verify_accept(tokV, confV, sigma, n_fill, dt, dm, p)
    assert acc.tolist() == [[1, 1, 1, 1, 1]] and ks[0] == 2 and nspec[0] == 2
    confV[0, 0, 0] = 0.75                                   # == tau at the slot node 1 speculates
    _, _, ks, nspec, _, acc = oracle.verify_accept(tokV, confV, sigma, n_fill, dt, dm, p)
    assert acc.tolist() == [[1, 0, 0, 0, 0]] and ks[0] == 0 and nspec[0] == 0


def test_accept_mode_policy_membership():
    # Mode 2: the speculated slot must also be one the policy would pick on the parent's node.
    conf = np.array([[0.5, 0.4, 0.3]])
    tok = np.array([[1, 2, 3]], dtype=np.int32)
    tokens = np.full((1, 3), MASK, dtype=np.int32)
    mask = np.ones((1, 3), dtype=np.int32)
    p = Policy(tau=0.95, k_min=1, k_max=1, depth=2, stride=1, accept_mode=2)
    sigma, n_fill, dt, dm = oracle.build_drafts(conf, tok, tokens, mask, p)
    assert sigma[0].tolist() == [0, 1, 2]
    tokV = np.repeat(tok[:, None, :], 2, axis=1)
    confV = np.array([[[0.6, 0.7, 0.1], [0.1, 0.1, 0.1]]])  # on the root, the policy would pick slot 1, not 0
    _, _, ks, _, _, _ = oracle.verify_accept(tokV, confV, sigma, n_fill, dt, dm, p)
    assert ks[0] == 0
    confV[0, 0] = [0.8, 0.7, 0.1]                           # now slot 0 ranks first on the root
    _, _, ks, _, _, _ = oracle.verify_accept(tokV, confV, sigma, n_fill, dt, dm, p)
    assert ks[0] == 1


def test_tau_one_commits_nothing_extra():
    rng = np.random.default_rng(33)
    B, M, D = 5, 8, 3
    conf, tok, tokens, mask = _rand_case(rng, B, M)
    p = Policy(tau=1.0, k_min=1, depth=D)
    sigma, n_fill, dt, dm = oracle.build_drafts(conf, tok, tokens, mask, p)
    tokV = np.repeat(tok[:, None, :], D, axis=1)
    confV = np.ones((B, D, M))
    t2, m2, ks, nspec, ncomm, _ = oracle.verify_accept(tokV, confV, sigma, n_fill, dt, dm, p)
    assert (ks == 0).all() and (ncomm == 0).all()
    assert (t2 == tokens).all() and (m2 == mask).all()


# ------------------------------------------------------------------ Algorithm 1 as a whole

class ToyModel:
    """A deterministic stand-in for p_theta: fixed target tokens; confidence of a masked slot grows
    with the number of already revealed slots and depends on the slot."""

    def __init__(self, M, seed=0, stable=True):
        rng = np.random.default_rng(seed)
        self.target = rng.integers(0, 500, size=M).astype(np.int32)
        self.base = rng.random(M)
        self.stable = stable
        self.calls = []

    def __call__(self, tokens, mask):
        tokens = np.atleast_2d(tokens)
        mask = np.atleast_2d(mask)
        K, M = mask.shape
        self.calls.append(K)
        revealed = (mask == 0).sum(axis=1, keepdims=True) / M
        conf = np.clip(0.2 + 0.6 * self.base[None, :] + 0.5 * revealed, 0, 0.999)
        tok = np.repeat(self.target[None, :], K, axis=0).copy()
        if not self.stable:
            tok[:, ::3] += (mask == 0).sum(axis=1, keepdims=True) % 2       # predictions drift with context
        return tok, conf


def test_greedy_collapse_one_token_per_call():
    # tau = 1, k = 1, no speculation: exactly one slot per forward pass, always the most confident one.
    M = 12
    model = ToyModel(M)
    p = Policy(tau=1.0, k_min=1, k_max=1, depth=1, mask_id=MASK)
    order = []

    def spy(tokens, mask):
        tok, conf = model(tokens, mask)
        order.append(int(np.argmax(np.where(np.atleast_2d(mask)[0] == 1, conf[0], -1))))
        return tok, conf

    tokens, calls, log = oracle.decode_block(spy, M, p)
    assert calls == M and all(n == 1 for n, *_ in log)
    assert (tokens == model.target).all()
    assert sorted(order) == list(range(M))                 # each call revealed its argmax slot


def test_tau_one_with_speculation_accepts_nothing():
    M = 10
    model = ToyModel(M)
    p = Policy(tau=1.0, k_min=1, k_max=1, depth=4, mask_id=MASK)
    tokens, calls, log = oracle.decode_block(model, M, p)
    assert all(n == 1 and ks == 0 and nc == 0 for n, ks, _, nc in log)
    assert len(log) == M


@pytest.mark.parametrize("k", [1, 2, 3, 5])
def test_fixed_k_needs_ceil_n_over_k_iterations(k):
    M = 16
    model = ToyModel(M)
    p = Policy(tau=1.0, k_min=k, k_max=k, depth=1, mask_id=MASK)
    _, calls, log = oracle.decode_block(model, M, p)
    assert calls == math.ceil(M / k) == len(log)


def test_one_token_per_depth_with_stable_predictions():
    # k = 1 per step, agreement-only acceptance, predictions that never change: every draft is
    # accepted, so each iteration reveals 1 + (D-1) slots (one per drafted iteration).
    M, D = 16, 4
    model = ToyModel(M)
    p = Policy(tau=1.0, k_min=1, k_max=1, depth=D, accept_mode=1, mask_id=MASK)
    tokens, calls, log = oracle.decode_block(model, M, p)
    assert (tokens == model.target).all()
    assert len(log) == math.ceil(M / D)
    assert all(ks == D - 1 and ns == D - 1 for _, ks, ns, _ in log[:-1])
    assert all(K in (1, D) for K in model.calls)           # verification is one batched call over all drafts


def test_loop_always_terminates_within_m_iterations():
    for seed in range(10):
        M = 24
        model = ToyModel(M, seed=seed, stable=False)
        p = Policy(tau=0.8, k_min=1, k_max=6, depth=3, stride=2, mask_id=MASK)
        tokens, calls, log = oracle.decode_block(model, M, p)
        assert len(log) <= M and (tokens != MASK).all()
        assert sum(n + nc for n, _, _, nc in log) == M      # every slot committed exactly once


# ---- the loop with one model call per iteration ------------------------------------------------

def test_one_pass_greedy_collapse_equals_two_pass_greedy():
    # tau = 1, k = 1, D = 1: nothing exceeds tau, so an iteration is "commit the most confident slot";
    # both arrangements of Algorithm 1 then make the same calls and reveal the same slots.
    M = 12
    p = Policy(tau=1.0, k_min=1, k_max=1, depth=1, mask_id=MASK)
    a = oracle.decode_block(ToyModel(M), M, p)
    b = oracle.decode_block_one_pass(ToyModel(M), M, p)
    assert (a[0] == b[0]).all() and a[1] == b[1] == M
    assert [n for n, *_ in a[2]] == [n for n, *_ in b[2]] == [1] * M


@pytest.mark.parametrize("k", [1, 2, 3, 5])
def test_one_pass_fixed_k_without_threshold_hits(k):
    # all confidences below tau: the extra commit never fires, each call reveals exactly k slots
    M = 16
    p = Policy(tau=1.0, k_min=k, k_max=k, depth=1, mask_id=MASK)
    tokens, calls, log = oracle.decode_block_one_pass(ToyModel(M), M, p)
    assert calls == math.ceil(M / k) and (tokens != MASK).all()


def test_one_pass_stable_predictions_accept_every_draft():
    # agreement-only acceptance and predictions that never change: each call accepts the deepest draft
    # (D-1 speculated slots) and the policy adds one more, so a call reveals D slots; the first call
    # verifies copies of the empty state and reveals 1.
    M, D = 17, 4
    model = ToyModel(M)
    p = Policy(tau=1.0, k_min=1, k_max=1, depth=D, accept_mode=1, mask_id=MASK)
    tokens, calls, log = oracle.decode_block_one_pass(model, M, p)
    assert (tokens == model.target).all()
    assert log[0] == (1, 0, 0, 0)
    assert all(ks == D - 1 and ns == D - 1 for _, ks, ns, _ in log[1:-1])
    assert calls == 1 + math.ceil((M - 1) / D)
    assert all(K == D for K in model.calls)                # every call is the batched pass over D drafts


def test_one_pass_every_slot_committed_once_and_never_more_calls_than_slots():
    for seed in range(10):
        M = 24
        model = ToyModel(M, seed=seed, stable=False)
        p = Policy(tau=0.8, k_min=1, k_max=6, depth=3, stride=2, mask_id=MASK)
        tokens, calls, log = oracle.decode_block_one_pass(model, M, p)
        assert calls == len(log) <= M and (tokens != MASK).all()
        assert sum(n + nc for n, _, _, nc in log) == M


def test_policy_validation():
    for bad in (Policy(k_min=0), Policy(k_min=3, k_max=2), Policy(depth=0), Policy(tau=float("nan")),
                Policy(accept_mode=5), Policy(stride=-1)):
        with pytest.raises(ValueError):
            bad.check()
