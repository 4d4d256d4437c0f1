"""Pins for the confidence oracle (Sec. 3.1: x^ = argmax_v p(v), c = max_v p(v)).

Nothing here compares the oracle with itself: each test checks it against a closed form,
a library routine on a case that reduces to it, brute force, or an invariant.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
import psd_inputs as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "softmax_closed_forms.txt")


def _bits(a):
    return gen.bf16_bits(np.asarray(a, dtype=np.float32))


def _golden_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, lg, am, pr = [x.strip() for x in line.split("|")]
            rows.append((name, [float(x) for x in lg.split()], int(am), float(pr)))
    return rows


@pytest.mark.parametrize("name,lg,am,pr", _golden_rows())
def test_row_stats_closed_forms(name, lg, am, pr):
    tok, conf, lse, gap = oracle.row_stats(lg)
    assert tok == am
    assert abs(conf - pr) < 1e-12
    # conf = exp(m - lse)
    assert abs(math.exp(max(lg) - lse) - conf) < 1e-14
    srt = sorted(lg, reverse=True)
    assert abs(gap - (srt[0] - srt[1])) < 1e-15


def test_all_equal_logits_give_uniform_and_lowest_index():
    # hidden = 0 makes every logit 0 whatever W is.
    V, H = 37, 8
    W = _bits(np.random.default_rng(0).normal(size=(V, H)))
    hid = _bits(np.zeros((3, H)))
    tok, conf, lse, gap = oracle.confidence(hid, W)
    assert (tok == 0).all()
    assert np.allclose(conf, 1.0 / V, rtol=0, atol=1e-15)
    assert np.allclose(lse, math.log(V), atol=1e-14)
    assert (gap == 0).all()


def test_one_hot_closed_form():
    # W = identity-like (V = H), hidden = a * e_j: logits are a at v = j and 0 elsewhere,
    # so conf = 1 / (1 + (V-1) e^-a) and the token is j.
    V = H = 16
    W = _bits(np.eye(V))
    for j, a in [(0, 1.0), (5, 2.5), (15, 8.0)]:
        hid = np.zeros((1, H), dtype=np.float32)
        hid[0, j] = a
        tok, conf, lse, gap = oracle.confidence(_bits(hid), W)
        assert tok[0] == j
        assert abs(conf[0] - 1.0 / (1.0 + (V - 1) * math.exp(-a))) < 1e-14
        assert abs(gap[0] - a) < 1e-15
    # negative a: every other entry ties at 0 -> lowest other index wins
    hid = np.zeros((1, H), dtype=np.float32)
    hid[0, 0] = -3.0
    tok, conf, _, gap = oracle.confidence(_bits(hid), W)
    assert tok[0] == 1 and gap[0] == 0.0
    assert abs(conf[0] - 1.0 / ((V - 1) + math.exp(-3.0))) < 1e-14


def test_hand_checkable_integers():
    # H = 2, V = 3: hidden (1, 2); W rows (1,0), (0,1), (1,1) -> logits (1, 2, 3).
    hid = _bits([[1.0, 2.0]])
    W = _bits([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]])
    lg = oracle.logits(hid, W)
    assert lg.tolist() == [[1.0, 2.0, 3.0]]
    tok, conf, lse, gap = oracle.confidence(hid, W)
    assert tok[0] == 2 and abs(conf[0] - 0.66524095577482) < 1e-13 and gap[0] == 1.0


def test_operand_orientation_not_transposed():
    # Non-square, asymmetric case with exactly representable values: logits[r, v] must pair
    # hidden row r with W row v (both contract over their last axis).
    hid = np.array([[1, 0, 2], [0, 3, 1]], dtype=np.float32)          # [2, 3]
    W = np.array([[1, 1, 0], [0, 2, 1], [4, 0, 0], [0, 0, 5]], dtype=np.float32)  # [4, 3]
    lg = oracle.logits(_bits(hid), _bits(W))
    expect = [[1, 2, 4, 10], [3, 7, 0, 5]]
    assert lg.tolist() == expect
    tok, _, _, _ = oracle.confidence(_bits(hid), _bits(W))
    assert tok.tolist() == [3, 1]


def test_against_library_softmax_float64():
    # A case that reduces to library routines: fp64 matmul + torch.softmax + max.
    rng = np.random.default_rng(7)
    R, H, V = 9, 64, 301
    hid = _bits(rng.normal(size=(R, H)))
    W = _bits(rng.normal(scale=0.3, size=(V, H)))
    tok, conf, lse, gap = oracle.confidence(hid, W)
    h64 = torch.from_numpy(gen.bf16_to_f64(hid))
    w64 = torch.from_numpy(gen.bf16_to_f64(W))
    lg = h64 @ w64.T
    p = torch.softmax(lg, dim=1)
    pm, am = p.max(dim=1)
    assert tok.tolist() == am.tolist()
    assert np.allclose(conf, pm.numpy(), rtol=1e-12, atol=0)
    assert np.allclose(lse, torch.logsumexp(lg, dim=1).numpy(), rtol=0, atol=1e-11)
    top2 = torch.topk(lg, 2, dim=1).values
    assert np.allclose(gap, (top2[:, 0] - top2[:, 1]).numpy(), atol=1e-11)


def test_softmax_sums_to_one_and_bounds():
    rng = np.random.default_rng(3)
    R, H, V = 5, 32, 200
    hid = _bits(rng.normal(size=(R, H)))
    W = _bits(rng.normal(size=(V, H)))
    lg = oracle.logits(hid, W)
    tok, conf, lse, _ = oracle.confidence(hid, W)
    for r in range(R):
        total = math.fsum(math.exp(x - lse[r]) for x in lg[r])
        assert abs(total - 1.0) < 1e-12
        assert abs(conf[r] - math.exp(lg[r].max() - lse[r])) < 1e-13
        assert 1.0 / V <= conf[r] <= 1.0
        assert lg[r, tok[r]] == lg[r].max()


def test_brute_force_tiny_vocab():
    # V <= 16, H <= 8, small integers: probabilities by exact enumeration in Python.
    rng = np.random.default_rng(11)
    for _ in range(20):
        H = int(rng.integers(1, 9))
        V = int(rng.integers(1, 17))
        hid = rng.integers(-2, 3, size=(2, H)).astype(np.float32)
        W = rng.integers(-2, 3, size=(V, H)).astype(np.float32)
        tok, conf, _, _ = oracle.confidence(_bits(hid), _bits(W))
        for r in range(2):
            lg = [sum(int(hid[r, j]) * int(W[v, j]) for j in range(H)) for v in range(V)]
            best = max(lg)
            denom = math.fsum(math.exp(x - best) for x in lg)
            assert tok[r] == lg.index(best)
            assert abs(conf[r] - 1.0 / denom) < 1e-14


def test_bf16_widening_is_exact():
    # bf16 values with a full 8-bit significand; products and the 2-term sum are exact in fp64.
    a, b = 1.0078125, -3.984375       # 1 + 2^-7, -(4 - 2^-6): both exact in bf16
    hid = _bits([[a, b]])
    assert gen.bf16_to_f64(hid).tolist() == [[a, b]]
    W = _bits([[b, a]])
    assert oracle.logits(hid, W)[0, 0] == a * b + b * a


def test_split_vocabulary_merge_matches_single_pass():
    # The (max, sum-exp, argmax) triple of a row can be merged over any split of the vocabulary:
    # merging the oracle's results on the pieces must reproduce its result on the whole.
    rng = np.random.default_rng(5)
    H, V = 16, 96
    hid = _bits(rng.normal(size=(4, H)))
    W = _bits(rng.normal(size=(V, H)))
    tok, conf, lse, _ = oracle.confidence(hid, W)
    for cuts in ([0, 96], [0, 1, 96], [0, 32, 64, 96], [0, 7, 50, 51, 96]):
        for r in range(4):
            parts = []
            for a, b in zip(cuts[:-1], cuts[1:]):
                t, c, l, _ = oracle.confidence(hid[r:r + 1], W[a:b])
                parts.append((l[0] + math.log(c[0]), l[0], t[0] + a))   # (max, lse, idx)
            m = max(p[0] for p in parts)
            idx = min(p[2] for p in parts if p[0] == m)
            total = m + math.log(math.fsum(math.exp(p[1] - m) for p in parts))
            assert idx == tok[r]
            assert abs(total - lse[r]) < 1e-12
            assert abs(math.exp(m - total) - conf[r]) < 1e-13
