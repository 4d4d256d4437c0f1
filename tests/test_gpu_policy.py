"""GPU parity of psd_select_unmask / psd_build_drafts / psd_verify_accept against the oracle on the
same inputs: every integer output bit-exact (Sec. 3.2, Eq. (1), Eq. (2), Algorithm 1)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_15609_b200 as psd
from psd_testlib import GpuChain, dev, f32, np_

pytestmark = pytest.mark.gpu
MASK_ID = 70000


def _case(seed, B, M, n_nodes=1, p_masked=0.6, quant=None, with_nan=False):
    rng = np.random.default_rng(seed)
    conf = rng.random((B, n_nodes, M)).astype(np.float32)
    if quant:
        conf = (np.round(conf * quant) / quant).astype(np.float32)      # many exact ties
    if with_nan:
        conf[rng.random(conf.shape) < 0.05] = np.nan
    tok = rng.integers(0, 60000, size=(B, n_nodes, M)).astype(np.int32)
    mask = (rng.random((B, M)) < p_masked).astype(np.int32)
    if B > 2:
        mask[0] = 0          # a finished block
        mask[1] = 1          # a fresh block
    tokens = np.where(mask == 1, MASK_ID, rng.integers(0, 60000, size=(B, M))).astype(np.int32)
    node = rng.integers(0, n_nodes, size=B).astype(np.int32)
    return conf, tok, tokens, mask, node


def _pols(tau, k_min, k_max, D, stride, mode=0):
    tau = f32(tau)
    return (oracle.Policy(tau=tau, k_min=k_min, k_max=k_max, depth=D, stride=stride, accept_mode=mode, mask_id=MASK_ID),
            psd.policy(tau=tau, k_min=k_min, k_max=k_max, depth=D, stride=stride, accept_mode=mode, mask_id=MASK_ID))


SHAPES = [(1, 32), (5, 1), (7, 33), (16, 64), (3, 100), (2, 1024), (64, 32)]
POLS = [(0.9, 1, 0, 4, 0), (0.5, 2, 5, 3, 2), (1.0, 1, 1, 1, 0), (-1.0, 1, 0, 6, 3), (0.8, 4, 4, 6, 4),
        (0.3, 1, 8, 64, 1)]


def _run_select(conf, tok, tokens, mask, node, n_nodes, pg):
    B, M = mask.shape
    g = GpuChain(B, M, 1)
    t_d, m_d = dev(tokens), dev(mask)
    psd.psd_select_unmask(dev(conf), dev(tok), t_d, m_d, pg, g.sel, g.n_sel, g.sel_pos,
                          node=None if node is None else dev(node), n_nodes=n_nodes)
    torch.cuda.synchronize()
    return np_(t_d), np_(m_d), np_(g.sel), np_(g.n_sel), np_(g.sel_pos)


@pytest.mark.parametrize("B,M", SHAPES)
@pytest.mark.parametrize("pol", POLS)
def test_select_unmask_parity(B, M, pol):
    tau, k_min, k_max, D, stride = pol
    for seed, quant, nan in ((1, None, False), (2, 8, False), (3, None, True)):
        n_nodes = 1 + seed % 3
        conf, tok, tokens, mask, node = _case(seed * 100 + M, B, M, n_nodes, quant=quant, with_nan=nan)
        po, pg = _pols(tau, k_min, k_max, D, stride)
        rows = np.arange(B)
        want = oracle.select_unmask(conf[rows, node], tok[rows, node], tokens, mask, po)
        got = _run_select(conf, tok, tokens, mask, node, n_nodes, pg)
        for w, g_, name in zip(want, got, ("tokens", "mask", "sel", "n_sel", "sel_pos")):
            assert np.array_equal(w, g_), name


def test_select_default_node_is_zero():
    conf, tok, tokens, mask, _ = _case(5, 4, 32, 3)
    po, pg = _pols(0.5, 1, 0, 2, 0)
    want = oracle.select_unmask(conf[:, 0], tok[:, 0], tokens, mask, po)
    got = _run_select(conf, tok, tokens, mask, None, 3, pg)
    for w, g_ in zip(want, got):
        assert np.array_equal(w, g_)


def _run_build(conf, tok, tokens, mask, node, n_nodes, pg, D):
    B, M = mask.shape
    g = GpuChain(B, M, D)
    psd.psd_build_drafts(dev(conf), dev(tok), dev(tokens), dev(mask), pg, g.sigma, g.n_fill, g.draft_tokens,
                         g.draft_mask, node=dev(node), n_nodes=n_nodes)
    torch.cuda.synchronize()
    return np_(g.sigma), np_(g.n_fill), np_(g.draft_tokens), np_(g.draft_mask)


@pytest.mark.parametrize("B,M", SHAPES)
@pytest.mark.parametrize("pol", POLS)
def test_build_drafts_parity(B, M, pol):
    tau, k_min, k_max, D, stride = pol
    for seed, quant, nan in ((11, None, False), (12, 4, True)):
        n_nodes = 1 + seed % 2
        conf, tok, tokens, mask, node = _case(seed * 100 + M, B, M, n_nodes, quant=quant, with_nan=nan)
        po, pg = _pols(tau, k_min, k_max, D, stride)
        rows = np.arange(B)
        want = oracle.build_drafts(conf[rows, node], tok[rows, node], tokens, mask, po)
        got = _run_build(conf, tok, tokens, mask, node, n_nodes, pg, D)
        for w, g_, name in zip(want, got, ("sigma", "n_fill", "draft_tokens", "draft_mask")):
            assert np.array_equal(w, g_), name


def _verify_inputs(seed, B, M, po, agree=0.85):
    rng = np.random.default_rng(seed)
    conf, tok, tokens, mask, _ = _case(seed, B, M, 1, p_masked=0.8)
    conf, tok = conf[:, 0], tok[:, 0]
    D = po.depth
    sigma, n_fill, dt, dm = oracle.build_drafts(conf, tok, tokens, mask, po)
    tokV = np.repeat(tok[:, None, :], D, axis=1).copy()
    tokV[rng.random(tokV.shape) > agree] += 1
    confV = (rng.random((B, D, M)) ** 0.25).astype(np.float32)
    return sigma, n_fill, dt, dm, tokV.astype(np.int32), confV


@pytest.mark.parametrize("B,M", SHAPES)
@pytest.mark.parametrize("pol", POLS)
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_verify_accept_parity(B, M, pol, mode):
    tau, k_min, k_max, D, stride = pol
    po, pg = _pols(tau, k_min, k_max, D, stride, mode)
    depths = set()
    for seed in (21, 22, 23):
        sigma, n_fill, dt, dm, tokV, confV = _verify_inputs(seed * 10 + M, B, M, po, agree=0.8 + 0.06 * (seed - 21))
        want = oracle.verify_accept(tokV, confV, sigma, n_fill, dt, dm, po)
        g = GpuChain(B, M, D)
        psd.psd_verify_accept(dev(tokV), dev(confV), dev(sigma), dev(n_fill), dev(dt), dev(dm), pg, g.tokens_out,
                              g.mask_out, g.k_star, g.n_spec, g.n_comm, g.accepted)
        torch.cuda.synchronize()
        got = (np_(g.tokens_out), np_(g.mask_out), np_(g.k_star), np_(g.n_spec), np_(g.n_comm), np_(g.accepted))
        for w, g_, name in zip(want, got, ("tokens", "mask", "k_star", "n_spec", "n_committed", "accepted")):
            assert np.array_equal(w, g_), name
        depths.update(want[2].tolist())
    if D >= 3 and mode == 1 and B >= 16 and stride <= 2:
        assert len(depths) >= 2          # the inputs exercise more than one acceptance depth


def test_verify_accept_without_accepted_output_and_degenerate_chains():
    po, pg = _pols(0.9, 1, 0, 1, 0)      # D = 1: the root only
    sigma, n_fill, dt, dm, tokV, confV = _verify_inputs(99, 4, 32, po)
    want = oracle.verify_accept(tokV, confV, sigma, n_fill, dt, dm, po)
    g = GpuChain(4, 32, 1)
    psd.psd_verify_accept(dev(tokV), dev(confV), dev(sigma), dev(n_fill), dev(dt), dev(dm), pg, g.tokens_out,
                          g.mask_out, g.k_star, g.n_spec, g.n_comm, None)
    torch.cuda.synchronize()
    assert np.array_equal(want[0], np_(g.tokens_out)) and np.array_equal(want[1], np_(g.mask_out))
    assert (np_(g.k_star) == 0).all() and np.array_equal(want[4], np_(g.n_comm))
