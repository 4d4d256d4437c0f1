"""Whole-step parity (Algorithm 1, one iteration): psd_step against the oracle.

Stage-forced (the gate): the oracle's integer stages are fed the GPU's own token ids and fp32
confidences (already checked against the fp64 oracle elsewhere), so every comparison the policy,
the drafts and the acceptance make is exact and every integer output must match bit for bit.
Free-running: the oracle runs end to end in fp64; a block is set aside (and counted) if one of its
rows got a different token id on the GPU (allowed only under a top-1/top-2 logit gap of 1e-2), if a
confidence of it lies within 1e-3 of tau, or if two confidences of a node whose ranking the step
uses (the stage-1 pass and node k*) are within a relative 5e-5; every other block must match bit
for bit.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_15609_b200 as psd
import psd_inputs as gen
from psd_testlib import (STEP_INT_OUTPUTS, bf16_dev, check_confidence, golden_confidence, gpu_prologue, gpu_step,
                         oracle_prologue, oracle_step, policies, ranking_margin_ok, step_buffers_from,
                         threshold_margin_ok, weights_cached)

pytestmark = pytest.mark.gpu


MEDIUM = gen.Config("medium", B=16, H=256, V=4096, M=32, D=4, frac=0.5, s_lo=2.0, s_hi=5.5, tau=0.85, k_min=1,
                    k_max=6, seed=11)


def _workload(name, D=None):
    cfg = MEDIUM if name == "medium" else gen.CONFIGS[name]
    if D is not None:
        cfg = gen.with_depth(cfg, D)
    if name in ("tiny", "medium"):
        wl = gen.make(cfg)
        return cfg, wl, bf16_dev(wl.W)
    W, w_dev = weights_cached(name)
    return cfg, gen.make(cfg, W), w_dev


CASES = [("tiny", None), ("medium", None), ("single_request", None), ("class_7b", None), ("batched_serving", None),
         ("deep_sweep", 1), ("deep_sweep", 2), ("deep_sweep", 4), ("deep_sweep", 8)]


@pytest.mark.parametrize("name,D", CASES)
def test_step_stage_forced(name, D):
    cfg, wl, w_dev = _workload(name, D)
    po, pg = policies(cfg)
    pro_g, chain = gpu_prologue(cfg, bf16_dev(wl.hidden_stage1), w_dev, pg)
    pro_o = oracle_prologue(cfg, pro_g["tok1"], pro_g["conf1"], po)
    for k in pro_o:
        assert np.array_equal(pro_o[k], pro_g[k]), f"prologue {k}"
    buf = step_buffers_from(chain, cfg, bf16_dev(wl.hidden_verify), w_dev)
    out_g = gpu_step(buf, cfg, pg)
    out_o = oracle_step(cfg, out_g["tokV"], out_g["confV"], pro_o, po)
    for k in STEP_INT_OUTPUTS:
        assert np.array_equal(out_o[k], out_g[k]), f"step {k}"
    # the workload must exercise the method: not every block may stop at the same depth, and the
    # policy must see confidences on both sides of tau
    if cfg.D > 1 and cfg.B >= 8:
        assert len(set(out_g["k_star"].tolist())) >= 2
    assert (out_g["confV"] > cfg.tau).any() and (out_g["confV"] < cfg.tau).any()
    assert (out_g["n_sel"] >= np.minimum(cfg.k_min, (out_o["mask"] + out_o["sel"]).sum(axis=1))).all()


@pytest.mark.parametrize("name", ["tiny", "medium", "single_request", "class_7b", "batched_serving", "deep_sweep"])
def test_step_free_running(name):
    cfg, wl, w_dev = _workload(name)
    po, pg = policies(cfg)
    B, M, D = cfg.B, cfg.M, cfg.D
    pro_g, chain = gpu_prologue(cfg, bf16_dev(wl.hidden_stage1), w_dev, pg)
    buf = step_buffers_from(chain, cfg, bf16_dev(wl.hidden_verify), w_dev)
    out_g = gpu_step(buf, cfg, pg)

    if name in ("class_7b", "batched_serving", "deep_sweep"):
        # minutes of oracle time: its outputs for exactly these input bytes are read from the file its own
        # script wrote (digests checked); everything after the confidences is computed here, live
        g = golden_confidence(name, wl)
        tok1, conf1, lse1, gap1 = g["token1"], g["conf1"], g["lse1"], g["gap1"]
        tokV, confV, lseV, gapV = g["token"], g["conf"], g["lse"], g["gap"]
    else:
        tok1, conf1, lse1, gap1 = oracle.confidence(wl.hidden_stage1, wl.W)
        tokV, confV, lseV, gapV = oracle.confidence(wl.hidden_verify, wl.W)
    check_confidence(pro_g["tok1"].reshape(-1), pro_g["conf1"].reshape(-1), None, tok1, conf1, lse1, gap1)
    check_confidence(out_g["tokV"].reshape(-1), out_g["confV"].reshape(-1), None, tokV, confV, lseV, gapV)
    tok1, conf1, gap1 = tok1.reshape(B, M), conf1.reshape(B, M), gap1.reshape(B, M)
    tokV, confV, gapV = tokV.reshape(B, D, M), confV.reshape(B, D, M), gapV.reshape(B, D, M)
    pro_o = oracle_prologue(cfg, tok1, conf1, po)
    out_o = oracle_step(cfg, tokV, confV, pro_o, po)

    compared = 0
    for b in range(B):
        ks = int(out_o["k_star"][b])
        clear = np.array_equal(pro_g["tok1"][b], tok1[b]) and np.array_equal(out_g["tokV"][b], tokV[b])
        clear = clear and threshold_margin_ok(conf1[b], po.tau) and threshold_margin_ok(confV[b], po.tau)
        clear = clear and ranking_margin_ok(conf1[b]) and ranking_margin_ok(confV[b, ks])
        if not clear:
            continue
        compared += 1
        for k in pro_o:
            assert np.array_equal(pro_o[k][b], pro_g[k][b]), f"prologue {k} block {b}"
        for k in STEP_INT_OUTPUTS:
            assert np.array_equal(out_o[k][b], out_g[k][b]), f"step {k} block {b}"
    print(f"free-running {name}: compared {compared} of {B} blocks")
    # with 64 slots per block and six or more nodes a block rarely has every decision outside the margins
    assert compared >= ((B + 1) // 2 if cfg.M * cfg.D <= 128 else 1)


def test_psd_step_equals_the_four_calls_and_is_deterministic():
    cfg, wl, w_dev = _workload("tiny")
    po, pg = policies(cfg)
    B, M, D = cfg.B, cfg.M, cfg.D
    hv = bf16_dev(wl.hidden_verify)
    runs = []
    for _ in range(2):
        _, chain = gpu_prologue(cfg, bf16_dev(wl.hidden_stage1), w_dev, pg)
        runs.append(gpu_step(step_buffers_from(chain, cfg, hv, w_dev), cfg, pg))
    for k in runs[0]:
        assert np.array_equal(runs[0][k], runs[1][k]), k

    # the same step as four separate calls
    _, g = gpu_prologue(cfg, bf16_dev(wl.hidden_stage1), w_dev, pg)
    tokV = torch.zeros(B, D, M, dtype=torch.int32, device="cuda")
    confV = torch.zeros(B, D, M, dtype=torch.float32, device="cuda")
    ws = torch.empty(psd.psd_workspace_bytes(cfg.rows, cfg.H, cfg.V), dtype=torch.uint8, device="cuda")
    psd.psd_confidence(hv, w_dev, tokV.view(-1), confV.view(-1), None, ws, None)
    psd.psd_verify_accept(tokV, confV, g.sigma, g.n_fill, g.draft_tokens, g.draft_mask, pg, g.tokens_out,
                          g.mask_out, g.k_star, g.n_spec, g.n_comm, None)
    psd.psd_select_unmask(confV, tokV, g.tokens_out, g.mask_out, pg, g.sel, g.n_sel, g.sel_pos, node=g.k_star,
                          n_nodes=D)
    psd.psd_build_drafts(confV, tokV, g.tokens_out, g.mask_out, pg, g.sigma, g.n_fill, g.draft_tokens,
                         g.draft_mask, node=g.k_star, n_nodes=D)
    torch.cuda.synchronize()
    sep = dict(k_star=g.k_star, n_spec_accepted=g.n_spec, n_committed=g.n_comm, tokens=g.tokens_out,
               mask=g.mask_out, sel=g.sel, n_sel=g.n_sel, sel_pos=g.sel_pos, sigma=g.sigma, n_fill=g.n_fill,
               draft_tokens=g.draft_tokens, draft_mask=g.draft_mask)
    for k, v in sep.items():
        assert np.array_equal(v.cpu().numpy(), runs[0][k]), k


@pytest.mark.parametrize("one_block", [False, True])
@pytest.mark.parametrize("name", ["tiny", "single_request"])
def test_psd_step_host_matches_device_step(name, one_block):
    cfg, wl, w_dev = _workload(name)
    po, pg = policies(cfg)
    B, M, D = cfg.B, cfg.M, cfg.D
    _, chain = gpu_prologue(cfg, bf16_dev(wl.hidden_stage1), w_dev, pg)
    hv_dev = bf16_dev(wl.hidden_verify)
    want = gpu_step(step_buffers_from(chain, cfg, hv_dev, w_dev), cfg, pg)

    hv_host = hv_dev.cpu().pin_memory()
    if one_block:   # every array a view of one pinned block: single copies in each direction
        hb = psd.host_step_buffers(B, M, D, hv_host, w_dev)
        n, off = psd.psd_step_host_block(B, M, D)
        assert hb.n_fill.data_ptr() - hb.sigma.data_ptr() == off[1] and off[0] == 0 and n >= off[14] + 4
    else:
        hb = psd.StepBuffers.allocate(B, M, D, cfg.H, hv_host, w_dev, "cpu", pin=True)
    hb.sigma.copy_(chain.sigma)
    hb.n_fill.copy_(chain.n_fill)
    hb.draft_tokens.copy_(chain.draft_tokens)
    hb.draft_mask.copy_(chain.draft_mask)
    staging = torch.empty(psd.psd_step_host_bytes(B, M, cfg.H, cfg.V, D), dtype=torch.uint8, device="cuda")
    assert psd.psd_step_host(hb, pg, staging) == 0
    for k in STEP_INT_OUTPUTS + ("tokV", "confV"):
        assert np.array_equal(getattr(hb, k).numpy(), want[k]), k


@pytest.mark.parametrize("name,one_block", [("class_7b", True), ("batched_serving", True), ("batched_serving", False)])
def test_psd_step_host_in_two_pieces(name, one_block):
    """2048 rows or more (batched_serving) go up in two pieces whose second copy overlaps the first piece's
    kernels; class_7b (1536 rows) stays in one piece.  Either way: token ids equal to the device-resident
    step's, confidences equal up to the rounding order of another tiling, and every integer output
    what the oracle's stages make of the host path's own confidences, bit for bit."""
    cfg, wl, w_dev = _workload(name)
    po, pg = policies(cfg)
    B, M, D = cfg.B, cfg.M, cfg.D
    pro_g, chain = gpu_prologue(cfg, bf16_dev(wl.hidden_stage1), w_dev, pg)
    hv_dev = bf16_dev(wl.hidden_verify)
    want = gpu_step(step_buffers_from(chain, cfg, hv_dev, w_dev), cfg, pg)
    hv_host = hv_dev.cpu().pin_memory()
    hb = (psd.host_step_buffers(B, M, D, hv_host, w_dev) if one_block else
          psd.StepBuffers.allocate(B, M, D, cfg.H, hv_host, w_dev, "cpu", pin=True))
    staging = torch.empty(psd.psd_step_host_bytes(B, M, cfg.H, cfg.V, D), dtype=torch.uint8, device="cuda")
    for _ in range(2):                       # twice: the second call reuses the staging area and the lane
        for k in ("sigma", "n_fill", "draft_tokens", "draft_mask"):
            getattr(hb, k).copy_(getattr(chain, k))
        assert psd.psd_step_host(hb, pg, staging) == 0
        tokV, confV = hb.tokV.numpy().copy(), hb.confV.numpy().copy()
        assert np.array_equal(tokV, want["tokV"])
        assert np.abs(confV - want["confV"]).max() <= 1e-5
        pro_o = {k: pro_g[k] for k in ("sigma", "n_fill", "draft_tokens", "draft_mask")}
        out_o = oracle_step(cfg, tokV, confV, pro_o, po)
        for k in STEP_INT_OUTPUTS:
            assert np.array_equal(out_o[k], getattr(hb, k).numpy()), k


def test_psd_step_can_be_captured_in_a_cuda_graph():
    """The step is two launches with by-value tensor maps and no host synchronisation, so a stream
    capture of it replays to the same outputs as direct calls."""
    cfg, wl, w_dev = _workload("tiny")
    po, pg = policies(cfg)
    _, chain = gpu_prologue(cfg, bf16_dev(wl.hidden_stage1), w_dev, pg)
    hv = bf16_dev(wl.hidden_verify)
    ws = torch.empty(psd.psd_workspace_bytes(cfg.rows, cfg.H, cfg.V), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ref = step_buffers_from(chain, cfg, hv, w_dev)
    for _ in range(3):
        psd.psd_step(ref, pg, ws, status)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    buf = step_buffers_from(chain, cfg, hv, w_dev)
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            psd.psd_step(buf, pg, ws, status, side)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for k in STEP_INT_OUTPUTS + ("tokV", "confV"):
        assert torch.equal(getattr(buf, k), getattr(ref, k)), k
