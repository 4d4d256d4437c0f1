"""Row compaction (Sec. 3.2 Stage 3 scores "each masked position" of each draft): psd_confidence with a
row list, and psd_step scoring only the rows of slots still masked in their draft.  Gates: the row-list
results against the fp64 oracle on the listed rows; the compacted step stage-forced against the
oracle's integer stages, bit for bit, over several consecutive steps as the blocks fill up."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_15609_b200 as psd
import psd_inputs as gen
from psd_testlib import (STEP_INT_OUTPUTS, bf16_dev, check_confidence, dev, gpu_prologue, np_, oracle_prologue,
                         oracle_step, policies, step_buffers_from, weights_cached)

pytestmark = pytest.mark.gpu


@pytest.fixture
def compaction():
    def turn(mode):
        assert psd.psd_set_tuning(psd.PSD_TUNE_COMPACT_ROWS, mode) == 0
    yield turn
    psd.psd_set_tuning(psd.PSD_TUNE_COMPACT_ROWS, 0)


def _conf_rows(h_dev, w_dev, row_ids, impl=0):
    n = len(row_ids)
    H, V = h_dev.shape[1], w_dev.shape[0]
    tok = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    conf = torch.zeros(n, dtype=torch.float32, device="cuda")
    lse = torch.zeros(n, dtype=torch.float32, device="cuda")
    ws = torch.empty(psd.psd_compact_workspace_bytes(n, H, V), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    prev = psd.psd_set_confidence_impl(impl)
    try:
        psd.psd_confidence(h_dev, w_dev, tok, conf, lse, ws, status, row_ids=dev(np.asarray(row_ids, dtype=np.int32)))
        torch.cuda.synchronize()
    finally:
        psd.psd_set_confidence_impl(prev)
    assert int(status.item()) == 0
    return np_(tok), np_(conf), np_(lse)


@pytest.mark.parametrize("impl", [0, 1, 3])
@pytest.mark.parametrize("n_list", [1, 77, 128, 300])
def test_confidence_with_a_row_list(n_list, impl):
    rng = np.random.default_rng(n_list)
    R, H, V = 500, 192, 3001
    W = gen.bf16_bits(rng.normal(scale=0.05, size=(V, H)).astype(np.float32))
    hid = rng.normal(size=(R, H)).astype(np.float32)
    Wf = gen.bf16_to_f64(W)
    for r in range(0, R, 2):
        t = int(rng.integers(0, V))
        hid[r] += (rng.uniform(3.0, 10.0) / float(Wf[t] @ Wf[t])) * Wf[t]
    hid = gen.bf16_bits(hid)
    rows = rng.integers(0, R, size=n_list)            # any order, repeats allowed
    rows[0] = R - 1
    tok_o, conf_o, lse_o, gap_o = oracle.confidence(hid[rows], W)
    tok_g, conf_g, lse_g = _conf_rows(bf16_dev(hid), bf16_dev(W), rows, impl)
    check_confidence(tok_g, conf_g, lse_g, tok_o, conf_o, lse_o, gap_o)


MEDIUM = gen.Config("medium_c", B=16, H=256, V=4096, M=32, D=4, frac=0.6, s_lo=2.0, s_hi=5.5, tau=0.7, k_min=1,
                    k_max=6, seed=12)


def _workload(name):
    if name == "medium":
        wl = gen.make(MEDIUM)
        return MEDIUM, wl, bf16_dev(wl.W)
    cfg = gen.CONFIGS[name]
    W, w_dev = weights_cached(name)
    return cfg, gen.make(cfg, W), w_dev


@pytest.mark.parametrize("name,mode", [("tiny", 2), ("medium", 2), ("medium", 1), ("single_request", 2),
                                       ("batched_serving", 1)])
def test_compacted_steps_stage_forced(name, mode, compaction):
    cfg, wl, w_dev = _workload(name)
    po, pg = policies(cfg)
    pro_g, chain = gpu_prologue(cfg, bf16_dev(wl.hidden_stage1), w_dev, pg)
    state = oracle_prologue(cfg, pro_g["tok1"], pro_g["conf1"], po)
    hv = bf16_dev(wl.hidden_verify)
    buf = step_buffers_from(chain, cfg, hv, w_dev)
    ws = torch.empty(psd.psd_compact_workspace_bytes(cfg.rows, cfg.H, cfg.V), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # the same steps without compaction, for the comparison of the predictions themselves
    ref = step_buffers_from(chain, cfg, hv, w_dev)
    scored_fraction = []
    for step in range(4 if cfg.rows <= 2048 else 2):
        masked_rows = np_(buf.draft_mask).reshape(-1) != 0
        compaction(0)
        psd.psd_step(ref, pg, ws, status)
        compaction(mode)
        buf.tokV.fill_(-5)
        buf.confV.fill_(-5.0)
        psd.psd_step(buf, pg, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        tokV, confV = np_(buf.tokV), np_(buf.confV)
        used = mode == 2 or cfg.rows > 128
        if used:
            # rows of committed slots were not scored and are left alone
            assert (tokV.reshape(-1)[~masked_rows] == -5).all()
        assert np.array_equal(tokV.reshape(-1)[masked_rows], np_(ref.tokV).reshape(-1)[masked_rows])
        assert np.allclose(confV.reshape(-1)[masked_rows], np_(ref.confV).reshape(-1)[masked_rows], rtol=1e-5, atol=0)
        want = oracle_step(cfg, tokV, confV.astype(np.float64), state, po)
        for k in STEP_INT_OUTPUTS:
            assert np.array_equal(want[k], np_(getattr(buf, k))), f"step {step}: {k}"
            assert np.array_equal(want[k], np_(getattr(ref, k))), f"step {step}: {k} (no compaction)"
        state = {k: want[k] for k in ("sigma", "n_fill", "draft_tokens", "draft_mask", "tokens", "mask")}
        scored_fraction.append(float(masked_rows.mean()))
    assert scored_fraction[-1] < scored_fraction[0] <= 1.0          # the blocks fill up, fewer rows are scored


def test_small_workspace_is_rejected(compaction):
    cfg, wl, w_dev = _workload("tiny")
    po, pg = policies(cfg)
    pro_g, chain = gpu_prologue(cfg, bf16_dev(wl.hidden_stage1), w_dev, pg)
    buf = step_buffers_from(chain, cfg, bf16_dev(wl.hidden_verify), w_dev)
    ws = torch.empty(psd.psd_workspace_bytes(cfg.rows, cfg.H, cfg.V), dtype=torch.uint8, device="cuda")
    compaction(2)
    with pytest.raises(psd.PsdError) as e:
        psd.psd_step(buf, pg, ws, None)
    assert e.value.code == psd.PSD_ERR_WORKSPACE
    compaction(0)
    psd.psd_step(buf, pg, ws, None)
    torch.cuda.synchronize()


@pytest.mark.parametrize("impl", [0, 1, 3])
@pytest.mark.parametrize("R,frac", [(1, 1.0), (130, 0.5), (300, 0.1), (300, 0.0), (700, 0.9)])
def test_confidence_masked(R, frac, impl):
    rng = np.random.default_rng(R + int(frac * 10))
    H, V = 128, 2500
    W = gen.bf16_bits(rng.normal(scale=0.05, size=(V, H)).astype(np.float32))
    hid = gen.bf16_bits((rng.normal(size=(R, H)) * rng.uniform(0.5, 6.0, size=(R, 1))).astype(np.float32))
    flags = (rng.random(R) < frac).astype(np.int32)
    tok = torch.full((R,), -7, dtype=torch.int32, device="cuda")
    conf = torch.full((R,), -7.0, dtype=torch.float32, device="cuda")
    lse = torch.full((R,), -7.0, dtype=torch.float32, device="cuda")
    ws = torch.empty(psd.psd_compact_workspace_bytes(R, H, V), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    prev = psd.psd_set_confidence_impl(impl)
    try:
        psd.psd_confidence_masked(bf16_dev(hid), bf16_dev(W), dev(flags), tok, conf, lse, ws, status)
        torch.cuda.synchronize()
    finally:
        psd.psd_set_confidence_impl(prev)
    assert int(status.item()) == 0
    tok, conf, lse = np_(tok), np_(conf), np_(lse)
    on = flags != 0
    assert (tok[~on] == -7).all() and (conf[~on] == -7.0).all() and (lse[~on] == -7.0).all()
    if on.any():
        tok_o, conf_o, lse_o, gap_o = oracle.confidence(hid[on], W)
        check_confidence(tok[on], conf[on], lse[on], tok_o, conf_o, lse_o, gap_o)


def test_host_step_with_compaction(compaction):
    """psd_step_host sizes its staging for the compacted path too."""
    cfg, wl, w_dev = _workload("medium")
    po, pg = policies(cfg)
    _, chain = gpu_prologue(cfg, bf16_dev(wl.hidden_stage1), w_dev, pg)
    hv_dev = bf16_dev(wl.hidden_verify)
    ref = step_buffers_from(chain, cfg, hv_dev, w_dev)
    ws = torch.empty(psd.psd_workspace_bytes(cfg.rows, cfg.H, cfg.V), dtype=torch.uint8, device="cuda")
    psd.psd_step(ref, pg, ws, None)
    torch.cuda.synchronize()
    hb = psd.host_step_buffers(cfg.B, cfg.M, cfg.D, hv_dev.cpu().pin_memory(), w_dev)
    for k in ("sigma", "n_fill", "draft_tokens", "draft_mask"):
        getattr(hb, k).copy_(getattr(chain, k))
    staging = torch.empty(psd.psd_step_host_bytes(cfg.B, cfg.M, cfg.H, cfg.V, cfg.D), dtype=torch.uint8, device="cuda")
    compaction(2)
    assert psd.psd_step_host(hb, pg, staging) == 0
    for k in STEP_INT_OUTPUTS:
        assert np.array_equal(getattr(hb, k).numpy(), np_(getattr(ref, k))), k
