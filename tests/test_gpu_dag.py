"""GPU parity of psd_build_drafts_dag / psd_verify_accept_dag against the oracle's draft-graph stages on
the same inputs: every integer output bit-exact (Sec. 3.2 Stages 2-3 with a multi-parent DAG; Eq. (2);
Algorithm 1 Stage 3), plus the chain as a special case and one pass through the real pipeline
(stand-in body -> psd_confidence on the K drafts -> acceptance)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_15609_b200 as psd
import psd_inputs as gen
from psd_testlib import bf16_dev, dev, f32, gpu_confidence, np_

pytestmark = pytest.mark.gpu
MASK_ID = 70000

GRAPHS = {
    "root_only": [set()],
    "diamond": [set(), {0}, {1}, {0, 1}],
    "calibrated_like": [set(), {0}, {0, 1}, {1}, {0, 2}, {0, 1, 2}, {0, 1, 2, 3}, {2, 3}, {0, 1, 2, 3, 4, 5}],
    "chain_stride3": oracle.chain_as_dag(6, 3),
    "deep_ranks": [set(), {63}, {0, 63}, {0, 31, 32, 63}, set(range(64)), set(range(0, 64, 2))],
}


def _random_graph(seed, K, max_rank):
    rng = np.random.default_rng(seed)
    nodes = [set()]
    while len(nodes) < K:
        size = int(rng.integers(1, min(max_rank, 8) + 1))
        nodes.append(set(int(x) for x in rng.choice(max_rank, size=size, replace=False)))
    return nodes


GRAPHS["random_64_nodes"] = _random_graph(7, 64, 24)
GRAPHS["random_20_nodes"] = _random_graph(8, 20, 10)


def _state(seed, B, M, p_masked):
    rng = np.random.default_rng(seed)
    conf = rng.random((B, 1, M)).astype(np.float32)
    conf[rng.random(conf.shape) < 0.1] = np.float32(0.5)              # exact ties
    tok = rng.integers(0, 60000, size=(B, 1, M)).astype(np.int32)
    mask = (rng.random((B, M)) < p_masked).astype(np.int32)
    if B > 2:
        mask[0] = 0
        mask[1] = 1
    tokens = np.where(mask == 1, MASK_ID, rng.integers(0, 60000, size=(B, M))).astype(np.int32)
    return conf, tok, tokens, mask


def _pols(tau, k_min, k_max, mode):
    tau = f32(tau)
    return (oracle.Policy(tau=tau, k_min=k_min, k_max=k_max, depth=1, accept_mode=mode, mask_id=MASK_ID),
            psd.policy(tau=tau, k_min=k_min, k_max=k_max, depth=1, accept_mode=mode, mask_id=MASK_ID))


def _gpu_build(conf, tok, tokens, mask, pg, g, K):
    B, M = mask.shape
    i32 = lambda *s: torch.full(s, -9, dtype=torch.int32, device="cuda")
    sigma, n_fill, dt, dm = i32(B, M), i32(B, K), i32(B, K, M), i32(B, K, M)
    psd.psd_build_drafts_dag(dev(conf), dev(tok), dev(tokens), dev(mask), pg, g, sigma, n_fill, dt, dm)
    torch.cuda.synchronize()
    return np_(sigma), np_(n_fill), np_(dt), np_(dm)


def _gpu_accept(tokV, confV, sigma, dt, dm, pg, g, K):
    B, M = sigma.shape
    i32 = lambda *s: torch.full(s, -9, dtype=torch.int32, device="cuda")
    tokens, mask, ks, ns, nc, acc = i32(B, M), i32(B, M), i32(B), i32(B), i32(B), i32(B, K)
    psd.psd_verify_accept_dag(dev(tokV), dev(confV), dev(sigma), dev(dt), dev(dm), pg, g, tokens, mask, ks, ns, nc, acc)
    torch.cuda.synchronize()
    return np_(tokens), np_(mask), np_(ks), np_(ns), np_(nc), np_(acc)


NAMES = ("tokens", "mask", "k_star", "n_spec_accepted", "n_committed", "accepted")


@pytest.mark.parametrize("B,M", [(1, 32), (9, 64), (4, 5), (3, 200), (2, 1024)])
@pytest.mark.parametrize("name", list(GRAPHS))
def test_build_and_accept_parity(name, B, M):
    ranks = GRAPHS[name]
    K = len(ranks)
    g = psd.psd_dag_init(ranks)
    for seed, p_masked, mode, tau in ((1, 0.9, 0, 0.5), (2, 0.5, 1, 0.5), (3, 0.8, 2, 0.6), (4, 0.15, 0, 0.3)):
        conf, tok, tokens, mask = _state(seed * 1000 + M + K, B, M, p_masked)
        po, pg = _pols(tau, 1 + seed % 2, 0 if seed % 2 else 6, mode)
        want = oracle.build_drafts_dag(conf[:, 0], tok[:, 0], tokens, mask, po, ranks)
        got = _gpu_build(conf, tok, tokens, mask, pg, g, K)
        for w, x, n in zip(want, got, ("sigma", "n_fill", "draft_tokens", "draft_mask")):
            assert np.array_equal(w, x), n
        sigma, n_fill, dt, dm = want
        rng = np.random.default_rng(seed)
        tokV = np.where(rng.random((B, K, M)) < 0.85, tok, 77777).astype(np.int32)
        confV = (rng.random((B, K, M)) * 0.7 + 0.3).astype(np.float32)
        want = oracle.verify_accept_dag(tokV, confV, sigma, dt, dm, po, ranks)
        got = _gpu_accept(tokV, confV, sigma, dt, dm, pg, g, K)
        for w, x, n in zip(want, got, NAMES):
            assert np.array_equal(w, x), f"{n} mode {mode}"


def test_explicit_edges_and_chain_equivalence():
    D, step, B, M = 5, 2, 12, 32
    ranks = oracle.chain_as_dag(D, step)
    edges = [(d - 1, d) for d in range(1, D)]
    g_path = psd.psd_dag_init(ranks, edges)
    g_full = psd.psd_dag_init(ranks)
    conf, tok, tokens, mask = _state(11, B, M, 0.8)
    tau = f32(0.55)
    po = oracle.Policy(tau=tau, k_min=step, depth=D, stride=step, mask_id=MASK_ID)
    pg = psd.policy(tau=tau, k_min=step, depth=D, stride=step, mask_id=MASK_ID)
    sigma, n_fill, dt, dm = _gpu_build(conf, tok, tokens, mask, pg, g_path, D)
    rng = np.random.default_rng(3)
    tokV = np.where(rng.random((B, D, M)) < 0.8, tok, 77777).astype(np.int32)
    confV = (rng.random((B, D, M)) * 0.6 + 0.4).astype(np.float32)
    # the chain entry points on the same data
    i32 = lambda *s: torch.full(s, -9, dtype=torch.int32, device="cuda")
    c_sigma, c_fill, c_dt, c_dm = i32(B, M), i32(B, D), i32(B, D, M), i32(B, D, M)
    psd.psd_build_drafts(dev(conf), dev(tok), dev(tokens), dev(mask), pg, c_sigma, c_fill, c_dt, c_dm)
    for a, b in zip((sigma, n_fill, dt, dm), (c_sigma, c_fill, c_dt, c_dm)):
        assert np.array_equal(a, np_(b))
    t, m, ks, ns, nc, acc = i32(B, M), i32(B, M), i32(B), i32(B), i32(B), i32(B, D)
    psd.psd_verify_accept(dev(tokV), dev(confV), c_sigma, c_fill, c_dt, c_dm, pg, t, m, ks, ns, nc, acc)
    torch.cuda.synchronize()
    chain = tuple(np_(x) for x in (t, m, ks, ns, nc, acc))
    path = _gpu_accept(tokV, confV, sigma, dt, dm, pg, g_path, D)
    for a, b, n in zip(chain, path, NAMES):
        assert np.array_equal(a, b), n
    full = _gpu_accept(tokV, confV, sigma, dt, dm, pg, g_full, D)
    want = oracle.verify_accept_dag(tokV, confV, sigma, dt, dm, po, ranks)
    for a, b, n in zip(want, full, NAMES):
        assert np.array_equal(a, b), n
    assert (full[3] >= path[3]).all() and (full[3] > path[3]).any()     # the extra edges rescue some nodes


def test_graph_through_the_pipeline():
    """Stage-1 pass -> policy -> drafts of a graph -> stand-in body -> psd_confidence on all K drafts ->
    acceptance; the oracle's integer stages get the GPU's own predictions (stage-forced)."""
    cfg = gen.Config("dagpipe", B=8, H=256, V=2048, M=32, D=1, frac=0.8, tau=0.6, k_min=1, k_max=6, seed=31)
    ranks = GRAPHS["calibrated_like"]
    K = len(ranks)
    g = psd.psd_dag_init(ranks)
    B, M, H = cfg.B, cfg.M, cfg.H
    W = gen.weights(cfg)
    table, *_ = gen.table_body(cfg, W)
    flat = table.reshape(-1, H)
    w_dev, t_dev = bf16_dev(W), bf16_dev(flat)
    tau = f32(cfg.tau)
    po = oracle.Policy(tau=tau, k_min=1, k_max=6, depth=1, mask_id=cfg.mask_id)
    pg = psd.policy(tau=tau, k_min=1, k_max=6, depth=1, mask_id=cfg.mask_id)
    user = psd.table_body_user(t_dev.view(B, M, 3, H), B)
    i32 = lambda *s: torch.full(s, -9, dtype=torch.int32, device="cuda")
    tokens = torch.full((B, M), cfg.mask_id, dtype=torch.int32, device="cuda")
    mask = torch.ones((B, M), dtype=torch.int32, device="cuda")
    hidden = torch.zeros(B * K * M, H, dtype=torch.bfloat16, device="cuda")
    psd.psd_table_body(user, mask, hidden)
    tok1, conf1, _ = gpu_confidence(hidden[:B * M], w_dev, want_lse=False)
    tok1, conf1 = tok1.reshape(B, 1, M), conf1.reshape(B, 1, M)
    sel, n_sel, sel_pos = i32(B, M), i32(B), i32(B, M)
    psd.psd_select_unmask(dev(conf1), dev(tok1), tokens, mask, pg, sel, n_sel, sel_pos)
    o_tokens, o_mask, *_ = oracle.select_unmask(conf1[:, 0], tok1[:, 0], np.full((B, M), cfg.mask_id, np.int32),
                                                np.ones((B, M), np.int32), po)
    assert np.array_equal(np_(tokens), o_tokens) and np.array_equal(np_(mask), o_mask)
    sigma, n_fill, dt, dm = i32(B, M), i32(B, K), i32(B, K, M), i32(B, K, M)
    psd.psd_build_drafts_dag(dev(conf1), dev(tok1), tokens, mask, pg, g, sigma, n_fill, dt, dm)
    want = oracle.build_drafts_dag(conf1[:, 0], tok1[:, 0], o_tokens, o_mask, po, ranks)
    for w, x in zip(want, (sigma, n_fill, dt, dm)):
        assert np.array_equal(w, np_(x))
    psd.psd_table_body(user, dm.view(B * K, M), hidden)
    tokV, confV, _ = gpu_confidence(hidden, w_dev, want_lse=False)
    tokV, confV = tokV.reshape(B, K, M), confV.reshape(B, K, M)
    got = _gpu_accept(tokV, confV, np_(sigma), np_(dt), np_(dm), pg, g, K)
    want = oracle.verify_accept_dag(tokV, confV, np_(sigma), np_(dt), np_(dm), po, ranks)
    for w, x, n in zip(want, got, NAMES):
        assert np.array_equal(w, x), n
    assert (got[2] > 0).any() and (got[5].sum(axis=1) < K).any()       # some nodes accepted, some rejected


def test_argument_errors():
    g = psd.psd_dag_init(GRAPHS["diamond"])
    with pytest.raises(psd.PsdError):
        psd.psd_dag_init([set()] * 65)
    with pytest.raises(psd.PsdError):
        psd.psd_dag_init([{1}, {1, 2}])
    with pytest.raises(psd.PsdError):
        psd.psd_dag_init([set(), {0}, {1}], edges=[(1, 2)])
    x = torch.zeros(1, 8, dtype=torch.int32, device="cuda")
    pg = psd.policy(tau=0.5, k_min=0)
    with pytest.raises(psd.PsdError) as e:
        psd.psd_verify_accept_dag(x, x.float(), x, x, x, pg, g, x, x, x, x, x)
    assert e.value.code == psd.PSD_ERR_POLICY


def test_step_dag_equals_its_stages():
    """psd_step_dag against the same stages called one by one (merge included), on evolving drafts."""
    cfg = gen.Config("dagstep", B=6, H=128, V=1500, M=32, D=1, frac=0.8, tau=0.6, k_min=1, k_max=5, seed=33)
    ranks = GRAPHS["calibrated_like"]
    K = len(ranks)
    g = psd.psd_dag_init(ranks)
    B, M, H, V = cfg.B, cfg.M, cfg.H, cfg.V
    W = gen.weights(cfg)
    table, *_ = gen.table_body(cfg, W)
    w_dev, t_dev = bf16_dev(W), bf16_dev(table.reshape(-1, H))
    user = psd.table_body_user(t_dev.view(B, M, 3, H), B)
    tau = f32(cfg.tau)
    po = oracle.Policy(tau=tau, k_min=1, k_max=5, depth=1, mask_id=cfg.mask_id)
    pg = psd.policy(tau=tau, k_min=1, k_max=5, depth=1, mask_id=cfg.mask_id)
    hidden = torch.zeros(B * K * M, H, dtype=torch.bfloat16, device="cuda")
    buf = psd.StepBuffers.allocate(B, M, K, H, hidden, w_dev, "cuda")
    buf.tokens.fill_(cfg.mask_id)
    buf.mask.fill_(1)
    buf.sigma.fill_(-1)
    buf.draft_tokens.fill_(cfg.mask_id)
    buf.draft_mask.fill_(1)
    ws = torch.empty(psd.psd_workspace_bytes(B * K * M, H, V), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for step in range(5):
        before = {k: np_(getattr(buf, k)) for k in ("sigma", "draft_tokens", "draft_mask")}
        psd.psd_table_body(user, buf.draft_mask.view(B * K, M), hidden)
        psd.psd_step_dag(buf, pg, g, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        tokV, confV = np_(buf.tokV), np_(buf.confV)
        tokens, mask, ks, ns, nc, _ = oracle.verify_accept_dag(tokV, confV, before["sigma"], before["draft_tokens"],
                                                               before["draft_mask"], po, ranks)
        rows = np.arange(B)
        tokens, mask, sel, n_sel, sel_pos = oracle.select_unmask(confV[rows, ks], tokV[rows, ks], tokens, mask, po)
        sigma, n_fill, dt, dm = oracle.build_drafts_dag(confV[rows, ks], tokV[rows, ks], tokens, mask, po, ranks)
        want = dict(k_star=ks, n_spec_accepted=ns, n_committed=nc, tokens=tokens, mask=mask, sel=sel, n_sel=n_sel,
                    sel_pos=sel_pos, sigma=sigma, n_fill=n_fill, draft_tokens=dt, draft_mask=dm)
        for k, v in want.items():
            assert np.array_equal(v, np_(getattr(buf, k))), f"step {step}: {k}"
