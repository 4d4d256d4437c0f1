"""The whole decoding loop on the GPU (psd_decode_blocks, Algorithm 1) against the oracle's loops.

The body is a table look-up (psd_inputs.table_body): no arithmetic, so the GPU's native body, a
Python callback body and the oracle's model read bit-identical hidden states.  The oracle runs each
block on its own in fp64; a block is set aside (and counted) if one of its table rows got a different
token id on the GPU (allowed only under a top-1/top-2 logit gap of 1e-2), or if, among the masked slots
of a sequence the oracle's loop scored, a confidence lies within 1e-3 of tau or two confidences are
within a relative 5e-5 (either could flip a decision between fp32 and fp64).  Every other block must
agree exactly: final tokens, forward passes charged to the block, and the per-iteration log (|T|, k*, n_spec_accepted, n_committed).
"""
import ctypes
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2605_15609_b200 as psd
import psd_inputs as gen
from psd_testlib import bf16_dev, check_confidence, gpu_confidence, ranking_margin_ok, threshold_margin_ok

pytestmark = pytest.mark.gpu


class Loop:
    """Device buffers of one psd_decode_blocks problem plus the oracle's view of the same table."""

    def __init__(self, cfg, max_iterations=None, ranks=None):
        if ranks is not None:                       # the drafts are the nodes of a graph
            from dataclasses import replace
            cfg = replace(cfg, D=len(ranks))
        self.cfg, self.ranks = cfg, ranks
        self.dag = psd.psd_dag_init(ranks) if ranks is not None else None
        B, M, D, H, V = cfg.B, cfg.M, cfg.D, cfg.H, cfg.V
        self.W = gen.weights(cfg)
        self.table, self.token, self.present, _ = gen.table_body(cfg, self.W)
        flat = self.table.reshape(-1, H)
        self.tok_o, self.conf_o, lse_o, self.gap_o = oracle.confidence(flat, self.W)
        self.w_dev, self.table_dev = bf16_dev(self.W), bf16_dev(flat)
        tok_g, conf_g, lse_g = gpu_confidence(self.table_dev, self.w_dev)
        check_confidence(tok_g, conf_g, lse_g, self.tok_o, self.conf_o, lse_o, self.gap_o)
        self.tok_g = tok_g
        self.max_it = max_iterations or (M + 2)
        hidden = torch.zeros(B * D * M, H, dtype=torch.bfloat16, device="cuda")
        self.buf = psd.StepBuffers.allocate(B, M, D, H, hidden, self.w_dev, "cuda")
        self.ws = torch.empty(psd.psd_compact_workspace_bytes(B * D * M, H, V), dtype=torch.uint8, device="cuda")
        self.scratch = torch.empty(psd.psd_decode_scratch_bytes(B, M), dtype=torch.uint8, device="cuda")
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.passes = torch.zeros(B, dtype=torch.int32, device="cuda")
        self.done = torch.zeros(B, dtype=torch.int32, device="cuda")
        self.trace = torch.zeros(self.max_it, B, 4, dtype=torch.int32, device="cuda")
        tau = float(np.float32(cfg.tau))
        self.pg = psd.policy(tau=tau, k_min=cfg.k_min, k_max=cfg.k_max, depth=D, stride=cfg.stride,
                             mask_id=cfg.mask_id)
        self.po = oracle.Policy(tau=tau, k_min=cfg.k_min, k_max=cfg.k_max, depth=D, stride=cfg.stride,
                                mask_id=cfg.mask_id)

    def reset(self):
        self.buf.tokens.fill_(self.cfg.mask_id)
        self.buf.mask.fill_(1)
        self.trace.zero_()

    def run_native(self, order):
        self.reset()
        user = psd.table_body_user(self.table_dev.view(self.cfg.B, self.cfg.M, 3, self.cfg.H), self.cfg.B)
        stats = psd.psd_decode_blocks(psd.table_body_address(), ctypes.addressof(user), self.buf, self.pg, order,
                                      self.max_it, self.scratch, self.ws, self.status, self.passes, self.done,
                                      self.trace, dag=self.dag)
        torch.cuda.synchronize()
        assert int(self.status.item()) == 0
        return stats

    def run_callback(self, order):
        """The same loop with a body written in Python (torch used only to gather table rows)."""
        self.reset()
        cfg, buf = self.cfg, self.buf
        B, M, D = cfg.B, cfg.M, cfg.D
        seen = []

        def body(tokens_ptr, mask_ptr, n_seq, m, hidden_ptr, stream_ptr):
            assert m == M and hidden_ptr == buf.hidden.data_ptr()
            if mask_ptr == buf.mask.data_ptr():
                mask, per_block = buf.mask, 1
            else:
                assert mask_ptr == buf.draft_mask.data_ptr() and n_seq == B * D
                mask, per_block = buf.draft_mask.view(B * D, M), D
            assert n_seq == B * per_block
            seen.append(n_seq)
            committed = (mask == 0).to(torch.int64)
            c = torch.zeros_like(committed)
            c[:, 1:] += committed[:, :-1]
            c[:, :-1] += committed[:, 1:]
            b = (torch.arange(n_seq, device="cuda") // per_block)[:, None]
            rows = ((b * M + torch.arange(M, device="cuda")[None, :]) * 3 + c).reshape(-1)
            buf.hidden[:n_seq * M] = self.table_dev.index_select(0, rows)
            return 0

        stats = psd.psd_decode_blocks(body, None, buf, self.pg, order, self.max_it, self.scratch, self.ws,
                                      self.status, self.passes, self.done, self.trace)
        torch.cuda.synchronize()
        assert int(self.status.item()) == 0
        return stats, seen

    def outputs(self):
        return (self.buf.tokens.cpu().numpy(), self.buf.mask.cpu().numpy(), self.passes.cpu().numpy(),
                self.done.cpu().numpy(), self.trace.cpu().numpy())

    def oracle_block(self, b, order):
        """The oracle's loop on block b.  Also reports whether every decision it took was clear of the
        fp32/fp64 margins: over the masked slots of every sequence of every model call, same token id
        on the GPU, no confidence within 1e-3 of tau, no two confidences within a relative 5e-5."""
        M = self.cfg.M
        clear = [True]

        def model(tokens, mask):
            mask = np.atleast_2d(mask)
            rows = gen.table_rows(mask, seq_per_block=mask.shape[0]) + b * M * 3
            for s in range(mask.shape[0]):
                r = rows[s][mask[s] != 0]
                if len(r) and not (np.array_equal(self.tok_g[r], self.tok_o[r])
                                   and threshold_margin_ok(self.conf_o[r], self.po.tau)
                                   and ranking_margin_ok(self.conf_o[r])):
                    clear[0] = False
            return self.tok_o[rows], self.conf_o[rows]

        fn = oracle.decode_block if order == psd.ORDER_TWO_PASSES else oracle.decode_block_one_pass
        return fn(model, M, self.po, node_ranks=self.ranks), clear[0]

    def compare(self, order, stats):
        cfg = self.cfg
        tokens, mask, passes, done, trace = self.outputs()
        assert stats.masked_left == 0 and (mask == 0).all() and (tokens != cfg.mask_id).all()
        set_aside, most_passes, k_stars = 0, 0, []
        for b in range(cfg.B):
            (tok_o, calls_o, log_o), clear = self.oracle_block(b, order)
            if not clear:
                set_aside += 1
                continue
            assert np.array_equal(tokens[b], tok_o), f"block {b}: final tokens"
            assert passes[b] == calls_o, f"block {b}: forward passes"
            assert done[b] == len(log_o) - 1, f"block {b}: resolving iteration"
            assert [tuple(r) for r in trace[:len(log_o), b].tolist()] == log_o, f"block {b}: per-iteration log"
            most_passes = max(most_passes, calls_o)
            k_stars += [ks for _, ks, _, _ in log_o]
        if order == psd.ORDER_ONE_PASS:
            assert stats.forward_passes == stats.iterations
        assert stats.iterations <= cfg.M
        return set_aside, most_passes, k_stars


CASES = {
    "threshold": gen.Config("loop_thr", B=6, H=256, V=1024, M=32, D=4, frac=0.7, s_lo=2.5, s_hi=3.5, tau=0.7,
                            k_min=1, k_max=8, seed=21),
    "no_speculation": gen.Config("loop_d1", B=3, H=256, V=1024, M=32, D=1, frac=0.7, s_lo=2.5, s_hi=3.5, tau=0.9,
                                 k_min=1, k_max=8, seed=22),
    "top_k": gen.Config("loop_topk", B=4, H=128, V=2000, M=32, D=3, frac=0.9, s_lo=2.5, s_hi=3.5, tau=0.5, k_min=2,
                        k_max=2, stride=2, seed=23),
    "long_block": gen.Config("loop_m64", B=2, H=256, V=1024, M=64, D=8, frac=0.8, s_lo=2.5, s_hi=3.5, tau=0.85,
                             k_min=1, k_max=0, seed=24),
}


@pytest.mark.parametrize("order", [psd.ORDER_TWO_PASSES, psd.ORDER_ONE_PASS])
@pytest.mark.parametrize("name", list(CASES))
def test_loop_matches_oracle(name, order):
    loop = Loop(CASES[name])
    stats = loop.run_native(order)
    set_aside, most_passes, k_stars = loop.compare(order, stats)
    assert set_aside <= loop.cfg.B // 2
    if loop.cfg.D > 1:
        assert max(k_stars) > 0                      # some speculation was accepted
        assert stats.iterations < loop.cfg.M         # fewer iterations than slots


GRAPH = [set(), {0}, {0, 1}, {1}, {0, 2}, {0, 1, 2}, {0, 1, 2, 3}, {2, 3}, {0, 1, 2, 3, 4, 5}]


@pytest.mark.parametrize("compact", [0, 2])
@pytest.mark.parametrize("order", [psd.ORDER_TWO_PASSES, psd.ORDER_ONE_PASS])
def test_loop_over_a_draft_graph(order, compact):
    """Algorithm 1 with a multi-parent draft graph in place of the chain, against the oracle's loop."""
    loop = Loop(CASES["threshold"], ranks=GRAPH)
    assert psd.psd_set_tuning(psd.PSD_TUNE_COMPACT_ROWS, compact) == 0
    try:
        stats = loop.run_native(order)
    finally:
        psd.psd_set_tuning(psd.PSD_TUNE_COMPACT_ROWS, 0)
    set_aside, _, k_stars = loop.compare(order, stats)
    assert set_aside <= loop.cfg.B // 2 and max(k_stars) > 0 and stats.iterations < loop.cfg.M


@pytest.mark.parametrize("order", [psd.ORDER_TWO_PASSES, psd.ORDER_ONE_PASS])
@pytest.mark.parametrize("name", ["threshold", "long_block"])
def test_loop_with_row_compaction(name, order):
    """The loop scoring only masked rows (psd_step's compaction, psd_confidence_masked): same parity bar."""
    loop = Loop(CASES[name])
    assert psd.psd_set_tuning(psd.PSD_TUNE_COMPACT_ROWS, 2) == 0
    try:
        stats = loop.run_native(order)
    finally:
        psd.psd_set_tuning(psd.PSD_TUNE_COMPACT_ROWS, 0)
    set_aside, _, k_stars = loop.compare(order, stats)
    assert set_aside <= loop.cfg.B // 2 and max(k_stars) > 0


@pytest.mark.parametrize("order", [psd.ORDER_TWO_PASSES, psd.ORDER_ONE_PASS])
def test_python_body_gives_the_same_loop(order):
    loop = Loop(CASES["threshold"])
    stats_n = loop.run_native(order)
    native = [x.copy() for x in loop.outputs()]
    stats_c, seen = loop.run_callback(order)
    for a, b in zip(native, loop.outputs()):
        assert np.array_equal(a, b)
    assert (stats_n.iterations, stats_n.forward_passes) == (stats_c.iterations, stats_c.forward_passes)
    assert len(seen) == stats_c.forward_passes
    B, D = loop.cfg.B, loop.cfg.D
    assert set(seen) <= ({B * D} if order == psd.ORDER_ONE_PASS else {B, B * D})


@pytest.mark.parametrize("order", [psd.ORDER_TWO_PASSES, psd.ORDER_ONE_PASS])
def test_greedy_collapse_one_slot_per_pass(order):
    # tau = 1, k = 1, no speculation: every forward pass reveals exactly one slot of every block
    from dataclasses import replace
    cfg = replace(CASES["no_speculation"], tau=1.0, k_min=1, k_max=1)
    loop = Loop(cfg)
    stats = loop.run_native(order)
    tokens, mask, passes, done, trace = loop.outputs()
    assert stats.iterations == stats.forward_passes == cfg.M and (passes == cfg.M).all()
    assert (trace[:cfg.M, :, 0] == 1).all() and (trace[:, :, 1:] == 0).all()
    loop.compare(order, stats)


def test_iteration_limit_and_argument_errors():
    loop = Loop(CASES["no_speculation"], max_iterations=2)
    stats = loop.run_native(psd.ORDER_TWO_PASSES)
    assert stats.iterations == 2 and stats.masked_left > 0
    assert int((loop.buf.mask != 0).sum().item()) == stats.masked_left
    with pytest.raises(psd.PsdError) as e:
        psd.psd_decode_blocks(psd.table_body_address(), None, loop.buf, loop.pg, 7, 4, loop.scratch, loop.ws)
    assert e.value.code == psd.PSD_ERR_UNSUPPORTED
    with pytest.raises(psd.PsdError) as e:
        psd.psd_decode_blocks(psd.table_body_address(), None, loop.buf, loop.pg, 0, 4, loop.scratch[:256], loop.ws)
    assert e.value.code == psd.PSD_ERR_WORKSPACE
    # a body that fails: its code comes back unchanged (native body, NULL user)
    with pytest.raises(psd.PsdError) as e:
        psd.psd_decode_blocks(psd.table_body_address(), None, loop.buf, loop.pg, 0, 4, loop.scratch, loop.ws)
    assert e.value.code == psd.PSD_ERR_NULL
