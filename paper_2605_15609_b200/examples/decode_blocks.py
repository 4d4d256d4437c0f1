#!/usr/bin/env python
"""Decode a batch of blocks with PSD end to end on one GPU: Algorithm 1 (psd_decode_blocks) with the
table look-up body standing in for the transformer, a chain of drafts or a small draft graph, with or
without row compaction.

    python -m paper_2605_15609_b200.examples.decode_blocks [--blocks 8] [--depth 4] [--graph] [--compact]

A real caller replaces the body: any function that, given token states on the device, writes their
final hidden states (see psd_body_fn in include/psd.h); everything after the body runs in this
library's kernels.
"""
from __future__ import annotations

import argparse
import ctypes
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import paper_2605_15609_b200 as psd  # noqa: E402
import psd_inputs as gen  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--blocks", type=int, default=8)
    ap.add_argument("--depth", type=int, default=4, help="chain nodes, root included (ignored with --graph)")
    ap.add_argument("--graph", action="store_true", help="use a small multi-parent draft graph instead of the chain")
    ap.add_argument("--compact", action="store_true", help="score only rows that are still masked")
    ap.add_argument("--tau", type=float, default=0.7)
    args = ap.parse_args()

    ranks = [set(), {0}, {1}, {0, 1}, {0, 1, 2}, {0, 1, 2, 3}] if args.graph else None
    D = len(ranks) if ranks else args.depth
    cfg = gen.Config("example", B=args.blocks, H=1024, V=32000, M=32, D=D, frac=0.8, tau=args.tau, k_min=1, k_max=8,
                     seed=1)
    B, M, H, V = cfg.B, cfg.M, cfg.H, cfg.V
    W = gen.weights(cfg)
    table, *_ = gen.table_body(cfg, W)
    dev = torch.device("cuda", 0)
    as_bf16 = lambda bits: torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)
    w_dev, table_dev = as_bf16(W), as_bf16(table.reshape(-1, H))

    hidden = torch.zeros(B * D * M, H, dtype=torch.bfloat16, device=dev)        # the body writes here
    buf = psd.StepBuffers.allocate(B, M, D, H, hidden, w_dev, dev)
    buf.tokens.fill_(cfg.mask_id)
    buf.mask.fill_(1)
    workspace = torch.empty(psd.psd_compact_workspace_bytes(B * D * M, H, V), dtype=torch.uint8, device=dev)
    scratch = torch.empty(psd.psd_decode_scratch_bytes(B, M), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    passes = torch.zeros(B, dtype=torch.int32, device=dev)
    policy = psd.policy(tau=args.tau, k_min=1, k_max=8, depth=D, mask_id=cfg.mask_id)
    dag = psd.psd_dag_init(ranks) if ranks else None
    psd.psd_set_tuning(psd.PSD_TUNE_COMPACT_ROWS, 2 if args.compact else 0)

    user = psd.table_body_user(table_dev.view(B, M, 3, H), B)                    # argument of the native body
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    stats = psd.psd_decode_blocks(psd.table_body_address(), ctypes.addressof(user), buf, policy,
                                  psd.ORDER_ONE_PASS, 4 * M, scratch, workspace, status, passes, dag=dag)
    stop.record()
    torch.cuda.synchronize()
    if int(status.item()) != 0:
        raise RuntimeError(psd.status_string(int(status.item())))
    p = passes.cpu().numpy()
    print(f"{B} blocks of {M} slots, {'graph of ' + str(D) + ' nodes' if ranks else 'chain of ' + str(D) + ' nodes'}: "
          f"{stats.iterations} iterations, {stats.forward_passes} forward passes, {start.elapsed_time(stop):.2f} ms")
    print(f"tokens per forward pass, per block: mean {float((M / p).mean()):.2f}, best {float((M / p).max()):.2f}")
    print("first block:", buf.tokens[0].tolist())


if __name__ == "__main__":
    main()
