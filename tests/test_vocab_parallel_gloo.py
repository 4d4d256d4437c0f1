"""The vocabulary split's exchange on CPU: two gloo ranks each reduce their range of the vocabulary to
per-row triples (computed here by the oracle's fp64 logits), all-gather them with the package's
gather_partials, and merge; every rank must arrive at the whole-vocabulary prediction."""
import os
import socket
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out, V=1000):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import torch
    import torch.distributed as dist

    import oracle
    import psd_inputs as gen
    from paper_2605_15609_b200.vocab_parallel import gather_partials, neutral_triple, shard_rows
    dist.init_process_group(backend="gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(0)                      # the same inputs on every rank
    R, H = 9, 64
    W = gen.bf16_bits(rng.normal(scale=0.2, size=(V, H)).astype(np.float32))
    hid = gen.bf16_bits(rng.normal(size=(R, H)).astype(np.float32))
    v0, v1 = shard_rows(V, world, rank)
    if v1 > v0:
        logits = oracle.logits(hid, W[v0:v1])           # [R, v1 - v0] fp64
        m = logits.max(axis=1)
        s = np.exp(logits - m[:, None]).sum(axis=1)
        a = logits.argmax(axis=1) + v0
        local = torch.from_numpy(np.stack([m.astype(np.float32).view(np.int32),
                                           s.astype(np.float32).view(np.int32), a.astype(np.int32)]))
    else:
        local = neutral_triple(R)                       # a rank without vocabulary rows still takes part
    allp = gather_partials(local).numpy()               # [world, 3, R]
    ms, ss, aa = allp[:, 0].view(np.float32).astype(np.float64), allp[:, 1].view(np.float32).astype(np.float64), allp[:, 2]
    best = ms.max(axis=0)
    total = (ss * np.exp(ms - best[None, :])).sum(axis=0)
    tok = np.array([min(aa[g, r] for g in range(world) if ms[g, r] == best[r]) for r in range(R)])
    tok_o, conf_o, _, _ = oracle.confidence(hid, W)
    out.put((rank, (v0, v1), bool((tok == tok_o).all()), float(np.abs(1.0 / total - conf_o).max())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_exchange_and_merge():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, sh0, ok0, e0), (r1, sh1, ok1, e1) = res
    assert sh0 == (0, 512) and sh1 == (512, 1000)
    assert ok0 and ok1 and e0 < 1e-6 and e1 < 1e-6


def test_more_ranks_than_ranges_of_sixteen_rows():
    # V = 20 gives two ranges of the vocabulary; the third rank holds none, contributes the neutral triple
    # (-inf, 0, INT32_MAX) and must neither stall the all-gather nor change the result
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 3, port, q, 20)) for r in range(3)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [(0, 16), (16, 20), (20, 20)]
    assert all(ok and err < 1e-6 for _, _, ok, err in res)


def test_shard_rows_cover_the_vocabulary():
    sys.path.insert(0, ROOT)
    from paper_2605_15609_b200.vocab_parallel import shard_rows
    for V in (1, 15, 16, 1000, 126464, 152064):
        for world in (1, 2, 3, 8):
            edges = [shard_rows(V, world, r) for r in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == V
            assert all(a[1] == b[0] for a, b in zip(edges, edges[1:]))
            assert all(v0 % 16 == 0 for v0, v1 in edges if v1 > v0)
            sizes = [v1 - v0 for v0, v1 in edges if v1 > v0]
            assert max(sizes) - min(sizes) <= 16 + 15 or len(sizes) < world
