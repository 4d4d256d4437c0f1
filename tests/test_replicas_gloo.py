"""The N > 1 plumbing on CPU: two gloo ranks line up, keep distinct batches and aggregate throughput as
(sum of units) / (max of times)."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2605_15609_b200 import replicas
    info = replicas.rank_info_from_env()
    assert replicas.init_process_group(info, backend="gloo")
    replicas.barrier(info)
    seed = replicas.replica_seed(2, info.rank)
    value, secs = replicas.aggregate_throughput(128.0 * (rank + 1), 0.5 + rank, info)
    mx = replicas.max_over_ranks(float(rank), info)
    out.put((rank, info.is_main, seed, value, secs, mx))
    replicas.barrier(info)
    import torch.distributed as dist
    dist.destroy_process_group()


def test_two_ranks_aggregate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, main0, seed0, v0, s0, m0), (r1, main1, seed1, v1, s1, m1) = res
    assert (r0, r1) == (0, 1) and main0 and not main1
    assert seed0 == 2 and seed1 == 1002
    assert s0 == s1 == 1.5                      # max over ranks
    assert v0 == v1 == (128.0 + 256.0) / 1.5    # all units over the slowest rank's time
    assert m0 == m1 == 1.0


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    from paper_2605_15609_b200 import replicas
    info = replicas.rank_info_from_env({})
    assert info.world_size == 1 and info.is_main
    assert replicas.init_process_group(info) is False
    assert replicas.aggregate_throughput(10.0, 2.0, info) == (5.0, 2.0)
