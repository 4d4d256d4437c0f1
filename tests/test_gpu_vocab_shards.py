"""The vocabulary split (psd_confidence_partial + psd_merge_partials) on one GPU: the shards of every
"rank" are computed one after the other on the same device, stacked as an all-gather would, and merged;
the result must meet the same bar against the fp64 oracle as the unsplit pass, whatever the split."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_15609_b200 as psd
import psd_inputs as gen
from paper_2605_15609_b200.vocab_parallel import VocabParallelHead, shard_rows
from psd_testlib import bf16_dev, check_confidence, gpu_confidence, np_

pytestmark = pytest.mark.gpu


def _inputs(seed, R, H, V):
    rng = np.random.default_rng(seed)
    W = gen.bf16_bits(rng.normal(scale=0.05, size=(V, H)).astype(np.float32))
    hid = rng.normal(size=(R, H)).astype(np.float32)
    Wf = gen.bf16_to_f64(W)
    for r in range(0, R, 2):
        t = int(rng.integers(0, V))
        hid[r] += (rng.uniform(3.0, 10.0) / float(Wf[t] @ Wf[t])) * Wf[t]
    return gen.bf16_bits(hid), W


@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("R,H,V", [(128, 256, 5000), (37, 128, 1000), (300, 64, 20011)])
def test_sharded_equals_whole(R, H, V, world):
    hid, W = _inputs(R + V + world, R, H, V)
    tok_o, conf_o, lse_o, gap_o = oracle.confidence(hid, W)
    h_dev, w_dev = bf16_dev(hid), bf16_dev(W)
    m = torch.zeros(world, R, dtype=torch.float32, device="cuda")
    s = torch.zeros(world, R, dtype=torch.float32, device="cuda")
    a = torch.zeros(world, R, dtype=torch.int32, device="cuda")
    covered = 0
    for rank in range(world):
        v0, v1 = shard_rows(V, world, rank)
        assert v0 == covered and v0 % 16 == 0
        covered = v1
        shard = w_dev[v0:v1]
        ws = torch.empty(psd.psd_workspace_bytes(R, H, v1 - v0), dtype=torch.uint8, device="cuda")
        psd.psd_confidence_partial(h_dev, shard, v0, m[rank], s[rank], a[rank], ws)
    assert covered == V
    tok = torch.zeros(R, dtype=torch.int32, device="cuda")
    conf = torch.zeros(R, dtype=torch.float32, device="cuda")
    lse = torch.zeros(R, dtype=torch.float32, device="cuda")
    psd.psd_merge_partials(m, s, a, tok, conf, lse)
    torch.cuda.synchronize()
    check_confidence(np_(tok), np_(conf), np_(lse), tok_o, conf_o, lse_o, gap_o)
    whole = gpu_confidence(h_dev, w_dev)
    assert np.array_equal(np_(tok), whole[0]) and np.abs(np_(conf) - whole[1]).max() < 1e-5
    am = np_(a)
    for rank in range(world):
        v0, v1 = shard_rows(V, world, rank)
        assert (am[rank] >= v0).all() and (am[rank] < v1).all()         # global indices inside the shard


def test_equal_maxima_across_shards_keep_the_lowest_index():
    H, V = 64, 640
    W = np.zeros((V, H), dtype=np.float32)
    W[5, 0] = W[333, 0] = W[600, 0] = 1.0                                # three identical best rows, three shards
    hid = np.zeros((4, H), dtype=np.float32)
    hid[:, 0] = 2.0
    h_dev, w_dev = bf16_dev(gen.bf16_bits(hid)), bf16_dev(gen.bf16_bits(W))
    world = 4
    m = torch.zeros(world, 4, dtype=torch.float32, device="cuda")
    s, a = torch.zeros_like(m), torch.zeros(world, 4, dtype=torch.int32, device="cuda")
    for rank in range(world):
        v0, v1 = shard_rows(V, world, rank)
        ws = torch.empty(psd.psd_workspace_bytes(4, H, v1 - v0), dtype=torch.uint8, device="cuda")
        psd.psd_confidence_partial(h_dev, w_dev[v0:v1], v0, m[rank], s[rank], a[rank], ws)
    tok = torch.zeros(4, dtype=torch.int32, device="cuda")
    conf = torch.zeros(4, dtype=torch.float32, device="cuda")
    psd.psd_merge_partials(m, s, a, tok, conf)
    torch.cuda.synchronize()
    assert (np_(tok) == 5).all()
    assert np.allclose(np_(conf), 1.0 / (3.0 + (V - 3) * np.exp(-2.0)), rtol=1e-5)


def test_head_object_single_process():
    R, H, V = 64, 128, 3000
    hid, W = _inputs(3, R, H, V)
    tok_o, conf_o, lse_o, gap_o = oracle.confidence(hid, W)
    head = VocabParallelHead(bf16_dev(W), 0, max_rows=128)
    tok = torch.zeros(R, dtype=torch.int32, device="cuda")
    conf = torch.zeros(R, dtype=torch.float32, device="cuda")
    lse = torch.zeros(R, dtype=torch.float32, device="cuda")
    head.confidence(bf16_dev(hid), tok, conf, lse)
    torch.cuda.synchronize()
    check_confidence(np_(tok), np_(conf), np_(lse), tok_o, conf_o, lse_o, gap_o)


def test_head_object_on_a_stream_that_is_not_current():
    """The partial pass, the gather and the merge must all be ordered on the stream that is passed in, not
    on torch's current stream: a long kernel is queued on the side stream first, so work that wrongly went
    to the current stream would run ahead of the partial pass and read triples that are not written yet."""
    R, H, V = 128, 256, 20000
    hid, W = _inputs(11, R, H, V)
    tok_o, conf_o, lse_o, gap_o = oracle.confidence(hid, W)
    head = VocabParallelHead(bf16_dev(W), 0, max_rows=R)
    h_dev = bf16_dev(hid)
    tok = torch.full((R,), -3, dtype=torch.int32, device="cuda")
    conf = torch.full((R,), -3.0, dtype=torch.float32, device="cuda")
    lse = torch.full((R,), -3.0, dtype=torch.float32, device="cuda")
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    big = torch.empty(1 << 28, dtype=torch.float32, device="cuda")
    with torch.cuda.stream(side):
        for _ in range(4):
            big.add_(1.0)                      # a few milliseconds of work ahead of the pass, on the side stream
    head.confidence(h_dev, tok, conf, lse, stream=side)
    side.synchronize()
    check_confidence(np_(tok), np_(conf), np_(lse), tok_o, conf_o, lse_o, gap_o)


def test_head_object_with_an_empty_range():
    R, H = 16, 64
    w = torch.zeros(0, H, dtype=torch.bfloat16, device="cuda")
    head = VocabParallelHead(w, 640, max_rows=R)
    tok = torch.zeros(R, dtype=torch.int32, device="cuda")
    conf = torch.zeros(R, dtype=torch.float32, device="cuda")
    # alone in its group the merged result is the neutral triple itself: the call must simply not fail
    head.confidence(torch.zeros(R, H, dtype=torch.bfloat16, device="cuda"), tok, conf)
    torch.cuda.synchronize()
    assert (np_(tok) == 2**31 - 1).all()
