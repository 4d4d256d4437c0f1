"""psd_confidence_static: the confidence pass for callers that cannot allocate device memory (their
process gave all HBM to its own pool, or they run inside another runtime's callback where cudaMalloc
is not allowed).  Its scratch is a fixed array inside the library, so the test checks that it gives
what psd_confidence gives with caller-provided scratch, bit for bit (same kernel, same tiles, same
merge order), twice in a row on different inputs (the array keeps the first call's contents), that
both agree with the fp64 CPU oracle under the usual tolerances, that a call after the first leaves the
device's free memory as it found it, and that problems larger than the array are refused.

Collected last on purpose: a failure here must not hide the other tests' results.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_15609_b200 as psd
import psd_inputs as gen
from psd_testlib import check_confidence

pytestmark = pytest.mark.gpu


def _inputs(seed, R, H, V):
    rng = np.random.default_rng(seed)
    W = gen.bf16_bits(rng.normal(scale=0.05, size=(V, H)).astype(np.float32))
    hid = rng.normal(size=(R, H)).astype(np.float32)
    Wf = gen.bf16_to_f64(W)
    for r in range(0, R, 2):
        t = int(rng.integers(0, V))
        hid[r] += (8.0 / float(Wf[t] @ Wf[t])) * Wf[t]
    to_dev = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    hid = gen.bf16_bits(hid)
    return to_dev(hid), to_dev(W), hid, W


def _both(hid, w):
    n, H = hid.shape
    V = w.shape[0]
    out = []
    for static in (False, True):
        tok = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        conf = torch.full((n,), -1.0, dtype=torch.float32, device="cuda")
        lse = torch.full((n,), -1.0, dtype=torch.float32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        if static:
            psd.psd_confidence_static(hid, w, tok, conf, lse, status)
        else:
            ws = torch.empty(psd.psd_workspace_bytes(n, H, V), dtype=torch.uint8, device="cuda")
            psd.psd_confidence(hid, w, tok, conf, lse, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        out.append((tok.cpu().numpy(), conf.cpu().numpy(), lse.cpu().numpy()))
    return out


def test_static_scratch_matches_caller_scratch_on_two_calls_in_a_row():
    # first call: many splits and rows; second call: a smaller problem that reuses a prefix of the
    # array still holding the first call's triples
    for seed, R, H, V in ((1, 200, 256, 20000), (2, 37, 128, 3001)):
        hid, w, hid_bits, w_bits = _inputs(seed, R, H, V)
        (tok_a, conf_a, lse_a), (tok_b, conf_b, lse_b) = _both(hid, w)
        # same kernel, same tile geometry, same merge order: not one bit may differ
        assert np.array_equal(tok_a, tok_b)
        assert np.array_equal(conf_a.view(np.uint32), conf_b.view(np.uint32))
        assert np.array_equal(lse_a.view(np.uint32), lse_b.view(np.uint32))
        # and both are right: the fp64 oracle of Sec. 3.1 on the same bytes
        tok_o, conf_o, lse_o, gap_o = oracle.confidence(hid_bits, w_bits)
        check_confidence(tok_b, conf_b, lse_b, tok_o, conf_o, lse_o, gap_o)


def test_static_scratch_calls_after_the_first_leave_free_memory_alone():
    hid, w, _, _ = _inputs(3, 64, 128, 4000)
    n = hid.shape[0]
    tok = torch.zeros(n, dtype=torch.int32, device="cuda")
    conf = torch.zeros(n, dtype=torch.float32, device="cuda")
    psd.psd_confidence_static(hid, w, tok, conf)      # the first call on a device may make the driver load
    torch.cuda.synchronize()                          # the module that holds the array
    free0, _ = torch.cuda.mem_get_info()
    psd.psd_confidence_static(hid, w, tok, conf)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0


def test_static_scratch_rejects_what_does_not_fit():
    assert psd.psd_workspace_bytes(8192, 4096, 126464) > psd.PSD_STATIC_SCRATCH_BYTES
    hid = torch.zeros(8192, 64, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(126464, 64, dtype=torch.bfloat16, device="cuda")
    tok = torch.zeros(8192, dtype=torch.int32, device="cuda")
    conf = torch.zeros(8192, dtype=torch.float32, device="cuda")
    with pytest.raises(psd.PsdError) as e:
        psd.psd_confidence_static(hid, w, tok, conf)
    assert e.value.code == psd.PSD_ERR_WORKSPACE
