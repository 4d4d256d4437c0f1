"""The give-up path of the tensor-core kernels, exercised without faulting, trapping or hanging anything:
with PSD_TUNE_SELFTEST_STALL on, the loader of every CTA (of every pair's leading CTA) waits, after its
first K-slice, on a barrier that nothing ever arrives on; the wait is bounded (PSD_TUNE_WAIT_LIMIT, set
to a fraction of a millisecond here), so it runs out, the CTA reports PSD_ERR_TIMEOUT through the status
word, every role of the CTA (and of its partner in a pair) leaves its loop, the copies and tensor-core
work already issued are waited for, tensor memory is freed and the kernel returns normally.  The call
after it, with the knobs back at their defaults, must give the oracle's results."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_15609_b200 as psd
import psd_inputs as gen
from psd_testlib import bf16_dev, check_confidence, gpu_confidence

pytestmark = pytest.mark.gpu

DEFAULT_WAIT_KCYCLES = 4_000_000


@pytest.mark.parametrize("impl,rows", [(2, 128), (3, 128), (2, 300), (3, 300)])
def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_fine(impl, rows):
    cfg = gen.CONFIGS["tiny"]
    wl = gen.make(cfg)
    hid = np.concatenate([wl.hidden_verify, wl.hidden_stage1, wl.hidden_verify])[:rows]
    h, w = bf16_dev(hid), bf16_dev(wl.W)
    n, H = h.shape
    V = w.shape[0]
    tok = torch.zeros(n, dtype=torch.int32, device="cuda")
    conf = torch.zeros(n, dtype=torch.float32, device="cuda")
    ws = torch.zeros(psd.psd_workspace_bytes(n, H, V), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    prev = psd.psd_set_confidence_impl(impl)
    assert psd.psd_set_tuning(psd.PSD_TUNE_WAIT_LIMIT, 400) == 0          # 400 000 cycles: about 0.2 ms
    assert psd.psd_set_tuning(psd.PSD_TUNE_SELFTEST_STALL, 1) == 0
    try:
        psd.psd_confidence(h, w, tok, conf, None, ws, status)               # returns normally ...
        torch.cuda.synchronize()                                            # ... and so does the kernel
    finally:
        psd.psd_set_tuning(psd.PSD_TUNE_SELFTEST_STALL, 0)
        psd.psd_set_tuning(psd.PSD_TUNE_WAIT_LIMIT, DEFAULT_WAIT_KCYCLES)
        psd.psd_set_confidence_impl(prev)
    assert int(status.item()) == psd.PSD_ERR_TIMEOUT
    # the context is intact: an ordinary call right after it matches the oracle
    tok_o, conf_o, lse_o, gap_o = oracle.confidence(hid, wl.W)
    tok_g, conf_g, lse_g = gpu_confidence(h, w, impl=impl)
    check_confidence(tok_g, conf_g, lse_g, tok_o, conf_o, lse_o, gap_o)


def test_an_error_code_in_the_status_word_is_not_turned_into_a_count():
    """A row with a NaN is counted in the status word only while the word holds no error."""
    cfg = gen.CONFIGS["tiny"]
    wl = gen.make(cfg)
    hid = wl.hidden_verify.copy()
    hid[5, 3] = 0x7FC0
    h, w = bf16_dev(hid), bf16_dev(wl.W)
    n, H = h.shape
    tok = torch.zeros(n, dtype=torch.int32, device="cuda")
    conf = torch.zeros(n, dtype=torch.float32, device="cuda")
    ws = torch.zeros(psd.psd_workspace_bytes(n, H, w.shape[0]), dtype=torch.uint8, device="cuda")
    status = torch.full((1,), psd.PSD_ERR_TIMEOUT, dtype=torch.int32, device="cuda")
    psd.psd_confidence(h, w, tok, conf, None, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == psd.PSD_ERR_TIMEOUT and np.isnan(conf.cpu().numpy()[5])
