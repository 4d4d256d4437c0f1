"""The C-ABI boundary without a GPU: the library loads, exports every symbol psd.h declares, and
rejects bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import pytest

import paper_2605_15609_b200 as psd
from paper_2605_15609_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "psd.h")


def _declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(psd_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_four_calls():
    names = _declared_symbols()
    for n in ("psd_confidence", "psd_select_unmask", "psd_build_drafts", "psd_verify_accept",
              "psd_workspace_bytes", "psd_status_string", "psd_step", "psd_step_host"):
        assert n in names


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(psd.LIB_PATH)
    for n in _declared_symbols():
        assert hasattr(lib, n), n


def test_debug_build_exports_the_same_symbols():
    from paper_2605_15609_b200 import build
    lib = ctypes.CDLL(build.build(debug=True))
    for n in _declared_symbols():
        assert hasattr(lib, n), n
    assert psd.status_string(psd.PSD_ERR_INTERNAL) == "a debug-build check inside a kernel failed"


def test_binding_has_the_same_names():
    for n in _declared_symbols():
        assert hasattr(binding, n) or n in ("psd_status_string",), n
    assert psd.status_string(0) == "ok"
    for code in range(-9, 1):
        assert psd.status_string(code) != "unknown status"
    assert psd.status_string(-99) == "unknown status"


def test_struct_layouts_match_the_header():
    assert ctypes.sizeof(psd.PsdPolicy) == 28
    assert ctypes.sizeof(psd.PsdStepIO) == 16 * ctypes.sizeof(ctypes.c_void_p)


def test_workspace_bytes():
    assert psd.psd_workspace_bytes(128, 4096, 126464) >= 12 * 128 * (126464 // 256 + 1)
    assert psd.psd_workspace_bytes(128, 4096, 126464) % 256 == 0
    for bad in ((0, 4096, 1000), (128, 100, 1000), (128, 32, 1000), (128, 4096, 0), (-1, 64, 10)):
        assert psd.psd_workspace_bytes(*bad) == 0
    assert psd.psd_step_host_bytes(1, 32, 4096, 126464, 4) > 128 * 4096 * 2
    assert psd.psd_step_host_bytes(1, 2000, 4096, 126464, 4) == 0
    assert psd.psd_step_host_bytes(1, 32, 4096, 126464, 65) == 0


FAKE = 0x10000  # a non-NULL, well-aligned address that is never dereferenced: validation fails first


def _conf(hidden=FAKE, w=FAKE, row_ids=None, n_rows=128, H=256, V=1024, tok=FAKE, conf=FAKE, lse=None, ws=FAKE,
          ws_bytes=1 << 30, status=None):
    return binding.LIB.psd_confidence(hidden, w, row_ids, n_rows, H, V, tok, conf, lse, ws, ws_bytes, status, None)


def test_confidence_argument_errors():
    assert _conf(hidden=None) == psd.PSD_ERR_NULL
    assert _conf(w=None) == psd.PSD_ERR_NULL
    assert _conf(tok=None) == psd.PSD_ERR_NULL
    assert _conf(ws=None) == psd.PSD_ERR_NULL
    # a row list needs the larger workspace (room for the dense copy of the listed rows)
    assert _conf(row_ids=FAKE, ws_bytes=psd.psd_workspace_bytes(128, 256, 1024)) == psd.PSD_ERR_WORKSPACE
    assert _conf(row_ids=FAKE + 2, ws_bytes=1 << 30) == psd.PSD_ERR_ALIGN
    assert psd.psd_compact_workspace_bytes(128, 256, 1024) >= psd.psd_workspace_bytes(128, 256, 1024) + 128 * 256 * 2
    assert psd.psd_compact_workspace_bytes(0, 256, 1024) == 0
    assert _conf(n_rows=0) == psd.PSD_ERR_SHAPE
    assert _conf(H=100) == psd.PSD_ERR_SHAPE
    assert _conf(H=0) == psd.PSD_ERR_SHAPE
    assert _conf(V=0) == psd.PSD_ERR_SHAPE
    assert _conf(hidden=FAKE + 2) == psd.PSD_ERR_ALIGN
    assert _conf(w=FAKE + 8) == psd.PSD_ERR_ALIGN
    assert _conf(ws=FAKE + 16) == psd.PSD_ERR_ALIGN
    assert _conf(conf=FAKE + 1) == psd.PSD_ERR_ALIGN
    assert _conf(ws_bytes=1024) == psd.PSD_ERR_WORKSPACE


def _pol(**kw):
    base = dict(tau=0.9, k_min=1, k_max=0, depth=2, stride=0, accept_mode=0, mask_id=0)
    base.update(kw)
    return psd.policy(**base)


BAD_POLICIES = [dict(k_min=0), dict(k_min=3, k_max=2), dict(depth=0), dict(depth=65), dict(stride=-1),
                dict(accept_mode=3), dict(accept_mode=-1), dict(tau=float("nan"))]


@pytest.mark.parametrize("kw", BAD_POLICIES)
def test_policy_errors(kw):
    L = binding.LIB
    p = _pol(**kw)
    assert L.psd_select_unmask(FAKE, FAKE, None, 1, FAKE, FAKE, 2, 32, p, FAKE, FAKE, FAKE, None) == psd.PSD_ERR_POLICY
    assert L.psd_build_drafts(FAKE, FAKE, None, 1, FAKE, FAKE, 2, 32, p, FAKE, FAKE, FAKE, FAKE, None) == psd.PSD_ERR_POLICY
    assert L.psd_verify_accept(FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 2, 32, p, FAKE, FAKE, FAKE, FAKE, FAKE, None,
                               None) == psd.PSD_ERR_POLICY


def test_block_shape_and_null_errors():
    L = binding.LIB
    p = _pol()
    assert L.psd_select_unmask(FAKE, FAKE, None, 1, FAKE, FAKE, 0, 32, p, FAKE, FAKE, FAKE, None) == psd.PSD_ERR_SHAPE
    assert L.psd_select_unmask(FAKE, FAKE, None, 1, FAKE, FAKE, 1, 1025, p, FAKE, FAKE, FAKE, None) == psd.PSD_ERR_SHAPE
    assert L.psd_select_unmask(FAKE, FAKE, None, 0, FAKE, FAKE, 1, 32, p, FAKE, FAKE, FAKE, None) == psd.PSD_ERR_SHAPE
    assert L.psd_select_unmask(None, FAKE, None, 1, FAKE, FAKE, 1, 32, p, FAKE, FAKE, FAKE, None) == psd.PSD_ERR_NULL
    assert L.psd_build_drafts(FAKE, FAKE, None, 1, FAKE, FAKE, 1, 0, p, FAKE, FAKE, FAKE, FAKE, None) == psd.PSD_ERR_SHAPE
    assert L.psd_build_drafts(FAKE, FAKE, None, 1, FAKE, None, 1, 32, p, FAKE, FAKE, FAKE, FAKE, None) == psd.PSD_ERR_NULL
    assert L.psd_verify_accept(FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 1, 32, p, FAKE, FAKE, None, FAKE, FAKE, None,
                               None) == psd.PSD_ERR_NULL
    io = psd.PsdStepIO()
    assert L.psd_step(ctypes.byref(io), 1, 32, 256, 1024, p, FAKE, 1 << 30, None, None) == psd.PSD_ERR_NULL
    assert L.psd_step(None, 1, 32, 256, 1024, p, FAKE, 1 << 30, None, None) == psd.PSD_ERR_NULL
    assert L.psd_step_host(None, 1, 32, 256, 1024, p, FAKE, 1 << 30, None, None) == psd.PSD_ERR_NULL
    assert L.psd_set_confidence_impl(7) == psd.PSD_ERR_SHAPE
    # knobs: bad values and unknown knobs are refused, good ones accepted and put back
    assert L.psd_set_tuning(psd.PSD_TUNE_WAIT_LIMIT, 0) == psd.PSD_ERR_SHAPE
    assert L.psd_set_tuning(psd.PSD_TUNE_WAIT_LIMIT, 4_000_000) == psd.PSD_OK
    assert L.psd_set_tuning(psd.PSD_TUNE_SELFTEST_STALL, 2) == psd.PSD_ERR_SHAPE
    assert L.psd_set_tuning(psd.PSD_TUNE_SELFTEST_STALL, 0) == psd.PSD_OK
    assert L.psd_set_tuning(psd.PSD_TUNE_PDL, 3) == psd.PSD_ERR_SHAPE
    assert L.psd_set_tuning(psd.PSD_TUNE_PDL, 1) == psd.PSD_OK
    assert L.psd_set_tuning(99, 0) == psd.PSD_ERR_UNSUPPORTED
    # psd_merge_partials checks alignment before it launches
    assert L.psd_merge_partials(FAKE + 2, FAKE, FAKE, 2, 8, FAKE, FAKE, None, None) == psd.PSD_ERR_ALIGN
    assert L.psd_merge_partials(FAKE, FAKE, FAKE, 2, 8, FAKE, FAKE + 1, None, None) == psd.PSD_ERR_ALIGN
    assert L.psd_confidence_kernel_name(128) == b"confidence_tc_kernel"
    assert L.psd_confidence_kernel_name(200) == b"confidence_tc2_kernel"
