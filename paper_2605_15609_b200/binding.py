"""ctypes binding of libpsd_b200.so: the same entry points as include/psd.h, argument marshalling only.

Tensor arguments are torch tensors (device tensors for the device entry points, pinned or plain
host tensors for ``psd_step_host``); every step of the path runs inside the library's CUDA
kernels.  There is no fallback: if the shared library cannot be loaded the import of this module
raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

from . import build as _build

_i32, _i64, _f32, _vp, _sz = ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t

PSD_OK = 0
PSD_ERR_NULL, PSD_ERR_SHAPE, PSD_ERR_ALIGN, PSD_ERR_WORKSPACE = -1, -2, -3, -4
PSD_ERR_POLICY, PSD_ERR_CUDA, PSD_ERR_UNSUPPORTED, PSD_ERR_TIMEOUT, PSD_ERR_INTERNAL = -5, -6, -7, -8, -9
PSD_MAX_M, PSD_MAX_DEPTH = 1024, 64
ACCEPT_AGREE_AND_CONF, ACCEPT_AGREE_ONLY, ACCEPT_AGREE_AND_POLICY = 0, 1, 2


class PsdPolicy(ctypes.Structure):
    """psd_policy_t"""
    _fields_ = [("tau", _f32), ("k_min", _i32), ("k_max", _i32), ("depth", _i32), ("stride", _i32),
                ("accept_mode", _i32), ("mask_id", _i32)]


class PsdStepIO(ctypes.Structure):
    """psd_step_io_t"""
    _fields_ = [(n, _vp) for n in ("hidden_bf16", "w_lm_bf16", "sigma", "n_fill", "draft_tokens", "draft_mask",
                                   "tokV", "confV", "tokens", "mask", "k_star", "n_spec_accepted",
                                   "n_committed", "sel", "n_sel", "sel_pos")]


class PsdDag(ctypes.Structure):
    """psd_dag_t"""
    _fields_ = [("n_nodes", _i32), ("reserved", _i32), ("ranks", ctypes.c_uint64 * 64),
                ("parents", ctypes.c_uint64 * 64)]


class PsdDecodeStats(ctypes.Structure):
    """psd_decode_stats_t"""
    _fields_ = [("iterations", _i32), ("forward_passes", _i32), ("masked_left", _i32)]


class PsdTableBody(ctypes.Structure):
    """psd_table_body_t"""
    _fields_ = [("table_bf16", _vp), ("B", _i32), ("H", _i32)]


# psd_body_fn
BODY_FN = ctypes.CFUNCTYPE(ctypes.c_int, _vp, _vp, _vp, _i32, _i32, _vp, _vp)
ORDER_TWO_PASSES, ORDER_ONE_PASS = 0, 1


class PsdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


def _load() -> ctypes.CDLL:
    # build() compares the library's time stamp with the sources' and recompiles when a source is newer,
    # so a stale library is never loaded silently
    # PSD_B200_DEBUG=1 in the environment selects the debug build of the library (device-side bounds and
    # ring-order checks that report PSD_ERR_INTERNAL through the status word); same entry points
    lib = ctypes.CDLL(_build.build(debug=DEBUG_BUILD))
    pol = PsdPolicy
    lib.psd_status_string.restype = ctypes.c_char_p
    lib.psd_status_string.argtypes = [ctypes.c_int]
    lib.psd_workspace_bytes.restype = _sz
    lib.psd_workspace_bytes.argtypes = [_i32, _i32, _i32]
    lib.psd_compact_workspace_bytes.restype = _sz
    lib.psd_compact_workspace_bytes.argtypes = [_i32, _i32, _i32]
    lib.psd_confidence.restype = ctypes.c_int
    lib.psd_confidence.argtypes = [_vp, _vp, _vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
    lib.psd_confidence_masked.restype = ctypes.c_int
    lib.psd_confidence_masked.argtypes = [_vp, _vp, _vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
    lib.psd_compact_rows_enabled.restype = ctypes.c_int
    lib.psd_compact_rows_enabled.argtypes = [_i32]
    lib.psd_confidence_partial.restype = ctypes.c_int
    lib.psd_confidence_partial.argtypes = [_vp, _vp, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
    lib.psd_merge_partials.restype = ctypes.c_int
    lib.psd_merge_partials.argtypes = [_vp, _vp, _vp, _i32, _i32, _vp, _vp, _vp, _vp]
    lib.psd_confidence_static.restype = ctypes.c_int
    lib.psd_confidence_static.argtypes = [_vp, _vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp]
    lib.psd_select_unmask.restype = ctypes.c_int
    lib.psd_select_unmask.argtypes = [_vp, _vp, _vp, _i32, _vp, _vp, _i32, _i32, pol, _vp, _vp, _vp, _vp]
    lib.psd_build_drafts.restype = ctypes.c_int
    lib.psd_build_drafts.argtypes = [_vp, _vp, _vp, _i32, _vp, _vp, _i32, _i32, pol, _vp, _vp, _vp, _vp, _vp]
    lib.psd_verify_accept.restype = ctypes.c_int
    lib.psd_verify_accept.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, pol, _vp, _vp, _vp, _vp, _vp,
                                      _vp, _vp]
    lib.psd_step.restype = ctypes.c_int
    lib.psd_step.argtypes = [ctypes.POINTER(PsdStepIO), _i32, _i32, _i32, _i32, pol, _vp, _sz, _vp, _vp]
    lib.psd_step_host_bytes.restype = _sz
    lib.psd_step_host_bytes.argtypes = [_i32, _i32, _i32, _i32, _i32]
    lib.psd_step_host_block.restype = _sz
    lib.psd_step_host_block.argtypes = [_i32, _i32, _i32, ctypes.POINTER(_sz)]
    lib.psd_step_host.restype = ctypes.c_int
    lib.psd_step_host.argtypes = [ctypes.POINTER(PsdStepIO), _i32, _i32, _i32, _i32, pol, _vp, _sz, _vp, _vp]
    lib.psd_dag_init.restype = ctypes.c_int
    lib.psd_dag_init.argtypes = [ctypes.POINTER(PsdDag), _i32, _vp, _vp]
    lib.psd_build_drafts_dag.restype = ctypes.c_int
    lib.psd_build_drafts_dag.argtypes = [_vp, _vp, _vp, _i32, _vp, _vp, _i32, _i32, pol, ctypes.POINTER(PsdDag), _vp,
                                         _vp, _vp, _vp, _vp]
    lib.psd_verify_accept_dag.restype = ctypes.c_int
    lib.psd_verify_accept_dag.argtypes = [_vp, _vp, _vp, _vp, _vp, _i32, _i32, pol, ctypes.POINTER(PsdDag), _vp, _vp,
                                          _vp, _vp, _vp, _vp, _vp]
    lib.psd_decode_scratch_bytes.restype = _sz
    lib.psd_decode_scratch_bytes.argtypes = [_i32, _i32]
    lib.psd_decode_blocks.restype = ctypes.c_int
    lib.psd_step_dag.restype = ctypes.c_int
    lib.psd_step_dag.argtypes = [ctypes.POINTER(PsdStepIO), _i32, _i32, _i32, _i32, pol, ctypes.POINTER(PsdDag), _vp,
                                 _sz, _vp, _vp]
    lib.psd_decode_blocks.argtypes = [_vp, _vp, ctypes.POINTER(PsdStepIO), _i32, _i32, _i32, _i32, pol,
                                      ctypes.POINTER(PsdDag), _i32, _i32,
                                      _vp, _sz, _vp, _sz, _vp, _vp, _vp, _vp, ctypes.POINTER(PsdDecodeStats), _vp]
    lib.psd_table_body.restype = ctypes.c_int
    lib.psd_table_body.argtypes = [_vp, _vp, _vp, _i32, _i32, _vp, _vp]
    lib.psd_set_confidence_impl.restype = ctypes.c_int
    lib.psd_set_confidence_impl.argtypes = [ctypes.c_int]
    lib.psd_set_tuning.restype = ctypes.c_int
    lib.psd_set_tuning.argtypes = [ctypes.c_int, ctypes.c_int]
    lib.psd_set_kernel_events.restype = ctypes.c_int
    lib.psd_set_kernel_events.argtypes = [_vp, _vp]
    lib.psd_confidence_kernel_name.restype = ctypes.c_char_p
    lib.psd_confidence_kernel_name.argtypes = [_i32]
    lib.psd_launch_count.restype = _i64
    lib.psd_launch_count.argtypes = []
    return lib


DEBUG_BUILD = os.environ.get("PSD_B200_DEBUG", "0") not in ("", "0")
LIB = _load()
LIB_PATH = _build.LIB_DEBUG if DEBUG_BUILD else _build.LIB


def status_string(code: int) -> str:
    return LIB.psd_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != PSD_OK:
        raise PsdError(code, where)


def _ptr(t):
    """Address of a tensor's first element, or None."""
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("psd binding: tensors must be contiguous")
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def policy(tau=0.9, k_min=1, k_max=0, depth=1, stride=0, accept_mode=0, mask_id=0) -> PsdPolicy:
    return PsdPolicy(float(tau), int(k_min), int(k_max), int(depth), int(stride), int(accept_mode), int(mask_id))


def psd_workspace_bytes(n_rows: int, H: int, V: int) -> int:
    return int(LIB.psd_workspace_bytes(n_rows, H, V))


def psd_compact_workspace_bytes(n_rows: int, H: int, V: int) -> int:
    return int(LIB.psd_compact_workspace_bytes(n_rows, H, V))


def psd_set_confidence_impl(impl: int) -> int:
    return int(LIB.psd_set_confidence_impl(int(impl)))


PSD_TUNE_BAND_BYTES = 1
PSD_TUNE_PDL = 2
PSD_TUNE_TILE_ORDER = 3
PSD_TUNE_COMPACT_ROWS = 4
PSD_TUNE_WAIT_LIMIT = 5
PSD_TUNE_SELFTEST_STALL = 6


def psd_set_tuning(knob: int, value: int) -> int:
    return int(LIB.psd_set_tuning(int(knob), int(value)))


def psd_set_kernel_events(start_event, stop_event) -> int:
    """torch.cuda.Event objects (already recorded once or created with enable_timing=True), or None."""
    def h(e):
        if e is None:
            return None
        return e.cuda_event if hasattr(e, "cuda_event") else int(e)
    return int(LIB.psd_set_kernel_events(h(start_event), h(stop_event)))


def psd_confidence_kernel_name(n_rows: int) -> str:
    """Name of the kernel the confidence pass launches for ``n_rows`` rows under the current setting."""
    return LIB.psd_confidence_kernel_name(int(n_rows)).decode()


def psd_launch_count() -> int:
    return int(LIB.psd_launch_count())


def psd_confidence(hidden, w_lm, out_token, out_conf, out_lse=None, workspace=None, status=None, stream=None,
                   row_ids=None):
    """hidden [n_rows, H] bf16, w_lm [V, H] bf16 -> out_token int32, out_conf fp32 (and out_lse) [n_rows]."""
    n_rows, H = hidden.shape
    if row_ids is not None:
        n_rows = row_ids.numel()
    V = w_lm.shape[0]
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(LIB.psd_confidence(_ptr(hidden), _ptr(w_lm), _ptr(row_ids), n_rows, H, V, _ptr(out_token),
                              _ptr(out_conf), _ptr(out_lse), _ptr(workspace), ws_bytes, _ptr(status),
                              _stream(stream)), "psd_confidence")


def psd_confidence_masked(hidden, w_lm, row_mask, out_token, out_conf, out_lse=None, workspace=None, status=None,
                          stream=None):
    """psd_confidence on the rows whose ``row_mask`` (int32, device, one entry per row of ``hidden``) is
    non-zero; the other rows' outputs are left untouched.  No host synchronisation."""
    n_rows, H = hidden.shape
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(LIB.psd_confidence_masked(_ptr(hidden), _ptr(w_lm), _ptr(row_mask), n_rows, H, w_lm.shape[0],
                                     _ptr(out_token), _ptr(out_conf), _ptr(out_lse), _ptr(workspace), ws_bytes,
                                     _ptr(status), _stream(stream)), "psd_confidence_masked")


def psd_compact_rows_enabled(n_rows: int) -> int:
    return int(LIB.psd_compact_rows_enabled(int(n_rows)))


def psd_confidence_partial(hidden, w_shard, v_offset, out_max, out_sumexp, out_arg, workspace, status=None,
                           stream=None):
    """Per-row (max, sum-exp, global argmax) over the vocabulary rows held in ``w_shard`` [V_shard, H]."""
    n_rows, H = hidden.shape
    _check(LIB.psd_confidence_partial(_ptr(hidden), _ptr(w_shard), n_rows, H, w_shard.shape[0], int(v_offset),
                                      _ptr(out_max), _ptr(out_sumexp), _ptr(out_arg), _ptr(workspace),
                                      workspace.numel() * workspace.element_size(), _ptr(status), _stream(stream)),
           "psd_confidence_partial")


def psd_merge_partials(max_, sumexp, arg, out_token, out_conf, out_lse=None, stream=None):
    """Merge [n_shards, n_rows] triples into token / confidence / lse per row."""
    n_shards, n_rows = max_.shape
    _check(LIB.psd_merge_partials(_ptr(max_), _ptr(sumexp), _ptr(arg), n_shards, n_rows, _ptr(out_token),
                                  _ptr(out_conf), _ptr(out_lse), _stream(stream)), "psd_merge_partials")


PSD_STATIC_SCRATCH_BYTES = 4 << 20


def psd_confidence_static(hidden, w_lm, out_token, out_conf, out_lse=None, status=None, stream=None):
    """psd_confidence for callers that cannot allocate: the scratch is a fixed array inside the
    library (PSD_STATIC_SCRATCH_BYTES); larger problems raise PSD_ERR_WORKSPACE.  Calls on one device
    must not overlap."""
    n_rows, H = hidden.shape
    _check(LIB.psd_confidence_static(_ptr(hidden), _ptr(w_lm), n_rows, H, w_lm.shape[0], _ptr(out_token),
                                     _ptr(out_conf), _ptr(out_lse), _ptr(status), _stream(stream)),
           "psd_confidence_static")


def psd_select_unmask(conf, tok, tokens, mask, p: PsdPolicy, sel, n_sel, sel_pos, node=None, n_nodes=1,
                      stream=None):
    B, M = mask.shape
    _check(LIB.psd_select_unmask(_ptr(conf), _ptr(tok), _ptr(node), n_nodes, _ptr(tokens), _ptr(mask), B, M, p,
                                 _ptr(sel), _ptr(n_sel), _ptr(sel_pos), _stream(stream)), "psd_select_unmask")


def psd_build_drafts(conf, tok, tokens, mask, p: PsdPolicy, sigma, n_fill, draft_tokens, draft_mask, node=None,
                     n_nodes=1, stream=None):
    B, M = mask.shape
    _check(LIB.psd_build_drafts(_ptr(conf), _ptr(tok), _ptr(node), n_nodes, _ptr(tokens), _ptr(mask), B, M, p,
                                _ptr(sigma), _ptr(n_fill), _ptr(draft_tokens), _ptr(draft_mask), _stream(stream)),
           "psd_build_drafts")


def psd_verify_accept(tokV, confV, sigma, n_fill, draft_tokens, draft_mask, p: PsdPolicy, tokens, mask, k_star,
                      n_spec_accepted, n_committed, accepted=None, stream=None):
    B, M = tokens.shape
    _check(LIB.psd_verify_accept(_ptr(tokV), _ptr(confV), _ptr(sigma), _ptr(n_fill), _ptr(draft_tokens),
                                 _ptr(draft_mask), B, M, p, _ptr(tokens), _ptr(mask), _ptr(k_star),
                                 _ptr(n_spec_accepted), _ptr(n_committed), _ptr(accepted), _stream(stream)),
           "psd_verify_accept")


_STEP_FIELDS = [n for n, _ in PsdStepIO._fields_]


@dataclass
class StepBuffers:
    """The tensors of one decoding step (psd_step_io_t), all on one device or all on the host
    (``w_lm`` always on the device)."""
    hidden: torch.Tensor
    w_lm: torch.Tensor
    sigma: torch.Tensor
    n_fill: torch.Tensor
    draft_tokens: torch.Tensor
    draft_mask: torch.Tensor
    tokV: torch.Tensor
    confV: torch.Tensor
    tokens: torch.Tensor
    mask: torch.Tensor
    k_star: torch.Tensor
    n_spec_accepted: torch.Tensor
    n_committed: torch.Tensor
    sel: torch.Tensor
    n_sel: torch.Tensor
    sel_pos: torch.Tensor

    def io(self) -> PsdStepIO:
        vals = [self.hidden, self.w_lm, self.sigma, self.n_fill, self.draft_tokens, self.draft_mask, self.tokV,
                self.confV, self.tokens, self.mask, self.k_star, self.n_spec_accepted, self.n_committed, self.sel,
                self.n_sel, self.sel_pos]
        return PsdStepIO(*[_ptr(v) for v in vals])

    @staticmethod
    def allocate(B, M, D, H, hidden, w_lm, device, pin=False):
        kw = dict(device=device)
        if pin:
            kw["pin_memory"] = True
        i32 = lambda *s: torch.zeros(*s, dtype=torch.int32, **kw)
        return StepBuffers(hidden=hidden, w_lm=w_lm, sigma=i32(B, M), n_fill=i32(B, D), draft_tokens=i32(B, D, M),
                           draft_mask=i32(B, D, M), tokV=i32(B, D, M),
                           confV=torch.zeros(B, D, M, dtype=torch.float32, **kw), tokens=i32(B, M), mask=i32(B, M),
                           k_star=i32(B), n_spec_accepted=i32(B), n_committed=i32(B), sel=i32(B, M), n_sel=i32(B),
                           sel_pos=i32(B, M))


def psd_step_host_block(B, M, D):
    """(bytes, offsets[15]) of the one-block host layout that psd_step_host moves with single copies."""
    off = (_sz * 15)()
    n = int(LIB.psd_step_host_block(B, M, D, off))
    return n, [int(x) for x in off]


def host_step_buffers(B, M, D, hidden, w_lm) -> StepBuffers:
    """StepBuffers whose arrays are views of ONE pinned host block laid out as psd_step_host_block says
    (``hidden``: a host tensor, ``w_lm``: a device tensor).  The block is kept alive by the views."""
    n, off = psd_step_host_block(B, M, D)
    block = torch.zeros(n, dtype=torch.uint8).pin_memory()

    def view(o, shape, dtype=torch.int32):
        count = 1
        for d in shape:
            count *= d
        return block[o:o + 4 * count].view(dtype).view(*shape)

    return StepBuffers(hidden=hidden, w_lm=w_lm, sigma=view(off[0], (B, M)), n_fill=view(off[1], (B, D)),
                       draft_tokens=view(off[2], (B, D, M)), draft_mask=view(off[3], (B, D, M)),
                       tokV=view(off[4], (B, D, M)), confV=view(off[5], (B, D, M), torch.float32),
                       tokens=view(off[6], (B, M)), mask=view(off[7], (B, M)), k_star=view(off[8], (B,)),
                       n_spec_accepted=view(off[9], (B,)), n_committed=view(off[10], (B,)), sel=view(off[11], (B, M)),
                       n_sel=view(off[12], (B,)), sel_pos=view(off[13], (B, M)))


def psd_step(buf: StepBuffers, p: PsdPolicy, workspace, status=None, stream=None):
    B, M = buf.tokens.shape
    H = buf.hidden.shape[1]
    V = buf.w_lm.shape[0]
    io = buf.io()
    _check(LIB.psd_step(ctypes.byref(io), B, M, H, V, p, _ptr(workspace),
                        workspace.numel() * workspace.element_size(), _ptr(status), _stream(stream)), "psd_step")


def psd_step_host_bytes(B, M, H, V, D) -> int:
    return int(LIB.psd_step_host_bytes(B, M, H, V, D))


def psd_step_host(buf: StepBuffers, p: PsdPolicy, staging, stream=None) -> int:
    """``buf`` holds host tensors (w_lm on the device).  Returns the device status word."""
    B, M = buf.tokens.shape
    H = buf.hidden.shape[1]
    V = buf.w_lm.shape[0]
    io = buf.io()
    st = _i32(0)
    _check(LIB.psd_step_host(ctypes.byref(io), B, M, H, V, p, _ptr(staging),
                             staging.numel() * staging.element_size(), ctypes.byref(st), _stream(stream)),
           "psd_step_host")
    return int(st.value)


def psd_decode_scratch_bytes(B: int, M: int) -> int:
    return int(LIB.psd_decode_scratch_bytes(B, M))


def psd_step_dag(buf: StepBuffers, p: PsdPolicy, g: PsdDag, workspace, status=None, stream=None):
    B, M = buf.tokens.shape
    io = buf.io()
    _check(LIB.psd_step_dag(ctypes.byref(io), B, M, buf.hidden.shape[1], buf.w_lm.shape[0], p, ctypes.byref(g),
                            _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(status),
                            _stream(stream)), "psd_step_dag")


def psd_decode_blocks(body, user, buf: StepBuffers, p: PsdPolicy, order: int, max_iterations: int, scratch,
                      workspace, status=None, passes=None, done_iteration=None, trace=None, stream=None, dag=None):
    """Algorithm 1 over the blocks of ``buf`` (device tensors; ``buf.hidden`` is scratch the body fills).

    ``body`` is either the address of a native ``psd_body_fn`` (an int, e.g. ``table_body_address()``)
    with ``user`` the address of its argument, or a Python callable
    ``body(tokens_ptr, mask_ptr, n_seq, M, hidden_ptr, stream_ptr) -> int``.  Returns PsdDecodeStats."""
    B, M = buf.tokens.shape
    H = buf.hidden.shape[1]
    V = buf.w_lm.shape[0]
    if callable(body):
        fn = body
        cb = BODY_FN(lambda u, t, m, n, mm, h, s: int(fn(t, m, n, mm, h, s)))
        body_ptr = ctypes.cast(cb, _vp)
    else:
        cb, body_ptr = None, _vp(int(body))
    io = buf.io()
    stats = PsdDecodeStats()
    code = LIB.psd_decode_blocks(body_ptr, user, ctypes.byref(io), B, M, H, V, p,
                                 ctypes.byref(dag) if dag is not None else None, int(order), int(max_iterations),
                                 _ptr(scratch), scratch.numel() * scratch.element_size(), _ptr(workspace),
                                 workspace.numel() * workspace.element_size(), _ptr(status), _ptr(passes),
                                 _ptr(done_iteration), _ptr(trace), ctypes.byref(stats), _stream(stream))
    del cb
    _check(code, "psd_decode_blocks")
    return stats


def table_body_address() -> int:
    """Address of the native stand-in body psd_table_body, to pass as ``body``."""
    return ctypes.cast(LIB.psd_table_body, _vp).value


def table_body_user(table, B: int) -> PsdTableBody:
    """psd_table_body_t for a device table [B, M, 3, H] bf16; keep the object alive during the call and
    pass ``ctypes.addressof(obj)`` as ``user``."""
    return PsdTableBody(_ptr(table), int(B), int(table.shape[-1]))


def psd_table_body(user: PsdTableBody, mask, hidden, stream=None):
    """One call of the stand-in body: ``mask`` [n_seq, M] int32 -> ``hidden`` [n_seq*M, H] bf16 (device)."""
    n_seq, M = mask.shape
    _check(LIB.psd_table_body(ctypes.addressof(user), None, _ptr(mask), n_seq, M, _ptr(hidden), _stream(stream)),
           "psd_table_body")


def psd_dag_init(node_ranks, edges=None) -> PsdDag:
    """A draft graph from node rank sets (node 0 = the root, empty) and, optionally, an edge list
    [(p, k), ...]; without one every strict-subset pair is an edge."""
    K = len(node_ranks)
    ranks = (ctypes.c_uint64 * max(K, 1))(*[sum(1 << int(j) for j in s) for s in node_ranks])
    par = None
    if edges is not None:
        words = [0] * K
        for q, k in edges:
            words[k] |= 1 << q
        par = (ctypes.c_uint64 * max(K, 1))(*words)
    g = PsdDag()
    _check(LIB.psd_dag_init(ctypes.byref(g), K, ctypes.cast(ranks, _vp), ctypes.cast(par, _vp) if par else None),
           "psd_dag_init")
    return g


def psd_build_drafts_dag(conf, tok, tokens, mask, p: PsdPolicy, g: PsdDag, sigma, n_fill, draft_tokens, draft_mask,
                         node=None, n_nodes=1, stream=None):
    B, M = mask.shape
    _check(LIB.psd_build_drafts_dag(_ptr(conf), _ptr(tok), _ptr(node), n_nodes, _ptr(tokens), _ptr(mask), B, M, p,
                                    ctypes.byref(g), _ptr(sigma), _ptr(n_fill), _ptr(draft_tokens), _ptr(draft_mask),
                                    _stream(stream)), "psd_build_drafts_dag")


def psd_verify_accept_dag(tokV, confV, sigma, draft_tokens, draft_mask, p: PsdPolicy, g: PsdDag, tokens, mask, k_star,
                          n_spec_accepted, n_committed, accepted=None, stream=None):
    B, M = tokens.shape
    _check(LIB.psd_verify_accept_dag(_ptr(tokV), _ptr(confV), _ptr(sigma), _ptr(draft_tokens), _ptr(draft_mask), B, M,
                                     p, ctypes.byref(g), _ptr(tokens), _ptr(mask), _ptr(k_star), _ptr(n_spec_accepted),
                                     _ptr(n_committed), _ptr(accepted), _stream(stream)), "psd_verify_accept_dag")
