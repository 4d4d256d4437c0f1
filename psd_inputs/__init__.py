"""Seeded synthetic workloads for the PSD hot path.

Input generation only: an LM-head matrix ``W[V, H]`` (bf16), and hidden states
``[rows, H]`` (bf16) made of unit Gaussian noise plus, on a fraction of rows, a
multiple of one row of ``W`` so that the row's softmax has a planted peak.  None of
the method's arithmetic lives here; the CPU oracle's tests and the CUDA path's tests
both read the bytes this module writes, and nothing else is shared between them.

bf16 arrays are returned as ``numpy.uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libpsd_gen.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile gen.c into libpsd_gen.so next to it (no-op when up to date)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        u64, i64, i32, f64, vp = (ctypes.c_uint64, ctypes.c_int64, ctypes.c_int32,
                                  ctypes.c_double, ctypes.c_void_p)
        lib.psd_gen_u64.restype = u64
        lib.psd_gen_u64.argtypes = [u64, u64, u64]
        lib.psd_gen_uniform.restype = f64
        lib.psd_gen_uniform.argtypes = [u64, u64, u64]
        lib.psd_gen_normal.restype = f64
        lib.psd_gen_normal.argtypes = [u64, u64, u64]
        lib.psd_gen_bf16.restype = ctypes.c_uint16
        lib.psd_gen_bf16.argtypes = [ctypes.c_float]
        lib.psd_gen_weights.restype = None
        lib.psd_gen_weights.argtypes = [u64, i64, i64, f64, i64, i64, vp]
        lib.psd_gen_peaks.restype = None
        lib.psd_gen_peaks.argtypes = [u64, i64, i64, i64, i64, f64, f64, f64, f64, vp, vp, vp]
        lib.psd_gen_hidden.restype = None
        lib.psd_gen_hidden.argtypes = [u64, i64, i64, i64, i64, i64, f64, i32, i64, i64,
                                       vp, vp, vp, vp, vp]
        _lib = lib
    return _lib


STREAM_MISC = 7
W_STD = 0.02


def uniform(seed: int, stream: int, idx: int) -> float:
    return _load().psd_gen_uniform(seed, stream, idx)


def normal(seed: int, stream: int, k: int) -> float:
    return _load().psd_gen_normal(seed, stream, k)


def bf16_bits(x) -> np.ndarray:
    """fp32 -> bf16 bit patterns (round to nearest even), vectorised."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    u = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_to_f64(bits) -> np.ndarray:
    """bf16 bit patterns -> float64, exact."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


@dataclass(frozen=True)
class Config:
    """One workload shape plus the policy parameters it is run with."""
    name: str
    B: int
    H: int
    V: int
    M: int
    D: int                 # chain nodes in the verify batch, root included
    frac: float            # planted-peak fraction
    s_lo: float = 4.0      # peak scale range (logit units, see gen.c gain_mode 1)
    s_hi: float = 4.0
    rho: float = 0.8       # probability that depth d keeps depth d-1's peak
    tau: float = 0.9
    k_min: int = 1
    k_max: int = 0         # 0 = no cap
    stride: int = 0        # 0 = k_min
    seed: int = 0
    gain_mode: int = 1
    mask_id: int = -1      # filled in __post_init__ when left negative: V (one past the vocabulary)

    def __post_init__(self):
        if self.mask_id < 0:
            object.__setattr__(self, "mask_id", self.V)

    @property
    def rows(self) -> int:
        return self.B * self.D * self.M


# The five workload shapes of the benchmark description, in its order.
CONFIGS = {
    "tiny": Config("tiny", B=1, H=256, V=1024, M=32, D=4, frac=0.5, tau=0.9, k_min=1, k_max=32, seed=0),
    "single_request": Config("single_request", B=1, H=4096, V=126464, M=32, D=4, frac=0.3,
                             tau=0.8, k_min=1, k_max=8, seed=2),
    "class_7b": Config("class_7b", B=8, H=3584, V=152064, M=32, D=6, frac=0.5, s_lo=1.0, s_hi=6.0,
                       tau=0.9, k_min=4, k_max=4, stride=4, seed=3),
    "batched_serving": Config("batched_serving", B=64, H=4096, V=126464, M=32, D=4, frac=0.4,
                              tau=0.9, k_min=1, k_max=16, seed=4),
    "deep_sweep": Config("deep_sweep", B=16, H=4096, V=126464, M=64, D=8, frac=0.6, rho=0.8,
                         tau=0.85, k_min=1, k_max=64, seed=5),
}


def with_depth(cfg: Config, D: int) -> Config:
    """The same workload at another draft depth (the depth sweep of ``deep_sweep``)."""
    from dataclasses import replace
    return replace(cfg, D=D, name=f"{cfg.name}_D{D}")


def weights(cfg: Config) -> np.ndarray:
    """``W[V, H]`` bf16 bits, ``N(0, 0.02^2)``."""
    out = np.empty((cfg.V, cfg.H), dtype=np.uint16)
    _load().psd_gen_weights(cfg.seed, cfg.V, cfg.H, W_STD, 0, cfg.V, out.ctypes.data)
    return out


@dataclass
class Workload:
    cfg: Config
    W: np.ndarray                  # [V, H] uint16 (bf16 bits)
    hidden_stage1: np.ndarray      # [B*M, H] uint16: the single-sequence pass that precedes drafting
    hidden_verify: np.ndarray      # [B*D*M, H] uint16: rows (b, d, i) of the batched verification pass
    present: np.ndarray            # [B, M, D+1] int32, level index l+1 (l = -1 is the stage-1 pass)
    token: np.ndarray              # [B, M, D+1] int32 planted vocabulary entry
    scale: np.ndarray              # [B, M, D+1] float64
    extra: dict = field(default_factory=dict)


def make(cfg: Config, W: np.ndarray | None = None) -> Workload:
    """Generate the full workload of ``cfg``. ``W`` may be passed in to avoid regenerating it."""
    lib = _load()
    if W is None:
        W = weights(cfg)
    B, M, D, H, V = cfg.B, cfg.M, cfg.D, cfg.H, cfg.V
    nl = D + 1
    present = np.empty((B, M, nl), dtype=np.int32)
    token = np.empty((B, M, nl), dtype=np.int32)
    scale = np.empty((B, M, nl), dtype=np.float64)
    lib.psd_gen_peaks(cfg.seed, B, M, nl, V, cfg.frac, cfg.rho, cfg.s_lo, cfg.s_hi,
                      present.ctypes.data, token.ctypes.data, scale.ctypes.data)
    w_rows = np.ascontiguousarray(W[token.reshape(-1)])           # [B*M*nl, H]
    h1 = np.empty((B * M, H), dtype=np.uint16)
    hv = np.empty((B * D * M, H), dtype=np.uint16)
    lib.psd_gen_hidden(cfg.seed, B, M, nl, H, V, W_STD, cfg.gain_mode, 0, 1,
                       present.ctypes.data, scale.ctypes.data, w_rows.ctypes.data,
                       h1.ctypes.data, None)
    lib.psd_gen_hidden(cfg.seed, B, M, nl, H, V, W_STD, cfg.gain_mode, 1, D,
                       present.ctypes.data, scale.ctypes.data, w_rows.ctypes.data,
                       hv.ctypes.data, None)
    return Workload(cfg, W, h1, hv, present, token, scale)


def random_state(seed: int, B: int, M: int, V: int, p_masked: float, mask_id: int):
    """A partially decoded block state: ``tokens[B, M]``, ``mask[B, M]`` int32 (1 = masked)."""
    lib = _load()
    tokens = np.empty((B, M), dtype=np.int32)
    mask = np.empty((B, M), dtype=np.int32)
    for b in range(B):
        for i in range(M):
            e = b * M + i
            mk = lib.psd_gen_uniform(seed, STREAM_MISC, 2 * e) <= p_masked
            tk = int(lib.psd_gen_uniform(seed, STREAM_MISC, 2 * e + 1) * V) % V
            mask[b, i] = 1 if mk else 0
            tokens[b, i] = mask_id if mk else tk
    return tokens, mask


# ----------------------------------------------------------------------------------------------
# A stand-in transformer body for the whole decoding loop: a table of hidden states.
# ----------------------------------------------------------------------------------------------

TABLE_LEVELS = 3


def table_body(cfg: Config, W: np.ndarray, seed: int | None = None):
    """Hidden states of a toy body whose output depends on the context only through the number of
    committed neighbours: ``table[b, i, c, :]`` (bf16 bits) is what slot ``i`` of block ``b`` sees when
    ``c`` of its neighbours ``i-1, i+1`` are committed.  A slot carries a planted peak with probability
    ``cfg.frac``; its scale starts in [2.75, 3.5] and grows by half a unit (2 nats) per committed
    neighbour, so that confidences cross the usual thresholds as the block fills, and its token
    changes from one level to the next with probability ``1 - cfg.rho`` (so that a draft built from an
    older prediction can be rejected).  Returns (table [B, M, 3, H] uint16, token [B, M, 3] int32,
    present [B, M] int32, scale [B, M, 3] float64)."""
    rng = np.random.default_rng(cfg.seed * 7919 + 17 if seed is None else seed)
    B, M, H, V, L = cfg.B, cfg.M, cfg.H, cfg.V, TABLE_LEVELS
    present = (rng.random((B, M)) < cfg.frac).astype(np.int32)
    s0 = rng.uniform(2.75, 3.5, size=(B, M))        # confidence 0.27 .. 0.88 with no committed neighbour
    scale = s0[:, :, None] + np.arange(L)[None, None, :] * 0.5
    token = np.empty((B, M, L), dtype=np.int32)
    token[:, :, 0] = rng.integers(0, V, size=(B, M))
    for c in range(1, L):
        keep = rng.random((B, M)) < cfg.rho
        token[:, :, c] = np.where(keep, token[:, :, c - 1], rng.integers(0, V, size=(B, M)))
    q = H * W_STD * W_STD
    table = np.empty((B, M, L, H), dtype=np.uint16)
    for b in range(B):
        for i in range(M):
            for c in range(L):
                z = rng.standard_normal(H).astype(np.float32)
                if present[b, i]:
                    w = bf16_to_f64(W[token[b, i, c]])
                    g = (np.log(V) + q / 2 + 4.0 * (scale[b, i, c] - 3.0)) / max(float(w @ w), 1e-12)
                    z = (z.astype(np.float64) + g * w).astype(np.float32)
                table[b, i, c] = bf16_bits(z)
    return table, token, present, scale


def table_rows(mask: np.ndarray, seq_per_block: int) -> np.ndarray:
    """Row of the flattened table ``[B*M*3, H]`` that each slot of ``mask[n_seq, M]`` reads:
    ``((b*M + i)*3 + c)`` with ``b = s // seq_per_block`` and ``c`` = committed neighbours of slot i."""
    mask = np.asarray(mask)
    n_seq, M = mask.shape
    committed = (mask == 0).astype(np.int64)
    c = np.zeros((n_seq, M), dtype=np.int64)
    c[:, 1:] += committed[:, :-1]
    c[:, :-1] += committed[:, 1:]
    b = (np.arange(n_seq) // seq_per_block)[:, None]
    i = np.arange(M)[None, :]
    return (b * M + i) * TABLE_LEVELS + c
