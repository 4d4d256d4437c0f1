#!/usr/bin/env python
"""Writes tests/golden/full_size_confidence_<workload>.npz: the fp64 oracle's (token, confidence, lse,
gap) of Sec. 3.1 for EVERY row of the verification batch (token, conf, lse, gap) and of the stage-1
pass (token1, conf1, lse1, gap1) of the three large workloads (class_7b, batched_serving,
deep_sweep), so that the GPU tests can hold every row of a full-size launch to the oracle without
spending minutes of host time per run.

Calls only oracle/ and the seeded input generator; nothing here comes from the CUDA path.  Each file
also stores SHA-256 digests of the exact input bytes (W and the hidden rows) the values were computed
from; a test that finds other digests for its regenerated inputs must not use the file.

    python tests/golden/make_full_size_confidence.py [workload ...]

About 2 x 8192 + 1536 rows at 25-50 rows/s: ten minutes or so on 8-16 cores.
"""
from __future__ import annotations

import hashlib
import os
import sys
import time

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import oracle  # noqa: E402
import psd_inputs as gen  # noqa: E402

WORKLOADS = ("class_7b", "batched_serving", "deep_sweep")


def digest(a: np.ndarray) -> str:
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()


def path_for(name: str) -> str:
    return os.path.join(HERE, f"full_size_confidence_{name}.npz")


def all_rows(name: str, what: str, hidden: np.ndarray, W: np.ndarray, chunk: int = 256):
    R = hidden.shape[0]
    tok = np.empty(R, dtype=np.int32)
    conf = np.empty(R, dtype=np.float64)
    lse = np.empty(R, dtype=np.float64)
    gap = np.empty(R, dtype=np.float64)
    t0 = time.perf_counter()
    for r0 in range(0, R, chunk):
        r1 = min(R, r0 + chunk)
        tok[r0:r1], conf[r0:r1], lse[r0:r1], gap[r0:r1] = oracle.confidence(hidden[r0:r1], W)
        print(f"{name} {what}: rows {r1}/{R}  {time.perf_counter() - t0:.0f} s", flush=True)
    return tok, conf, lse, gap.astype(np.float32)


def write(name: str) -> str:
    cfg = gen.CONFIGS[name]
    wl = gen.make(cfg)
    out = path_for(name)
    ids = dict(sha256_W=np.array(digest(wl.W)), sha256_hidden=np.array(digest(wl.hidden_verify)),
               sha256_hidden1=np.array(digest(wl.hidden_stage1)),
               shape=np.array([cfg.rows, cfg.H, cfg.V], dtype=np.int64))
    have = {}
    if os.path.exists(out):          # parts this script wrote earlier from the same input bytes are kept
        with np.load(out) as old:
            if str(old["sha256_W"]) == str(ids["sha256_W"]):
                if str(old["sha256_hidden"]) == str(ids["sha256_hidden"]):
                    have.update({k: old[k] for k in ("token", "conf", "lse", "gap")})
                if "sha256_hidden1" in old and str(old["sha256_hidden1"]) == str(ids["sha256_hidden1"]):
                    have.update({k: old[k] for k in ("token1", "conf1", "lse1", "gap1")})
    if "token" not in have:
        have.update(zip(("token", "conf", "lse", "gap"), all_rows(name, "verification batch", wl.hidden_verify, wl.W)))
    if "token1" not in have:
        have.update(zip(("token1", "conf1", "lse1", "gap1"), all_rows(name, "stage-1 pass", wl.hidden_stage1, wl.W)))
    np.savez_compressed(out, **have, **ids)
    return out


if __name__ == "__main__":
    for n in (sys.argv[1:] or WORKLOADS):
        print(write(n))
