#!/usr/bin/env python
"""Benchmark of the PSD per-step hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

A step is one pass of the whole path over one batch of synthetic input: psd_confidence on all
B*D*M rows of the verification batch, then psd_verify_accept, psd_select_unmask and
psd_build_drafts (psd_step), on one stream.  The metric is masked positions scored and accepted
per second = B*D*M / t_step.  Rank 0 prints ONE JSON line.

Without --config the line's own result is the largest single-GPU workload (batched_serving: 8192
rows, bound by the bf16 tensor pipe) and the key "single_request" holds the same measurements of
the 128-row workload (bound by the one pass over W in HBM), so that one run covers both regimes.
A timed region is exactly K steps; it is repeated until --min-seconds of device time have passed
and the median region is reported with the spread.

For N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs an independent
replica on its own batch: no data-path collective, weak scaling.

--impl reference times the CPU oracle (the only "reference implementation" of this path) on the
host cores, on bounded samples of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
from dataclasses import replace

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "masked positions scored+accepted/sec per step"
UNIT = "positions/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the fused kernel, from the ncu captures
# summarised under profiles/, keyed by (workload, kernel): a capture of another kernel does not count.
NCU_TRAFFIC = {
    ("single_request", "confidence_tc_kernel"): (1.0413e9, "profiles/confidence_tc_single_request.md"),
    ("batched_serving", "confidence_tc_kernel"): (2.1491e9, "profiles/confidence_tc_batched_serving.md"),
    ("single_request_B2", "confidence_tc2_kernel"): (1.0534e9, "profiles/confidence_tc2_256_rows.md"),
    ("single_request_B8", "confidence_tc_kernel"): (1.0492e9, "profiles/confidence_tc_1024_rows.md"),
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._period = period_s
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def sample(self):
        if self._nv is None:
            return
        try:
            mhz = int(self._nv.nvmlDeviceGetClockInfo(self._h, self._nv.NVML_CLOCK_SM))
            bits = int(self._nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
        except Exception:
            return
        self.samples.append(mhz)
        for bit, name in self.REASONS.items():
            if bits & bit:
                self.reasons.add(name)

    def _run(self):
        while not self._stop.is_set():
            self.sample()
            self._stop.wait(self._period)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": (statistics.median(self.samples) if self.samples else None),
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


def algorithmic_bytes(cfg) -> float:
    """Bytes the method has to move per launch of the fused kernel: W once, the hidden rows once,
    and 12 bytes of result per row.  Logits are not counted: the method never materialises them."""
    R = cfg.rows
    return float(cfg.V) * cfg.H * 2 + float(R) * cfg.H * 2 + 12.0 * R


def algorithmic_flops(cfg) -> float:
    return 2.0 * cfg.rows * cfg.V * cfg.H


def sustained_copy_gbs(device, seconds=0.5):
    """A STREAM-style copy (b.copy_(a), 512 MiB each way) run back to back for `seconds`: read + write
    bytes per second under the same sustained conditions as the timed regions.  Context for the HBM-bound
    figure, printed beside the fraction of the pod file's (burst) copy bandwidth."""
    import torch
    n = 256 << 20
    a = torch.empty(n, dtype=torch.bfloat16, device=device)
    b = torch.empty(n, dtype=torch.bfloat16, device=device)
    a.fill_(1.0)
    for _ in range(3):
        b.copy_(a)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps, total = 0, 0.0
    while total < seconds and reps < 100000:
        e0.record()
        for _ in range(20):
            b.copy_(a)
        e1.record()
        torch.cuda.synchronize()
        total += e0.elapsed_time(e1) * 1e-3
        reps += 20
    del a, b
    return 2.0 * n * 2 * reps / total / 1e9


def ridge_rows(peaks) -> float:
    return peaks["bf16_tflops"] * 1e12 / (peaks["hbm_gbs"] * 1e9)


# ------------------------------------------------------------------------------------ shared by both arms

def config_dict(cfg, n_gpus):
    """The `config` object of the JSON line: the same keys and values in the library arm and in the
    reference arm, so that the two lines can be matched."""
    return {"workload": cfg.name, "B": cfg.B, "D": cfg.D, "M": cfg.M, "H": cfg.H, "V": cfg.V, "rows": cfg.rows,
            "policy": {"tau": cfg.tau, "k_min": cfg.k_min, "k_max": cfg.k_max, "stride": cfg.stride},
            "parallelism": f"replicas x{n_gpus}",
            "l2": f"inputs larger than L2: W is {cfg.V * cfg.H * 2 / 1e6:.0f} MB and is re-read every step"}


def resolve_config(name, blocks=0):
    import psd_inputs as gen
    if name.startswith("deep_sweep_D"):
        cfg = gen.with_depth(gen.CONFIGS["deep_sweep"], int(name.rsplit("D", 1)[1]))
    else:
        cfg = gen.CONFIGS[name]
    if blocks > 0:
        cfg = replace(cfg, B=blocks, name=f"{cfg.name}_B{blocks}")
    return cfg


# ------------------------------------------------------------------------------------ reference arm

def oracle_sample_rate(cfg, wl, n_rows):
    """Times the oracle on the first n_rows rows of the verification batch; returns seconds."""
    import oracle
    t0 = time.perf_counter()
    oracle.confidence(wl.hidden_verify[:n_rows], wl.W)
    return time.perf_counter() - t0


def oracle_full_step(cfg, wl, n_blocks, po):
    """The oracle's whole step on the first n_blocks blocks: stage-1 pass, policy, drafts,
    verification pass, acceptance, policy on node k*, next drafts.  Returns (seconds of the step
    proper, rows scored by the step)."""
    import oracle
    B, M, D = n_blocks, cfg.M, cfg.D
    tok1, conf1, _, _ = oracle.confidence(wl.hidden_stage1[:B * M], wl.W)
    tokens = np.full((B, M), cfg.mask_id, dtype=np.int32)
    mask = np.ones((B, M), dtype=np.int32)
    tokens, mask, *_ = oracle.select_unmask(conf1.reshape(B, M), tok1.reshape(B, M), tokens, mask, po)
    sigma, n_fill, dt, dm = oracle.build_drafts(conf1.reshape(B, M), tok1.reshape(B, M), tokens, mask, po)
    t0 = time.perf_counter()
    tokV, confV, _, _ = oracle.confidence(wl.hidden_verify[:B * D * M], wl.W)
    tokV, confV = tokV.reshape(B, D, M), confV.reshape(B, D, M)
    tokens, mask, ks, _, _, _ = oracle.verify_accept(tokV, confV, sigma, n_fill, dt, dm, po)
    rows = np.arange(B)
    tokens, mask, *_ = oracle.select_unmask(confV[rows, ks], tokV[rows, ks], tokens, mask, po)
    oracle.build_drafts(confV[rows, ks], tokV[rows, ks], tokens, mask, po)
    return time.perf_counter() - t0, B * D * M


def oracle_policy(cfg):
    import oracle
    return oracle.Policy(tau=float(np.float32(cfg.tau)), k_min=cfg.k_min, k_max=cfg.k_max, depth=cfg.D,
                         stride=cfg.stride, mask_id=cfg.mask_id)


def cpu_baseline(cfg, wl, budget_s=15.0):
    """The oracle as it stands, on the host cores, on a bounded sample of the workload."""
    import oracle
    probe_rows = min(4, cfg.rows)
    t_probe = oracle_sample_rate(cfg, wl, probe_rows)
    per_row = t_probe / probe_rows
    rows_per_block = cfg.D * cfg.M
    n_blocks = int(max(1, min(cfg.B, budget_s / max(per_row * rows_per_block, 1e-9))))
    secs, rows = oracle_full_step(cfg, wl, n_blocks, oracle_policy(cfg))
    return {"value": rows / secs, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": f"whole step on the first {n_blocks} of {cfg.B} blocks ({rows} of {cfg.rows} rows, "
                      f"all {cfg.V} vocabulary entries), {secs:.2f} s"}


def reference_workload(args, cfg, total_budget):
    """The CPU oracle on one workload: K timed steps after W warm-ups, each step a bounded sample of
    the workload sized so that all of them fit `total_budget` seconds.  Returns the result object."""
    import oracle
    import psd_inputs as gen
    wl = gen.make(cfg)
    t_probe = oracle_sample_rate(cfg, wl, 1)
    rows_per_step = int(max(1, min(cfg.rows, total_budget / max(t_probe, 1e-9) / (args.steps + args.warmup))))
    rows_per_block = cfg.D * cfg.M
    po = oracle_policy(cfg)
    whole_blocks = rows_per_step >= rows_per_block
    n_blocks = min(cfg.B, rows_per_step // rows_per_block) if whole_blocks else 0

    def one_step():
        if whole_blocks:
            return oracle_full_step(cfg, wl, n_blocks, po)
        t0 = time.perf_counter()
        oracle.confidence(wl.hidden_verify[:rows_per_step], wl.W)
        return time.perf_counter() - t0, rows_per_step

    for _ in range(args.warmup):
        one_step()
    secs = rows = 0.0
    for _ in range(args.steps):
        s, r = one_step()
        secs += s
        rows += r
    value = rows / secs
    sample = (f"each step = the whole oracle step on {n_blocks} of {cfg.B} block(s)" if whole_blocks else
              f"each step = the oracle's confidence computation on {rows_per_step} row(s) "
              f"(fewer than one block of {rows_per_block}; the integer stages need whole blocks)")
    sample += f"; {int(rows / args.steps)} of {cfg.rows} rows per step"
    return {"value": value, "unit": UNIT, "ms_per_step": 1e3 * secs / args.steps,
            "config": config_dict(cfg, args.gpus),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def run_reference(args, names):
    """--impl reference: the CPU oracle on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return 0
    budgets = [150.0] if len(names) == 1 else [100.0] + [50.0] * (len(names) - 1)
    results = [reference_workload(args, resolve_config(n, args.blocks), b) for n, b in zip(names, budgets)]
    top = results[0]
    line = {"impl": "reference", "metric": METRIC, "value": top["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": top["ms_per_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": top["config"], "cpu_baseline": top["cpu_baseline"], "e2e": top["e2e"],
            "gpu_launches": 0}
    for r in results[1:]:
        line[r["config"]["workload"]] = r
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------------ our arm

BAD_REASONS = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}


def measure_workload(args, cfg, info, device, peaks, peaks_kind, with_cpu_baseline):
    """All measurements of one workload on this rank's GPU; rank 0 gets the result object back."""
    import torch

    import paper_2605_15609_b200 as psd
    import psd_inputs as gen
    from paper_2605_15609_b200 import replicas

    # Every replica holds the same W; each rank has its own batch of blocks.
    W = gen.weights(cfg)
    wl = gen.make(replace(cfg, seed=replicas.replica_seed(cfg.seed, info.rank)), W)
    B, M, D, H, V, R = cfg.B, cfg.M, cfg.D, cfg.H, cfg.V, cfg.rows
    pg = psd.policy(tau=float(np.float32(cfg.tau)), k_min=cfg.k_min, k_max=cfg.k_max, depth=D, stride=cfg.stride,
                    mask_id=cfg.mask_id)

    def bf16(bits, pin=False):
        t = torch.from_numpy(bits.view(np.int16))
        if pin:
            return t.pin_memory().view(torch.bfloat16)
        return t.to(device).view(torch.bfloat16)

    w_dev, h1_dev, hv_dev = bf16(wl.W), bf16(wl.hidden_stage1), bf16(wl.hidden_verify)
    ws = torch.empty(psd.psd_workspace_bytes(R, H, V), dtype=torch.uint8, device=device)
    status = torch.zeros(1, dtype=torch.int32, device=device)
    stream = torch.cuda.current_stream()

    # Untimed prologue: stage-1 pass -> policy -> first drafts.
    buf = psd.StepBuffers.allocate(B, M, D, H, hv_dev, w_dev, device)
    tok1 = torch.zeros(B * M, dtype=torch.int32, device=device)
    conf1 = torch.zeros(B * M, dtype=torch.float32, device=device)
    psd.psd_confidence(h1_dev, w_dev, tok1, conf1, None, ws, status)
    buf.tokens.fill_(cfg.mask_id)
    buf.mask.fill_(1)
    c1, t1 = conf1.view(B, 1, M), tok1.view(B, 1, M)
    psd.psd_select_unmask(c1, t1, buf.tokens, buf.mask, pg, buf.sel, buf.n_sel, buf.sel_pos)
    psd.psd_build_drafts(c1, t1, buf.tokens, buf.mask, pg, buf.sigma, buf.n_fill, buf.draft_tokens, buf.draft_mask)
    torch.cuda.synchronize()
    first = {k: getattr(buf, k).clone() for k in ("sigma", "n_fill", "draft_tokens", "draft_mask")}

    def timed_region(step_fn, n):
        """Exactly n steps between two events on the launching stream, barrier + synchronize on both
        sides; returns this region's duration as the max over ranks."""
        replicas.barrier(info, device)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(n):
            step_fn(i)
        e1.record(stream)
        torch.cuda.synchronize()
        replicas.barrier(info, device)
        return replicas.max_over_ranks(e0.elapsed_time(e1) * 1e-3, info, device)

    def repeated(step_fn, n):
        """The n-step region repeated until args.min_seconds of device time have passed (at least 3
        times); all ranks run the same number of repeats because they share the max-over-ranks times."""
        times = []
        while len(times) < 3 or (sum(times) < args.min_seconds and len(times) < 5000):
            times.append(timed_region(step_fn, n))
        return times

    def spread(times, n):
        return {"ms_per_step_median": 1e3 * statistics.median(times) / n, "ms_per_step_min": 1e3 * min(times) / n,
                "ms_per_step_max": 1e3 * max(times) / n, "ms_per_step_first": 1e3 * times[0] / n,
                "repeats": len(times), "steps_per_repeat": n,
                "timed_seconds": sum(times)}

    # ---- device-resident steps: the headline value
    for _ in range(args.warmup):
        psd.psd_step(buf, pg, ws, status, stream)
    remeasured = False
    while True:
        sampler = ClockSampler(physical_gpu_index(info.local_rank))
        launches0 = psd.psd_launch_count()
        sampler.start()
        times = repeated(lambda i: psd.psd_step(buf, pg, ws, status, stream), args.steps)
        sampler.sample()
        sampler.stop()
        launches = psd.psd_launch_count() - launches0
        # a measurement that saw a hardware or thermal slowdown is taken again, once
        bad = BAD_REASONS & set(sampler.summary()["reasons"])
        bad_anywhere = replicas.max_over_ranks(1.0 if bad else 0.0, info, device) > 0   # all ranks decide alike
        if not bad_anywhere or remeasured:
            break
        remeasured = True
        time.sleep(2.0)
    if int(status.item()) != 0:
        code = int(status.item())
        raise RuntimeError("device status: " + (psd.status_string(code) if code < 0 else f"{code} non-finite rows"))
    secs_region = statistics.median(times)
    rows_all = replicas.sum_over_ranks(float(R) * args.steps, info, device)
    value = rows_all / secs_region
    timed_total = sum(times)

    if args.profile_only:
        return {"profile_only": True, "workload": cfg.name, "ms_per_step": 1e3 * secs_region / args.steps,
                "gpu_launches": launches}

    # ---- the same steps again with an event pair around the fused kernel of every step
    # (as many steps as the timed regions held, so that the board is in the same sustained state; at most
    # 4096 event pairs)
    n_k = max(8, min(args.steps * len(times), 4096))
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_k)]
    for a, b in evs:          # torch creates the CUDA event on first record; the library re-records it later
        a.record(stream)
        b.record(stream)

    def instrumented(i):
        psd.psd_set_kernel_events(*evs[i])
        psd.psd_step(buf, pg, ws, status, stream)

    secs_instr = timed_region(instrumented, n_k)
    kernel_ms = [a.elapsed_time(b) for a, b in evs]
    kernel_s = statistics.fmean(kernel_ms) * 1e-3

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside)
    hv_host = bf16(wl.hidden_verify, pin=True)
    hb = psd.host_step_buffers(B, M, D, hv_host, w_dev)     # one pinned block: single copies each way
    for k, v in first.items():
        getattr(hb, k).copy_(v)
    staging = torch.empty(psd.psd_step_host_bytes(B, M, H, V, D), dtype=torch.uint8, device=device)
    for _ in range(3):
        psd.psd_step_host(hb, pg, staging, stream)
    times_e2e = repeated(lambda i: psd.psd_step_host(hb, pg, staging, stream), args.steps)
    e2e_value = rows_all / statistics.median(times_e2e)
    # bytes actually moved per step: hidden plus the one block up (draft state, and the output slots and the
    # zeroed status word that travel with it), the same block down
    _, off = psd.psd_step_host_block(B, M, D)
    h2d = R * H * 2 + off[14] + 4
    d2h = off[14] + 4

    if not info.is_main:
        return None

    tensor_bound = R > ridge_rows(peaks)
    kernel_name = psd.psd_confidence_kernel_name(R)
    if tensor_bound:
        # back-to-back tensor-bound steps for over a second sit at the board's power cap: the sustained
        # cuBLAS figure is the like-for-like peak there, the burst figure otherwise; both fractions are given
        sustained = timed_total > 1.0
        peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
        achieved = algorithmic_flops(cfg) / kernel_s / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "peak_kind": f"{'sustained' if sustained else 'burst'} bf16, of {peaks_kind}",
                "frac_of_burst": achieved / peaks["bf16_tflops"],
                "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"]}
    else:
        peak = peaks["hbm_gbs"]
        achieved = algorithmic_bytes(cfg) / kernel_s / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_kind": f"copy bandwidth, of {peaks_kind}"}
        # the same kind of copy, sustained for half a second in this process right after the timed regions
        copy_now = sustained_copy_gbs(device)
        roof["copy_gbs_sustained_this_run"] = copy_now
        roof["frac_of_copy_sustained_this_run"] = achieved / copy_now
    traffic = NCU_TRAFFIC.get((cfg.name, kernel_name))
    roof["traffic"] = traffic[0] if traffic else None
    roof["traffic_source"] = (f"ncu capture summarised in {traffic[1]}; not measured by this run" if traffic else
                              "no ncu capture of this kernel on this workload")
    roof["kernel"] = kernel_name
    roof["kernel_ms"] = kernel_s * 1e3
    roof["kernel_ms_min"] = min(kernel_ms)
    roof["kernel_ms_max"] = max(kernel_ms)
    roof["kernel_launches_timed"] = n_k
    roof["step_ms_while_instrumented"] = 1e3 * secs_instr / n_k
    roof["algorithmic_bytes"] = algorithmic_bytes(cfg)
    roof["algorithmic_flops"] = algorithmic_flops(cfg)

    res = {"value": value, "unit": UNIT, "ms_per_step": 1e3 * secs_region / args.steps,
           "timing": spread(times, args.steps), "config": config_dict(cfg, info.world_size),
           "clocks": dict(sampler.summary(), remeasured=remeasured),
           "e2e": dict({"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                        "ms_per_step": 1e3 * statistics.median(times_e2e) / args.steps, "steps": args.steps},
                       **{"timing": spread(times_e2e, args.steps)}),
           "gpu_launches": launches // len(times), "gpu_launches_all_repeats": launches, "roofline": roof}
    if with_cpu_baseline:
        res["cpu_baseline"] = cpu_baseline(cfg, wl)
    return res


def apply_tuning(specs):
    """--tune KNOB=VALUE pairs -> library settings; returns what was set, for the record."""
    import paper_2605_15609_b200 as psd
    knobs = {"band_bytes": psd.PSD_TUNE_BAND_BYTES, "pdl": psd.PSD_TUNE_PDL, "tile_order": psd.PSD_TUNE_TILE_ORDER,
             "compact_rows": psd.PSD_TUNE_COMPACT_ROWS}
    done = {}
    for spec in specs:
        name, _, value = spec.partition("=")
        value = int(value)
        if name == "kernel":
            rc = psd.psd_set_confidence_impl(value)
            rc = 0 if rc >= 0 else rc
        elif name in knobs:
            rc = psd.psd_set_tuning(knobs[name], value)
        else:
            raise SystemExit(f"--tune: unknown knob {name!r}")
        if rc != 0:
            raise SystemExit(f"--tune {spec}: {psd.status_string(rc)}")
        done[name] = value
    return done


def run_ours(args, names):
    import torch

    from paper_2605_15609_b200 import replicas

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    info = replicas.rank_info_from_env()
    torch.cuda.set_device(info.local_rank)
    device = torch.device("cuda", info.local_rank)
    replicas.init_process_group(info)
    peaks, peaks_kind = load_peaks()
    tuning = apply_tuning(args.tune)

    results = []
    for i, name in enumerate(names):
        cfg = resolve_config(name, args.blocks)
        results.append(measure_workload(args, cfg, info, device, peaks, peaks_kind, with_cpu_baseline=(i == 0)))
        torch.cuda.empty_cache()
    if not info.is_main:
        return 0
    top = results[0]
    if args.profile_only:
        print(json.dumps(top), flush=True)
        return 0
    line = {"metric": METRIC, "value": top["value"], "unit": UNIT, "n_gpus": info.world_size, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": top["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic"}
    line.update({k: top[k] for k in ("config", "timing", "clocks", "e2e", "gpu_launches", "gpu_launches_all_repeats",
                                     "roofline", "cpu_baseline")})
    for r in results[1:]:
        line[r["config"]["workload"]] = r
    if tuning:
        line["tuning"] = tuning
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------------ whole loop

def run_loop(args, cfg):
    """--loop: Algorithm 1 as a whole (psd_decode_blocks) with the table look-up body standing in for
    the transformer.  Reports time per iteration and the tokens-per-forward-pass of this synthetic
    body (a property of the toy body, printed as context: the paper's figures come from real models)."""
    import ctypes

    import torch

    import paper_2605_15609_b200 as psd
    import psd_inputs as gen

    torch.cuda.set_device(0)
    B, M, D, H, V = cfg.B, cfg.M, cfg.D, cfg.H, cfg.V
    W = gen.weights(cfg)
    table, *_ = gen.table_body(cfg, W)
    dev = torch.device("cuda", 0)
    bf = lambda bits: torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)
    w_dev, t_dev = bf(W), bf(table.reshape(-1, H))
    hidden = torch.zeros(B * D * M, H, dtype=torch.bfloat16, device=dev)
    buf = psd.StepBuffers.allocate(B, M, D, H, hidden, w_dev, dev)
    ws = torch.empty(psd.psd_compact_workspace_bytes(B * D * M, H, V), dtype=torch.uint8, device=dev)
    psd.psd_set_tuning(psd.PSD_TUNE_COMPACT_ROWS, 1 if args.compact else 0)
    scratch = torch.empty(psd.psd_decode_scratch_bytes(B, M), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    passes = torch.zeros(B, dtype=torch.int32, device=dev)
    pg = psd.policy(tau=float(np.float32(cfg.tau)), k_min=cfg.k_min, k_max=cfg.k_max, depth=D, stride=cfg.stride,
                    mask_id=cfg.mask_id)
    user = psd.table_body_user(t_dev.view(B, M, 3, H), B)
    order = psd.ORDER_ONE_PASS if args.loop == "one_pass" else psd.ORDER_TWO_PASSES
    stream = torch.cuda.current_stream()

    def decode():
        buf.tokens.fill_(cfg.mask_id)
        buf.mask.fill_(1)
        return psd.psd_decode_blocks(psd.table_body_address(), ctypes.addressof(user), buf, pg, order, 4 * M, scratch,
                                     ws, status, passes, None, None, stream)

    for _ in range(max(3, min(args.warmup, 5))):
        decode()
    n = max(3, min(args.steps, 50))
    launches0 = psd.psd_launch_count()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    its = fwd = 0
    for _ in range(n):
        st = decode()
        its += st.iterations
        fwd += st.forward_passes
    e1.record(stream)
    torch.cuda.synchronize()
    secs = e0.elapsed_time(e1) * 1e-3
    p = passes.cpu().numpy()
    line = {"metric": "blocks decoded end to end (Algorithm 1 loop, table look-up body)", "value": B * M * n / secs,
            "unit": "tokens/s", "n_gpus": 1, "steps": n, "ms_per_block_batch": 1e3 * secs / n,
            "us_per_iteration": 1e6 * secs / max(its, 1), "iterations_per_decode": its / n,
            "forward_passes_per_decode": fwd / n, "tokens_per_forward_pass_mean": float((M / np.maximum(p, 1)).mean()),
            "order": args.loop, "compact_rows": bool(args.compact), "dtype": "bf16", "data": "synthetic",
            "config": {"workload": cfg.name, "B": B, "D": D, "M": M, "H": H, "V": V},
            "gpu_launches": psd.psd_launch_count() - launches0, "status": int(status.item())}
    print(json.dumps(line), flush=True)
    return 0


DEFAULT_WORKLOADS = ("batched_serving", "single_request")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default=None,
                    help="one workload: tiny, single_request, class_7b, batched_serving, deep_sweep[_D1|_D2|_D4]. "
                         "Default: batched_serving (8192 rows, tensor bound) as the line's own result, with "
                         "single_request (128 rows, HBM bound) measured the same way under the key of that name")
    ap.add_argument("--blocks", type=int, default=0,
                    help="override the workload's number of blocks B (rows = B*D*M), e.g. to sweep row counts "
                         "across the HBM/tensor ridge; the printed config names the override")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="the K-step timed region is repeated until this much device time has passed (at least "
                         "3 times); the line reports the median region and the spread")
    ap.add_argument("--tune", action="append", default=[], metavar="KNOB=VALUE",
                    help="set a performance knob of the library before measuring (band_bytes, pdl, tile_order, "
                         "compact_rows, or kernel for psd_set_confidence_impl); the line records it under \"tuning\"")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--loop", default=None, choices=["one_pass", "two_passes"],
                    help="time the whole decoding loop (psd_decode_blocks) instead of one step; an extra "
                         "measurement, not the headline metric")
    ap.add_argument("--compact", action="store_true",
                    help="with --loop: score only the rows of slots that are still masked")
    ap.add_argument("--profile-only", action="store_true",
                    help="for runs under a profiler: device-resident steps only (no instrumented pass, no "
                         "end-to-end pass, no CPU baseline); the printed line is not a benchmark result")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.profile_only:
        args.min_seconds = 0.0
    names = [args.config] if args.config else list(DEFAULT_WORKLOADS)
    if args.impl == "reference":
        return run_reference(args, names)
    if args.loop:
        return run_loop(args, resolve_config(names[-1], args.blocks))
    return run_ours(args, names)


if __name__ == "__main__":
    sys.exit(main())
