#!/usr/bin/env python
"""Benchmark of the FastMMoE MoE-layer hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload all|C0|C1|C2|C2x4|C3|C4|C1_fp8|C2_fp8|C3_fp8]
                    [--impl reference]

One "step" = one pass of the whole hot path over one batch of synthetic tokens:
router + top-k + gates, permute-by-expert, grouped SwiGLU expert GEMMs + shared
experts, weighted combine, then routing-aware pruning of the layer output with that
layer's routing probabilities (fmmoe_moe_forward_prune); for the 24-layer stack a step
is the whole stack (fmmoe_stack_forward).

The default (`--workload all`) prints ONE JSON line whose top-level fields are the
largest single-layer workload (the batch of four Qwen3-MoE-style sequences, 14,336
tokens) and whose `configs` object holds one record per other workload (C0, C1, C2,
C3, C4, C1-C3 once more with their expert matrices stored as FP8, and the paper's two
three-stage pruning schedules on stacks of the matching layer shape), each with its own
timing, clocks, roofline and end-to-end figure.

Timing: a block is exactly K steps between two CUDA events, with a barrier and a
device synchronisation on both sides.  Whatever K is, blocks are repeated until the
workload has at least `--min-seconds` of timed GPU work; the reported step time is the
MEDIAN block (the best block and the SM clock of every block are given beside it).
`--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import gc
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "MoE-layer prefill tokens/s"
UNIT = "tokens/s"
LAYER_WORKLOADS = ("C0", "C1", "C2", "C2x4", "C3")
# the paper's own three-stage schedules (Appendix A) at 50 % overall retention, attention-guided, on a stack of the
# matching layer shape: name -> (backbone family, overall retention)
PAPER_STACKS = {"S_internvl_50": ("internvl3.5", 0.5), "S_deepseek_50": ("deepseek-vl2", 0.5)}
WORKLOADS = ("all",) + LAYER_WORKLOADS + ("C1_fp8", "C2_fp8", "C3_fp8", "C4") + tuple(PAPER_STACKS)
HEADLINE = "C2x4"
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}   # the nominal peaks the metric names (8 TB/s, dense bf16)

# DRAM bytes (read + written) one launch of a kernel moved under the profiler, per workload.
# Each figure comes from one capture of that kernel on that workload; an entry is removed (null in
# the output) when its kernel changes after the capture.
NCU_TRAFFIC_BYTES = {
    "C2x4": {"gemm1": 1101.6e6, "gemm2": 723.2e6, "route": 60.4e6, "finalize": 296.1e6},   # ffn_tc_kernel<0/1>, route_tc, finalize_pair
    "C1": {"gemm1": 824.8e6, "gemm2": 469.9e6, "finalize": 51.6e6},                         # ffn_tc_kernel<0/1>, finalize_pair
    "C2": {"gemm1": 870.4e6, "gemm2": 477.2e6},                                             # ffn_tc_kernel<0/1>
    "C1_fp8": {"gemm1": 501.7e6, "gemm2": 293.8e6},                                         # ffn_sm_kernel<0/1, 1>
}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "tf_burst": float(d["bf16_tflops"]),
                "tf_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "tf_burst": 1590.0, "tf_sustained": 1400.0, "source": "fallback"}


def workload_cfg(name):
    from paper_2511_17885_b200 import inputs as I
    cfg = I.CONFIGS[name]
    # pruning stage of the step: the workload's own 50%-retention setting (C3/C2: the sweep's middle point)
    prune = None
    for pc in cfg.prune:
        if abs(pc.retain - 0.5) < 1e-9:
            prune = pc
    if prune is None and cfg.prune:
        prune = cfg.prune[0]
    return cfg, prune


def describe(name, cfg, prune):
    return {"workload": f"{name}: {cfg.name}, {cfg.batch} x ({cfg.n_vis} visual + {cfg.n_text} text) tokens, "
                        f"H={cfg.hidden} E={cfg.n_experts} I={cfg.inter} shared={cfg.n_shared} K={cfg.top_k} "
                        f"K_v={cfg.top_k_vis} (reduction on); then pruning to {int(prune.retain * 100)}% "
                        f"(W={prune.window}, gamma={prune.gamma}, attention-free score)",
            "tokens_per_step": cfg.n_tokens,
            "l2": "inputs larger than L2: every step streams the layer's expert weights "
                  f"({weight_bytes(cfg) / 1e6:.0f} MB) from HBM" if weight_bytes(cfg) > 126e6 else
                  f"the layer's weights ({weight_bytes(cfg) / 1e6:.1f} MB) fit in L2: a launch-latency workload, "
                  "timed with the L2 warm"}


def weight_bytes(cfg):
    e = 2 if cfg.dtype == "bf16" else 4
    return (3 * cfg.hidden * cfg.inter * cfg.n_experts + 3 * cfg.hidden * cfg.shared_inter * cfg.n_shared
            + cfg.n_experts * cfg.hidden) * e


# ------------------------------------------------------------------ algorithmic work per launch
def kernel_work(cfg, kernel, P, touched, prune_rows=None, w_elem=None):
    """(bytes, flops) one launch of `kernel` must move / compute for this workload.
    P = routed pairs, touched = experts with at least one row, prune_rows = (rows read, rows written) of the
    compaction pass, w_elem = bytes per stored expert-matrix element (1 for the FP8 weight stream)."""
    e = 2 if cfg.dtype == "bf16" else 4
    we = e if w_elem is None else w_elem
    T, H, E, I_, Ns, Is, K = cfg.n_tokens, cfg.hidden, cfg.n_experts, cfg.inter, cfg.n_shared, cfg.shared_inter, cfg.top_k
    if kernel == "gemm1":
        b = touched * 2 * H * I_ * we + Ns * 2 * H * Is * we + T * H * e + (P * I_ + Ns * T * Is) * e
        f = 4 * H * I_ * P + 4 * H * Is * Ns * T
    elif kernel == "gemm2":
        b = touched * H * I_ * we + Ns * H * Is * we + (P * I_ + Ns * T * Is) * e + T * H * e
        f = 2 * H * I_ * P + 2 * H * Is * Ns * T
    elif kernel == "route":
        b = T * H * e + E * H * e + T * K * 8 + T * E * 4
        f = 2 * T * H * E
    elif kernel == "permute":
        b = T * K * 4 + 3 * P * 4
        f = 0
    elif kernel == "finalize":
        b = T * H * 4 + T * H * e
        f = 0
    elif kernel == "prune_score":
        b = cfg.batch * cfg.n_vis * E * 4
        f = 0
    elif kernel == "prune_compact" and prune_rows is not None:
        b = (prune_rows[0] + prune_rows[1]) * H * e
        f = 0
    else:
        b, f = 0, 0
    return float(b), float(f)


# ------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock, board power and clock-event reasons while the timed region runs (read-only NVML)."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index):
        self.samples, self.times, self.reasons, self.max_mhz, self.ok = [], [], set(), None, False
        self.power_w = []
        self._stop = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM))
            try:
                self.power_limit_w = pynvml.nvmlDeviceGetEnforcedPowerLimit(self.dev) / 1000.0
            except Exception:
                self.power_limit_w = None
            self.ok = True
        except Exception:
            self.ok = False
        self.th = None

    def sample_once(self):
        if not self.ok:
            return
        try:
            mhz = int(self.nv.nvmlDeviceGetClockInfo(self.dev, self.nv.NVML_CLOCK_SM))
            self.samples.append(mhz)
            self.times.append(time.perf_counter())
            try:
                self.power_w.append(self.nv.nvmlDeviceGetPowerUsage(self.dev) / 1000.0)
            except Exception:
                pass
            try:
                r = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.dev))
            except Exception:
                r = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.dev))
            for bit, name in self.REASONS.items():
                if r & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self.sample_once()
            time.sleep(0.002)

    def start(self):
        if self.ok:
            self.th = threading.Thread(target=self._run, daemon=True)
            self.th.start()

    def stop(self):
        self._stop.set()
        if self.th is not None:
            self.th.join(timeout=2)

    def median_between(self, t0, t1):
        v = [m for m, t in zip(self.samples, self.times) if t0 <= t <= t1]
        return float(np.median(v)) if v else None

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w": float(np.median(self.power_w)) if self.power_w else None,
                "power_limit_w": getattr(self, "power_limit_w", None)}


def settle_clocks(step, index, min_s=0.4, max_s=3.0):
    """Untimed load before the timed region, after the W warm-up steps: a GPU that has been idle ramps its SM
    clock over the first tenths of a second of work.  Runs `step` until the SM clock reads >= 95 % of its
    maximum or a power/thermal cap is active (read-only NVML), for at least min_s and at most max_s seconds."""
    import torch
    probe = ClockSampler(index)
    t0 = time.perf_counter()
    while True:
        for _ in range(8):
            step()
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        if dt >= max_s:
            break
        if dt >= min_s:
            if not probe.ok:
                break
            probe.samples.clear(); probe.reasons.clear()
            probe.sample_once()
            if probe.reasons or (probe.samples and probe.samples[-1] >= 0.95 * probe.max_mhz):
                break
    return time.perf_counter() - t0


def timed_blocks(step, K, min_seconds, clocks, D, dev, max_blocks=400):
    """Blocks of exactly K steps, each between two CUDA events on the current stream with a barrier and a
    device synchronisation on both sides; repeated until min_seconds of timed GPU work has accumulated.
    Block times are the MAX over ranks.  Returns per-block seconds and the median SM clock of each block."""
    import torch
    secs, mhz = [], []
    total, n_blocks = 0.0, None
    while True:
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        D.barrier(); torch.cuda.synchronize()
        t0 = time.perf_counter()
        ev0.record()
        for _ in range(K):
            step()
        ev1.record()
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        D.barrier()
        s = D.max_over_ranks(ev0.elapsed_time(ev1) * 1e-3, dev)
        secs.append(s)
        mhz.append(clocks.median_between(t0, t1))
        total += s
        if n_blocks is None:     # every rank runs the same number of blocks: decided from the first (max over ranks) time
            n_blocks = int(min(max_blocks, max(3, math.ceil(min_seconds / max(s, 1e-6)))))
        if len(secs) >= n_blocks:
            break
    return secs, mhz


def block_stats(secs, mhz, K):
    per_step = np.array(secs) / K
    med = float(np.median(per_step))
    m = [x for x in mhz if x is not None]
    med_mhz = float(np.median(m)) if m else None
    return {"blocks": len(secs), "steps_per_block": K, "gpu_seconds_timed": float(np.sum(secs)),
            "ms_per_step_median": med * 1e3, "ms_per_step_best": float(per_step.min()) * 1e3,
            "ms_per_step_p90": float(np.percentile(per_step, 90)) * 1e3,
            "sm_mhz_median_of_blocks": med_mhz,
            "sm_mhz_min_max_of_blocks": [float(min(m)), float(max(m))] if m else None,
            # step time x SM clock: comparable between runs that sat at different power-capped clocks
            "ms_x_mhz": med * 1e3 * med_mhz if med_mhz else None}, med


# ------------------------------------------------------------------ oracle timing
def oracle_sample(name, cfg, prune, frac, fp8=False):
    """Inputs of a bounded sample: the first `frac` of every sequence's visual and text tokens."""
    from paper_2511_17885_b200 import inputs as I
    x, mask, seq_off, n_vis = I.make_tokens(cfg)
    w = I.make_weights(cfg)
    if fp8:      # the values the FP8 bytes and block scales represent
        w, _ = I.weights_to_fp8(w)
    idx = []
    for b in range(cfg.batch):
        lo = int(seq_off[b])
        nv = max(prune.window * 4, int(cfg.n_vis * frac))
        nt = max(1, int(cfg.n_text * frac))
        idx += list(range(lo, lo + min(nv, cfg.n_vis))) + list(range(lo + cfg.n_vis, lo + cfg.n_vis + min(nt, cfg.n_text)))
    idx = np.array(idx)
    xs, ms = x[idx], mask[idx]
    per = len(idx) // cfg.batch
    so = np.arange(cfg.batch + 1, dtype=np.int64) * per
    nvs = np.array([int(ms[so[b]:so[b + 1]].sum()) for b in range(cfg.batch)], np.int64)
    return xs, ms, so, nvs, w


def oracle_step(cfg, prune, xs, ms, so, nvs, w):
    from oracle import fmmoe_oracle as O
    from paper_2511_17885_b200 import inputs as I
    r = O.moe_forward(xs, ms, w, cfg.top_k, cfg.top_k_vis, True)
    O.prune_visual(r["out"], ms, r["probs"], None, so, I.retain_counts(nvs, prune.retain), prune.window,
                   prune.alpha, prune.gamma)


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        nt = [i.get("num_threads", 0) for i in threadpool_info() if i.get("user_api") == "blas"]
        if nt:
            return int(max(nt))
    except Exception:
        pass
    return 1


def time_oracle(name, cfg, prune, frac, steps, warmup, one_thread_frac=None, fp8=False):
    xs, ms, so, nvs, w = oracle_sample(name, cfg, prune, frac, fp8)
    for _ in range(warmup):
        oracle_step(cfg, prune, xs, ms, so, nvs, w)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(cfg, prune, xs, ms, so, nvs, w)
    dt = time.perf_counter() - t0
    threads = blas_threads()
    sample = (f"{xs.shape[0]} of {cfg.n_tokens} tokens of the workload (first {frac:.3g} of each sequence's visual "
              f"and text tokens), route + experts + combine + pruning, fp64 numpy, {steps} pass(es); `cores` = BLAS "
              f"threads used, of {len(os.sched_getaffinity(0))} host cores available")
    one = None
    if one_thread_frac:
        try:
            from threadpoolctl import threadpool_limits
            xs1, ms1, so1, nvs1, _ = oracle_sample(name, cfg, prune, one_thread_frac)
            with threadpool_limits(limits=1):
                t1 = time.perf_counter()
                oracle_step(cfg, prune, xs1, ms1, so1, nvs1, w)
                one = xs1.shape[0] / (time.perf_counter() - t1)
        except Exception:
            one = None
    return xs.shape[0] * steps / dt, dt / max(steps, 1), threads, sample, one


def cpu_baseline_for(name, cfg, prune):
    frac = 1.0 if cfg.n_tokens <= 4096 else 4096.0 / cfg.n_tokens
    v, spp, cores, sample, one = time_oracle(name, cfg, prune, frac, 3, 0, one_thread_frac=frac / 8)
    return {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample, "value_1_thread": one}


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return 0
    name = HEADLINE if args.workload == "all" else args.workload
    fp8 = name.endswith("_fp8")
    name = name[:-4] if fp8 else name
    cfg, prune = workload_cfg(name)
    frac = 1.0 if cfg.n_tokens <= 4096 else 4096.0 / cfg.n_tokens
    value, spp, cores, sample, _ = time_oracle(name, cfg, prune, frac, max(args.steps, 1), min(args.warmup, 1), fp8=fp8)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": spp * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": describe(name, cfg, prune),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------ one layer workload on the GPU
def roofline_of(kernel, b, f, per_launch_s, peaks, traffic):
    t_hbm, t_tc = b / (peaks["hbm_gbs"] * 1e9), f / (peaks["tf_sustained"] * 1e12)
    if t_hbm >= t_tc:
        roof = {"bound": "hbm", "achieved": b / per_launch_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "peak_nominal": NOMINAL["hbm_gbs"]}
    else:
        roof = {"bound": "tensor", "achieved": f / per_launch_s / 1e12, "peak": peaks["tf_sustained"], "unit": "TFLOP/s",
                "peak_nominal": NOMINAL["bf16_tflops"]}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["frac_of_nominal"] = roof["achieved"] / roof["peak_nominal"]
    roof["traffic"] = traffic
    roof.update({"kernel": kernel, "us_per_launch": per_launch_s * 1e6, "algorithmic_bytes": b, "algorithmic_flops": f,
                 "peak_source": peaks["source"] + (" (sustained bf16)" if roof["bound"] == "tensor" else " (copy)"),
                 "tensor_tflops": f / per_launch_s / 1e12, "hbm_gbs": b / per_launch_s / 1e9})
    return roof


def measure_layer(name, args, D, rank, local, world, peaks, with_cpu, fp8=False):
    import torch
    from paper_2511_17885_b200 import binding as B
    from paper_2511_17885_b200.workload import LayerWorkload
    dev = f"cuda:{local}"
    cfg, prune = workload_cfg(name)
    h = B.Handle(local)
    wl = LayerWorkload(cfg, h, device=local, prune=prune, token_seed=D.token_seed_for_rank(cfg.seed, rank),
                       fp8_weights=fp8)
    K, W = max(args.steps, 1), max(args.warmup, 3)
    if args.plain:      # for profilers: warm-up and K steps of the device-resident path, nothing else
        for _ in range(args.warmup + K):
            wl.step()
        torch.cuda.synchronize()
        h.check_status("plain run")
        return {"value": 0.0, "ms_per_step": 0.0, "dtype": cfg.dtype, "config": describe(name, cfg, prune), "plain": True}
    for _ in range(W):
        wl.step()
    settle_s = settle_clocks(wl.step, local)
    h.check_status("warm-up")
    P, touched = wl.routing_stats()

    # ---- device-resident timed blocks (no instrumentation inside)
    clocks = ClockSampler(local)
    clocks.start()
    n0 = h.launch_count()
    secs, mhz = timed_blocks(wl.step, K, args.min_seconds, clocks, D, dev)
    launches = (h.launch_count() - n0) // len(secs)
    h.check_status("timed region")
    stats, step_s = block_stats(secs, mhz, K)
    value = cfg.n_tokens * world / step_s

    # ---- per-kernel durations: the same step with every kernel launch between two CUDA events on the
    # launching stream (the layer and the pruning stage as two calls on one stream, so that a pair brackets
    # one kernel).  Short kernels that can be repeated without changing their result are issued 50 times
    # inside their pair, which amortises the launch latency a pair adds to a 10-30 us kernel.
    h.profile_reset()
    h.profile_enable(50)
    kp = max(3, min(K, 10))
    for _ in range(kp):
        wl.step(fused=False)
    torch.cuda.synchronize()
    h.profile_enable(0)
    prof = h.profile_read()
    h.check_status("instrumented region")

    # ---- end to end: host buffers in, host buffers out.  K independent batches in pinned host memory per
    # block; every one is uploaded, computed and downloaded (layer output and pruned rows) inside the timed
    # block, three in flight (upload of batch i beside the layer of batch i-1 and the downloads of batch i-2).
    for i in range(3):
        wl.step_host_async(i)
    wl.drain_host()
    counter = [0]

    def e2e_block_step():
        wl.step_host_async(counter[0]); counter[0] += 1

    def e2e_block(Kb):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        D.barrier(); torch.cuda.synchronize()
        tw0 = time.perf_counter()
        e0.record()
        for _ in range(Kb):
            e2e_block_step()
        wl.drain_host()                      # host-side wait: every result is in host memory
        e1.record()
        torch.cuda.synchronize()
        tw1 = time.perf_counter()
        D.barrier()
        return D.max_over_ranks(max(e0.elapsed_time(e1) * 1e-3, tw1 - tw0), dev), (tw0, tw1)

    e_secs, e_mhz = [], []
    first, span = e2e_block(K)
    e_secs.append(first); e_mhz.append(clocks.median_between(*span))
    for _ in range(int(min(200, max(2, math.ceil(args.min_seconds / max(first, 1e-6))))) - 1):
        s, span = e2e_block(K)
        e_secs.append(s); e_mhz.append(clocks.median_between(*span))
    e_stats, e_step_s = block_stats(e_secs, e_mhz, K)
    h.check_status("end-to-end region")
    # the same without overlap: one batch at a time, the stream synchronised after every download
    for _ in range(2):
        wl.step_host()
    torch.cuda.synchronize()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ks = max(3, min(K, 20))
    s0.record()
    for _ in range(ks):
        wl.step_host()
    s1.record()
    torch.cuda.synchronize(); D.barrier()
    e2e_serial = cfg.n_tokens * world / (D.max_over_ranks(s0.elapsed_time(s1) * 1e-3, dev) / ks)
    h.check_status("end-to-end region (one batch at a time)")
    clocks.stop()

    # ---- rooflines
    w_elem = 1 if fp8 else None
    t_out = int(wl.last["x_out"].shape[0]) if wl.last is not None else 0
    merged = wl.merged_rows() if wl.last is not None else 0
    prune_rows = (t_out + merged * (prune.window - 1), t_out)
    kernels = {}
    tot_ms = max(sum(v["ms"] for v in prof.values()), 1e-12)
    for k, v in prof.items():
        if not v["launches"]:
            continue
        per_launch_s = v["ms"] * 1e-3 / v["launches"]
        b, f = kernel_work(cfg, k, P, touched, prune_rows, w_elem)
        kernels[k] = {"us_per_launch": per_launch_s * 1e6, "launches_per_step": v["launches"] / kp,
                      "us_per_step": v["ms"] * 1e3 / kp, "share": v["ms"] / tot_ms,
                      "algorithmic_bytes": b, "hbm_gbs": b / per_launch_s / 1e9 if b else None,
                      "frac_of_hbm_peak": b / per_launch_s / 1e9 / peaks["hbm_gbs"] if b else None,
                      "tensor_tflops": f / per_launch_s / 1e12 if f else None}
    dom = max(prof, key=lambda k: prof[k]["ms"])
    per_launch_s = prof[dom]["ms"] * 1e-3 / max(prof[dom]["launches"], 1)
    b, f = kernel_work(cfg, dom, P, touched, prune_rows, w_elem)
    roof = roofline_of(dom, b, f, per_launch_s, peaks, NCU_TRAFFIC_BYTES.get(name, {}).get(dom))
    # whole step against the slower of (activated FLOPs at tensor peak, algorithmic bytes at HBM bandwidth)
    e = 2 if cfg.dtype == "bf16" else 4
    tot_b = sum(kernel_work(cfg, k, P, touched, None, w_elem)[0] for k in ("route", "gemm1", "gemm2")) - 2 * cfg.n_tokens * cfg.hidden * e
    tot_f = sum(kernel_work(cfg, k, P, touched)[1] for k in ("route", "gemm1", "gemm2"))
    t_hbm, t_tc = tot_b / (peaks["hbm_gbs"] * 1e9), tot_f / (peaks["tf_sustained"] * 1e12)
    t_step = max(t_hbm, t_tc)
    t_step_nom = max(tot_b / (NOMINAL["hbm_gbs"] * 1e9), tot_f / (NOMINAL["bf16_tflops"] * 1e12))

    conf = describe(name, cfg, prune)
    if fp8:
        conf["workload"] += ("; expert matrices stored as FP8 E4M3 bytes with one power-of-two scale per 128x128 block "
                             "(activations, accumulation and outputs as in the bf16 layer)")
        conf["l2"] = conf["l2"].replace(f"({weight_bytes(cfg) / 1e6:.0f} MB)", f"({weight_bytes(cfg) / 2e6:.0f} MB as FP8)")
    conf.update({"routed_pairs": P, "experts_touched": touched, "parallelism": f"replicas x{world} (no collective)"})
    rec = {"value": value, "unit": UNIT, "ms_per_step": step_s * 1e3, "timing": stats, "dtype": cfg.dtype,
           "config": conf,
           "clocks": dict(clocks.summary(), settle_s=round(settle_s, 2)),
           "e2e": {"value": cfg.n_tokens * world / e_step_s, "unit": UNIT, "h2d_bytes_per_step": wl.h2d_bytes(),
                   "d2h_bytes_per_step": wl.d2h_bytes(), "batches_in_flight": wl.PIPE_DEPTH, "timing": e_stats,
                   "value_one_batch_at_a_time": e2e_serial},
           "gpu_launches": int(launches * K),
           "roofline": roof,
           "step_roofline": {"frac": t_step / step_s, "frac_of_nominal": t_step_nom / step_s,
                             "bound": "hbm" if t_hbm >= t_tc else "tensor", "t_bound_us": t_step * 1e6,
                             "algorithmic_bytes": tot_b, "activated_flops": tot_f, "peak_source": peaks["source"]},
           "kernels": kernels}
    if with_cpu:
        rec["cpu_baseline"] = cpu_baseline_for(name, cfg, prune)
    del wl
    h.close()
    gc.collect(); torch.cuda.empty_cache()
    return rec


# ------------------------------------------------------------------ the 24-layer stack (C4)
def stack_describe(sc, n_layers, label="C4", attention=False):
    lc = sc.layer
    st = ", ".join(f"after layer {l}: to {pc.retain * 100:.1f}% (W={pc.window}, gamma={pc.gamma}"
                   + (f", alpha={pc.alpha}" if attention else "") + ")"
                   for l, pc in sorted(sc.prune_after.items()))
    score = ("attention-guided score, A_hat of Eq. 7 from fmmoe_attention_importance on stand-in queries / keys inside "
             "the step" if attention else "attention-free score")
    return {"workload": f"{label}: {n_layers} MoE layers of the {lc.name} shape with residual adds (attention layers omitted), "
                        f"{lc.batch} x ({lc.n_vis} visual + {lc.n_text} text) tokens, H={lc.hidden} E={lc.n_experts} "
                        f"I={lc.inter} shared={lc.n_shared} K={lc.top_k}, K_v={lc.top_k_vis} from layer {sc.reduce_from}; "
                        f"pruning {st}; {score}",
            "tokens_per_step": lc.n_tokens,
            "l2": f"inputs larger than L2: {n_layers} x {weight_bytes(lc) / 1e6:.0f} MB of distinct layer weights"}


def stack_flops(lc, shapes):
    """Activated MoE FLOPs of the stack (router + routed pairs + shared experts), per kernel class."""
    H, E, I_, Ns, Is = lc.hidden, lc.n_experts, lc.inter, lc.n_shared, lc.shared_inter
    g1 = sum(4 * H * I_ * P + 4 * H * Is * Ns * T for T, P in shapes)
    g2 = sum(2 * H * I_ * P + 2 * H * Is * Ns * T for T, P in shapes)
    rt = sum(2 * T * H * E for T, P in shapes)
    return float(g1), float(g2), float(rt)


def oracle_stack_sample(sc, n_layers_sample=2, n_tok=512):
    """Bounded CPU sample for the stack: the first n_tok tokens of sequence 0 through the first layers."""
    from paper_2511_17885_b200 import inputs as I
    from oracle import fmmoe_oracle as O
    lc = sc.layer
    x, mask, seq_off, n_vis = I.make_tokens(lc)
    idx = np.concatenate([np.arange(n_tok - 32), np.arange(lc.n_vis, lc.n_vis + 32)])
    xs, ms = x[idx].astype(np.float64), mask[idx]
    ws = []
    for l in range(n_layers_sample):
        w = I.stack_layer_weights_torch(sc, l, "cpu")
        ws.append({k: (None if v is None else v.float().numpy()) for k, v in w.items()})
    t0 = time.perf_counter()
    for l in range(n_layers_sample):
        r = O.moe_forward(xs, ms, ws[l], lc.top_k, lc.top_k_vis, l >= sc.reduce_from, add_residual=True)
        xs = r["out"]
    dt = time.perf_counter() - t0
    return len(idx), n_layers_sample, dt


def stack_cpu_baseline(sc, n_layers):
    n_tok, nl, dt = oracle_stack_sample(sc)
    # tokens/s through the whole stack, extrapolated from nl layers to n_layers
    value = n_tok / (dt * n_layers / nl)
    sample = (f"{n_tok} tokens of sequence 0 through the first {nl} of {n_layers} layers (router, experts, combine, "
              f"residual; fp64 numpy; no pruning stage falls in these layers), time scaled by {n_layers}/{nl}; "
              f"`cores` = BLAS threads used, of {len(os.sched_getaffinity(0))} host cores available")
    return {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample}


def measure_stack(args, D, rank, local, world, peaks, with_cpu, sc=None, label="C4", attention=False):
    import torch
    from paper_2511_17885_b200 import binding as B
    from paper_2511_17885_b200 import inputs as I
    from paper_2511_17885_b200.workload import StackWorkload
    dev = f"cuda:{local}"
    paper = sc is not None
    sc = I.C4 if sc is None else sc
    n_layers = sc.n_layers if paper else (args.layers or sc.n_layers)
    h = B.Handle(local)
    wl = StackWorkload(sc, h, device=local, token_seed=D.token_seed_for_rank(sc.layer.seed, rank), n_layers=n_layers,
                       attention=attention)
    K, W = max(1, min(args.steps, 10)), max(args.warmup, 3)      # a stack step is 24 layers: at most 10 per block
    if args.plain:      # for profilers
        for _ in range(args.warmup + K):
            wl.step()
        torch.cuda.synchronize()
        h.check_status("plain run")
        return {"value": 0.0, "ms_per_step": 0.0, "dtype": sc.layer.dtype, "config": stack_describe(sc, n_layers, label, attention), "plain": True}
    for _ in range(min(W, 5)):
        wl.step()
    settle_s = settle_clocks(wl.step, local, min_s=0.2)
    h.check_status("warm-up")
    if not bool(torch.isfinite(wl.x_out.float()).all()):
        raise SystemExit("bench.py: the stack's output is not finite")
    out_std = float(wl.x_out.float().std())
    clocks = ClockSampler(local)
    clocks.start()
    n0 = h.launch_count()
    secs, mhz = timed_blocks(wl.step, K, args.min_seconds, clocks, D, dev)
    launches = (h.launch_count() - n0) // len(secs)
    h.check_status("timed region")
    stats, step_s = block_stats(secs, mhz, K)
    value = wl.n_tokens * world / step_s
    # instrumented pass
    h.profile_reset(); h.profile_enable(1)
    kp = 2
    for _ in range(kp):
        wl.step()
    torch.cuda.synchronize()
    h.profile_enable(0)
    prof = h.profile_read()
    # end to end: independent batches from pinned host memory, two in flight; then one batch at a time
    for i in range(2):
        wl.step_host_async(i)
    wl.drain_host()
    ke = max(4, K)
    D.barrier(); torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.perf_counter()
    e0.record()
    n_e2e = 0
    while True:
        for i in range(ke):
            wl.step_host_async(n_e2e + i)
        n_e2e += ke
        if (time.perf_counter() - t_wall0) >= args.min_seconds or n_e2e >= 400:
            break
    wl.drain_host()
    e1.record()
    torch.cuda.synchronize(); D.barrier()
    e2e_secs = D.max_over_ranks(max(e0.elapsed_time(e1) * 1e-3, time.perf_counter() - t_wall0), dev)
    e2e_value = wl.n_tokens * world * n_e2e / e2e_secs
    h.check_status("end-to-end region")
    wl.step_host()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record()
    for _ in range(4):
        wl.step_host()
    s1.record()
    torch.cuda.synchronize(); D.barrier()
    e2e_serial = wl.n_tokens * world / (D.max_over_ranks(s0.elapsed_time(s1) * 1e-3, dev) / 4)
    h.check_status("end-to-end region (one batch at a time)")
    clocks.stop()

    shapes = wl.layer_shapes()
    g1, g2, rt = stack_flops(sc.layer, shapes)
    dom = max(prof, key=lambda k: prof[k]["ms"])
    per_launch_s = prof[dom]["ms"] * 1e-3 / max(prof[dom]["launches"], 1)
    flops_per_launch = {"gemm1": g1, "gemm2": g2, "route": rt}.get(dom, 0.0) / n_layers
    # bytes per launch of the dominant kernel, mean over the layers (every expert counted as touched)
    lc = sc.layer
    e = 2
    H, E, I_, Ns, Is = lc.hidden, lc.n_experts, lc.inter, lc.n_shared, lc.shared_inter
    if dom == "gemm1":
        bytes_per_launch = sum(E * 2 * H * I_ * e + Ns * 2 * H * Is * e + T * H * e + (P * I_ + Ns * T * Is) * e for T, P in shapes) / n_layers
    elif dom == "gemm2":
        bytes_per_launch = sum(E * H * I_ * e + Ns * H * Is * e + (P * I_ + Ns * T * Is) * e + T * H * e for T, P in shapes) / n_layers
    else:
        bytes_per_launch = 0.0
    roof = roofline_of(dom, bytes_per_launch, flops_per_launch, per_launch_s, peaks, NCU_TRAFFIC_BYTES.get(label, {}).get(dom))
    roof["note"] = "per-launch figures are the mean over the stack's layers (their token counts differ)"
    t_bound = max((g1 + g2 + rt) / (peaks["tf_sustained"] * 1e12), n_layers * weight_bytes(sc.layer) / (peaks["hbm_gbs"] * 1e9))
    t_bound_nom = max((g1 + g2 + rt) / (NOMINAL["bf16_tflops"] * 1e12), n_layers * weight_bytes(sc.layer) / (NOMINAL["hbm_gbs"] * 1e9))
    tot_ms = max(sum(x["ms"] for x in prof.values()), 1e-12)
    kernels = {k: {"us_per_step": v["ms"] * 1e3 / kp, "launches_per_step": v["launches"] / kp, "share": v["ms"] / tot_ms}
               for k, v in prof.items() if v["launches"]}

    # the unreduced, unpruned comparison run (K experts for every token, all tokens in every layer)
    dense = None
    if not args.no_dense and not paper:
        del wl.x_out
        wd = StackWorkload.__new__(StackWorkload)
        wd.__dict__.update(wl.__dict__)
        wd.dense, wd.reduce_from, wd.stages = True, n_layers + 1, []
        wd.out_off, wd.out_vis = B.fmmoe_stack_output_layout([], n_layers, wl.seq_off, wl.n_vis)
        wd.x_out = torch.empty((wd.out_off[-1], sc.layer.hidden), dtype=wl.x.dtype, device=dev)
        wd.mask_out = torch.empty(wd.out_off[-1], dtype=torch.uint8, device=dev)
        for _ in range(2):
            wd.step()
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        d0.record()
        nd = 5
        for _ in range(nd):
            wd.step()
        d1.record()
        torch.cuda.synchronize()
        dg1, dg2, drt = stack_flops(sc.layer, wd.layer_shapes())
        dense = {"ms_per_step": d0.elapsed_time(d1) / nd, "moe_flops": dg1 + dg2 + drt,
                 "activated_flops_saved": 1.0 - (g1 + g2 + rt) / (dg1 + dg2 + drt),
                 "time_saved": 1.0 - step_s * 1e3 / (d0.elapsed_time(d1) / nd)}
        h.check_status("dense-k run")
        del wd

    conf = stack_describe(sc, n_layers, label, attention)
    conf.update({"parallelism": f"replicas x{world} (no collective)", "tokens_per_layer": [t for t, _ in shapes],
                 "final_tokens": wl.out_off[-1], "output_std": out_std,
                 "weights": "N(0, 0.02^2); down-projections N(0, (0.02/sqrt(2*layers))^2) so that the norm-free "
                            "residual stack stays at unit scale"})
    rec = {"value": value, "unit": UNIT, "ms_per_step": step_s * 1e3, "timing": stats, "dtype": sc.layer.dtype,
           "config": conf, "clocks": dict(clocks.summary(), settle_s=round(settle_s, 2)),
           "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": wl.h2d_bytes(),
                   "d2h_bytes_per_step": wl.d2h_bytes(), "batches_in_flight": wl.PIPE_DEPTH, "batches_timed": n_e2e,
                   "value_one_batch_at_a_time": e2e_serial},
           "gpu_launches": int(launches * K), "roofline": roof,
           "step_roofline": {"frac": t_bound / step_s, "frac_of_nominal": t_bound_nom / step_s,
                             "bound": "tensor" if (g1 + g2 + rt) / (peaks["tf_sustained"] * 1e12) >= n_layers * weight_bytes(sc.layer) / (peaks["hbm_gbs"] * 1e9) else "hbm",
                             "t_bound_us": t_bound * 1e6, "activated_flops": g1 + g2 + rt, "peak_source": peaks["source"]},
           "kernels": kernels, "dense_k_unpruned": dense}
    if with_cpu:
        rec["cpu_baseline"] = stack_cpu_baseline(sc, n_layers)
    del wl
    h.close()
    gc.collect(); torch.cuda.empty_cache()
    return rec


def run_stack_reference(args):
    if int(os.environ.get("RANK", 0)) != 0:
        return 0
    from paper_2511_17885_b200 import inputs as I
    paper = args.workload in PAPER_STACKS
    sc = I.paper_stack(*PAPER_STACKS[args.workload]) if paper else I.C4
    n_layers = sc.n_layers if paper else (args.layers or sc.n_layers)
    cb = stack_cpu_baseline(sc, n_layers)
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sc.layer.n_tokens / cb["value"] * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": stack_describe(sc, n_layers, args.workload, paper), "cpu_baseline": cb,
            "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------ the CUDA arm
def run_ours(args):
    import torch
    from paper_2511_17885_b200 import dist as D
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no CPU fallback")
    rank, local, world = D.init("nccl") if int(os.environ.get("WORLD_SIZE", 1)) > 1 else (0, 0, 1)
    torch.cuda.set_device(local)
    peaks = load_peaks()
    head = HEADLINE if args.workload == "all" else args.workload
    others = [w for w in ("C0", "C1", "C2", "C3", "C4") if w != head] if args.workload == "all" else []
    with_cpu = rank == 0 and world == 1 and not args.no_cpu_baseline and not args.plain

    def measure(name, cpu):
        if name == "C4":
            return measure_stack(args, D, rank, local, world, peaks, cpu)
        if name in PAPER_STACKS:
            from paper_2511_17885_b200 import inputs as I
            model, retain = PAPER_STACKS[name]
            return measure_stack(args, D, rank, local, world, peaks, False, sc=I.paper_stack(model, retain), label=name,
                                 attention=True)
        if name.endswith("_fp8"):
            return measure_layer(name[:-4], args, D, rank, local, world, peaks, cpu, fp8=True)
        return measure_layer(name, args, D, rank, local, world, peaks, cpu)

    rec = measure(head, with_cpu)
    configs = {}
    if args.workload == "all":     # the weight-stream-bound workloads once more with FP8 expert weights
        others = others[:-1] + ["C1_fp8", "C2_fp8", "C3_fp8"] + others[-1:] + list(PAPER_STACKS)
    for name in others:
        configs[name] = measure(name, False)
    if rank == 0:
        line = {"metric": METRIC, "value": rec["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": rec["ms_per_step"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": rec["dtype"], "data": "synthetic"}
        for k, v in rec.items():
            if k not in line:
                line[k] = v
        line.setdefault("cpu_baseline", None)
        if configs:
            line["configs"] = configs
        print(json.dumps(line))
    D.shutdown()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all", choices=WORKLOADS)
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="timed GPU work per workload and per region: blocks of --steps steps are repeated until it is reached")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--plain", action="store_true",
                    help="run --warmup + --steps steps of the device-resident path and exit (what a profiler is pointed at)")
    ap.add_argument("--layers", type=int, default=0, help="C4 only: run the first N layers of the stack")
    ap.add_argument("--no-dense", action="store_true", help="C4 only: skip the unreduced, unpruned comparison run")
    args = ap.parse_args()
    if args.impl == "reference":
        sys.exit(run_stack_reference(args) if (args.workload == "C4" or args.workload in PAPER_STACKS) else run_reference(args))
    sys.exit(run_ours(args))


if __name__ == "__main__":
    main()
