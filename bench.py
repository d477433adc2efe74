#!/usr/bin/env python
"""Benchmark of hard-routed FFF inference (FORWARD_I) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config NAME] [--leg NAME]

One step = one pass of the whole path (tree descent, leaf bucketing, grouped leaf evaluation with
un-permuting write-back) over one batch of synthetic tokens.  Prints ONE JSON line (rank 0).

  value      tokens/s with inputs resident in HBM: CUDA events around a region of exactly K steps, max over
             ranks; the region is repeated back to back (R times, at least 0.25 s in all) and the median
             region is the headline, the fastest one is reported beside it
  e2e        tokens/s through fff_forward_infer_host: pinned host x -> device, forward, y and leaf_idx -> host
  roofline   dominant kernel: algorithmic bytes per launch / mean launch time (events recorded by the library
             on the launching stream inside the timed region) against the measured HBM copy bandwidth
  path_roofline  whole path: max(FLOPs / tensor peak, algorithmic bytes / HBM bandwidth) / time per step
  cpu_baseline   the float64 CPU oracle timed on this machine's cores (rank 0, N = 1 only)

With N > 1 (torchrun) every rank runs the same workload on its own GPU: tokens are independent, weights
are replicated, there is no collective on the data path ("weak" scaling of replicas).

--impl reference times the CPU oracle instead (there is no other implementation of the paper here).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2308_14711_b200 import replicas, workloads as wl  # noqa: E402

DEFAULT_CONFIG = "vit_d8_l12_bf16"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
L2_BYTES_NOMINAL = 126 * 1024 * 1024      # used only when the device attribute cannot be read
MIN_TIMED_SECONDS = 0.25                  # the K-step region is repeated until the timed span is at least this long
METRIC = "FFF hard-inference tokens/sec"
UNIT = "tokens/s"


# ------------------------------------------------------------------------------------------- peaks
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    except Exception:
        return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
                "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, torch_device_index: int, period_s: float = 0.02):
        self.samples, self.period, self._stop, self._thr, self.h = [], period_s, threading.Event(), None, None
        self.sm_max = None
        try:
            import pynvml
            import torch
            self.nv = pynvml
            pynvml.nvmlInit()
            try:
                uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode() if not uuid.startswith("GPU-")
                                                          else uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(torch_device_index)
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.h = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                self.samples.append((time.perf_counter(), mhz, mask))
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.h is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self, t0=None, t1=None) -> dict:
        if self._thr is not None:
            self._stop.set()
            self._thr.join()
        inside = [s for s in self.samples if t0 is None or t0 <= s[0] <= t1]
        note = None
        if not inside:
            inside, note = self.samples, "no sample fell inside the timed region; all samples of the run used"
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": [], "note": "NVML unavailable"}
        mask = 0
        for s in inside:
            mask |= s[2]
        out = {"sm_mhz": statistics.median(s[1] for s in inside), "sm_max_mhz": self.sm_max,
               "reasons": sorted(n for b, n in self.REASONS.items() if mask & b), "samples": len(inside)}
        if note:
            out["note"] = note
        return out


def csrc_digest() -> str:
    """sha256 over the CUDA sources: ncu counters are only quoted for the kernels they were taken from."""
    import hashlib
    h = hashlib.sha256()
    base = os.path.join(ROOT, "paper_2308_14711_b200", "csrc")
    for d, _, files in sorted(os.walk(base)):
        for f in sorted(files):
            with open(os.path.join(d, f), "rb") as fh:
                h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(kernel: str, workload: str):
    """dram read + write bytes per launch from the committed ncu capture, or None if the kernels changed since."""
    try:
        with open(os.path.join(ROOT, "profiles", "ncu_traffic.json")) as f:
            rec = json.load(f)
        if rec.get("csrc_digest") != csrc_digest():
            return None, "kernel sources changed since the ncu capture in profiles/"
        v = rec["kernels"].get(f"{kernel}@{workload}")
        return (v, rec.get("note")) if v is not None else (None, "no ncu capture of this kernel on this workload")
    except Exception:
        return None, "no ncu capture committed"


# ------------------------------------------------------------------------------------------- byte / flop model
def path_flops(cfg: wl.FFFConfig, B: int) -> float:
    return 2.0 * B * (cfg.depth * cfg.D + cfg.leaf_width * cfg.D + cfg.leaf_width * cfg.O)


def leaf_param_bytes(cfg: wl.FFFConfig) -> int:
    l, D, O, e = cfg.leaf_width, cfg.D, cfg.O, cfg.elem_bytes
    return (l * D + l + O * l + O) * e


def path_bytes(cfg: wl.FFFConfig, B: int, leaves_touched: int) -> float:
    """x in + y out + all node weights and biases + parameters of the distinct leaves touched + leaf_idx out."""
    e = cfg.elem_bytes
    return B * (cfg.D + cfg.O) * e + cfg.n_nodes * (cfg.D + 1) * e + leaves_touched * leaf_param_bytes(cfg) + 4 * B


def kernel_bytes(name: str, cfg: wl.FFFConfig, B: int, leaves_touched: int) -> float:
    """Algorithmic bytes one launch of the named kernel must move."""
    e = cfg.elem_bytes
    if name.startswith("fused_forward"):                       # the whole path in one launch
        return path_bytes(cfg, B, leaves_touched)
    if name.startswith("tree_descent"):
        return B * cfg.D * e + cfg.n_nodes * (cfg.D + 1) * e + 4 * B
    if name.startswith("leaf_bucketing+grouped_leaf_ff"):      # bucketing done by the leaf kernel's prologue
        return 8 * B + 8 * cfg.n_leaves + kernel_bytes("grouped_leaf_ff", cfg, B, leaves_touched)
    if name.startswith("leaf_bucketing") or name.startswith("leaf_histogram"):
        return 8 * B + 8 * cfg.n_leaves
    if name.startswith("grouped_leaf_ff") or name.startswith("descent_tail+leaf_ff"):   # the tail's node rows: O(B) more
        return B * (cfg.D + cfg.O) * e + leaves_touched * leaf_param_bytes(cfg) + 8 * B
    return 0.0


# ------------------------------------------------------------------------------------------- our arm
def make_device_case(cfg: wl.FFFConfig, seed: int, n_sets: int):
    import torch
    from paper_2308_14711_b200.binding import FFFLayer
    td = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    w = wl.make_weights(cfg, seed)
    dev = {k: torch.from_numpy(v).to(td).cuda() for k, v in w.items()}
    if cfg.depth == 0:
        dev["node_w"] = dev["node_b"] = None
    layer = FFFLayer(cfg.D, cfg.O, cfg.depth, cfg.leaf_width, cfg.activation, cfg.dtype, **dev)
    layer.reserve(cfg.B)
    del dev
    xs_host = [wl.TokenSource(cfg, seed + i).x for i in range(n_sets)]
    xs = [torch.from_numpy(a).to(td).cuda() for a in xs_host]
    ys = [torch.empty((cfg.B, cfg.O), dtype=td, device="cuda") for _ in range(n_sets)]
    ls = [torch.empty((cfg.B,), dtype=torch.int32, device="cuda") for _ in range(n_sets)]
    return layer, w, xs_host, xs, ys, ls, td


def l2_bytes() -> int:
    try:
        import torch
        return int(torch.cuda.get_device_properties(torch.cuda.current_device()).L2_cache_size)
    except Exception:
        return L2_BYTES_NOMINAL


def n_buffer_sets(cfg: wl.FFFConfig) -> int:
    per_set = cfg.B * (cfg.D + cfg.O) * cfg.elem_bytes
    return max(2, min(64, int(np.ceil(2.5 * l2_bytes() / per_set))))


def time_device(layer, xs, ys, ls, steps: int, warmup: int, profile: bool, min_seconds: float = 0.0):
    """Regions of exactly `steps` forwards on resident inputs, rotating buffer sets, each between two CUDA
    events on the launching stream; repeated back to back until the span lasts min_seconds.
    Returns (list of ms per region, launches of one region, profile, t0, t1)."""
    import torch
    n = len(xs)
    for i in range(warmup):
        layer.forward_infer(xs[i % n], ys[i % n], ls[i % n])
    torch.cuda.synchronize()
    if profile:
        layer.profile_begin(steps)
    regions, launches = [], 0
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    while True:
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches = 0
        start.record()
        for i in range(steps):
            layer.forward_infer(xs[i % n], ys[i % n], ls[i % n])
            launches += layer.last_launch_count()
        stop.record()
        regions.append((start, stop))
        if profile or len(regions) >= 4096 or time.perf_counter() - t0 >= min_seconds:
            break
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    prof = layer.profile_end() if profile else None
    return [a.elapsed_time(b) for a, b in regions], launches, prof, t0, t1


def dominant_kernel_roofline(prof, cfg, B, leaves_touched, peaks, steps, ms_prof):
    """The roofline object of the launch that takes longest, from the per-launch events of a profiled pass."""
    kernels, prof_steps = prof
    if not kernels:
        return None
    name, kms = max(kernels, key=lambda kv: kv[1])
    kb = kernel_bytes(name, cfg, B, leaves_touched)
    achieved = kb / (kms * 1e-3) / 1e9
    traffic, traffic_note = ncu_traffic(name, cfg.name)
    return {"bound": "hbm", "kernel": name, "achieved": round(achieved, 1), "peak": peaks["hbm_gbs"],
            "unit": "GB/s", "frac": round(achieved / peaks["hbm_gbs"], 4), "traffic": traffic,
            "peak_source": peaks["source"], "kernel_ms": round(kms, 5), "algorithmic_bytes": int(kb),
            "launches_ms": {f"{i}:{n}": round(m, 5) for i, (n, m) in enumerate(kernels)},
            "profiled_steps": prof_steps, "profiled_ms_per_step": round(ms_prof / steps, 5),
            "traffic_note": traffic_note}


def run_ours(args, rank: int, world: int, local_rank: int):
    import torch
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(v: float) -> float:
        return replicas.max_over_ranks(v, dist, "cuda")

    peaks = measured_peaks()
    cfg = wl.CONFIGS[args.config]
    B = cfg.B
    n_sets = n_buffer_sets(cfg)
    layer, w_host, xs_host, xs, ys, ls, td = make_device_case(cfg, seed=rank * 1000, n_sets=n_sets)

    sampler = ClockSampler(local_rank)
    sampler.start()
    barrier()
    region_ms, launches, _, t0, t1 = time_device(layer, xs, ys, ls, args.steps, args.warmup, profile=False,
                                                 min_seconds=MIN_TIMED_SECONDS)
    barrier()
    clocks = sampler.stop(t0, t1)
    # every rank ran its own number of regions; the median region of each rank, then the max over ranks
    ms = max_over_ranks(statistics.median(region_ms))
    ms_min = max_over_ranks(min(region_ms))
    # the same K steps once more with one CUDA event after every launch (recorded by the library on the
    # launching stream): per-kernel durations for the roofline.  Kept out of the headline region because
    # the extra events lengthen the gaps between these short kernels.
    prof_ms, _, prof, _, _ = time_device(layer, xs, ys, ls, args.steps, 3, profile=True)
    status = layer.last_status()
    ms_per_step = ms / args.steps
    value = replicas.whole_job_throughput(B, args.steps, world, ms)

    leaves_touched = int(torch.unique(ls[0]).numel())
    roofline = dominant_kernel_roofline(prof, cfg, B, leaves_touched, peaks, args.steps, prof_ms[0])
    pb, pf = path_bytes(cfg, B, leaves_touched), path_flops(cfg, B)
    t_roof_ms = max(pf / (peaks["bf16_tflops"] * 1e12), pb / (peaks["hbm_gbs"] * 1e9)) * 1e3
    path_roofline = {"bound": "hbm" if pb / (peaks["hbm_gbs"] * 1e9) >= pf / (peaks["bf16_tflops"] * 1e12) else "tensor",
                     "flops": pf, "algorithmic_bytes": int(pb), "leaves_touched": leaves_touched,
                     "roofline_ms": round(t_roof_ms, 5), "frac": round(t_roof_ms / ms_per_step, 4),
                     "frac_at_8TBs": round(max(pf / 2.25e15, pb / 8e12) * 1e3 / ms_per_step, 4)}

    # end to end: host buffers in, host buffers out, through the C ABI
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    xh = [torch.from_numpy(a).to(td).pin_memory() for a in xs_host[:2]]
    yh = torch.empty((B, cfg.O), dtype=td).pin_memory()
    lh = torch.empty((B,), dtype=torch.int32).pin_memory()
    for i in range(3):
        layer.forward_infer_host(xh[i % 2], yh, lh)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(e2e_steps):
        layer.forward_infer_host(xh[i % 2], yh, lh)
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1))
    e2e = {"value": world * B * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "steps": e2e_steps,
           "ms_per_step": round(e2e_ms / e2e_steps, 5),
           "h2d_bytes_per_step": B * cfg.D * cfg.elem_bytes, "d2h_bytes_per_step": B * cfg.O * cfg.elem_bytes + 4 * B}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": ms_per_step, "ms_per_step_min": ms_min / args.steps, "timed_regions": len(region_ms),
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": cfg.dtype, "data": "synthetic",
           "config": {"workload": cfg.name, "D": cfg.D, "O": cfg.O, "depth": cfg.depth, "leaf_width": cfg.leaf_width,
                      "activation": cfg.activation, "tokens_per_step_per_gpu": B, "x": cfg.x_kind,
                      "margin_resampling": False,
                      "l2": f"inputs larger than L2: {n_sets} rotating x/y buffer sets of "
                            f"{B * (cfg.D + cfg.O) * cfg.elem_bytes / 1e6:.0f} MB",
                      "parallelism": "replicas only" if world > 1 else "single GPU"},
           "path_roofline": path_roofline, "roofline": roofline,
           "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "device_status": status}

    if rank == 0 and world == 1:
        if not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(cfg, w_host, xs_host[0], budget_s=args.cpu_budget)
            # the oracle's own count of distinct leaves reached by buffer set 0 (the GPU's count sizes path_roofline)
            path_roofline["leaves_touched_oracle"] = out["cpu_baseline"].pop("leaves_touched")
        if not args.no_per_config:
            out["per_config"] = per_config_table(args, peaks, skip={cfg.name: (ms_per_step, path_roofline)})
            # four layers of the ViT-shaped configuration as one stack (the paper's transformer use of the layer)
            out["stack"] = stack_bench(wl.CONFIGS["vit_d8_l12_bf16"], 4, max(5, min(args.steps, 50)))
            out["forward_train"] = train_bench(wl.CONFIGS["vit_d8_l12_bf16"], max(3, min(args.steps, 10)), peaks)
            out["w8"] = w8_bench(wl.CONFIGS["wide_d11_l32_bf16"], max(5, min(args.steps, 50)), peaks)
    layer.close()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out), flush=True)


def per_config_table(args, peaks, skip):
    """Resident-input throughput and whole-path roofline fraction of all five configurations."""
    import torch
    rows = {}
    for name in wl.CONFIG_ORDER:
        cfg = wl.CONFIGS[name]
        if name in skip:
            ms_step, pr = skip[name]
        else:
            n_sets = n_buffer_sets(cfg)
            layer, _, _, xs, ys, ls, _ = make_device_case(cfg, seed=0, n_sets=n_sets)
            steps = max(5, min(args.steps, 200))
            region_ms, _, _, _, _ = time_device(layer, xs, ys, ls, steps, max(3, min(args.warmup, 10)), profile=False,
                                                min_seconds=MIN_TIMED_SECONDS / 2)
            ms_step = statistics.median(region_ms) / steps
            touched = int(torch.unique(ls[0]).numel())
            pb, pf = path_bytes(cfg, cfg.B, touched), path_flops(cfg, cfg.B)
            t_roof = max(pf / (peaks["bf16_tflops"] * 1e12), pb / (peaks["hbm_gbs"] * 1e9)) * 1e3
            pr = {"algorithmic_bytes": int(pb), "leaves_touched": touched, "roofline_ms": round(t_roof, 5),
                  "frac": round(t_roof / ms_step, 4),
                  "frac_at_8TBs": round(max(pf / 2.25e15, pb / 8e12) * 1e3 / ms_step, 4)}
            # the per-launch split and the dominant kernel's roofline, as for the headline workload
            psteps = min(steps, 50)
            prof_ms, _, prof, _, _ = time_device(layer, xs, ys, ls, psteps, 3, profile=True)
            pr["roofline"] = dominant_kernel_roofline(prof, cfg, cfg.B, touched, peaks, psteps, prof_ms[0])
            layer.close()
            del layer, xs, ys, ls
            torch.cuda.empty_cache()
        rows[name] = {"tokens_per_s": cfg.B / (ms_step * 1e-3), "ms_per_step": round(ms_step, 5),
                      "roofline_frac": pr["frac"], "roofline_frac_at_8TBs": pr["frac_at_8TBs"],
                      "leaves_touched": pr["leaves_touched"], "algorithmic_bytes": pr["algorithmic_bytes"]}
        if pr.get("roofline"):
            rows[name]["roofline"] = pr["roofline"]
    return rows


def stack_bench(cfg: wl.FFFConfig, n_layers: int, steps: int) -> dict:
    """n_layers layers of one configuration as a stack (layer normalisation + residual connections between them),
    as plain launches and as a recorded CUDA graph: time per stack forward on resident inputs."""
    import torch
    from paper_2308_14711_b200.binding import FFFLayer, FFFStack
    td = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    layers = []
    for k in range(n_layers):
        w = wl.make_weights(cfg, 100 + k)
        dev = {n: torch.from_numpy(v).to(td).cuda() for n, v in w.items()}
        layers.append(FFFLayer(cfg.D, cfg.O, cfg.depth, cfg.leaf_width, cfg.activation, cfg.dtype, **dev))
        del dev
    stack = FFFStack(layers, layer_norm=True, residual=True)
    n_sets = n_buffer_sets(cfg)
    xs = [torch.from_numpy(wl.TokenSource(cfg, 200 + i).x).to(td).cuda() for i in range(n_sets)]
    ys = [torch.empty_like(x) for x in xs]
    side = torch.cuda.Stream()
    out = {"layers": n_layers, "workload": cfg.name, "tokens": cfg.B}
    for mode in ("plain", "graph"):
        stack.set_graph(mode == "graph")
        with torch.cuda.stream(side):
            for _ in range(3):                      # warm-up; with the graph on, the second call of a set records it
                for i in range(1 if mode == "graph" else n_sets):
                    stack.forward(xs[i], ys[i], want_leaf_idx=False, stream=side)
            side.synchronize()
            regions = []
            t_begin = time.perf_counter()
            while True:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(side)
                for i in range(steps):
                    # (the recording is tied to one set of addresses: the graph arm re-runs set 0, whose 155 MB
                    # per layer pair still exceed L2 together with the buffers between the layers)
                    j = 0 if mode == "graph" else i % n_sets
                    stack.forward(xs[j], ys[j], want_leaf_idx=False, stream=side)
                e1.record(side)
                regions.append((e0, e1))
                if time.perf_counter() - t_begin >= MIN_TIMED_SECONDS / 2 or len(regions) >= 256:
                    break
            side.synchronize()
        ms = statistics.median(a.elapsed_time(b) for a, b in regions) / steps
        out[f"ms_per_forward_{mode}"] = round(ms, 5)
        if mode == "graph":
            out["replayed"] = bool(stack.last_was_replay())
        else:
            out["launches_per_forward"] = stack.last_launch_count()
    out["tokens_per_s"] = cfg.B / (min(out["ms_per_forward_plain"], out["ms_per_forward_graph"]) * 1e-3)
    stack.close()
    for l in layers:
        l.close()
    return out


def w8_bench(cfg: wl.FFFConfig, steps: int, peaks) -> dict:
    """The hard forward of one configuration with its leaf weights stored as 8-bit floats (fff_create_w8): time per
    step on resident inputs, and the algorithmic bytes with the leaf weights at one byte each."""
    import torch
    from paper_2308_14711_b200.binding import FFFLayer
    w = wl.make_weights(cfg, 0)
    c1, s1, _ = wl.quantize_e4m3(w["w1"])
    c2, s2, _ = wl.quantize_e4m3(w["w2"])

    def bf(a):
        return torch.from_numpy(a).to(torch.bfloat16).cuda()
    layer = FFFLayer(cfg.D, cfg.O, cfg.depth, cfg.leaf_width, cfg.activation, "bf16", bf(w["node_w"]), bf(w["node_b"]),
                     torch.from_numpy(c1).cuda(), bf(w["b1"]), torch.from_numpy(c2).cuda(), bf(w["b2"]),
                     w1_scale=torch.from_numpy(s1).cuda(), w2_scale=torch.from_numpy(s2).cuda())
    layer.reserve(cfg.B)
    n = n_buffer_sets(cfg)
    xs = [torch.from_numpy(wl.TokenSource(cfg, i).x).to(torch.bfloat16).cuda() for i in range(n)]
    ys = [torch.empty((cfg.B, cfg.O), dtype=torch.bfloat16, device="cuda") for _ in range(n)]
    ls = [torch.empty((cfg.B,), dtype=torch.int32, device="cuda") for _ in range(n)]
    regions, _, _, _, _ = time_device(layer, xs, ys, ls, steps, 5, profile=False, min_seconds=MIN_TIMED_SECONDS / 2)
    ms = statistics.median(regions) / steps
    touched = int(torch.unique(ls[0]).numel())
    l, D, O = cfg.leaf_width, cfg.D, cfg.O
    pb = cfg.B * (D + O) * 2 + cfg.n_nodes * (D + 1) * 2 + touched * ((l * D + O * l) * 1 + (l + O) * 2 + 8) + 4 * cfg.B
    status = layer.last_status()
    layer.close()
    return {"workload": cfg.name, "leaf_weights": "e4m3 codes + one float32 scale per leaf", "ms_per_step": round(ms, 5),
            "tokens_per_s": cfg.B / (ms * 1e-3), "algorithmic_bytes": int(pb), "device_status": status,
            "roofline_frac": round(pb / (peaks["hbm_gbs"] * 1e9) * 1e3 / ms, 4)}


def train_bench(cfg: wl.FFFConfig, steps: int, peaks) -> dict:
    """FORWARD_T (all leaves, soft mixture, node entropies) of one configuration: a dense contraction, so its
    roofline is the tensor peak.  FLOPs = 2 B (nodes D + hidden D + (hidden + leaves, padded to 64) O)."""
    import torch
    layer, _, _, xs, _, _, _ = make_device_case(cfg, 0, 2)
    for i in range(3):
        layer.forward_train(xs[i % 2], want_mixture=False, want_entropy=True)
    torch.cuda.synchronize()
    regions = []
    t_begin = time.perf_counter()
    while True:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            layer.forward_train(xs[i % 2], want_mixture=False, want_entropy=True)
        e1.record()
        regions.append((e0, e1))
        if time.perf_counter() - t_begin >= MIN_TIMED_SECONDS / 2 or len(regions) >= 64:
            break
    torch.cuda.synchronize()
    ms = statistics.median(a.elapsed_time(b) for a, b in regions) / steps
    hidden = cfg.n_leaves * cfg.leaf_width
    kp = (hidden + cfg.n_leaves + 63) // 64 * 64
    flops = 2.0 * cfg.B * (cfg.n_nodes * cfg.D + hidden * cfg.D + kp * cfg.O)
    achieved = flops / (ms * 1e-3) / 1e12
    status = layer.last_status()
    layer.close()
    return {"workload": cfg.name, "tokens": cfg.B, "ms_per_step": round(ms, 5), "tokens_per_s": cfg.B / (ms * 1e-3),
            "flops": flops, "device_status": status,
            "roofline": {"bound": "tensor", "achieved": round(achieved, 1), "peak": peaks["bf16_tflops_sustained"],
                         "unit": "TFLOP/s", "frac": round(achieved / peaks["bf16_tflops_sustained"], 4),
                         "peak_source": peaks["source"] + " (sustained bf16: several GEMMs back to back)", "traffic": None}}


# ------------------------------------------------------------------------------------------- CPU oracle legs
def n_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(cfg, w_host, x_host, budget_s: float = 20.0) -> dict:
    """The float64 oracle as it stands, on this machine's cores, on a bounded prefix of the batch."""
    from oracle import fff_oracle as orc
    cores = n_cores()
    net = orc.Net.from_config(cfg, w_host)
    probe = min(cfg.B, 256)
    t = time.perf_counter()
    orc.forward_i(net, x_host[:probe], threads=cores)
    per_tok = (time.perf_counter() - t) / probe
    n = int(max(probe, min(cfg.B, budget_s / max(per_tok, 1e-9))))
    # about 10 s of CPU work: the whole batch (or the prefix that fits the budget), as many passes as that takes
    # (sized from one untimed pass: the short probe above overestimates the per-token cost)
    t = time.perf_counter()
    orc.forward_i(net, x_host[:n], threads=cores)
    passes = int(max(1, min(500, 10.0 / max(time.perf_counter() - t, 1e-6))))
    t = time.perf_counter()
    for _ in range(passes):
        orc.forward_i(net, x_host[:n], threads=cores)
    dt = time.perf_counter() - t
    n1 = max(64, n // max(cores, 1))
    t = time.perf_counter()
    orc.forward_i(net, x_host[:n1], threads=1)
    dt1 = time.perf_counter() - t
    touched = int(np.unique(orc.descend(net, x_host, threads=cores)[0]).size)
    return {"leaves_touched": touched, "value": n * passes / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {n} of {cfg.B} tokens of {cfg.name}, {passes} passes, float64 C oracle, {cores} threads",
            "seconds": round(dt, 3), "single_thread_value": n1 / dt1, "single_thread_sample_tokens": n1}


def run_reference(args, rank: int, world: int):
    """The reference arm: the CPU oracle (the only other implementation of the paper available here)."""
    if rank != 0:
        return
    from oracle import fff_oracle as orc
    cfg = wl.CONFIGS[args.config]
    cores = n_cores()
    w = wl.make_weights(cfg, 0)
    net = orc.Net.from_config(cfg, w)
    x = wl.TokenSource(cfg, 0).x
    # per-token cost from one untimed pass over a few thousand tokens (a shorter probe overestimates it: thread start-up)
    probe = min(x.shape[0], 4096)
    orc.forward_i(net, x[:probe], threads=cores)
    t = time.perf_counter()
    orc.forward_i(net, x[:probe], threads=cores)
    per_tok = (time.perf_counter() - t) / probe
    total_steps = args.steps + args.warmup
    # the GPU arm's batch when all steps then fit about two minutes, else the prefix that does
    n = int(max(32, min(x.shape[0], (120.0 / total_steps) / max(per_tok, 1e-9))))
    for _ in range(args.warmup):
        orc.forward_i(net, x[:n], threads=cores)
    t = time.perf_counter()
    for _ in range(args.steps):
        orc.forward_i(net, x[:n], threads=cores)
    dt = time.perf_counter() - t
    value = n * args.steps / dt
    sample = f"each step: first {n} of {cfg.B} tokens of {cfg.name}, float64 C oracle, {cores} threads"
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": cfg.name, "D": cfg.D, "O": cfg.O, "depth": cfg.depth, "leaf_width": cfg.leaf_width,
                      "activation": cfg.activation, "tokens_per_step": n},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default=DEFAULT_CONFIG, choices=wl.CONFIG_ORDER)
    ap.add_argument("--e2e-steps", type=int, default=30)
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true")
    ap.add_argument("--leg", default="path", choices=["path", "forward_train", "stack", "w8"],
                    help="path: the benchmark line; forward_train / stack: only that extra measurement of --config (for profiling)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
    elif args.leg != "path":
        import torch
        torch.cuda.set_device(local_rank)
        cfg = wl.CONFIGS[args.config]
        if args.leg == "forward_train":
            out = train_bench(cfg, max(1, min(args.steps, 10)), measured_peaks())
        elif args.leg == "w8":
            out = w8_bench(cfg, max(1, min(args.steps, 50)), measured_peaks())
        else:
            out = stack_bench(cfg, 4, max(1, min(args.steps, 50)))
        if rank == 0:
            print(json.dumps({"leg": args.leg, **out}), flush=True)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
