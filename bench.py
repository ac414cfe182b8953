#!/usr/bin/env python
"""Benchmark of the EAD gate step (one step = compaction, LM-head contraction with the
fused entropy / arg-max epilogue, merge, window + dwell + threshold update) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME|all] [--repeats R]
                    [--temperature T] [--impl ours|reference]

Prints ONE JSON line (rank 0).  The headline workload is the LLaMA-shaped B = 1 latency
configuration: `value` is gate steps per second over all GPUs with the inputs resident in
HBM (W warm-up steps, then EXACTLY K timed steps, the timed region repeated R >= 10 times
from the same checkpointed state, median reported, every repeat listed); `e2e` is the same
through the host-buffer entry point (`ead_run_host`), host<->device copies inside the timed
region; `roofline` is the LM-head kernel's achieved fraction of the binding bound, its
duration measured with CUDA events around every launch; `cpu_baseline` is the fp64 CPU
oracle timed on a bounded sample of the same workload.

Without `--config` (or with `--config all`) the same line carries `per_config`: one entry
per benchmark configuration (LLaMA-shaped B = 1 on the large head, on the small head and
switching; B = 64; Qwen-shaped B = 256; B = 1024 with 0 / 25 / 50 / 100 % of the rows on the
large head; two rows with temperature sampling), each measured by the same protocol with
at least 32 warm-up steps (so that the mix of heads is the configuration's, not that of
Algorithm 1's first d_min tokens) and at least 32 timed steps per repeat.  `--config NAME`
measures that configuration alone.

With N > 1 every rank runs an independent replica of the headline workload (the path has no
cross-sequence term and is not sharded); `per_config` is reported by single-GPU runs only.  `--impl reference` times the CPU oracle alone
(there is no reference implementation of this path): rank 0 only, a bounded number of steps.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from workloads import configs, synth  # noqa: E402

METRIC = "ead_gate_steps_per_s"
UNIT = "steps/s"
HEADLINE = "llama_b1"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# Configurations of the `per_config` list: (workload, temperature).
PER_CONFIG = [("llama_b1", 0.0), ("llama_b1_small_only", 0.0), ("llama_b1_switching", 0.0),
              ("llama_b64", 0.0), ("qwen_b256", 0.0), ("qwen_b1024_f0", 0.0), ("qwen_b1024_f25", 0.0),
              ("qwen_b1024_f50", 0.0), ("qwen_b1024_f100", 0.0), ("llama_b1", 1.0), ("qwen_b1024_f0", 1.0)]
PER_CONFIG_MIN_WARMUP = 32
PER_CONFIG_MIN_STEPS = 32
MIN_REPEATS = 10
MAX_REPEATS = 40
TARGET_TIMED_SECONDS = 0.25          # repeats are added until the timed regions sum to this

# dram__bytes_read.sum + dram__bytes_write.sum of one LM-head launch, from the ncu captures
# committed under profiles/ (file named beside each figure), keyed by workload and by the
# heads that served rows in the captured launch.  An entry is None once the kernel it was
# taken from has changed.  A run reports the figure only for the share of its timed steps
# with the same live heads; workloads whose steps differ mix the per-head figures.
NCU_DRAM_BYTES_PER_LAUNCH = {
    ("llama_b1", "large"): (1.05726e9, "profiles/lmhead_small_kernel_llama_b1_ncu_full.md"),
    ("llama_b1", "small"): (5.3285e8, "profiles/lmhead_small_kernel_llama_b1_small_only_ncu_counters.md"),
    ("llama_b64", "both"): (1.5823e9, "profiles/lmhead_small_kernel_llama_b64_ncu_full.md"),
    ("qwen_b256", "both"): (2.0305e9, "profiles/lmhead_dual_kernel_qwen_configs_ncu_counters.md"),
    ("qwen_b1024", "small"): (4.7428e8, "profiles/lmhead_dual_kernel_qwen_configs_ncu_counters.md"),
    # with both heads live the traffic depends on how the large head's row blocks fall into units
    # (one pass over its weights per kind of unit): keyed by configuration, not by family
    ("qwen_b1024_f25", "both"): (2.0606e9, "profiles/lmhead_dual_kernel_qwen_configs_ncu_counters.md"),
    ("qwen_b1024_f50", "both"): (2.9448e9, "profiles/lmhead_dual_kernel_qwen_configs_ncu_counters.md"),
    ("qwen_b1024", "large"): (1.6573e9, "profiles/lmhead_dual_kernel_qwen_configs_ncu_counters.md"),
}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


# ----------------------------------------------------------------------------- clocks
_REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
            0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
            0x2: "applications_clocks_setting", 0x10: "sync_boost"}


class ClockSampler:
    """Reads SM clock and clock-event reasons of this process's GPU through NVML (read
    only) every few milliseconds while the timed regions run."""

    def __init__(self, uuid: str | None, period_s: float = 0.004):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            h = None
            for cand in (("GPU-" + uuid, uuid) if uuid else ()):
                try:
                    h = pynvml.nvmlDeviceGetHandleByUUID(cand)
                    break
                except Exception:
                    h = None
            self._h = h if h is not None else pynvml.nvmlDeviceGetHandleByIndex(0)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _loop(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in _REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        return {"sm_mhz": int(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------- helpers
def step_costs(cfg, used: np.ndarray):
    """Algorithmic bytes and flops of each step from the model that served each row:
    one read of every head that has at least one row plus the active hidden rows; one
    multiply-add per (row, vocabulary entry, hidden element) of the active head."""
    n_large = used.sum(axis=1).astype(np.int64)
    n_small = cfg.B - n_large
    wb = [2 * cfg.V * cfg.H_small, 2 * cfg.V * cfg.H_large]
    bytes_ = ((n_small > 0) * wb[0] + (n_large > 0) * wb[1]
              + 2 * (n_small * cfg.H_small + n_large * cfg.H_large))
    flops = 2 * cfg.V * (n_small * cfg.H_small + n_large * cfg.H_large)
    return bytes_.astype(np.float64), flops.astype(np.float64)


def aggregate_over_ranks(elapsed_ms: float, steps: int, dist=None):
    """Whole-job rate: every rank did `steps` steps; time = max over ranks."""
    world = 1
    t = float(elapsed_ms)
    if dist is not None and dist.is_initialized():
        import torch
        world = dist.get_world_size()
        dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
        buf = torch.tensor([t], dtype=torch.float64, device=dev)
        dist.all_reduce(buf, op=dist.ReduceOp.MAX)
        t = float(buf.item())
    return world * steps / (t * 1e-3), t, world


def roofline_of(bytes_per_launch: float, flops_per_launch: float, kernel_s: float, step_s: float,
                peaks: dict) -> dict:
    """Binding bound of one LM-head launch and the achieved fraction of it.  The bound is the
    slower of (algorithmic bytes / measured copy rate) and (flops / measured sustained bf16
    rate); tensor-bound rows also state the fraction of the burst rate."""
    t_hbm = bytes_per_launch / (peaks["hbm_gbs"] * 1e9)
    t_mma = flops_per_launch / (peaks["bf16_tflops_sustained"] * 1e12)
    if t_hbm >= t_mma:
        r = {"bound": "hbm", "achieved": bytes_per_launch / kernel_s / 1e9, "peak": peaks["hbm_gbs"],
             "unit": "GB/s"}
        r["frac"] = r["achieved"] / r["peak"]
        r["frac_of_burst"] = None
        r["step_frac"] = bytes_per_launch / step_s / 1e9 / peaks["hbm_gbs"]
        r["step_frac_of_burst"] = None
        r["peak_source"] = peaks["source"] + " (copy rate)"
    else:
        r = {"bound": "tensor", "achieved": flops_per_launch / kernel_s / 1e12,
             "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s"}
        r["frac"] = r["achieved"] / r["peak"]
        r["frac_of_burst"] = r["achieved"] / peaks["bf16_tflops"]
        r["step_frac"] = flops_per_launch / step_s / 1e12 / peaks["bf16_tflops_sustained"]
        r["step_frac_of_burst"] = flops_per_launch / step_s / 1e12 / peaks["bf16_tflops"]
        r["peak_burst"] = peaks["bf16_tflops"]
        r["peak_source"] = peaks["source"] + " (sustained bf16; burst beside it)"
    r["bound_us"] = {"hbm": t_hbm * 1e6, "tensor_sustained": t_mma * 1e6}
    return r


def ncu_traffic(cfg, used: np.ndarray):
    """DRAM bytes per LM-head launch of this run's mix of steps from the committed ncu
    captures, or None when no (current) capture covers it."""
    family = "qwen_b1024" if cfg.name.startswith("qwen_b1024") else \
        "llama_b1" if cfg.name.startswith("llama_b1") else cfg.name
    n_large = used.sum(axis=1)
    kinds = np.where(n_large == 0, 0, np.where(n_large == cfg.B, 2, 1))     # small / both / large
    total, files = 0.0, set()
    for code, kind in ((0, "small"), (1, "both"), (2, "large")):
        share = float((kinds == code).mean())
        if share == 0.0:
            continue
        entry = NCU_DRAM_BYTES_PER_LAUNCH.get((cfg.name, kind)) or NCU_DRAM_BYTES_PER_LAUNCH.get((family, kind))
        if entry is None:
            return None, None
        total += share * entry[0]
        files.add(entry[1])
    return total, sorted(files)


def oracle_sample(cfg, wl, budget_s: float, max_steps: int, skip: int):
    """Times the CPU oracle as it stands on steps [skip, skip + n) of the workload, all rows.
    The oracle always starts from Algorithm 1's initial state, so the first `skip` steps
    are run (and timed) separately and their time subtracted."""
    from oracle import ead_oracle as O
    kw = dict(w=cfg.w, d_min=cfg.d_min, tau=float(np.float32(cfg.tau)), unit=cfg.unit,
              start_model=cfg.start_model)

    def timed(T):
        t0 = time.perf_counter()
        out = O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, T=T, **kw)
        return time.perf_counter() - t0, out

    skip = min(skip, wl.T - 1)
    t_skip, _ = timed(skip)
    t_probe, probe = timed(skip + 1)
    per_step = max(t_probe - t_skip, t_skip / max(skip, 1), 1e-4)
    if float(probe["used"][skip].mean()) < 0.5:            # probed on the small head: later steps may cost
        per_step *= max(1.0, cfg.H_large / cfg.H_small)    # as much as the large one
    n = int(max(1, min(max_steps, wl.T - skip, (budget_s - t_skip) / per_step)))
    t_all, out = timed(skip + n)
    dt = max(t_all - t_skip, 1e-9)
    return n / dt, n, dt, O.num_threads(), float(out["used"][skip:].mean())


def pinned(a: np.ndarray):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else a)
    return t.pin_memory()


def config_keys(cfg) -> dict:
    """The `config` object: the same keys in both arms."""
    return {"workload": cfg.name, "B": cfg.B, "V": cfg.V, "H_small": cfg.H_small, "H_large": cfg.H_large,
            "w": cfg.w, "d_min": cfg.d_min, "tau": cfg.tau}


class WorkloadCache:
    """Host inputs by what determines their bits, so that configurations that differ only in
    the threshold or the start model share one draw."""

    def __init__(self):
        self._heads, self._hidden = {}, {}

    def get(self, cfg, T):
        hk = (cfg.seed, cfg.V, cfg.H_small, cfg.H_large)
        if hk not in self._heads:
            self._heads = {hk: (synth.lm_head(cfg.seed, 0, cfg.V, cfg.H_small),
                                synth.lm_head(cfg.seed, 1, cfg.V, cfg.H_large))}     # keep one pair only
        xk = hk + (cfg.B, T, cfg.stay_easy, cfg.stay_hard, cfg.p_hard0, cfg.s_easy, cfg.s_hard)
        if xk not in self._hidden:
            wl = synth.Workload(cfg, T=T, heads=False)
            self._hidden = {xk: wl}
        h = self._hidden[xk]
        return HostInputs(cfg, T, h.h_small, h.h_large, *self._heads[hk])


class HostInputs:
    """bf16 bit patterns of one configuration's inputs (host memory)."""

    def __init__(self, cfg, T, h_small, h_large, W_small, W_large):
        self.cfg, self.T = cfg, T
        self.h_small, self.h_large, self.W_small, self.W_large = h_small, h_large, W_small, W_large


# ----------------------------------------------------------------------------- arms
def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    K, W = args.steps, args.warmup
    budget = float(args.cpu_seconds if args.cpu_seconds is not None else 60.0)
    wl = synth.Workload(cfg, T=min(W + K, cfg.T))
    rate, n, dt, cores, fl = oracle_sample(cfg, wl, budget, K, skip=W)
    sample = (f"steps {W}..{W + n} of the {K} timed steps, all {cfg.B} rows, oracle as it stands "
              f"(large-head share {fl:.2f}), {dt:.1f} s")
    line = {"impl": "reference", "metric": METRIC, "value": rate, "unit": UNIT, "n_gpus": args.gpus,
            "steps": K, "warmup": W, "ms_per_step": 1e3 / rate, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_keys(cfg),
            "seq_tokens_per_s": rate * cfg.B,
            "cpu_baseline": {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": rate, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


class Runtime:
    """Process-wide pieces of the GPU arm: torch, the binding, the process group."""

    def __init__(self):
        import torch
        import torch.distributed as dist
        from paper_2502_06833_b200 import binding as E
        self.torch, self.dist, self.E = torch, dist, E
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
        torch.cuda.set_device(self.local)
        if self.world > 1:
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local))
        self.uuid = str(torch.cuda.get_device_properties(self.local).uuid)
        self.peaks = load_peaks()
        self.cache = WorkloadCache()

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def max_over_ranks(self, ms: float, steps: int):
        return aggregate_over_ranks(ms, steps, self.dist if self.world > 1 else None)

    def close(self):
        if self.world > 1:
            self.dist.destroy_process_group()


def measure(rt: Runtime, cfg, K: int, W: int, repeats: int | None, temperature: float = 0.0) -> dict:
    """One configuration by the protocol of the module docstring.  Returns the measurements;
    `wl` (host inputs) rides along for the CPU-oracle leg."""
    torch, E = rt.torch, rt.E
    T_total = W + K
    wl = rt.cache.get(cfg, T_total)
    hs_pin, hl_pin = pinned(wl.h_small), pinned(wl.h_large)
    W_small = pinned(wl.W_small).cuda().view(torch.bfloat16)
    W_large = pinned(wl.W_large).cuda().view(torch.bfloat16)
    hs = hs_pin.cuda().view(torch.bfloat16)
    hl = hl_pin.cuda().view(torch.bfloat16)
    B = cfg.B
    used = torch.zeros(T_total, B, dtype=torch.uint8, device="cuda")
    tok = torch.zeros(T_total, B, dtype=torch.int32, device="cuda")
    Hd = torch.zeros(T_total, B, dtype=torch.float32, device="cuda")
    Hbar = torch.zeros(T_total, B, dtype=torch.float32, device="cuda")
    nxt = torch.zeros(T_total, B, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    ctx = E.ead_create(B=B, V=cfg.V, H_small=cfg.H_small, H_large=cfg.H_large, w=cfg.w,
                       d_min=cfg.d_min, tau=cfg.tau, unit=cfg.unit, start_model=cfg.start_model,
                       W_small=W_small, W_large=W_large, device=rt.local, stream=stream.cuda_stream,
                       temperature=temperature, seed=cfg.seed)

    def outs(t0):
        return (tok[t0:], Hd[t0:], Hbar[t0:], used[t0:], nxt[t0:])

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    # W warm-up steps; the state they leave is the start of every timed region
    E.ead_run(ctx, W, hs, hl, *outs(0))
    rt.barrier()
    blob = E.ead_get_state(ctx)

    def timed_device():
        E.ead_set_state(ctx, blob)
        rt.barrier()
        e0.record()
        E.ead_run(ctx, K, hs[W:], hl[W:], *outs(W))
        e1.record()
        rt.barrier()
        return rt.max_over_ranks(e0.elapsed_time(e1), K)[1]

    o_host = [torch.empty(T_total, B, dtype=d).pin_memory()
              for d in (torch.int32, torch.float32, torch.float32, torch.uint8, torch.uint8)]

    def timed_host():
        E.ead_set_state(ctx, blob)
        rt.barrier()
        e0.record()
        E.ead_run_host(ctx, K, hs_pin[W:], hl_pin[W:], *[o[W:] for o in o_host])
        e1.record()
        rt.barrier()
        return rt.max_over_ranks(e0.elapsed_time(e1), K)[1]

    with ClockSampler(rt.uuid) as clocks:
        # ---- device-resident: exactly K timed steps per repeat
        l0 = E.ead_kernel_launches(ctx)
        first = timed_device()
        launches = E.ead_kernel_launches(ctx) - l0
        n_rep = repeats if repeats else int(min(MAX_REPEATS, max(MIN_REPEATS, math.ceil(
            TARGET_TIMED_SECONDS * 1e3 / max(first, 1e-3)))))
        if rt.world > 1:                                   # every rank must take the same count
            buf = torch.tensor([n_rep], dtype=torch.int64, device="cuda")
            rt.dist.all_reduce(buf, op=rt.dist.ReduceOp.MAX)
            n_rep = int(buf.item())
        dev_ms = [first] + [timed_device() for _ in range(n_rep - 1)]
        used_np = used.cpu().numpy()
        status = E.ead_status(ctx)

        # ---- the LM-head kernel alone: events around every launch over the same K steps
        k_rep = min(n_rep, MIN_REPEATS)
        kern = []
        for _ in range(k_rep):
            E.ead_set_state(ctx, blob)
            kern.append(E.ead_run_timed(ctx, K, hs[W:], hl[W:], *outs(W)))
        assert np.array_equal(used.cpu().numpy(), used_np), "timed replay diverged from the graph run"

        # ---- end to end through the host-buffer entry point (pinned host memory)
        timed_host()                                       # allocates the staging buffers
        host_ms = [timed_host() for _ in range(k_rep)]
        assert np.array_equal(o_host[3].numpy()[W:], used_np[W:]), "host-buffer run diverged from the device run"
    info = E.ead_launch_info(ctx)
    E.ead_destroy(ctx)

    t_ms = float(np.median(dev_ms))
    bytes_s, flops_s = step_costs(cfg, used_np[W:])
    t_kernel = float(np.median([k["lmhead_ms"] for k in kern])) * 1e-3 / K          # seconds per launch
    roof = roofline_of(bytes_s.mean(), flops_s.mean(), t_kernel, t_ms * 1e-3 / K, rt.peaks)
    traffic, files = ncu_traffic(cfg, used_np[W:])
    roof["traffic"] = traffic
    roof["traffic_source"] = files
    roof.update({"kernel": "ead_lmhead_small_kernel" if B <= 128 else "ead_lmhead_dual_kernel",
                 "kernel_us_per_launch": t_kernel * 1e6,
                 "algorithmic_bytes_per_launch": bytes_s.mean(), "flops_per_launch": flops_s.mean(),
                 "other_kernels_us_per_step": float(np.median(
                     [k["compact_ms"] + k["merge_gate_ms"] for k in kern])) * 1e3 / K})
    e2e_ms = float(np.median(host_ms))
    return {"cfg": cfg, "wl": wl, "K": K, "W": W, "temperature": temperature,
            "world": rt.world, "ms": t_ms, "repeat_ms": dev_ms, "value": rt.world * K / (t_ms * 1e-3),
            "e2e_value": rt.world * K / (e2e_ms * 1e-3), "e2e_repeat_ms": host_ms,
            "h2d": 2 * B * (cfg.H_small + cfg.H_large), "d2h": B * (4 + 4 + 4 + 1 + 1),
            "launches": int(launches), "roofline": roof, "clocks": clocks.summary(),
            "large_head_share": float(used_np[W:].mean()), "launch": info, "status": status,
            "weights_gb_per_step": bytes_s.mean() / 1e9}


def per_config_entry(m: dict) -> dict:
    cfg = m["cfg"]
    name = cfg.name if m["temperature"] == 0.0 else f"{cfg.name}@T={m['temperature']:g}"
    return {"workload": name, "B": cfg.B, "temperature": m["temperature"],
            "large_head_share": m["large_head_share"], "steps": m["K"], "warmup": m["W"],
            "repeats": len(m["repeat_ms"]), "ms_per_step": m["ms"] / m["K"],
            "ms_per_step_min": min(m["repeat_ms"]) / m["K"], "ms_per_step_max": max(m["repeat_ms"]) / m["K"],
            "value": m["value"], "unit": UNIT, "seq_tokens_per_s": m["value"] * cfg.B,
            "roofline": m["roofline"],
            "e2e": {"value": m["e2e_value"], "unit": UNIT, "h2d_bytes_per_step": m["h2d"],
                    "d2h_bytes_per_step": m["d2h"]},
            "clocks": m["clocks"], "gpu_launches": m["launches"], "launch": m["launch"],
            "status_word": m["status"]}


def run_ours(args):
    rt = Runtime()
    # the per-configuration list is a single-GPU report: with N > 1 every rank would only repeat it
    everything = args.config in (None, "all") and rt.world == 1
    head_cfg = configs.ALL[HEADLINE if everything else args.config]
    W = max(3, args.warmup)
    K = args.steps if args.steps is not None else max(1, head_cfg.T - W)
    head = measure(rt, head_cfg, K, W, args.repeats, args.temperature)

    # ---- CPU oracle beside it (rank 0, single GPU runs only)
    cpu = None
    if rt.rank == 0 and rt.world == 1 and not args.no_cpu_baseline:
        budget = float(args.cpu_seconds if args.cpu_seconds is not None else 15.0)
        # the sample is sized by the time budget, not by K: a short timed region would otherwise
        # leave the oracle a fraction of a second (inputs of up to 1 GB for the extra steps)
        per_step_bytes = 2 * head_cfg.B * (head_cfg.H_small + head_cfg.H_large)
        T_cpu = int(min(head_cfg.T, max(W + K, W + min(2048, (1 << 30) // per_step_bytes))))
        wl_cpu = head["wl"] if T_cpu <= W + K else rt.cache.get(head_cfg, T_cpu)
        rate, n, dt, cores, fl = oracle_sample(head_cfg, wl_cpu, budget, T_cpu - W, skip=W)
        cpu = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"steps {W}..{W + n} of the same workload, all {head_cfg.B} rows "
                         f"(large-head share {fl:.2f}), {dt:.1f} s"}

    rows = []
    if everything:
        for name, temp in PER_CONFIG:
            cfg = configs.ALL[name]
            Wc = max(W, PER_CONFIG_MIN_WARMUP)
            if args.steps is not None:
                Kc = max(args.steps, PER_CONFIG_MIN_STEPS)
            else:
                Kc = 256 if cfg.B == 1 else 64
            Kc = min(Kc, cfg.T - Wc)
            rows.append(per_config_entry(measure(rt, cfg, Kc, Wc, args.repeats, temp)))

    if rt.rank == 0:
        roof = head["roofline"]
        line = {"metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": head["world"], "steps": K,
                "warmup": W, "ms_per_step": head["ms"] / K, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": config_keys(head_cfg),
                "temperature": args.temperature,
                "repeats": len(head["repeat_ms"]), "repeat_ms": head["repeat_ms"],
                "timing": "median over the repeats of one timed region of exactly `steps` steps, "
                          "each restarted from the state after `warmup` steps; max over ranks per repeat",
                "large_head_share": head["large_head_share"],
                "l2": "inputs larger than L2: every step streams %.2f GB of weights" % head["weights_gb_per_step"],
                "multi_gpu": "replicas only" if head["world"] > 1 else "single GPU",
                "launch": head["launch"],
                "seq_tokens_per_s": head["value"] * head_cfg.B,
                "clocks": head["clocks"],
                "e2e": {"value": head["e2e_value"], "unit": UNIT, "h2d_bytes_per_step": head["h2d"],
                        "d2h_bytes_per_step": head["d2h"]},
                "gpu_launches": head["launches"],
                "roofline": roof,
                "cpu_baseline": cpu,
                "status_word": head["status"]}
        if everything:
            line["per_config"] = rows
            line["per_config_protocol"] = (
                "same protocol as the headline; at least %d warm-up steps so that the share of rows on the "
                "large head is the configuration's, at least %d timed steps per repeat; fractions are of the "
                "binding bound (copy rate, or sustained bf16 rate with the fraction of burst beside it)"
                % (PER_CONFIG_MIN_WARMUP, PER_CONFIG_MIN_STEPS))
        print(json.dumps(line), flush=True)
    rt.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=32)
    ap.add_argument("--config", default=None, choices=sorted(configs.ALL) + ["all"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--repeats", type=int, default=None)
    ap.add_argument("--temperature", type=float, default=0.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=None)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        cfg = configs.ALL[HEADLINE if args.config in (None, "all") else args.config]
        if args.steps is None:
            args.steps = max(1, cfg.T - args.warmup)
        run_reference(args, cfg)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
