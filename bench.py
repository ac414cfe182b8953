#!/usr/bin/env python
"""Benchmark of the EAD gate step (one step = compaction, LM-head contraction with the
fused entropy / arg-max epilogue, merge, window + dwell + threshold update) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is gate steps per second over all GPUs with the
inputs resident in HBM; `e2e` is the same through the host-buffer entry point
(`ead_run_host`), host<->device copies inside the timed region; `roofline` is the
LM-head kernel's achieved fraction of the binding bound, its duration measured with CUDA
events around every launch; `cpu_baseline` is the fp64 CPU oracle timed on a bounded
sample of the same workload.  With N > 1 every rank runs an independent replica of the
workload (the path has no cross-sequence term and is not sharded).

`--impl reference` times the CPU oracle alone (there is no reference implementation of
this path): rank 0 only, a bounded number of steps.
"""
from __future__ import annotations

import argparse
import json
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
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per LM-head launch from the committed ncu
# capture of the same kernel (profiles/), keyed by config; None until captured for the
# kernel as it stands.
NCU_TRAFFIC_BYTES_PER_LAUNCH = {"llama_b1": 1.05726e9, "llama_b1_small_only": 5.3285e8, "llama_b64": 1.5823e9,
                                "qwen_b256": 2.0374e9, "qwen_b1024_f0": 4.7419e8, "qwen_b1024_f25": 2.0679e9,
                                "qwen_b1024_f50": 2.0830e9, "qwen_b1024_f100": 1.5878e9}


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
    only) every few milliseconds while the timed region runs."""

    def __init__(self, uuid: str | None, period_s: float = 0.01):
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
    t_probe, _ = timed(skip + 1)
    per_step = max(t_probe - t_skip, t_skip / max(skip, 1), 1e-4)
    n = int(max(1, min(max_steps, wl.T - skip, (budget_s - t_skip) / per_step)))
    t_all, out = timed(skip + n)
    dt = max(t_all - t_skip, 1e-9)
    return n / dt, n, dt, O.num_threads(), float(out["used"][skip:].mean())


def pinned(a: np.ndarray):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else a)
    return t.pin_memory()


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
            "config": {"workload": cfg.name, "B": cfg.B, "V": cfg.V, "H_small": cfg.H_small,
                       "H_large": cfg.H_large, "w": cfg.w, "d_min": cfg.d_min, "tau": cfg.tau},
            "seq_tokens_per_s": rate * cfg.B,
            "cpu_baseline": {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": rate, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_ours(args, cfg):
    import torch
    import torch.distributed as dist
    from paper_2502_06833_b200 import binding as E

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    K, W = args.steps, args.warmup
    T_total = W + K
    peaks = load_peaks()

    wl = synth.Workload(cfg, T=T_total)
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
                       W_small=W_small, W_large=W_large, device=local, stream=stream.cuda_stream)

    def outs(t0):
        return (tok[t0:], Hd[t0:], Hbar[t0:], used[t0:], nxt[t0:])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident: W warm-up steps, then exactly K timed steps
    E.ead_run(ctx, W, hs, hl, *outs(0))
    barrier()
    l0 = E.ead_kernel_launches(ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    uuid = str(torch.cuda.get_device_properties(local).uuid)
    with ClockSampler(uuid) as clocks:
        e0.record()
        E.ead_run(ctx, K, hs[W:], hl[W:], *outs(W))
        e1.record()
        barrier()
    launches = E.ead_kernel_launches(ctx) - l0
    status = E.ead_status(ctx)
    value, t_ms, world_seen = aggregate_over_ranks(e0.elapsed_time(e1), K, dist if world > 1 else None)
    used_np = used.cpu().numpy()

    # ---- the LM-head kernel alone: events around every launch over the same K steps
    E.ead_reset(ctx)
    E.ead_run(ctx, W, hs, hl, *outs(0))
    kms = E.ead_run_timed(ctx, K, hs[W:], hl[W:], *outs(W))
    assert np.array_equal(used.cpu().numpy(), used_np), "timed replay diverged from the graph run"
    bytes_s, flops_s = step_costs(cfg, used_np[W:])
    t_kernel = kms["lmhead_ms"] * 1e-3 / K                      # seconds per launch
    t_hbm = bytes_s.mean() / (peaks["hbm_gbs"] * 1e9)
    t_mma = flops_s.mean() / (peaks["bf16_tflops_sustained"] * 1e12)
    if t_hbm >= t_mma:
        roof = {"bound": "hbm", "achieved": bytes_s.mean() / t_kernel / 1e9, "peak": peaks["hbm_gbs"],
                "unit": "GB/s"}
    else:
        roof = {"bound": "tensor", "achieved": flops_s.mean() / t_kernel / 1e12,
                "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = NCU_TRAFFIC_BYTES_PER_LAUNCH.get(cfg.name)
    roof.update({"kernel": "ead_lmhead_small_kernel" if B <= 128 else "ead_lmhead_kernel", "kernel_us_per_launch": t_kernel * 1e6,
                 "algorithmic_bytes_per_launch": bytes_s.mean(), "flops_per_launch": flops_s.mean(),
                 "peak_source": peaks["source"] + (" (sustained bf16)" if roof["bound"] == "tensor" else ""),
                 "step_frac": (bytes_s.mean() / (t_ms * 1e-3 / K) / 1e9 / peaks["hbm_gbs"]) if roof["bound"] == "hbm"
                 else (flops_s.mean() / (t_ms * 1e-3 / K) / 1e12 / peaks["bf16_tflops_sustained"]),
                 "other_kernels_us_per_step": (kms["compact_ms"] + kms["merge_gate_ms"]) * 1e3 / K})

    # ---- end to end through the host-buffer entry point (pinned host memory)
    o_host = [torch.empty(T_total, B, dtype=d).pin_memory()
              for d in (torch.int32, torch.float32, torch.float32, torch.uint8, torch.uint8)]
    E.ead_reset(ctx)
    E.ead_run_host(ctx, W, hs_pin, hl_pin, *[o[:W] for o in o_host])
    barrier()
    e0.record()
    E.ead_run_host(ctx, K, hs_pin[W:], hl_pin[W:], *[o[W:] for o in o_host])
    e1.record()
    barrier()
    e2e_value, _, _ = aggregate_over_ranks(e0.elapsed_time(e1), K, dist if world > 1 else None)
    assert np.array_equal(o_host[3].numpy(), used_np), "host-buffer run diverged from the device run"
    h2d = 2 * B * (cfg.H_small + cfg.H_large)
    d2h = B * (4 + 4 + 4 + 1 + 1)
    info = E.ead_launch_info(ctx)
    E.ead_destroy(ctx)

    # ---- CPU oracle beside it (rank 0, single GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        budget = float(args.cpu_seconds if args.cpu_seconds is not None else 15.0)
        rate, n, dt, cores, fl = oracle_sample(cfg, wl, budget, K, skip=W)
        cpu = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"steps {W}..{W + n} of the same workload, all {B} rows "
                         f"(large-head share {fl:.2f}), {dt:.1f} s"}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world_seen, "steps": K,
                "warmup": W, "ms_per_step": t_ms / K, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": cfg.name, "B": B, "V": cfg.V, "H_small": cfg.H_small,
                           "H_large": cfg.H_large, "w": cfg.w, "d_min": cfg.d_min, "tau": cfg.tau,
                           "large_head_share": float(used_np[W:].mean()),
                           "l2": "inputs larger than L2: every step streams %.2f GB of weights"
                                 % (bytes_s.mean() / 1e9),
                           "multi_gpu": "replicas only" if world_seen > 1 else "single GPU",
                           "launch": info},
                "seq_tokens_per_s": value * B,
                "clocks": clocks.summary(),
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": d2h},
                "gpu_launches": int(launches),
                "roofline": roof,
                "cpu_baseline": cpu,
                "status_word": status}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=32)
    ap.add_argument("--config", default="llama_b1", choices=sorted(configs.ALL))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=None)
    args = ap.parse_args()
    cfg = configs.ALL[args.config]
    if args.warmup < 3:
        args.warmup = 3
    if args.steps is None:
        args.steps = max(1, cfg.T - args.warmup)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
