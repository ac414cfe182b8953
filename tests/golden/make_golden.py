"""Writes the stored oracle results of the full-size configurations.

Calls only ``oracle/`` and ``workloads/`` (never the CUDA path).  Every file holds the
oracle's outputs for a stated set of (row, step) cells of one configuration:
``head`` = all B rows for the first ``T_head`` steps, ``rows`` = a few rows for the
whole ``T``.  Rows are independent in Algorithm 1, so these cells are exactly what a
full run would give.  Usage:

    python tests/golden/make_golden.py [name ...]      # default: every plan below
"""
from __future__ import annotations

import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import ead_oracle as O  # noqa: E402
from workloads import configs, synth  # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))

# name -> (config, overrides, T_head over all rows, rows run for the full T, T)
PLANS = {
    "llama_b1": (configs.LLAMA_B1, {}, 0, [0], 2048),
    "llama_b1_switching": (configs.LLAMA_B1_SWITCHING, {}, 0, [0], 2048),
    "llama_b64": (configs.LLAMA_B64, {}, 12, [0, 9, 18, 27, 36, 45, 54, 63], 1024),
    "qwen_b256": (configs.QWEN_B256, {}, 12, [0, 85, 170, 255], 512),
    "qwen_b1024_f0": (configs.STRESS_0, {}, 2, [0, 1023], 256),
    "qwen_b1024_f25": (configs.STRESS_25, {}, 12, [0, 341, 682, 1023], 256),
    "qwen_b1024_f50": (configs.STRESS_50, {}, 0, [0, 146, 292, 438, 584, 730, 876, 1023], 256),
    "qwen_b1024_f100": (configs.STRESS_100, {}, 2, [0, 1023], 256),
    "qwen_b1024_w1": (configs.STRESS_50, dict(w=1, d_min=1), 0, [0, 511, 1023], 256),
    "qwen_b1024_w20": (configs.STRESS_50, dict(w=20, d_min=10), 0, [0, 511, 1023], 256),
    # window and dwell sweep on the 25 % mix ((w, d_min) = (5, 10) is qwen_b1024_f25 itself)
    "qwen_b1024_f25_w1_d1": (configs.STRESS_25, dict(w=1, d_min=1), 0, [0, 511, 1023], 256),
    "qwen_b1024_f25_w1_d10": (configs.STRESS_25, dict(w=1, d_min=10), 0, [0, 511, 1023], 256),
    "qwen_b1024_f25_w5_d1": (configs.STRESS_25, dict(w=5, d_min=1), 0, [0, 511, 1023], 256),
    "qwen_b1024_f25_w20_d1": (configs.STRESS_25, dict(w=20, d_min=1), 0, [0, 511, 1023], 256),
    "qwen_b1024_f25_w20_d10": (configs.STRESS_25, dict(w=20, d_min=10), 0, [0, 511, 1023], 256),
    # Algorithm 1's sampling lines at the benchmark shapes (temperature and seed in SAMPLING)
    "llama_b1_sampled": (configs.LLAMA_B1_SWITCHING, {}, 0, [0], 256),
    "llama_b64_sampled": (configs.LLAMA_B64, {}, 2, [5, 58], 96),
    "qwen_b1024_f50_sampled": (configs.STRESS_50, {}, 0, [3, 700], 64),
}

# name -> (temperature, seed of the random stream); every other plan is greedy
SAMPLING = {
    "llama_b1_sampled": (0.8, 0x5EED0001),
    "llama_b64_sampled": (1.0, 0x5EED0002),
    "qwen_b1024_f50_sampled": (1.3, 0x5EED0003),
}


def make(name: str) -> None:
    cfg, over, T_head, rows, T = PLANS[name]
    cfg = cfg.with_(**over)
    temperature, rng_seed = SAMPLING.get(name, (0.0, 0))
    t0 = time.time()
    wl = synth.Workload(cfg, T=T)
    kw = dict(w=cfg.w, d_min=cfg.d_min, tau=float(np.float32(cfg.tau)), unit=cfg.unit,
              start_model=cfg.start_model, temperature=temperature, seed=rng_seed)
    out = {}
    if T_head:
        o = O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, T=T_head, **kw)
        out.update({"head_" + k: v for k, v in o.items()})
    o = O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, rows=rows, T=T, **kw)
    out.update({"rows_" + k: v for k, v in o.items()})
    meta = dict(B=cfg.B, T=T, V=cfg.V, H_small=cfg.H_small, H_large=cfg.H_large, w=cfg.w,
                d_min=cfg.d_min, tau=float(np.float32(cfg.tau)), unit=cfg.unit,
                start_model=cfg.start_model, seed=cfg.seed, T_head=T_head, temperature=temperature,
                rng_seed=rng_seed)
    np.savez_compressed(os.path.join(HERE, f"oracle_{name}.npz"),
                        meta=np.array(repr(meta)), **out)
    cells = T_head * cfg.B + len(rows) * T
    print(f"{name}: {cells} cells in {time.time() - t0:.0f} s, large-head share of the full rows "
          f"{out['rows_used'].mean():.3f}", flush=True)


if __name__ == "__main__":
    for n in (sys.argv[1:] or list(PLANS)):
        make(n)
