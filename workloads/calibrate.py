"""Chooses the thresholds of the batched configurations (run once; results are frozen in
``workloads/configs.py``).

The large-head share of a run depends on tau only through how many "hard" entropies must
sit in the window before its mean crosses tau, so a cheap surrogate suffices: (1) the CPU
oracle evaluates a few real cells per (model, regime) of the configuration to get the
entropy level and spread there; (2) the regime chains of the configuration are replayed
through the oracle's window / dwell / threshold rule with entropies drawn from those levels;
(3) the tau whose simulated share is closest to the target is reported, together with the
share.  Usage: ``python -m workloads.calibrate llama_b64 0.43``.
"""
from __future__ import annotations

import sys

import numpy as np

from oracle import ead_oracle as O
from workloads import configs, synth


def entropy_levels(cfg, cells: int = 6):
    """mean / std of the entropy per (model, regime) from real oracle cells."""
    heads = [synth.lm_head(cfg.seed, 0, cfg.V, cfg.H_small), synth.lm_head(cfg.seed, 1, cfg.V, cfg.H_large)]
    r = np.repeat(np.array([[0], [1]], dtype=np.uint8), cells, axis=1)        # [2, cells]
    lv = np.zeros((2, 2, 2))
    for m, H in enumerate((cfg.H_small, cfg.H_large)):
        h = synth.hidden_states(cfg.seed + 1000, m, r, H, cfg.s_easy, cfg.s_hard)
        for reg in range(2):
            e = [O.entropy(O.logits(heads[m], h[reg, k])) for k in range(cells)]
            lv[m, reg] = (np.mean(e), np.std(e))
    return lv


def simulated_share(cfg, lv, tau: float, rows: int = 64) -> float:
    r = synth.regimes(cfg.seed, cfg.T, cfg.B, cfg.stay_easy, cfg.stay_hard, cfg.p_hard0)
    rng = np.random.default_rng(0)
    rows = min(rows, cfg.B)
    used = 0
    for b in range(rows):
        st = O.GateState(cfg.T, cfg.start_model)
        for t in range(cfg.T):
            m = st.model.value
            used += m
            mu, sd = lv[m, r[t, b]]
            st.step(rng.normal(mu, sd), cfg.w, cfg.d_min, tau)
    return used / (rows * cfg.T)


def main():
    cfg = configs.ALL[sys.argv[1]]
    target = float(sys.argv[2])
    lv = entropy_levels(cfg)
    print("entropy mean/std [model][regime]:\n", lv)
    easy, hard = lv[:, 0, 0].max(), lv[:, 1, 0].min()
    best = None
    for k in np.arange(0.5, cfg.w + 0.5, 0.5):              # between the k-hard-in-window levels
        tau = float(np.float32(easy + (hard - easy) * k / cfg.w))
        share = simulated_share(cfg, lv, tau)
        print(f"tau {tau:.4f}: simulated large-head share {share:.3f}")
        if best is None or abs(share - target) < abs(best[1] - target):
            best = (tau, share)
    print("closest:", best)


if __name__ == "__main__":
    main()
