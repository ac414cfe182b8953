"""Full-size configurations, in the launch configuration the benchmark times, against
stored oracle results (tests/golden/oracle_*.npz, written by tests/golden/make_golden.py,
which calls only the oracle).  The GPU runs the whole batch for the whole T; compared are
all rows over the first steps and a few rows over every step (rows are independent)."""
import ast
import functools
import os

import numpy as np
import pytest

from workloads import synth

from gpu_util import GpuGate, compare

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
sys_path_golden = os.path.join(GOLDEN)


def _plans():
    import importlib.util
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(GOLDEN, "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod.PLANS, mod.SAMPLING


PLANS, SAMPLING = _plans()


@functools.lru_cache(maxsize=2)
def _head(seed, which, V, H):
    return synth.lm_head(seed, which, V, H)


@functools.lru_cache(maxsize=2)
def _hidden(chain, T):
    """Hidden states by what determines their bits: configurations that differ only in the
    threshold, the window or the dwell share one draw."""
    cfg = chain[0]
    return synth.Workload(cfg, T=T, heads=False)


def _chain_key(cfg):
    return (cfg.with_(name="", tau=0.0, w=1, d_min=1, start_model=0, note=""),)


@pytest.mark.parametrize("name", sorted(PLANS))
def test_full_size_against_stored_oracle(name):
    cfg, over, T_head, rows, T = PLANS[name]
    cfg = cfg.with_(**over)
    z = np.load(os.path.join(GOLDEN, f"oracle_{name}.npz"))
    meta = ast.literal_eval(str(z["meta"]))
    assert meta["B"] == cfg.B and meta["T"] == T and meta["V"] == cfg.V and meta["w"] == cfg.w
    assert meta["d_min"] == cfg.d_min and meta["seed"] == cfg.seed
    assert meta["tau"] == float(np.float32(cfg.tau)), "stored oracle run used another threshold"

    wl = _hidden(_chain_key(cfg), T)
    Ws, Wl = _head(cfg.seed, 0, cfg.V, cfg.H_small), _head(cfg.seed, 1, cfg.V, cfg.H_large)
    temperature, rng_seed = SAMPLING.get(name, (0.0, 0))
    assert meta.get("temperature", 0.0) == temperature and meta.get("rng_seed", 0) == rng_seed
    with GpuGate(cfg, Ws, Wl, temperature=temperature, seed=rng_seed) as g:
        info = g.E.ead_launch_info(g.ctx)
        out = g.run(wl.h_small, wl.h_large, "run")
    assert info["ctas"] >= 100

    ora_rows = {k[5:]: z[k] for k in z.files if k.startswith("rows_")}
    log = compare(out, ora_rows, cfg.tau)
    cells = log["cells"]
    if T_head:
        ora_head = {k[5:]: z[k] for k in z.files if k.startswith("head_")}
        log_h = compare({k: v[:T_head] for k, v in out.items()}, ora_head, cfg.tau)
        cells += log_h["cells"]
        for k in ("token_near_ties", "switch_near_ties"):
            log[k] += log_h[k]
        log["max_H_err"] = max(log["max_H_err"], log_h["max_H_err"])
    print(f"{name}: {cells} cells compared, max |dH| {log['max_H_err']:.2e}, "
          f"token near-ties {log['token_near_ties']}, switch near-ties {log['switch_near_ties']}, "
          f"large-head share {out['used'].mean():.3f}")
    assert cells >= 0.9 * (T_head * cfg.B + len(rows) * T)
    assert len(log["token_near_ties"]) + len(log["switch_near_ties"]) <= 3
