"""Parity of the CUDA library (called through its C ABI) with the CPU oracle."""
import numpy as np
import pytest

from oracle import ead_oracle as O
from workloads import configs, synth

from gpu_util import GpuGate, compare

pytestmark = pytest.mark.gpu


def _oracle(cfg, wl, rows=None, T=None):
    return O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, w=cfg.w, d_min=cfg.d_min,
                 tau=float(np.float32(cfg.tau)), unit=cfg.unit, start_model=cfg.start_model,
                 rows=rows, T=T)


@pytest.mark.parametrize("name", ["tiny", "tiny_switching"])
def test_tiny_config_full_parity(name):
    cfg = configs.ALL[name]
    wl = synth.Workload(cfg)
    ora = _oracle(cfg, wl)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        out = g.run(wl.h_small, wl.h_large, "run")
    log = compare(out, ora, cfg.tau)
    assert log["cells"] >= cfg.B * cfg.T - 8
    if name == "tiny":
        assert out["used"][:, 0].tolist() == [0] * 10 + [1] * (cfg.T - 10)
    else:
        assert 0.05 < out["used"].mean() < 0.95
