"""Helpers of the GPU parity tests: run the CUDA library through its C ABI on a
seeded workload and compare with the CPU oracle under the stated tolerances."""
from __future__ import annotations

import numpy as np

H_TOL_NATS = 2e-3          # per-step entropy, absolute
GAP_TIE = 1e-3             # logit gap below which a token mismatch is a logged near-tie
TAU_TIE = 1e-4             # |Hbar - tau| below which a switch mismatch is a logged near-tie


def to_dev_bf16(bits: np.ndarray):
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


class GpuGate:
    """Owns the device copies of one workload and a library context."""

    def __init__(self, cfg, W_small_bits, W_large_bits, stream=None, temperature=0.0, seed=0,
                 eos_token=-1):
        import torch
        from paper_2502_06833_b200 import binding as E
        self.E, self.torch, self.cfg = E, torch, cfg
        self.W_small = to_dev_bf16(W_small_bits)
        self.W_large = to_dev_bf16(W_large_bits)
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        self.ctx = E.ead_create(B=cfg.B, V=cfg.V, H_small=cfg.H_small, H_large=cfg.H_large, w=cfg.w,
                                d_min=cfg.d_min, tau=cfg.tau, unit=cfg.unit,
                                start_model=cfg.start_model, W_small=self.W_small,
                                W_large=self.W_large, device=torch.cuda.current_device(),
                                stream=self.stream.cuda_stream, temperature=temperature, seed=seed,
                                eos_token=eos_token,
                                V_large=0 if W_large_bits.shape[0] == cfg.V else W_large_bits.shape[0])

    def close(self):
        if self.ctx:
            self.E.ead_destroy(self.ctx)
            self.ctx = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    def _outs(self, T):
        torch, B = self.torch, self.cfg.B
        return dict(tok=torch.full((T, B), -7, dtype=torch.int32, device="cuda"),
                    H=torch.full((T, B), -7.0, dtype=torch.float32, device="cuda"),
                    Hbar=torch.full((T, B), -7.0, dtype=torch.float32, device="cuda"),
                    used=torch.full((T, B), 9, dtype=torch.uint8, device="cuda"),
                    next=torch.full((T, B), 9, dtype=torch.uint8, device="cuda"))

    @staticmethod
    def _np(o):
        return {k: v.cpu().numpy() for k, v in o.items()}

    def run(self, h_small_bits, h_large_bits, mode="run"):
        """mode: "run" (ead_run), "step" (T x ead_step), "host" (ead_run_host)."""
        E, torch = self.E, self.torch
        T = h_small_bits.shape[0]
        if mode == "host":
            B = self.cfg.B
            o = dict(tok=np.full((T, B), -7, np.int32), H=np.full((T, B), -7, np.float32),
                     Hbar=np.full((T, B), -7, np.float32), used=np.full((T, B), 9, np.uint8),
                     next=np.full((T, B), 9, np.uint8))
            E.ead_run_host(self.ctx, T, np.ascontiguousarray(h_small_bits),
                           np.ascontiguousarray(h_large_bits), o["tok"], o["H"], o["Hbar"],
                           o["used"], o["next"])
            E.ead_status(self.ctx)
            return o
        hs, hl = to_dev_bf16(h_small_bits), to_dev_bf16(h_large_bits)
        o = self._outs(T)
        with torch.cuda.stream(self.stream):
            if mode == "run":
                E.ead_run(self.ctx, T, hs, hl, o["tok"], o["H"], o["Hbar"], o["used"], o["next"])
            else:
                for t in range(T):
                    E.ead_step(self.ctx, hs[t], hl[t], o["tok"][t], o["H"][t], o["Hbar"][t],
                               o["used"][t], o["next"][t])
        E.ead_status(self.ctx)
        return self._np(o)


def compare(gpu: dict, ora: dict, tau: float, rows=None, unit: int = 0):
    """Element-by-element comparison of GPU outputs [T, B] with oracle outputs
    [T, len(rows)].  Tokens and switch decisions must be identical except at
    provable near-ties, which are returned as a log; after a near-tie on a
    switch decision the row's later steps are not compared (its state has
    legitimately forked)."""
    rows = ora["rows"] if rows is None else np.asarray(rows)
    T = ora["H"].shape[0]
    scale = 1.0 if unit == 0 else 1.0 / np.log(2.0)
    log = dict(token_near_ties=[], switch_near_ties=[], cells=0, max_H_err=0.0)
    for k, b in enumerate(rows):
        for t in range(T):
            assert gpu["used"][t, b] == ora["used"][t, k], f"model_used differs at t={t} row={b}"
            if np.isnan(ora["H"][t, k]):           # ended sequence or non-finite logits: same report
                assert np.isnan(gpu["H"][t, b]) and np.isnan(gpu["Hbar"][t, b]) and gpu["tok"][t, b] == -1
                assert gpu["next"][t, b] == ora["next"][t, k]
                log["cells"] += 1
                continue
            errH = abs(float(gpu["H"][t, b]) - ora["H"][t, k])
            assert errH <= H_TOL_NATS * scale, f"H differs by {errH} at t={t} row={b}"
            log["max_H_err"] = max(log["max_H_err"], errH)
            errB = abs(float(gpu["Hbar"][t, b]) - ora["Hbar"][t, k])
            assert errB <= H_TOL_NATS * scale, f"Hbar differs by {errB} at t={t} row={b}"
            if gpu["tok"][t, b] != ora["tok"][t, k]:
                assert ora["gap"][t, k] < GAP_TIE, (
                    f"token differs at t={t} row={b}: {gpu['tok'][t, b]} vs {ora['tok'][t, k]}, "
                    f"gap {ora['gap'][t, k]}")
                log["token_near_ties"].append((t, int(b), float(ora["gap"][t, k])))
            log["cells"] += 1
            if gpu["next"][t, b] != ora["next"][t, k]:
                d = abs(ora["Hbar"][t, k] - tau)
                assert d < TAU_TIE * scale, f"switch differs at t={t} row={b}, |Hbar - tau| = {d}"
                log["switch_near_ties"].append((t, int(b), float(d)))
                break
    return log
