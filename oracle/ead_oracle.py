"""ctypes front end of the fp64 CPU oracle (``ead_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark.  It neither imports nor is imported by the
CUDA package.  Marshalling only; every formula lives in the C file, next to
the citation of the passage it follows.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "ead_oracle.c")
_LIB = os.path.join(_DIR, "libead_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _p(a, ctype):
    return None if a is None else a.ctypes.data_as(C.POINTER(ctype))


def lib():
    global _lib
    if _lib is None:
        # EAD_ORACLE_LIB: another build of this file's C source, for the test that plants
        # mistakes in copies of the oracle and checks that the pins notice
        L = C.CDLL(os.environ.get("EAD_ORACLE_LIB") or build())
        L.oracle_entropy.restype = C.c_double
        L.oracle_entropy.argtypes = [C.POINTER(C.c_double), C.c_int64, C.c_int,
                                     C.POINTER(C.c_double)]
        L.oracle_greedy.restype = C.c_int64
        L.oracle_greedy.argtypes = [C.POINTER(C.c_double), C.c_int64, C.POINTER(C.c_double)]
        L.oracle_logits.restype = None
        L.oracle_logits.argtypes = [C.POINTER(C.c_uint16), C.c_int64, C.c_int64,
                                    C.POINTER(C.c_uint16), C.POINTER(C.c_double)]
        L.oracle_gate_trace.restype = None
        L.oracle_gate_trace.argtypes = [C.POINTER(C.c_double), C.c_int64, C.c_int32, C.c_int32,
                                        C.c_double, C.c_int32, C.POINTER(C.c_double),
                                        C.POINTER(C.c_uint8), C.POINTER(C.c_uint8),
                                        C.POINTER(C.c_int32)]
        L.oracle_gate_step.restype = C.c_double
        L.oracle_gate_step.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_int64),
                                       C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.c_double,
                                       C.c_int32, C.c_int32, C.c_double]
        L.oracle_run.restype = None
        L.oracle_run.argtypes = ([C.c_int64] * 6 + [C.c_int32, C.c_int32, C.c_double, C.c_int32,
                                                    C.c_int32]
                                 + [C.POINTER(C.c_uint16)] * 4
                                 + [C.POINTER(C.c_int64), C.c_int64]
                                 + [C.POINTER(C.c_int32), C.POINTER(C.c_double),
                                    C.POINTER(C.c_double), C.POINTER(C.c_uint8),
                                    C.POINTER(C.c_uint8), C.POINTER(C.c_double),
                                    C.POINTER(C.c_int32), C.c_double, C.c_uint64, C.c_int32])
        L.oracle_philox4x32.restype = None
        L.oracle_philox4x32.argtypes = [C.POINTER(C.c_uint32)] * 3
        L.oracle_uniform.restype = C.c_double
        L.oracle_uniform.argtypes = [C.c_uint64, C.c_int64, C.c_int64, C.c_int64]
        L.oracle_sample.restype = C.c_int64
        L.oracle_sample.argtypes = [C.POINTER(C.c_double), C.c_int64, C.c_double, C.c_uint64,
                                    C.c_int64, C.c_int64, C.POINTER(C.c_double)]
        L.oracle_parameter_ratio.restype = C.c_double
        L.oracle_parameter_ratio.argtypes = [C.c_double, C.c_double, C.c_double]
        L.oracle_usage.restype = None
        L.oracle_usage.argtypes = [C.POINTER(C.c_uint8), C.POINTER(C.c_uint8), C.POINTER(C.c_int32),
                                   C.c_int64, C.POINTER(C.c_int64), C.POINTER(C.c_int64),
                                   C.POINTER(C.c_int64)]
        L.oracle_num_threads.restype = C.c_int
        L.oracle_num_threads.argtypes = []
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def entropy(z, unit: int = 0, return_p: bool = False):
    z = np.ascontiguousarray(z, dtype=np.float64)
    p = np.empty_like(z) if return_p else None
    H = lib().oracle_entropy(_p(z, C.c_double), z.size, int(unit), _p(p, C.c_double))
    return (H, p) if return_p else H


def greedy(z):
    """(token, gap between the two largest logits)."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    gap = C.c_double()
    tok = lib().oracle_greedy(_p(z, C.c_double), z.size, C.byref(gap))
    return int(tok), float(gap.value)


def logits(W_bits, h_bits):
    W_bits = np.ascontiguousarray(W_bits, dtype=np.uint16)
    h_bits = np.ascontiguousarray(h_bits, dtype=np.uint16)
    V, H = W_bits.shape
    assert h_bits.shape == (H,)
    z = np.empty(V, dtype=np.float64)
    lib().oracle_logits(_p(W_bits, C.c_uint16), V, H, _p(h_bits, C.c_uint16), _p(z, C.c_double))
    return z


def gate_trace(H_seq, w: int, d_min: int, tau: float, start_model: int = 0):
    """Window / dwell / threshold part of Algorithm 1 on a given entropy sequence."""
    H_seq = np.ascontiguousarray(H_seq, dtype=np.float64)
    T = H_seq.size
    Hbar = np.empty(T, dtype=np.float64)
    used = np.empty(T, dtype=np.uint8)
    nxt = np.empty(T, dtype=np.uint8)
    c_after = np.empty(T, dtype=np.int32)
    lib().oracle_gate_trace(_p(H_seq, C.c_double), T, int(w), int(d_min), float(tau),
                            int(start_model), _p(Hbar, C.c_double), _p(used, C.c_uint8),
                            _p(nxt, C.c_uint8), _p(c_after, C.c_int32))
    return dict(Hbar=Hbar, used=used, next=nxt, c_after=c_after)


def parameter_ratio(usage_large: float, P_small: float, P_large: float) -> float:
    """Average parameters per forward pass relative to the large model (Table 1 footnote)."""
    return float(lib().oracle_parameter_ratio(float(usage_large), float(P_small), float(P_large)))


def usage(used, nxt, tok=None):
    """(tokens by the small model, tokens by the large model, switches) of one [T] trace; with
    ``tok`` given, steps whose token is -1 (sequence already ended) are not counted."""
    used = np.ascontiguousarray(used, dtype=np.uint8)
    nxt = np.ascontiguousarray(nxt, dtype=np.uint8)
    tok = None if tok is None else np.ascontiguousarray(tok, dtype=np.int32)
    a, b, c = C.c_int64(), C.c_int64(), C.c_int64()
    lib().oracle_usage(_p(used, C.c_uint8), _p(nxt, C.c_uint8), _p(tok, C.c_int32), used.size,
                       C.byref(a), C.byref(b), C.byref(c))
    return int(a.value), int(b.value), int(c.value)


class GateState:
    """State of one sequence for step-by-step use of the window / dwell / threshold rule."""

    def __init__(self, capacity: int, start_model: int = 0):
        self.hist = np.zeros(max(1, capacity), dtype=np.float64)
        self.n = C.c_int64(0)
        self.c = C.c_int32(0)
        self.model = C.c_int32(start_model)

    def step(self, H: float, w: int, d_min: int, tau: float) -> float:
        """Feeds one entropy; returns the rolling mean; ``self.model.value`` is the next model."""
        return float(lib().oracle_gate_step(_p(self.hist, C.c_double), C.byref(self.n),
                                            C.byref(self.c), C.byref(self.model), float(H),
                                            int(w), int(d_min), float(tau)))


def philox4x32(ctr, key):
    c = (C.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (C.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (C.c_uint32 * 4)()
    lib().oracle_philox4x32(c, k, o)
    return [int(x) for x in o]


def uniform(seed: int, row: int, step: int, i: int) -> float:
    return float(lib().oracle_uniform(int(seed), int(row), int(step), int(i)))


def sample(z, temperature: float, seed: int, row: int, step: int):
    """(token drawn from softmax(z / T), gap between the two largest perturbed values)."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    gap = C.c_double()
    tok = lib().oracle_sample(_p(z, C.c_double), z.size, float(temperature), int(seed), int(row),
                              int(step), C.byref(gap))
    return int(tok), float(gap.value)


def run(W_small, W_large, h_small, h_large, *, w: int, d_min: int, tau: float, unit: int = 0,
        start_model: int = 0, rows=None, T: int | None = None, temperature: float = 0.0,
        seed: int = 0, eos_token: int = -1):
    """Algorithm 1 (greedy) on bf16 bit-pattern inputs.

    ``h_small``/``h_large`` are ``[T, B, H]`` uint16; ``rows`` selects which of
    the B independent sequences to run (default: all).  Outputs are
    ``[T, len(rows)]``.
    """
    W_small = np.ascontiguousarray(W_small, dtype=np.uint16)
    W_large = np.ascontiguousarray(W_large, dtype=np.uint16)
    h_small = np.ascontiguousarray(h_small, dtype=np.uint16)
    h_large = np.ascontiguousarray(h_large, dtype=np.uint16)
    Tfull, B, Hs = h_small.shape
    Hl = h_large.shape[2]
    assert h_large.shape[:2] == (Tfull, B)
    V = W_small.shape[0]
    Vl = W_large.shape[0]
    assert W_small.shape == (V, Hs) and W_large.shape == (Vl, Hl)
    T = Tfull if T is None else int(T)
    assert 0 <= T <= Tfull
    rows = np.arange(B, dtype=np.int64) if rows is None else np.ascontiguousarray(rows, np.int64)
    n = rows.size
    out = dict(tok=np.empty((T, n), np.int32), H=np.empty((T, n), np.float64),
               Hbar=np.empty((T, n), np.float64), used=np.empty((T, n), np.uint8),
               next=np.empty((T, n), np.uint8), gap=np.empty((T, n), np.float64),
               c_after=np.empty((T, n), np.int32), rows=rows)
    lib().oracle_run(B, T, V, Vl, Hs, Hl, int(w), int(d_min), float(tau), int(unit),
                     int(start_model),
                     _p(W_small, C.c_uint16), _p(W_large, C.c_uint16),
                     _p(h_small, C.c_uint16), _p(h_large, C.c_uint16),
                     _p(rows, C.c_int64), n,
                     _p(out["tok"], C.c_int32), _p(out["H"], C.c_double),
                     _p(out["Hbar"], C.c_double), _p(out["used"], C.c_uint8),
                     _p(out["next"], C.c_uint8), _p(out["gap"], C.c_double),
                     _p(out["c_after"], C.c_int32), float(temperature), int(seed), int(eos_token))
    return out


if __name__ == "__main__":
    print(build(force=True))
