"""Seeded synthetic inputs for the EAD gate step.

This module only *draws inputs*: LM-head weight matrices, regime chains and
hidden states, all as bf16 bit patterns (uint16).  It holds none of the
method's arithmetic (no logits, softmax, entropy, window or switch rule), so
it can feed both the CPU oracle and the CUDA path without coupling them.

Randomness is counter based: every tensor is cut into fixed-size chunks and
chunk ``k`` of tensor ``tid`` under ``seed`` is drawn from
``Philox(key=[seed, tid], counter=[k, 0, 0, 0])``.  Any chunk can therefore be
regenerated alone, in any order, and the bits do not depend on how many
chunks a caller asks for.

Recipe (per workload):
  * ``W_m[i, j] ~ N(0, 1/H_m)`` for both heads, rounded once to bf16 (RNE).
  * per sequence an independent two-state chain easy/hard: initial state
    Bernoulli(1/2), then stay with probability ``stay_easy`` / ``stay_hard``.
  * ``h_m[t, b, :] = s(regime[t, b]) * u`` with ``u ~ N(0, I)`` drawn
    independently for the small and the large model, ``s = s_easy`` or
    ``s_hard``, rounded once to bf16 (RNE).
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

TID_W_SMALL = 1
TID_W_LARGE = 2
TID_H_SMALL = 3
TID_H_LARGE = 4
TID_REGIME = 5

_W_CHUNK_ROWS = 2048      # vocab rows per Philox stream
_H_CHUNK_STEPS = 8        # time steps per Philox stream


def _map_chunks(fn, n_chunks: int) -> None:
    """Run ``fn(k)`` for every chunk index; chunks are independent streams, so
    the order and the number of threads do not change the bits."""
    workers = min(n_chunks, os.cpu_count() or 1, 16)
    if workers <= 1:
        for k in range(n_chunks):
            fn(k)
        return
    with ThreadPoolExecutor(workers) as ex:
        list(ex.map(fn, range(n_chunks)))


def _gen(seed: int, tid: int, chunk: int) -> np.random.Generator:
    bitgen = np.random.Philox(key=[int(seed), int(tid)], counter=[int(chunk), 0, 0, 0])
    return np.random.Generator(bitgen)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round to nearest even); returns uint16 bits.

    The inputs here are finite normals, so NaN payload handling is not needed.
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def lm_head(seed: int, which: int, V: int, H: int) -> np.ndarray:
    """bf16 bits of ``W[V, H]`` (row major, one row per vocabulary entry).

    ``which`` = 0 for the small model's head, 1 for the large model's.
    """
    tid = TID_W_SMALL if which == 0 else TID_W_LARGE
    out = np.empty((V, H), dtype=np.uint16)
    scale = np.float32(1.0 / np.sqrt(float(H)))

    def fill(k: int) -> None:
        r0 = k * _W_CHUNK_ROWS
        r1 = min(V, r0 + _W_CHUNK_ROWS)
        # always draw a whole chunk so the bits do not depend on V's tail
        x = _gen(seed, tid, k).standard_normal((_W_CHUNK_ROWS, H), dtype=np.float32)
        out[r0:r1] = f32_to_bf16_bits(x[: r1 - r0] * scale)

    _map_chunks(fill, (V + _W_CHUNK_ROWS - 1) // _W_CHUNK_ROWS)
    return out


def regimes(seed: int, T: int, B: int, stay_easy: float, stay_hard: float,
            p_hard0: float = 0.5) -> np.ndarray:
    """Regime chain ``r[T, B]`` (uint8): 0 = easy, 1 = hard."""
    u = _gen(seed, TID_REGIME, 0).random((T + 1, B))
    r = np.empty((T, B), dtype=np.uint8)
    cur = (u[0] < p_hard0).astype(np.uint8)
    for t in range(T):
        if t > 0:
            stay = np.where(cur == 0, stay_easy, stay_hard)
            flip = u[t] >= stay
            cur = np.where(flip, 1 - cur, cur).astype(np.uint8)
        r[t] = cur
    return r


def hidden_states(seed: int, which: int, r: np.ndarray, H: int,
                  s_easy: float, s_hard: float) -> np.ndarray:
    """bf16 bits of ``h[T, B, H]`` for one model given the regime chain ``r[T, B]``."""
    tid = TID_H_SMALL if which == 0 else TID_H_LARGE
    T, B = r.shape
    out = np.empty((T, B, H), dtype=np.uint16)
    s = np.where(r == 0, np.float32(s_easy), np.float32(s_hard)).astype(np.float32)

    def fill(k: int) -> None:
        t0 = k * _H_CHUNK_STEPS
        t1 = min(T, t0 + _H_CHUNK_STEPS)
        u = _gen(seed, tid, k).standard_normal((_H_CHUNK_STEPS, B, H), dtype=np.float32)
        out[t0:t1] = f32_to_bf16_bits(u[: t1 - t0] * s[t0:t1, :, None])

    _map_chunks(fill, (T + _H_CHUNK_STEPS - 1) // _H_CHUNK_STEPS)
    return out


class Workload:
    """All inputs of one configuration, as bf16 bit patterns on the host."""

    def __init__(self, cfg, T: int | None = None, heads: bool = True):
        self.cfg = cfg
        self.T = int(cfg.T if T is None else T)
        self.regime = regimes(cfg.seed, self.T, cfg.B, cfg.stay_easy, cfg.stay_hard,
                              cfg.p_hard0)
        self.h_small = hidden_states(cfg.seed, 0, self.regime, cfg.H_small,
                                     cfg.s_easy, cfg.s_hard)
        self.h_large = hidden_states(cfg.seed, 1, self.regime, cfg.H_large,
                                     cfg.s_easy, cfg.s_hard)
        if heads:
            self.W_small = lm_head(cfg.seed, 0, cfg.V, cfg.H_small)
            self.W_large = lm_head(cfg.seed, 1, cfg.V, cfg.H_large)
        else:
            self.W_small = self.W_large = None
