"""ctypes binding of ``include/ead.h``: same names, argument marshalling only.

PyTorch is used by callers for device memory and streams; every step of the
gate path runs inside the CUDA library.  Tensors are passed as raw device
pointers (``tensor.data_ptr()``), bf16 matrices as ``torch.bfloat16``.
"""
from __future__ import annotations

import ctypes as C
import os

_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_DIR, "libead_b200.so")

EAD_OK = 0
EAD_EINVALID_ARG = -1
EAD_EALIGNMENT = -2
EAD_ECUDA = -3
EAD_EUNSUPPORTED_ARCH = -4
EAD_EDEVICE_FAULT = -5
EAD_ESTATE = -6
EAD_ELIMIT = -7
EAD_STATIC_MAX_B = 128
EAD_STATIC_MAX_H = 8192
EAD_STATUS_NONFINITE = 0x1
EAD_STATUS_WAIT_EXPIRED = 0x2
EAD_STATUS_BAD_COUNT = 0x4
EAD_STATUS_SHARD_MISMATCH = 0x8
EAD_SHARD_RECORD_BYTES = 32
EAD_SHARD_MAX = 16

SYMBOLS = ["ead_create", "ead_step", "ead_run", "ead_run_host", "ead_run_timed", "ead_reset", "ead_status",
           "ead_state_size", "ead_get_state", "ead_set_state", "ead_kernel_launches",
           "ead_launch_info", "ead_destroy", "ead_strerror", "ead_head_entropy_static",
           "ead_plan_split", "ead_plan_units", "ead_usage", "ead_parameter_ratio", "ead_set_done", "ead_get_done",
           "ead_shard_range", "ead_shard_partials", "ead_shard_gate", "ead_shard_connect",
           "ead_shard_exchange_bytes"]


class EadConfig(C.Structure):
    _fields_ = [("B", C.c_int32), ("V", C.c_int32), ("H_small", C.c_int32), ("H_large", C.c_int32),
                ("w", C.c_int32), ("d_min", C.c_int32), ("tau", C.c_float), ("unit", C.c_int32),
                ("start_model", C.c_int32), ("device", C.c_int32), ("stream", C.c_void_p),
                ("temperature", C.c_float), ("seed", C.c_uint64), ("eos_token", C.c_int32),
                ("V_large", C.c_int32), ("shard_count", C.c_int32), ("vocab_offset_small", C.c_int32),
                ("vocab_offset_large", C.c_int32)]


class EadError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


_lib = None


def lib() -> C.CDLL:
    """Loads the CUDA library; fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2502_06833_b200.build` "
                              "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        vp, i32p, f32p, u8p = C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p
        L.ead_create.restype = C.c_int
        L.ead_create.argtypes = [C.POINTER(EadConfig), vp, vp, C.POINTER(C.c_void_p)]
        L.ead_step.restype = C.c_int
        L.ead_step.argtypes = [vp, vp, vp, i32p, f32p, f32p, u8p, u8p]
        for name in ("ead_run", "ead_run_host"):
            f = getattr(L, name)
            f.restype = C.c_int
            f.argtypes = [vp, C.c_int32, vp, vp, i32p, f32p, f32p, u8p, u8p]
        L.ead_run_timed.restype = C.c_int
        L.ead_run_timed.argtypes = [vp, C.c_int32, vp, vp, i32p, f32p, f32p, u8p, u8p,
                                    C.POINTER(C.c_float)]
        L.ead_reset.restype = C.c_int
        L.ead_reset.argtypes = [vp]
        L.ead_status.restype = C.c_int
        L.ead_status.argtypes = [vp, C.POINTER(C.c_uint32)]
        L.ead_state_size.restype = C.c_size_t
        L.ead_state_size.argtypes = [vp]
        L.ead_get_state.restype = C.c_int
        L.ead_get_state.argtypes = [vp, vp, C.c_size_t]
        L.ead_set_state.restype = C.c_int
        L.ead_set_state.argtypes = [vp, vp, C.c_size_t]
        L.ead_kernel_launches.restype = C.c_int64
        L.ead_kernel_launches.argtypes = [vp]
        L.ead_launch_info.restype = C.c_int
        L.ead_launch_info.argtypes = [vp, C.POINTER(C.c_int32), C.c_int32]
        L.ead_destroy.restype = None
        L.ead_destroy.argtypes = [vp]
        L.ead_head_entropy_static.restype = C.c_int
        L.ead_head_entropy_static.argtypes = [vp, vp, C.c_int32, C.c_int32, C.c_int32, i32p, f32p, vp,
                                              C.c_int32, vp]
        L.ead_set_done.restype = C.c_int
        L.ead_set_done.argtypes = [vp, vp]
        L.ead_get_done.restype = C.c_int
        L.ead_get_done.argtypes = [vp, vp]
        L.ead_usage.restype = C.c_int
        L.ead_usage.argtypes = [vp, C.POINTER(C.c_uint64), vp]
        L.ead_parameter_ratio.restype = C.c_double
        L.ead_parameter_ratio.argtypes = [C.c_uint64, C.c_uint64, C.c_double, C.c_double]
        L.ead_plan_split.restype = C.c_int
        L.ead_plan_split.argtypes = [C.c_int32] * 4 + [C.POINTER(C.c_int32)]
        L.ead_plan_units.restype = C.c_int
        L.ead_plan_units.argtypes = [C.c_int32] * 5 + [C.POINTER(C.c_int32)]
        L.ead_shard_range.restype = C.c_int
        L.ead_shard_range.argtypes = [C.c_int32] * 3 + [C.POINTER(C.c_int32)] * 2
        L.ead_shard_exchange_bytes.restype = C.c_size_t
        L.ead_shard_exchange_bytes.argtypes = [C.c_int32, C.c_int32]
        L.ead_shard_connect.restype = C.c_int
        L.ead_shard_connect.argtypes = [vp, C.c_int32, C.POINTER(C.c_void_p)]
        L.ead_shard_partials.restype = C.c_int
        L.ead_shard_partials.argtypes = [vp, vp, vp, vp]
        L.ead_shard_gate.restype = C.c_int
        L.ead_shard_gate.argtypes = [vp, vp, C.c_int32, i32p, f32p, f32p, u8p, u8p]
        L.ead_strerror.restype = C.c_char_p
        L.ead_strerror.argtypes = [C.c_int]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().ead_strerror(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != EAD_OK:
        raise EadError(code, where)


def _ptr(t):
    """Device (or host) address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def ead_create(*, B, V, H_small, H_large, w, d_min, tau, W_small, W_large, unit=0, start_model=0,
               device=0, stream=0, temperature=0.0, seed=0, eos_token=-1, V_large=0, shard_count=0,
               vocab_offset_small=0, vocab_offset_large=0):
    """Returns an opaque context handle (int).  ``W_*`` are device bf16 ``[V, H]``; they are
    borrowed, keep them alive until ``ead_destroy``."""
    cfg = EadConfig(B, V, H_small, H_large, w, d_min, float(tau), unit, start_model, device,
                    C.c_void_p(int(stream)), float(temperature), int(seed), int(eos_token), int(V_large),
                    int(shard_count), int(vocab_offset_small), int(vocab_offset_large))
    out = C.c_void_p()
    _check(lib().ead_create(C.byref(cfg), _ptr(W_small), _ptr(W_large), C.byref(out)), "ead_create")
    return out.value


def ead_step(ctx, h_small, h_large, tok=None, H=None, Hbar=None, model_used=None, next_model=None):
    _check(lib().ead_step(ctx, _ptr(h_small), _ptr(h_large), _ptr(tok), _ptr(H), _ptr(Hbar),
                          _ptr(model_used), _ptr(next_model)), "ead_step")


def ead_run(ctx, T, h_small_seq, h_large_seq, tok=None, H=None, Hbar=None, model_used=None,
            next_model=None):
    _check(lib().ead_run(ctx, int(T), _ptr(h_small_seq), _ptr(h_large_seq), _ptr(tok), _ptr(H),
                         _ptr(Hbar), _ptr(model_used), _ptr(next_model)), "ead_run")


def ead_run_host(ctx, T, h_small_seq, h_large_seq, tok=None, H=None, Hbar=None, model_used=None,
                 next_model=None):
    """All buffers are HOST memory (numpy arrays or CPU tensors, ideally pinned)."""
    _check(lib().ead_run_host(ctx, int(T), _ptr(h_small_seq), _ptr(h_large_seq), _ptr(tok), _ptr(H),
                              _ptr(Hbar), _ptr(model_used), _ptr(next_model)), "ead_run_host")


def ead_run_timed(ctx, T, h_small_seq, h_large_seq, tok=None, H=None, Hbar=None, model_used=None,
                  next_model=None) -> dict:
    """ead_run with CUDA events around every kernel; returns summed milliseconds per kernel."""
    ms = (C.c_float * 3)()
    _check(lib().ead_run_timed(ctx, int(T), _ptr(h_small_seq), _ptr(h_large_seq), _ptr(tok), _ptr(H),
                               _ptr(Hbar), _ptr(model_used), _ptr(next_model), ms), "ead_run_timed")
    return dict(compact_ms=ms[0], lmhead_ms=ms[1], merge_gate_ms=ms[2])


def ead_reset(ctx):
    _check(lib().ead_reset(ctx), "ead_reset")


def ead_status(ctx, raise_on_fault: bool = True) -> int:
    word = C.c_uint32()
    rc = lib().ead_status(ctx, C.byref(word))
    if rc != EAD_OK and (raise_on_fault or rc != EAD_EDEVICE_FAULT):
        raise EadError(rc, f"ead_status (status word {word.value:#x})")
    return int(word.value)


def ead_state_size(ctx) -> int:
    return int(lib().ead_state_size(ctx))


def ead_get_state(ctx) -> bytes:
    n = ead_state_size(ctx)
    buf = C.create_string_buffer(n)
    _check(lib().ead_get_state(ctx, C.cast(buf, C.c_void_p), n), "ead_get_state")
    return buf.raw


def ead_set_state(ctx, blob: bytes) -> None:
    buf = C.create_string_buffer(bytes(blob), len(blob))
    _check(lib().ead_set_state(ctx, C.cast(buf, C.c_void_p), len(blob)), "ead_set_state")


def ead_kernel_launches(ctx) -> int:
    return int(lib().ead_kernel_launches(ctx))


def ead_launch_info(ctx) -> dict:
    a = (C.c_int32 * 4)()
    _check(lib().ead_launch_info(ctx, a, 4), "ead_launch_info")
    return dict(ctas=a[0], stages=a[1], a_rows=a[2], smem_bytes=a[3])


def ead_head_entropy_static(W, h, B, V, H, tok=None, H_out=None, status=None, device=0, stream=0):
    """Entropy (nats) and greedy token of one LM head for a dense batch, for callers that
    may not allocate device memory: the library uses a scratch array compiled into it
    (B <= EAD_STATIC_MAX_B, H <= EAD_STATIC_MAX_H).  All buffers are device memory owned
    by the caller; asynchronous on ``stream``."""
    _check(lib().ead_head_entropy_static(_ptr(W), _ptr(h), int(B), int(V), int(H), _ptr(tok),
                                         _ptr(H_out), _ptr(status), int(device),
                                         C.c_void_p(int(stream))), "ead_head_entropy_static")


def ead_set_done(ctx, done) -> None:
    """``done``: uint8 numpy array [B] of 0/1 (host memory)."""
    _check(lib().ead_set_done(ctx, _ptr(done)), "ead_set_done")


def ead_get_done(ctx, B: int):
    import numpy as np
    out = np.zeros(B, dtype=np.uint8)
    _check(lib().ead_get_done(ctx, _ptr(out)), "ead_get_done")
    return out


def ead_usage(ctx, per_row=None) -> dict:
    """Tokens produced by each model and switches since the last reset (summed over rows);
    ``per_row`` may be a uint32 numpy array of shape [3, B] to receive the per-row counters."""
    a = (C.c_uint64 * 3)()
    _check(lib().ead_usage(ctx, a, _ptr(per_row)), "ead_usage")
    return dict(tokens_small=int(a[0]), tokens_large=int(a[1]), switches=int(a[2]))


def ead_parameter_ratio(tokens_small, tokens_large, P_small, P_large) -> float:
    return float(lib().ead_parameter_ratio(int(tokens_small), int(tokens_large), float(P_small),
                                           float(P_large)))


def ead_plan_split(cta, G, n_rows, V) -> dict:
    a = (C.c_int32 * 6)()
    _check(lib().ead_plan_split(int(cta), int(G), int(n_rows), int(V), a), "ead_plan_split")
    return dict(active=a[0], row_block=a[1], slot=a[2], col_begin=a[3], col_end=a[4], group=a[5])


def ead_plan_units(cta, G, n_rows, V, two_blocks=True) -> dict:
    a = (C.c_int32 * 13)()
    _check(lib().ead_plan_units(int(cta), int(G), int(n_rows), int(V), int(bool(two_blocks)), a), "ead_plan_units")
    return dict(active=a[0], two_blocks=a[1], row_block=a[2], slot=a[3], group=a[4], rounds=a[5],
                tail_col0=a[6], tail_cols=a[7], thin16=a[8], tile_n=a[9], n_hi=a[10], w_hi=a[11], w_lo=a[12])


def ead_shard_range(V, n_shards, shard) -> tuple:
    """Rows ``[begin, end)`` of a head of V rows held by ``shard`` of ``n_shards``."""
    b, e = C.c_int32(), C.c_int32()
    _check(lib().ead_shard_range(int(V), int(n_shards), int(shard), C.byref(b), C.byref(e)), "ead_shard_range")
    return int(b.value), int(e.value)


def ead_shard_exchange_bytes(B, n_shards) -> int:
    return int(lib().ead_shard_exchange_bytes(int(B), int(n_shards)))


def ead_shard_connect(ctx, shard, exchange) -> None:
    """``exchange``: one device address (or tensor) per shard, as addressable from this GPU."""
    ptrs = (C.c_void_p * len(exchange))(*[_ptr(e) for e in exchange])
    _check(lib().ead_shard_connect(ctx, int(shard), ptrs), "ead_shard_connect")


def ead_shard_partials(ctx, h_small, h_large, records) -> None:
    _check(lib().ead_shard_partials(ctx, _ptr(h_small), _ptr(h_large), _ptr(records)), "ead_shard_partials")


def ead_shard_gate(ctx, all_records, n_shards, tok=None, H=None, Hbar=None, model_used=None,
                   next_model=None) -> None:
    _check(lib().ead_shard_gate(ctx, _ptr(all_records), int(n_shards), _ptr(tok), _ptr(H), _ptr(Hbar),
                                _ptr(model_used), _ptr(next_model)), "ead_shard_gate")


def ead_destroy(ctx) -> None:
    if ctx:
        lib().ead_destroy(ctx)
