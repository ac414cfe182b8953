"""One rank's side of the vocabulary-sharded gate step (several GPUs, one sequence batch).

Eq. 1-2 are sums over the vocabulary and the token is a maximum over it, so every rank can
keep only a slice of the rows of both LM heads: it computes the statistics of its slice
(``ead_shard_partials``), the ranks all-gather their ``[B]`` records of 32 bytes, and every
rank merges all slices in rank order and runs the window / dwell / threshold rule of
Algorithm 1 itself (``ead_shard_gate``).  The per-sequence state is then identical on all
ranks, bit for bit, with no other traffic.

This module is marshalling only.  The records travel in one of two ways:

* ``connect`` / ``connect_symmetric``: every rank's exchange buffer is mapped on every GPU; the
  kernels store their records straight into all of them and wait for the others' to arrive, so
  ``step`` / ``run`` are single library calls (``run`` replays CUDA graphs of whole steps).
* otherwise ``step`` all-gathers the records with ``torch.distributed`` between the two halves
  of the step (NCCL between GPUs; it is ordered between the library's kernels because the
  context is created on the stream that is current here).
"""
from __future__ import annotations

from . import binding as _binding

RECORD_FLOATS = _binding.EAD_SHARD_RECORD_BYTES // 4


def shard_rows(V: int, world: int, rank: int, engine=_binding) -> tuple:
    """Rows ``[begin, end)`` of a head of V rows that ``rank`` of ``world`` holds."""
    return engine.ead_shard_range(V, world, rank)


def shard_of(W, world: int, rank: int, engine=_binding):
    """The slice of a full head ``W`` (``[V, H]``, contiguous) that ``rank`` holds: a view."""
    b, e = shard_rows(W.shape[0], world, rank, engine)
    return W[b:e]


class VocabParallelGate:
    """Gate step over a vocabulary split across the ranks of a process group.

    ``W_small`` / ``W_large`` are this rank's slices (``shard_of``); ``V_small`` / ``V_large`` the
    full vocabulary sizes.  Every rank must pass the same hyper-parameters and, at each step,
    the same hidden states.
    """

    def __init__(self, *, B, V_small, V_large, H_small, H_large, w, d_min, tau, W_small, W_large,
                 rank, world, group=None, unit=0, start_model=0, temperature=0.0, seed=0,
                 eos_token=-1, device=None, engine=_binding, dist=None, torch=None):
        if torch is None:
            import torch
        if dist is None:
            import torch.distributed as dist
        self.torch, self.dist, self.E = torch, dist, engine
        self.B, self.rank, self.world, self.group = int(B), int(rank), int(world), group
        bs, es = shard_rows(V_small, world, rank, engine)
        bl, el = shard_rows(V_large, world, rank, engine)
        if W_small.shape[0] != es - bs or W_large.shape[0] != el - bl:
            raise ValueError(f"rank {rank} of {world} holds rows [{bs}, {es}) of the small head and "
                             f"[{bl}, {el}) of the large head; got {W_small.shape[0]} and {W_large.shape[0]} rows")
        self.W_small, self.W_large = W_small, W_large            # borrowed by the context: keep alive
        dev = W_small.device if device is None else device
        on_gpu = getattr(dev, "type", "cpu") == "cuda"
        stream = torch.cuda.current_stream(dev).cuda_stream if on_gpu else 0
        self.records = torch.zeros((self.B, RECORD_FLOATS), dtype=torch.float32, device=dev)
        self.all_records = torch.zeros((self.world, self.B, RECORD_FLOATS), dtype=torch.float32, device=dev)
        self.connected = False
        self.exchange = None
        self.ctx = engine.ead_create(B=B, V=es - bs, V_large=el - bl, H_small=H_small, H_large=H_large, w=w,
                                     d_min=d_min, tau=tau, unit=unit, start_model=start_model,
                                     W_small=W_small, W_large=W_large,
                                     device=dev.index if on_gpu and dev.index is not None else 0,
                                     stream=stream, temperature=temperature, seed=seed, eos_token=eos_token,
                                     shard_count=world, vocab_offset_small=bs, vocab_offset_large=bl)

    def connect(self, exchange) -> None:
        """``exchange[r]``: rank r's exchange buffer (``ead_shard_exchange_bytes`` bytes, zeroed) as a
        tensor or an address that is valid on this GPU; ``exchange[self.rank]`` is this rank's own."""
        if len(exchange) != self.world:
            raise ValueError(f"need {self.world} exchange buffers, got {len(exchange)}")
        self.E.ead_shard_connect(self.ctx, self.rank, list(exchange))
        self.exchange = exchange                                 # keep the mappings alive
        self.connected = True

    def connect_symmetric(self, symm=None) -> None:
        """Allocates the exchange buffers in ``torch`` symmetric memory (peer-mapped over NVLink)
        and connects to them.  Collective over the group.  ``symm``: the symmetric-memory module
        (default ``torch.distributed._symmetric_memory``)."""
        if symm is None:
            import torch.distributed._symmetric_memory as symm
        torch, dist = self.torch, self.dist
        nbytes = self.E.ead_shard_exchange_bytes(self.B, self.world)
        dev = self.records.device
        buf = symm.empty(nbytes, dtype=torch.uint8, device=dev)
        handle = symm.rendezvous(buf, dist.group.WORLD if self.group is None else self.group)
        buf.zero_()
        if getattr(dev, "type", "cpu") == "cuda":
            torch.cuda.synchronize(dev)
        dist.barrier(group=self.group)                           # nobody stores before everybody has cleared
        self._symm = (buf, handle)
        self.connect([int(handle.buffer_ptrs[r]) for r in range(self.world)])

    def run(self, T, h_small_seq, h_large_seq, tok=None, H=None, Hbar=None, model_used=None, next_model=None):
        """T steps on device-resident ``[T, B, H]`` hidden states (connected ranks only)."""
        if not self.connected:
            raise RuntimeError("run() needs connect() or connect_symmetric() first")
        self.E.ead_run(self.ctx, T, h_small_seq, h_large_seq, tok, H, Hbar, model_used, next_model)

    def step(self, h_small, h_large, tok=None, H=None, Hbar=None, model_used=None, next_model=None):
        """One gate step for all B sequences; outputs as ``ead_step`` (identical on every rank)."""
        if self.connected:
            self.E.ead_step(self.ctx, h_small, h_large, tok, H, Hbar, model_used, next_model)
            return
        self.E.ead_shard_partials(self.ctx, h_small, h_large, self.records)
        if self.world == 1:
            self.all_records[0].copy_(self.records)
        else:
            self.dist.all_gather_into_tensor(self.all_records.view(-1), self.records.view(-1), group=self.group)
        self.E.ead_shard_gate(self.ctx, self.all_records, self.world, tok, H, Hbar, model_used, next_model)

    def status(self) -> int:
        return self.E.ead_status(self.ctx)

    def reset(self) -> None:
        self.E.ead_reset(self.ctx)

    def close(self) -> None:
        if self.ctx:
            self.E.ead_destroy(self.ctx)
            self.ctx = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()
