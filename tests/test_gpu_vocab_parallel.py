"""Vocabulary-sharded gate step against the (unsharded) oracle.

One GPU stands in for the n GPUs: the n shard contexts live on it and take each phase of a
step one after the other (all partials, then the gather by plain copies, then all gates), so no
kernel ever waits for another.  What must hold: every shard ends each step with identical
outputs, bit for bit, and those outputs are the oracle's full-vocabulary results.
"""
import math
import time

import numpy as np
import pytest

from oracle import ead_oracle as O
from workloads import synth
from workloads.configs import EADConfig

from gpu_util import compare, to_dev_bf16

pytestmark = pytest.mark.gpu


def _cfg(**kw):
    base = dict(name="case", B=4, T=20, H_small=64, H_large=128, V=1000, tau=5.2, w=3, d_min=2,
                seed=11, stay_easy=0.8, stay_hard=0.8)
    base.update(kw)
    return EADConfig(**base)


def _mid_tau(V):
    return 0.5 * (math.log(V) + (math.log(V) - 4.5))


class Shards:
    """n shard contexts of one workload on the current GPU."""

    def __init__(self, cfg, W_small_bits, W_large_bits, n, peer=False, **kw):
        import torch
        from paper_2502_06833_b200 import binding as E
        from paper_2502_06833_b200 import vocab_parallel as VP
        self.E, self.torch, self.cfg, self.n = E, torch, cfg, n
        Ws, Wl = to_dev_bf16(W_small_bits), to_dev_bf16(W_large_bits)
        self.full = (Ws, Wl)
        self.gates = [VP.VocabParallelGate(B=cfg.B, V_small=Ws.shape[0], V_large=Wl.shape[0],
                                           H_small=cfg.H_small, H_large=cfg.H_large, w=cfg.w, d_min=cfg.d_min,
                                           tau=cfg.tau, unit=cfg.unit, start_model=cfg.start_model,
                                           W_small=VP.shard_of(Ws, n, r), W_large=VP.shard_of(Wl, n, r),
                                           rank=r, world=n, **kw) for r in range(n)]
        self.all = torch.zeros((n, cfg.B, VP.RECORD_FLOATS), dtype=torch.float32, device="cuda")
        self.peer = peer
        if peer:                                                     # every shard's buffer is "peer memory" here
            nbytes = E.ead_shard_exchange_bytes(cfg.B, n)
            assert nbytes == 2 * n * cfg.B * E.EAD_SHARD_RECORD_BYTES
            self.exchange = [torch.zeros(nbytes, dtype=torch.uint8, device="cuda") for _ in range(n)]
            for g in self.gates:
                g.connect(self.exchange)

    def close(self):
        for g in self.gates:
            g.close()

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

    def run(self, h_small_bits, h_large_bits):
        """Returns one output dict per shard."""
        E = self.E
        T = h_small_bits.shape[0]
        hs, hl = to_dev_bf16(h_small_bits), to_dev_bf16(h_large_bits)
        outs = [self._outs(T) for _ in self.gates]
        for t in range(T):
            for r, g in enumerate(self.gates):                       # phase 1 on every shard
                E.ead_shard_partials(g.ctx, hs[t], hl[t], None if self.peer else self.all[r])
            for g, o in zip(self.gates, outs):                       # phase 2 on every shard
                E.ead_shard_gate(g.ctx, None if self.peer else self.all, self.n, o["tok"][t], o["H"][t],
                                 o["Hbar"][t], o["used"][t], o["next"][t])
        for g in self.gates:
            g.status()
        return [{k: v.cpu().numpy() for k, v in o.items()} for o in outs]


def _same_on_all_shards(outs):
    for o in outs[1:]:
        for k in ("tok", "used", "next"):
            assert np.array_equal(o[k], outs[0][k]), k
        for k in ("H", "Hbar"):
            assert np.array_equal(o[k].view(np.uint32), outs[0][k].view(np.uint32)), k


@pytest.mark.parametrize("B,V,Vl,Hs,Hl,n", [
    (1, 1100, 1100, 64, 128, 2),        # the latency case: one sequence, ragged last tile
    (5, 4100, 4100, 256, 512, 3),       # uneven deal of 33 tiles over 3 shards
    (12, 2500, 1900, 128, 64, 4),       # the two heads have different vocabularies
    (40, 3000, 3000, 64, 128, 2),       # 17..128 sequences: the transposing epilogue
    (150, 1700, 1700, 64, 64, 2),       # > 128 sequences: batch on the MMA's M side, two row blocks
    (3, 1024, 1024, 64, 64, 8),         # one tile per shard
    (7, 900, 900, 64, 128, 1),          # a single shard is the unsharded path with a record in between
])
@pytest.mark.parametrize("peer", [False, True], ids=["caller_exchange", "kernel_exchange"])
def test_sharded_step_equals_the_oracle(B, V, Vl, Hs, Hl, n, peer):
    cfg = _cfg(B=B, V=V, H_small=Hs, H_large=Hl, tau=_mid_tau(V))
    wl = synth.Workload(cfg)
    W_large = wl.W_large if Vl == V else synth.lm_head(cfg.seed + 17, 1, Vl, Hl)
    ora = O.run(wl.W_small, W_large, wl.h_small, wl.h_large, w=cfg.w, d_min=cfg.d_min,
                tau=float(np.float32(cfg.tau)))
    with Shards(cfg, wl.W_small, W_large, n, peer=peer) as sh:
        outs = sh.run(wl.h_small, wl.h_large)
    _same_on_all_shards(outs)
    compare(outs[0], ora, cfg.tau)
    assert 0.0 < ora["used"].mean() < 1.0                            # both heads took part


@pytest.mark.parametrize("B,V,n,temp", [(3, 1300, 2, 1.0), (40, 2600, 3, 0.8), (140, 1100, 2, 1.3)])
def test_sharded_sampling_draws_the_oracle_tokens(B, V, n, temp):
    """The random stream is indexed by the full-vocabulary index, so a slice that starts at
    row v0 must use the words of rows v0.. ; with that the draws are those of one GPU."""
    cfg = _cfg(B=B, V=V, tau=_mid_tau(V), T=12)
    wl = synth.Workload(cfg)
    seed = 0xFEDCBA9876543210
    ora = O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, w=cfg.w, d_min=cfg.d_min,
                tau=float(np.float32(cfg.tau)), temperature=temp, seed=seed)
    with Shards(cfg, wl.W_small, wl.W_large, n, peer=(n == 3), temperature=temp, seed=seed) as sh:
        outs = sh.run(wl.h_small, wl.h_large)
    _same_on_all_shards(outs)
    log = compare(outs[0], ora, cfg.tau)
    assert len(log["token_near_ties"]) <= 2
    assert outs[0]["tok"].max() >= V // 2                            # tokens beyond the first slice occur


def test_sharded_end_of_sequence_uses_full_vocabulary_indices():
    cfg = _cfg(B=6, V=1200, T=24, tau=_mid_tau(1200))
    wl = synth.Workload(cfg)
    free = O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, w=cfg.w, d_min=cfg.d_min,
                 tau=float(np.float32(cfg.tau)))
    late = free["tok"][4:12]
    toks, counts = np.unique(late[late >= 640], return_counts=True)  # a token of the second slice
    eos = int(toks[np.argmax(counts)])
    ora = O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, w=cfg.w, d_min=cfg.d_min,
                tau=float(np.float32(cfg.tau)), eos_token=eos)
    ended = np.isnan(ora["H"][-1])
    assert ended.any() and not ended.all()
    with Shards(cfg, wl.W_small, wl.W_large, 2, eos_token=eos) as sh:
        outs = sh.run(wl.h_small, wl.h_large)
        for g in sh.gates:
            assert np.array_equal(sh.E.ead_get_done(g.ctx, cfg.B).astype(bool), ended)
    _same_on_all_shards(outs)
    compare(outs[0], ora, cfg.tau)


def test_records_from_another_step_are_refused():
    """A shard that is one step behind hands over records with the wrong step number: the gate
    reports it in the status word and leaves the state alone."""
    cfg = _cfg(B=4, V=1000, T=4, tau=_mid_tau(1000))
    wl = synth.Workload(cfg)
    with Shards(cfg, wl.W_small, wl.W_large, 2) as sh:
        E, torch = sh.E, sh.torch
        sh.run(wl.h_small[:2], wl.h_large[:2])                       # two good steps
        stale = sh.all.clone()                                       # records of step 1
        g = sh.gates[0]
        hs, hl = to_dev_bf16(wl.h_small[2]), to_dev_bf16(wl.h_large[2])
        before = E.ead_get_state(g.ctx)
        E.ead_shard_partials(g.ctx, hs, hl, sh.all[0])               # step 2 on shard 0 only
        stale[0].copy_(sh.all[0])
        H = torch.zeros(cfg.B, dtype=torch.float32, device="cuda")
        E.ead_shard_gate(g.ctx, stale, 2, None, H, None, None, None)
        with pytest.raises(E.EadError) as err:
            E.ead_status(g.ctx)
        assert err.value.code == E.EAD_ESTATE
        assert np.isnan(H.cpu().numpy()).all()
        after = E.ead_get_state(g.ctx)
        # windows, counters and flags are those of before the step; only the step count moved on
        assert bytes(before)[16:] == bytes(after)[16:]


def test_a_shard_that_never_delivers_ends_the_wait_with_a_status():
    """Failure detection without a fault: shard 1 stays silent, so the step word that shard 0's
    gate polls is never set.  Its wait must give up after its limit (2 s), report
    EAD_STATUS_WAIT_EXPIRED, leave the per-sequence state alone, and the context must stay
    usable: after a reset and a fresh connect both shards run the workload to the oracle's
    results."""
    cfg = _cfg(B=3, V=1000, T=12, tau=_mid_tau(1000))
    wl = synth.Workload(cfg)
    ora = O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, w=cfg.w, d_min=cfg.d_min,
                tau=float(np.float32(cfg.tau)))
    with Shards(cfg, wl.W_small, wl.W_large, 2, peer=True) as sh:
        E, torch = sh.E, sh.torch
        g0 = sh.gates[0]
        hs, hl = to_dev_bf16(wl.h_small), to_dev_bf16(wl.h_large)
        before = E.ead_get_state(g0.ctx)
        H = torch.zeros(cfg.B, dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        t0 = time.time()
        E.ead_shard_partials(g0.ctx, hs[0], hl[0], None)             # shard 0 delivers to both buffers
        E.ead_shard_gate(g0.ctx, None, 2, None, H, None, None, None)  # ... and waits for shard 1 in vain
        word = E.ead_status(g0.ctx, raise_on_fault=False)
        waited = time.time() - t0
        assert word & E.EAD_STATUS_WAIT_EXPIRED
        with pytest.raises(E.EadError) as err:
            E.ead_status(g0.ctx)
        assert err.value.code == E.EAD_EDEVICE_FAULT
        assert 1.5 < waited < 20.0, waited
        assert np.isnan(H.cpu().numpy()).all()                       # reported like a row without a result
        after = E.ead_get_state(g0.ctx)
        assert bytes(before)[16:] == bytes(after)[16:]               # windows, counters, flags untouched
        # a second wait on the same context does not stall again: the expiry is sticky
        t1 = time.time()
        E.ead_shard_partials(g0.ctx, hs[0], hl[0], None)
        E.ead_shard_gate(g0.ctx, None, 2, None, H, None, None, None)
        E.ead_status(g0.ctx, raise_on_fault=False)
        assert time.time() - t1 < 1.0
        # recovery: clear the state and the status, renumber the exchange, run for real
        torch.cuda.synchronize()
        for x in sh.exchange:
            x.zero_()                                                # connect expects fresh buffers
        for g in sh.gates:
            g.reset()
            g.connect(sh.exchange)
        assert E.ead_status(g0.ctx) == 0
        outs = sh.run(wl.h_small, wl.h_large)
    _same_on_all_shards(outs)
    compare(outs[0], ora, cfg.tau)


def test_plain_calls_are_refused_on_a_sharded_context_and_vice_versa():
    cfg = _cfg(B=2, V=512, T=2, tau=_mid_tau(512))
    wl = synth.Workload(cfg)
    from gpu_util import GpuGate
    with Shards(cfg, wl.W_small, wl.W_large, 2) as sh, GpuGate(cfg, wl.W_small, wl.W_large) as plain:
        E, torch = sh.E, sh.torch
        hs, hl = to_dev_bf16(wl.h_small[0]), to_dev_bf16(wl.h_large[0])
        with pytest.raises(E.EadError) as err:
            E.ead_step(sh.gates[0].ctx, hs, hl)
        assert err.value.code == E.EAD_EINVALID_ARG
        with pytest.raises(E.EadError) as err:
            E.ead_shard_partials(plain.ctx, hs, hl, sh.all[0])
        assert err.value.code == E.EAD_EINVALID_ARG
        with pytest.raises(E.EadError) as err:
            E.ead_shard_gate(sh.gates[0].ctx, sh.all, 3)
        assert err.value.code == E.EAD_EINVALID_ARG


@pytest.mark.parametrize("B,V", [(1, 1500), (9, 2100), (60, 1300), (200, 1000)])
def test_whole_runs_through_the_exchange_buffer_of_a_single_shard(B, V):
    """With one shard the peer path needs no second GPU: ead_run replays its graphs of three
    kernels per step (compaction, LM head, merge + store of the records + wait + gate) for more
    steps than one graph holds, across a reset, and must give the oracle's results."""
    cfg = _cfg(B=B, V=V, tau=_mid_tau(V), T=70)
    wl = synth.Workload(cfg)
    ora = O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, w=cfg.w, d_min=cfg.d_min,
                tau=float(np.float32(cfg.tau)))
    with Shards(cfg, wl.W_small, wl.W_large, 1, peer=True) as sh:
        g, E, torch = sh.gates[0], sh.E, sh.torch
        hs, hl = to_dev_bf16(wl.h_small), to_dev_bf16(wl.h_large)
        o = sh._outs(cfg.T)
        g.run(cfg.T, hs, hl, o["tok"], o["H"], o["Hbar"], o["used"], o["next"])
        g.status()
        first = {k: v.cpu().numpy() for k, v in o.items()}
        g.reset()                                                    # the numbering of exchanged records carries on
        o2 = sh._outs(7)
        g.run(7, hs, hl, o2["tok"], o2["H"], o2["Hbar"], o2["used"], o2["next"])
        g.reset()                                                    # 77 exchanges so far: step 0 now lands in the other buffer
        o3 = sh._outs(cfg.T)
        for t in range(cfg.T):                                       # step by step through ead_step
            g.step(hs[t], hl[t], o3["tok"][t], o3["H"][t], o3["Hbar"][t], o3["used"][t], o3["next"][t])
        g.status()
        third = {k: v.cpu().numpy() for k, v in o3.items()}
        assert E.ead_kernel_launches(g.ctx) >= 3 * (2 * cfg.T + 7)
    compare(first, ora, cfg.tau)
    for k in ("tok", "used", "next"):
        assert np.array_equal(first[k], third[k]), k
    assert np.array_equal(first["H"].view(np.uint32), third["H"].view(np.uint32))


def test_stepping_calls_need_a_connected_context():
    cfg = _cfg(B=2, V=512, T=2, tau=_mid_tau(512))
    wl = synth.Workload(cfg)
    with Shards(cfg, wl.W_small, wl.W_large, 2) as sh:
        E = sh.E
        hs, hl = to_dev_bf16(wl.h_small), to_dev_bf16(wl.h_large)
        for call in (lambda: E.ead_run(sh.gates[0].ctx, 2, hs, hl),
                     lambda: E.ead_shard_partials(sh.gates[0].ctx, hs[0], hl[0], None),
                     lambda: E.ead_shard_gate(sh.gates[0].ctx, None, 2)):
            with pytest.raises(E.EadError) as err:
                call()
            assert err.value.code == E.EAD_EINVALID_ARG


# torch's symmetric memory with a process group of ONE rank on the one GPU there is: the real
# allocator, rendezvous and pointer table behind `connect_symmetric`, then whole runs through the
# buffer it returned.  (Several ranks would need several GPUs; kernels of different ranks that
# wait for one another never share a GPU here.)
_SYMM_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r}); sys.path.insert(0, os.path.join({root!r}, "tests"))
os.environ["MASTER_ADDR"] = "127.0.0.1"; os.environ["MASTER_PORT"] = "29741"
import numpy as np, torch, torch.distributed as dist
torch.cuda.set_device(0)
dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
from paper_2502_06833_b200 import binding as E, vocab_parallel as VP
from oracle import ead_oracle as O
from workloads import synth
from workloads.configs import EADConfig
from gpu_util import compare, to_dev_bf16
cfg = EADConfig(name="case", B=5, T=40, H_small=64, H_large=128, V=1500, tau=6.2, w=3, d_min=2, seed=11,
                stay_easy=0.8, stay_hard=0.8)
wl = synth.Workload(cfg)
ora = O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, w=cfg.w, d_min=cfg.d_min, tau=float(np.float32(cfg.tau)))
Ws, Wl = to_dev_bf16(wl.W_small), to_dev_bf16(wl.W_large)
gate = VP.VocabParallelGate(B=cfg.B, V_small=cfg.V, V_large=cfg.V, H_small=cfg.H_small, H_large=cfg.H_large, w=cfg.w,
                            d_min=cfg.d_min, tau=cfg.tau, W_small=Ws, W_large=Wl, rank=0, world=1)
gate.connect_symmetric()
buf, handle = gate._symm
assert buf.numel() == E.ead_shard_exchange_bytes(cfg.B, 1) and int(handle.buffer_ptrs[0]) == buf.data_ptr()
hs, hl = to_dev_bf16(wl.h_small), to_dev_bf16(wl.h_large)
T, B = cfg.T, cfg.B
o = dict(tok=torch.zeros((T, B), dtype=torch.int32, device="cuda"), H=torch.zeros((T, B), device="cuda"),
         Hbar=torch.zeros((T, B), device="cuda"), used=torch.zeros((T, B), dtype=torch.uint8, device="cuda"),
         next=torch.zeros((T, B), dtype=torch.uint8, device="cuda"))
gate.run(T, hs, hl, o["tok"], o["H"], o["Hbar"], o["used"], o["next"])
assert gate.status() == 0
log = compare({{k: v.cpu().numpy() for k, v in o.items()}}, ora, cfg.tau)
assert log["cells"] == T * B and 0 < ora["used"].mean() < 1
assert buf.view(torch.int32).reshape(2, 1, B, 8)[:, 0, :, 7].max().item() == T      # the records went through it
gate.close()
dist.destroy_process_group()
print("symmetric ok")
"""


def test_connect_symmetric_on_real_symmetric_memory_with_one_rank(tmp_path):
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script = tmp_path / "symm_worker.py"
    script.write_text(_SYMM_WORKER.format(root=root))
    res = subprocess.run([sys.executable, str(script)], capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and "symmetric ok" in res.stdout, (res.stdout + res.stderr)[-3000:]
