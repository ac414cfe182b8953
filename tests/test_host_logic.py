"""CPU-only checks of the host side: the C-ABI library loads and exports what
include/ead.h declares, argument validation, the CTA work split, bench helpers and the
multi-process aggregation (gloo, world size 2)."""
import os
import re
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def E():
    from paper_2502_06833_b200 import build
    build.build()
    from paper_2502_06833_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(E):
    hdr = open(os.path.join(ROOT, "include", "ead.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(ead_[a-z_]+)\s*\(", hdr))
    assert declared, "no declarations found"
    lib = E.lib()
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared but not exported"
    assert declared == set(E.SYMBOLS)


def test_strerror_names_every_code(E):
    for code in range(0, -8, -1):
        assert E.strerror(code) != "unknown error"
    assert E.strerror(-99) == "unknown error"


def test_create_rejects_bad_arguments_before_touching_the_gpu(E):
    good = dict(B=4, V=100, H_small=64, H_large=128, w=5, d_min=10, tau=2.0, W_small=4096,
                W_large=8192)
    for bad, code in [(dict(B=0), E.EAD_EINVALID_ARG), (dict(B=5000), E.EAD_EINVALID_ARG),
                      (dict(V=0), E.EAD_EINVALID_ARG), (dict(w=0), E.EAD_EINVALID_ARG),
                      (dict(w=65), E.EAD_EINVALID_ARG), (dict(unit=2), E.EAD_EINVALID_ARG),
                      (dict(start_model=3), E.EAD_EINVALID_ARG),
                      (dict(W_small=None), E.EAD_EINVALID_ARG),
                      (dict(H_small=60), E.EAD_EALIGNMENT), (dict(H_large=4), E.EAD_EINVALID_ARG),
                      (dict(W_large=8200), E.EAD_EALIGNMENT)]:
        with pytest.raises(E.EadError) as err:
            E.ead_create(**{**good, **bad})
        assert err.value.code == code, (bad, err.value.code)


def test_null_context_is_an_error_not_a_crash(E):
    for fn, args in [(E.ead_reset, (None,)), (E.ead_step, (None, 16, 16)),
                     (E.ead_run, (None, 1, 16, 16))]:
        with pytest.raises(E.EadError) as err:
            fn(*args)
        assert err.value.code == E.EAD_EINVALID_ARG
    E.ead_destroy(None)
    assert E.lib().ead_state_size(None) == 0


def test_static_entry_point_limits_are_checked_on_the_host(E):
    with pytest.raises(E.EadError) as err:
        E.ead_head_entropy_static(4096, 8192, E.EAD_STATIC_MAX_B + 1, 100, 64)
    assert err.value.code == E.EAD_ELIMIT
    with pytest.raises(E.EadError) as err:
        E.ead_head_entropy_static(4096, 8192, 4, 100, 60)
    assert err.value.code == E.EAD_EALIGNMENT


@pytest.mark.parametrize("G,n,V", [(148, 1, 128256), (148, 64, 128256), (148, 192, 152064),
                                   (148, 1024, 152064), (148, 4096, 1000), (148, 5, 37),
                                   (148, 129, 4100), (132, 300, 5000), (8, 1000, 257)])
def test_work_split_covers_every_column_once_per_row_block(E, G, n, V):
    R = (n + 127) // 128
    cover = np.zeros((R, (V + 15) // 16 * 16), dtype=np.int32)
    spans, slots = [], {}
    for cta in range(G):
        s = E.ead_plan_split(cta, G, n, V)
        if not s["active"]:
            assert s["col_begin"] == s["col_end"]
            continue
        assert s["col_begin"] % 16 == 0 and s["col_end"] % 16 == 0
        assert 0 <= s["row_block"] < R and 0 <= s["slot"] < s["group"] <= 160
        cover[s["row_block"], s["col_begin"]:s["col_end"]] += 1
        spans.append(s["col_end"] - s["col_begin"])
        assert slots.setdefault((s["row_block"], s["slot"]), cta) == cta
    assert (cover == 1).all(), "a column is missed or served twice"
    assert max(spans) - min(spans) <= 16          # balanced to one 16-column unit
    assert len(slots) == R * max(1, G // R)


@pytest.mark.parametrize("G,n,V", [(148, 129, 152064), (148, 256, 152064), (148, 1024, 152064), (148, 266, 152064),
                                   (148, 440, 152064), (148, 4096, 1000), (148, 300, 37), (132, 700, 5000),
                                   (148, 128, 3000), (20, 1000, 257), (148, 532, 152064), (148, 320, 152064),
                                   (148, 321, 152064), (148, 385, 3000), (148, 257, 100)])
@pytest.mark.parametrize("two", [True, False])
def test_unit_split_covers_every_column_once_per_row_block(E, G, n, V, two):
    """Units of two row blocks or of one block each; on a head of three blocks a last block of at
    most 64 rows rides along with the two-block unit as a thin third block on narrower tiles, and
    with a fuller last block the head is served one block per unit.  Every (row block, column) is served
    by exactly one CTA; a unit's members share its whole rounds of tiles round-robin and cut the
    rest evenly, so they finish within one tile of one another; CTAs are dealt out by unit cost."""
    R = (n + 127) // 128
    last = n - (R - 1) * 128
    vpad = (V + 15) // 16 * 16
    cover = np.zeros((R, vpad), dtype=np.int32)
    groups, work = {}, {}
    for cta in range(G):
        s = E.ead_plan_units(cta, G, n, V, two)
        if not s["active"]:
            continue
        assert 0 <= s["slot"] < s["group"]
        blocks = [s["row_block"], s["row_block"] + 1] if s["two_blocks"] else [s["row_block"]]
        if s["thin16"]:
            assert s["two_blocks"] and last <= s["thin16"] <= 64 and s["thin16"] - last < 16
            blocks.append(s["row_block"] + 2)
        tn = s["tile_n"]
        assert tn == 256 - s["thin16"]
        assert s["row_block"] % 2 == 0 or not s["two_blocks"]
        for rb in blocks:
            assert 0 <= rb < R
            mine = 0
            for k in range(s["rounds"]):
                hi = min(k, s["n_hi"])
                wk = s["w_hi"] if k < s["n_hi"] else s["w_lo"]
                assert 16 <= wk <= tn and wk % 16 == 0
                c0 = s["group"] * (hi * s["w_hi"] + (k - hi) * s["w_lo"]) + s["slot"] * wk
                assert c0 < vpad
                cover[rb, c0:min(vpad, c0 + wk)] += 1
                mine += min(vpad, c0 + wk) - c0
            if s["tail_cols"]:
                assert s["tail_cols"] % 16 == 0 and s["tail_col0"] % 16 == 0 and 0 < s["tail_cols"] <= tn
                cover[rb, s["tail_col0"]:s["tail_col0"] + s["tail_cols"]] += 1
        key = (s["row_block"], s["two_blocks"], s["thin16"])
        groups.setdefault(key, set()).add(s["slot"])
        work.setdefault(key, []).append(mine + s["tail_cols"])
        if s["rounds"] and (s["w_hi"], s["w_lo"]) != (tn, tn):   # a share in few pieces: all of about the same width
            assert s["rounds"] <= 8 and s["w_hi"] == s["w_lo"] + 16 and (R >= 3 or s["two_blocks"])
            assert s["tail_cols"] == 0 or s["w_lo"] - 16 <= s["tail_cols"] <= s["w_lo"] or s["slot"] == s["group"] - 1 \
                or s["tail_col0"] + s["tail_cols"] == vpad
    assert (cover == 1).all(), "a column of a row block is missed or served twice"
    for key, w in work.items():
        if V >= 256 * len(w):                                    # enough columns for whole rounds
            assert max(w) - min([x for x in w if x] or [0]) <= 256, (key, sorted(set(w)))
    kinds = {k: len(v) for k, v in groups.items()}
    duals = [v for (rb, two_, thin), v in kinds.items() if two_ and not thin]
    thins = [v for (rb, two_, thin), v in kinds.items() if thin]
    singles = [v for (rb, two_, thin), v in kinds.items() if not two_]
    if two and R == 3 and last <= 64:
        want = (0, 1, 0)
    elif two and R != 3:
        want = (R // 2, 0, R % 2)
    else:
        want = (0, 0, R)
    assert (len(duals), len(thins), len(singles)) == want
    assert len(set(duals)) <= 1 and len(set(singles)) <= 1       # units of a kind are alike
    if duals and singles and G >= 40:
        assert 0.4 <= singles[0] / duals[0] <= 0.75             # about 5 : 9
    if thins:
        assert thins == [G] and not duals and not singles       # a unit with a thin block has the head to itself
    assert sum(duals) + sum(thins) + sum(singles) <= G
    with pytest.raises(E.EadError):
        E.ead_plan_units(0, 4, 1000, 257, two)                   # eight row blocks, four CTAs


def test_work_split_needs_a_cta_per_row_block(E):
    with pytest.raises(E.EadError) as err:
        E.ead_plan_split(0, 4, 1000, 257)
    assert err.value.code == E.EAD_EINVALID_ARG


def test_work_split_of_an_empty_head(E):
    s = E.ead_plan_split(0, 148, 0, 1000)
    assert s["active"] == 0 and s["col_begin"] == s["col_end"]


def test_bench_roofline_picks_the_binding_bound_and_states_both_tensor_fractions():
    sys.path.insert(0, ROOT)
    import bench
    peaks = {"hbm_gbs": 6000.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1200.0, "source": "measured"}
    # 1.2 GB and 1.2 GFLOP in 250 us: 200 us of HBM time against 1 us of tensor time -> HBM bound
    r = bench.roofline_of(1.2e9, 1.2e9, 250e-6, 300e-6, peaks)
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["frac_of_burst"] is None
    assert r["achieved"] == pytest.approx(4800.0) and r["frac"] == pytest.approx(0.8)
    assert r["step_frac"] == pytest.approx(1.2e9 / 300e-6 / 1e9 / 6000.0)
    assert r["bound_us"]["hbm"] == pytest.approx(200.0) and r["bound_us"]["tensor_sustained"] == pytest.approx(1.0)
    # 0.5 GB and 1.2 TFLOP in 1.25 ms: 83 us against 1000 us -> tensor bound, both fractions
    r = bench.roofline_of(0.5e9, 1.2e12, 1.25e-3, 1.5e-3, peaks)
    assert r["bound"] == "tensor" and r["peak"] == 1200.0 and r["peak_burst"] == 1600.0
    assert r["frac"] == pytest.approx(0.8) and r["frac_of_burst"] == pytest.approx(0.6)
    assert r["step_frac"] == pytest.approx(1.2e12 / 1.5e-3 / 1e12 / 1200.0)
    assert r["frac"] == pytest.approx(r["achieved"] / r["peak"])


def test_bench_ncu_traffic_follows_the_heads_that_were_live():
    sys.path.insert(0, ROOT)
    import bench
    from workloads import configs
    tab = bench.NCU_DRAM_BYTES_PER_LAUNCH
    cfg = configs.LLAMA_B1
    used = np.array([[0]] * 5 + [[1]] * 15, dtype=np.uint8)           # 25 % small-head steps, 75 % large
    got, files = bench.ncu_traffic(cfg, used)
    want = 0.25 * tab[("llama_b1", "small")][0] + 0.75 * tab[("llama_b1", "large")][0]
    assert got == pytest.approx(want) and len(files) == 2 and all(f.startswith("profiles/") for f in files)
    for f in files:
        assert os.path.exists(os.path.join(ROOT, f)), f
    cfg = configs.STRESS_25
    used = np.zeros((4, cfg.B), dtype=np.uint8)
    used[:, :300] = 1                                                   # both heads live in every step
    got, files = bench.ncu_traffic(cfg, used)
    assert got == pytest.approx(tab[("qwen_b1024_f25", "both")][0])     # mixed steps: keyed by configuration
    assert tab[("qwen_b1024_f50", "both")][0] > 1.3 * got               # ... because the unit layout sets the traffic
    used[:] = 1
    assert bench.ncu_traffic(cfg, used)[0] == pytest.approx(tab[("qwen_b1024", "large")][0])
    assert bench.ncu_traffic(configs.TINY, np.zeros((2, 4), dtype=np.uint8)) == (None, None)   # never captured


def test_bench_arms_describe_the_workload_with_the_same_keys():
    sys.path.insert(0, ROOT)
    import bench
    from workloads import configs
    keys = set(bench.config_keys(configs.LLAMA_B1))
    assert keys == {"workload", "B", "V", "H_small", "H_large", "w", "d_min", "tau"}
    src = open(os.path.join(ROOT, "bench.py")).read()
    assert src.count('"config": config_keys(') == 2                     # the reference arm and ours


def test_bench_step_costs():
    sys.path.insert(0, ROOT)
    import bench
    from workloads import configs
    cfg = configs.LLAMA_B64
    used = np.zeros((3, cfg.B), dtype=np.uint8)
    used[1, :10] = 1
    used[2, :] = 1
    b, f = bench.step_costs(cfg, used)
    ws, wl = 2 * cfg.V * cfg.H_small, 2 * cfg.V * cfg.H_large
    assert b[0] == ws + 2 * 64 * cfg.H_small
    assert b[1] == ws + wl + 2 * (54 * cfg.H_small + 10 * cfg.H_large)
    assert b[2] == wl + 2 * 64 * cfg.H_large
    assert f[1] == 2 * cfg.V * (54 * cfg.H_small + 10 * cfg.H_large)


_GLOO_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
value, t, world = bench.aggregate_over_ranks(10.0 * (rank + 1), 100, dist)
assert world == 2 and abs(t - 20.0) < 1e-9 and abs(value - 2 * 100 / 0.020) < 1e-6, (value, t, world)
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_aggregation_over_two_ranks_takes_the_slowest(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_GLOO_WORKER.format(root=ROOT))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29631", str(script)]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert res.returncode == 0, res.stdout + res.stderr
    assert res.stdout.count("ok") == 2


def test_parameter_ratio_matches_the_table_footnote(E):
    """Host arithmetic of the library against two rows of the paper's Table 1 (Qwen 14B vs
    1.5B at 25.6 % usage -> 33.6 %; LLaMA 3B vs 1B at 16.0 % -> 44.0 %) and the end points."""
    assert 100 * E.ead_parameter_ratio(744, 256, 1.5, 14) == pytest.approx(33.6, abs=0.1)
    assert 100 * E.ead_parameter_ratio(84, 16, 1, 3) == pytest.approx(44.0, abs=0.05)
    assert E.ead_parameter_ratio(10, 0, 3, 11) == pytest.approx(3 / 11)
    assert E.ead_parameter_ratio(0, 10, 3, 11) == 1.0


def test_shard_ranges_cover_the_vocabulary_in_whole_tiles(E):
    for V, n in [(128256, 8), (152064, 4), (1100, 2), (1024, 8), (129, 2), (5, 1)]:
        cuts = [E.ead_shard_range(V, n, r) for r in range(n)]
        assert cuts[0][0] == 0 and cuts[-1][1] == V
        for (b0, e0), (b1, _) in zip(cuts, cuts[1:]):
            assert e0 == b1
        for b, e in cuts:
            assert b % 128 == 0 and e > b
        tiles = [-(-(e - b) // 128) for b, e in cuts]
        assert max(tiles) - min(tiles) <= 1                       # dealt out evenly
    with pytest.raises(E.EadError) as err:                        # 9 tiles cannot feed 10 shards
        E.ead_shard_range(1100, 10, 0)
    assert err.value.code == E.EAD_EINVALID_ARG
    with pytest.raises(E.EadError):
        E.ead_shard_range(1100, 2, 2)


# Two gloo ranks drive VocabParallelGate with a numpy stand-in for the CUDA library (same call
# names and record layout).  What is under test is the glue: slice bounds, the order of the
# gathered records, and that merging per-slice statistics in rank order gives the
# full-vocabulary entropy and arg max of the oracle.
_VP_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
sys.path.insert(0, os.path.join({root!r}, "tests"))
import numpy as np, torch, torch.distributed as dist
from paper_2502_06833_b200 import binding, vocab_parallel as VP
from oracle import ead_oracle as O

LOG2E = 1.4426950408889634

class FakeEngine:
    EAD_SHARD_RECORD_BYTES = 32
    ead_shard_range = staticmethod(binding.ead_shard_range)
    def ead_create(self, **kw):
        self.kw = kw
        self.step = 0
        return self
    def ead_shard_partials(self, ctx, h_small, h_large, records):
        W, off = self.kw["W_small"].double().numpy(), self.kw["vocab_offset_small"]   # every row starts on M_S
        z = h_small.double().numpy() @ W.T                                              # [B, slice]
        m = z.max(1)
        e = np.exp(z - m[:, None])
        rec = records.numpy()
        rec[:, 0], rec[:, 1], rec[:, 2] = m, e.sum(1), (e * (z - m[:, None])).sum(1) * LOG2E
        ints = rec.view(np.int32)
        ints[:, 3] = z.argmax(1) + off
        ints[:, 6], ints[:, 7] = 0, self.step
    def ead_shard_gate(self, ctx, all_records, n, tok, H, Hbar, used, nxt):
        a = all_records.numpy().astype(np.float64)
        ai = all_records.numpy().view(np.int32)
        assert n == self.kw["shard_count"] and (ai[:, :, 7] == self.step).all()
        B = a.shape[1]
        for b in range(B):
            m, s, t, idx = -1e30, 0.0, 0.0, 2**31 - 1
            for r in range(n):
                qm, qs, qt, qi = a[r, b, 0], a[r, b, 1], a[r, b, 2], int(ai[r, b, 3])
                M = max(m, qm)
                da, db = (m - M) * LOG2E, (qm - M) * LOG2E
                ea, eb = 2.0 ** da, 2.0 ** db
                s, t = ea * s + eb * qs, ea * (da * s + t) + eb * (db * qs + qt)
                idx = idx if m > qm else qi if qm > m else min(idx, qi)
                m = M
            H[b] = np.log(s) - t / (s * LOG2E)
            tok[b] = idx
        self.step += 1
    def ead_destroy(self, ctx): pass

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
rng = np.random.default_rng(5)
V, Hd, B = 1100, 32, 3
W = torch.from_numpy(rng.integers(-24, 25, (V, Hd)) / 16.0).float()          # exact in bf16 and float32
h = torch.from_numpy(rng.integers(-16, 17, (B, Hd)) / 8.0).float()
Wl = torch.zeros((V, 8))
gate = VP.VocabParallelGate(B=B, V_small=V, V_large=V, H_small=Hd, H_large=8, w=5, d_min=10, tau=1.0,
                            W_small=VP.shard_of(W, world, rank), W_large=VP.shard_of(Wl, world, rank),
                            rank=rank, world=world, engine=FakeEngine(), device=torch.device("cpu"))
assert gate.W_small.shape[0] == (512 if rank == 0 else 588)        # 9 tiles: 4 + 5 (ragged)
tok = torch.zeros(B, dtype=torch.int32); H = torch.zeros(B, dtype=torch.float32)
gate.step(h, torch.zeros((B, 8)), tok, H)
# records arrived in rank order: slice r's arg max lies in slice r
ints = gate.all_records.numpy().view(np.int32)
for r in range(world):
    b, e = VP.shard_rows(V, world, r)
    assert ((ints[r, :, 3] >= b) & (ints[r, :, 3] < e)).all()
z = h.double().numpy() @ W.double().numpy().T
for b in range(B):
    assert abs(float(H[b]) - O.entropy(z[b])) < 1e-6, (float(H[b]), O.entropy(z[b]))
    assert int(tok[b]) == O.greedy(z[b])[0]
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_vocab_parallel_glue_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "vp_worker.py"
    script.write_text(_VP_WORKER.format(root=ROOT))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29633", str(script)]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert res.returncode == 0, res.stdout + res.stderr
    assert res.stdout.count("ok") == 2


# The same two ranks through the other route: exchange buffers that every rank can address
# (here: files mapped by both processes), `connect()` with one buffer per rank in rank order,
# then whole steps by `run()`.  The stand-in engine stores its record into every rank's buffer,
# step word last, and polls its own buffer for the others', as the CUDA kernels do.
_VP_CONNECTED_WORKER = r"""
import os, sys, time
sys.path.insert(0, {root!r})
import numpy as np, torch, torch.distributed as dist
from paper_2502_06833_b200 import binding, vocab_parallel as VP
from oracle import ead_oracle as O

LOG2E = 1.4426950408889634
TMP = {tmp!r}

class FakeEngine:
    EAD_SHARD_RECORD_BYTES = 32
    ead_shard_range = staticmethod(binding.ead_shard_range)
    def ead_shard_exchange_bytes(self, B, n):
        return 2 * n * B * 32
    def ead_create(self, **kw):
        self.kw, self.xstep, self.connected_to = kw, 0, None
        return self
    def ead_shard_connect(self, ctx, shard, exchange):
        assert len(exchange) == self.kw["shard_count"]
        self.shard, self.connected_to, self.xstep = shard, list(exchange), 0
    def _record(self, h_small):
        W, off = self.kw["W_small"].double().numpy(), self.kw["vocab_offset_small"]
        z = h_small.double().numpy() @ W.T
        m = z.max(1)
        e = np.exp(z - m[:, None])
        rec = np.zeros((z.shape[0], 8), dtype=np.float32)
        rec[:, 0], rec[:, 1], rec[:, 2] = m, e.sum(1), (e * (z - m[:, None])).sum(1) * LOG2E
        rec.view(np.int32)[:, 3] = z.argmax(1) + off
        return rec
    def ead_step(self, ctx, h_small, h_large, tok, H, Hbar, used, nxt):
        n, B = self.kw["shard_count"], self.kw["B"]
        rec, step1, par = self._record(h_small), self.xstep + 1, self.xstep & 1
        for buf in self.connected_to:                       # every shard's buffer, own one included
            v = buf.reshape(2, n, B, 8)
            v[par, self.shard, :, :7] = rec[:, :7]
            buf.flush()
            v.view(np.int32)[par, self.shard, :, 7] = step1  # the step word goes last
            buf.flush()
        mine = self.connected_to[self.shard].reshape(2, n, B, 8)
        t0 = time.time()
        while not (mine.view(np.int32)[par, :, :, 7] == step1).all():
            assert time.time() - t0 < 60, "a shard never delivered"
            time.sleep(0.001)
        a, ai = mine[par].astype(np.float64), mine.view(np.int32)[par]
        for b in range(B):
            m, s, t, idx = -1e30, 0.0, 0.0, 2**31 - 1
            for r in range(n):
                qm, qs, qt, qi = a[r, b, 0], a[r, b, 1], a[r, b, 2], int(ai[r, b, 3])
                M = max(m, qm)
                da, db = (m - M) * LOG2E, (qm - M) * LOG2E
                ea, eb = 2.0 ** da, 2.0 ** db
                s, t = ea * s + eb * qs, ea * (da * s + t) + eb * (db * qs + qt)
                idx = idx if m > qm else qi if qm > m else min(idx, qi)
                m = M
            H[b] = np.log(s) - t / (s * LOG2E)
            tok[b] = idx
        self.xstep += 1
    def ead_run(self, ctx, T, hs, hl, tok, H, Hbar, used, nxt):
        for t in range(T):
            self.ead_step(ctx, hs[t], hl[t], tok[t], H[t], None, None, None)
    def ead_destroy(self, ctx): pass

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
rng = np.random.default_rng(7)
V, Hd, B, T = 1100, 32, 3, 5
W = torch.from_numpy(rng.integers(-24, 25, (V, Hd)) / 16.0).float()
h = torch.from_numpy(rng.integers(-16, 17, (T, B, Hd)) / 8.0).float()
Wl = torch.zeros((V, 8))
eng = FakeEngine()
gate = VP.VocabParallelGate(B=B, V_small=V, V_large=V, H_small=Hd, H_large=8, w=5, d_min=10, tau=1.0,
                            W_small=VP.shard_of(W, world, rank), W_large=VP.shard_of(Wl, world, rank),
                            rank=rank, world=world, engine=eng, device=torch.device("cpu"))
try:
    gate.run(1, h, torch.zeros((T, B, 8)))
    raise SystemExit("run() before connect() must be refused")
except RuntimeError:
    pass
nbytes = eng.ead_shard_exchange_bytes(B, world)
own = np.memmap(os.path.join(TMP, f"xchg_{{rank}}.bin"), dtype=np.float32, mode="w+", shape=(nbytes // 4,))
own[:] = 0
own.flush()
dist.barrier()                                              # every buffer exists and is clear
bufs = [own if r == rank else np.memmap(os.path.join(TMP, f"xchg_{{r}}.bin"), dtype=np.float32, mode="r+",
                                        shape=(nbytes // 4,)) for r in range(world)]
gate.connect(bufs)
assert eng.shard == rank and eng.connected_to[rank] is own
tok = torch.zeros((T, B), dtype=torch.int32); H = torch.zeros((T, B), dtype=torch.float32)
gate.run(T - 1, h, torch.zeros((T, B, 8)), tok, H)
gate.step(h[T - 1], torch.zeros((B, 8)), tok[T - 1], H[T - 1])   # a connected step is one call as well
for t in range(T):
    z = h[t].double().numpy() @ W.double().numpy().T
    for b in range(B):
        assert abs(float(H[t, b]) - O.entropy(z[b])) < 1e-6, (t, b)
        assert int(tok[t, b]) == O.greedy(z[b])[0]
# what the last two steps left in this rank's buffer: source r's arg max lies in slice r
ints = own.reshape(2, world, B, 8).view(np.int32)
for r in range(world):
    b0, e0 = VP.shard_rows(V, world, r)
    assert ((ints[:, r, :, 3] >= b0) & (ints[:, r, :, 3] < e0)).all()
assert sorted(ints[:, :, :, 7].reshape(2, -1)[:, 0].tolist()) == [T - 1, T]
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_vocab_parallel_connected_route_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "vp_connected_worker.py"
    script.write_text(_VP_CONNECTED_WORKER.format(root=ROOT, tmp=str(tmp_path)))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29635", str(script)]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert res.returncode == 0, res.stdout + res.stderr
    assert res.stdout.count("ok") == 2


def test_connect_symmetric_against_a_stand_in_for_symmetric_memory():
    """`connect_symmetric` in the order that keeps it safe: allocate, rendezvous over the right
    group, clear the buffer, barrier (nobody stores before everybody has cleared), and only then
    hand the peers' addresses to the library, in rank order."""
    import torch
    from paper_2502_06833_b200 import binding, vocab_parallel as VP

    log = []

    class Engine:
        EAD_SHARD_RECORD_BYTES = 32
        ead_shard_range = staticmethod(binding.ead_shard_range)

        def ead_shard_exchange_bytes(self, B, n):
            return 2 * n * B * 32

        def ead_create(self, **kw):
            return 1

        def ead_shard_connect(self, ctx, shard, exchange):
            log.append(("connect", shard, list(exchange), bool((buffers[0] == 0).all())))

        def ead_destroy(self, ctx):
            pass

    buffers = []

    class Handle:
        buffer_ptrs = [0x1000, 0x2000, 0x3000]

    class Symm:
        @staticmethod
        def empty(n, dtype, device):
            log.append(("empty", n, dtype, str(device)))
            buffers.append(torch.full((n,), 255, dtype=dtype))
            return buffers[-1]

        @staticmethod
        def rendezvous(buf, group):
            log.append(("rendezvous", buf is buffers[-1], group))
            return Handle

    class Dist:
        class group:
            WORLD = "world-group"

        @staticmethod
        def barrier(group=None):
            log.append(("barrier", group, bool((buffers[0] == 0).all())))

    W = torch.zeros((384, 8))
    gate = VP.VocabParallelGate(B=4, V_small=1100, V_large=1100, H_small=8, H_large=8, w=5, d_min=10, tau=1.0,
                                W_small=W[:384], W_large=W[:384], rank=1, world=3, group="sub-group",
                                engine=Engine(), dist=Dist, device=torch.device("cpu"))
    gate.connect_symmetric(symm=Symm)
    assert [e[0] for e in log] == ["empty", "rendezvous", "barrier", "connect"]
    assert log[0][1] == 2 * 3 * 4 * 32 and log[0][2] == torch.uint8
    assert log[1] == ("rendezvous", True, "sub-group")
    assert log[2] == ("barrier", "sub-group", True)                 # cleared before the barrier
    assert log[3] == ("connect", 1, [0x1000, 0x2000, 0x3000], True)
    assert gate.connected
    log.clear()
    gate2 = VP.VocabParallelGate(B=4, V_small=1100, V_large=1100, H_small=8, H_large=8, w=5, d_min=10, tau=1.0,
                                 W_small=W[:384], W_large=W[:384], rank=0, world=3, engine=Engine(), dist=Dist,
                                 device=torch.device("cpu"))
    gate2.connect_symmetric(symm=Symm)
    assert log[1][2] == "world-group" and log[2][1] is None         # default group
