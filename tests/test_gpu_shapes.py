"""Parity with the oracle on small shapes that span several tiles, ragged tails, several
row blocks and both heads in one step; and the properties that hold at any size."""
import math

import numpy as np
import pytest

from oracle import ead_oracle as O
from workloads import synth
from workloads.configs import EADConfig

from gpu_util import GpuGate, compare

pytestmark = pytest.mark.gpu


def _cfg(**kw):
    base = dict(name="case", B=4, T=24, H_small=64, H_large=128, V=1000, tau=5.2, w=3, d_min=2,
                seed=7, stay_easy=0.8, stay_hard=0.8)
    base.update(kw)
    return EADConfig(**base)


def _oracle(cfg, wl, rows=None, T=None):
    return O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, w=cfg.w, d_min=cfg.d_min,
                 tau=float(np.float32(cfg.tau)), unit=cfg.unit, start_model=cfg.start_model,
                 rows=rows, T=T)


def _mid_tau(V):
    """A threshold between the entropy modes of the generator for vocabulary size V."""
    return 0.5 * (math.log(V) + (math.log(V) - 4.5))


SHAPES = [
    # B, V, H_small, H_large        what it exercises
    (1, 1000, 64, 128),           # single row, V not a multiple of 16
    (3, 257, 72, 200),            # tiny ragged V, hidden sizes that are not multiples of 64
    (5, 4100, 256, 512),          # ragged tail after full 256-wide tiles
    (37, 16, 8, 16),              # fewer vocabulary units than CTAs, smallest hidden sizes
    (8, 40000, 128, 64),          # several 256-wide tiles per CTA; large head narrower than small
    (130, 3000, 64, 128),         # two row blocks, the second with 2 rows
    (300, 5000, 128, 256),        # three row blocks shared by both heads
    (150, 2000, 64, 128),         # one pair block per head, the second CTA of each pair mostly without rows
    (256, 2500, 128, 64),         # both heads together fill exactly one pair block
    (520, 1500, 64, 64),          # up to three pair blocks on one head, ragged last vocabulary tile
    (700, 9000, 192, 320),        # full 256-wide tiles, hidden sizes that are multiples of 64
    (300, 700, 64, 3072),         # large head long enough for two-block units: one unit of two blocks + a short third
    (520, 1100, 3072, 3136),      # both heads in two-block units, up to four blocks on a head, ragged last tile
    (200, 600, 3072, 64),         # the small head in two-block units (one unit: 128 rows + the rest)
    (128, 2048, 64, 64),          # exactly one full row block
    (100, 2300, 128, 64),         # four chunks of sequences in the 17..128 variant, the last ragged
    (17, 700, 64, 128),           # smallest batch of that variant
]


@pytest.mark.parametrize("B,V,Hs,Hl", SHAPES)
def test_small_shapes_full_parity(B, V, Hs, Hl):
    cfg = _cfg(B=B, V=V, H_small=Hs, H_large=Hl, tau=_mid_tau(V), T=20 if B > 64 else 28)
    wl = synth.Workload(cfg)
    ora = _oracle(cfg, wl)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        out = g.run(wl.h_small, wl.h_large, "run")
    log = compare(out, ora, cfg.tau)
    assert log["cells"] >= 0.9 * cfg.B * cfg.T
    if V > 16:
        assert 0.02 < out["used"].mean() < 0.98, "the case should exercise both heads"


@pytest.mark.parametrize("w,d_min,start", [(1, 1, 0), (1, 0, 1), (20, 10, 0), (5, 3, 1), (64, 1, 0)])
def test_window_and_dwell_variants(w, d_min, start):
    cfg = _cfg(B=6, V=1500, T=48, w=w, d_min=d_min, start_model=start, tau=_mid_tau(1500))
    wl = synth.Workload(cfg)
    ora = _oracle(cfg, wl)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        out = g.run(wl.h_small, wl.h_large, "run")
    compare(out, ora, cfg.tau)


def test_bits_convention_gives_the_nats_switch_trace():
    cfg = _cfg(B=5, V=2000, T=40, tau=_mid_tau(2000))
    wl = synth.Workload(cfg)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        nats = g.run(wl.h_small, wl.h_large, "run")
    cfg_b = cfg.with_(unit=1, tau=cfg.tau / math.log(2.0))
    ora_b = _oracle(cfg_b, wl)
    with GpuGate(cfg_b, wl.W_small, wl.W_large) as g:
        bits = g.run(wl.h_small, wl.h_large, "run")
    compare(bits, ora_b, cfg_b.tau, unit=1)
    assert np.array_equal(bits["used"], nats["used"]) and np.array_equal(bits["tok"], nats["tok"])
    np.testing.assert_allclose(bits["H"], nats["H"] / math.log(2.0), rtol=2e-6)


def test_step_run_and_host_entry_points_agree_bit_for_bit():
    cfg = _cfg(B=9, V=3000, T=70, tau=_mid_tau(3000))        # 70 = 2 graph chunks of 32 + 6 single steps
    wl = synth.Workload(cfg)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        a = g.run(wl.h_small, wl.h_large, "run")
        g.E.ead_reset(g.ctx)
        b = g.run(wl.h_small, wl.h_large, "step")
        g.E.ead_reset(g.ctx)
        c = g.run(wl.h_small, wl.h_large, "host")
        g.E.ead_reset(g.ctx)
        d1 = g.run(wl.h_small[:33], wl.h_large[:33], "run")      # a run continues where the last ended
        d2 = g.run(wl.h_small[33:], wl.h_large[33:], "run")
    for k in ("tok", "H", "Hbar", "used", "next"):
        assert np.array_equal(a[k], b[k]), k
        assert np.array_equal(a[k], c[k]), k
        assert np.array_equal(a[k], np.concatenate([d1[k], d2[k]])), k
    assert 0.05 < a["used"].mean() < 0.95


def test_checkpoint_and_resume():
    cfg = _cfg(B=7, V=1200, T=40, tau=_mid_tau(1200))
    wl = synth.Workload(cfg)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        full = g.run(wl.h_small, wl.h_large, "run")
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        g.run(wl.h_small[:17], wl.h_large[:17], "run")
        blob = g.E.ead_get_state(g.ctx)
        assert len(blob) == g.E.ead_state_size(g.ctx)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        g.E.ead_set_state(g.ctx, blob)
        rest = g.run(wl.h_small[17:], wl.h_large[17:], "run")
        with pytest.raises(g.E.EadError) as err:
            g.E.ead_set_state(g.ctx, blob[:-4])
        assert err.value.code == g.E.EAD_ESTATE
        # a damaged blob: a negative window fill count or dwell counter would index outside the
        # row's window on the device; it must be refused and leave the context as it was
        pad = (4 - cfg.B % 4) % 4
        off_c = 16 + 2 * (cfg.B + pad)
        for off in (off_c + 4 * 2, off_c + 4 * cfg.B + 4 * 3):          # c[2], nfill[3]
            bad = bytearray(blob)
            bad[off:off + 4] = np.int32(-1).tobytes()
            with pytest.raises(g.E.EadError) as err:
                g.E.ead_set_state(g.ctx, bytes(bad))
            assert err.value.code == g.E.EAD_ESTATE
        assert g.E.ead_get_state(g.ctx)[16:] != blob[16:]                # the rest of the run moved it on
    for k in ("tok", "H", "Hbar", "used", "next"):
        assert np.array_equal(full[k][17:], rest[k]), k


def test_rows_are_independent_and_permutation_equivariant():
    cfg = _cfg(B=12, V=2500, T=30, tau=_mid_tau(2500))
    wl = synth.Workload(cfg)
    perm = np.random.default_rng(3).permutation(cfg.B)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        a = g.run(wl.h_small, wl.h_large, "run")
        g.E.ead_reset(g.ctx)
        b = g.run(wl.h_small[:, perm], wl.h_large[:, perm], "run")
    for k in ("tok", "used", "next"):
        assert np.array_equal(a[k][:, perm], b[k]), k
    # the compacted position of a row changes with the batch around it, the arithmetic per row does not
    np.testing.assert_array_equal(a["H"][:, perm], b["H"])
    sub = cfg.with_(B=5)
    with GpuGate(sub, wl.W_small, wl.W_large) as g:
        c = g.run(wl.h_small[:, :5], wl.h_large[:, :5], "run")
    assert np.array_equal(c["tok"], a["tok"][:, :5]) and np.array_equal(c["used"], a["used"][:, :5])
    np.testing.assert_allclose(c["H"], a["H"][:, :5], atol=1e-5)


def test_non_finite_hidden_state_is_reported_and_leaves_the_row_untouched():
    cfg = _cfg(B=4, V=900, T=12, tau=_mid_tau(900))
    wl = synth.Workload(cfg)
    hs, hl = wl.h_small.copy(), wl.h_large.copy()
    hs[5, 2, 3] = 0x7FC0            # bf16 NaN in row 2 at step 5 (both models, whichever is active)
    hl[5, 2, 3] = 0x7FC0
    hs[7, 1, 0] = 0x7F80            # +inf in row 1 at step 7
    hl[7, 1, 0] = 0x7F80
    ora = O.run(wl.W_small, wl.W_large, hs, hl, w=cfg.w, d_min=cfg.d_min,
                tau=float(np.float32(cfg.tau)))
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        E = g.E
        from gpu_util import to_dev_bf16
        import torch
        d_hs, d_hl = to_dev_bf16(hs), to_dev_bf16(hl)
        o = g._outs(cfg.T)
        E.ead_run(g.ctx, cfg.T, d_hs, d_hl, o["tok"], o["H"], o["Hbar"], o["used"], o["next"])
        word = E.ead_status(g.ctx)
        out = g._np(o)
    assert word == E.EAD_STATUS_NONFINITE
    for (t, b) in ((5, 2), (7, 1)):
        assert math.isnan(out["H"][t, b]) and math.isnan(out["Hbar"][t, b]) and out["tok"][t, b] == -1
        assert math.isnan(ora["H"][t, b]) and ora["tok"][t, b] == -1
        assert out["used"][t, b] == out["next"][t, b] == ora["used"][t, b]
    ok = np.isfinite(ora["H"])
    assert np.array_equal(np.isfinite(out["H"]), ok)
    assert np.array_equal(out["tok"], ora["tok"]) and np.array_equal(out["used"], ora["used"])
    assert np.array_equal(out["next"], ora["next"])
    np.testing.assert_allclose(out["H"][ok], ora["H"][ok], atol=2e-3)
    np.testing.assert_allclose(out["Hbar"][ok], ora["Hbar"][ok], atol=2e-3)


def test_closed_forms_on_the_gpu():
    """Uniform logits (zero hidden state) give ln V; a one-hot-like row gives ~0 and its index."""
    V, H = 3000, 64
    cfg = _cfg(B=2, V=V, H_small=H, H_large=H, T=1, tau=99.0)
    W = np.zeros((V, H), dtype=np.float32)
    W[:, 0] = 0.0
    W[1234, 1] = 8.0
    Wb = synth.f32_to_bf16_bits(W)
    h = np.zeros((1, 2, H), dtype=np.float32)
    h[0, 1, 1] = 8.0                                   # row 1: logit 64 at column 1234, 0 elsewhere
    hb = synth.f32_to_bf16_bits(h)
    with GpuGate(cfg, Wb, Wb) as g:
        out = g.run(hb, hb, "run")
    assert out["H"][0, 0] == pytest.approx(math.log(V), abs=1e-5)
    assert out["tok"][0, 0] == 0                       # all equal: lowest index
    assert 0.0 <= out["H"][0, 1] < 1e-6 and out["tok"][0, 1] == 1234


def test_largest_batch_and_zero_steps():
    cfg = _cfg(B=1024, V=600, H_small=16, H_large=8, T=4, tau=_mid_tau(600), d_min=1, w=1)
    wl = synth.Workload(cfg)
    ora = _oracle(cfg, wl)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        g.E.ead_run(g.ctx, 0, 16, 16)                  # T = 0 is a no-op
        out = g.run(wl.h_small, wl.h_large, "run")
    compare(out, ora, cfg.tau)


@pytest.mark.parametrize("Hl", [192, 3072])
@pytest.mark.parametrize("B", [129, 192, 193, 256, 320])
def test_last_row_block_at_the_half_tile_boundary(B, Hl):
    """Every row on the large head, so its last row block has B - 128 (- 128) rows: 1, 64 and 65
    rows straddle the switch between the M = 64 and the M = 128 tile; 256 has no short block,
    320 a 64-row one after two full blocks."""
    cfg = _cfg(B=B, V=2100 if Hl < 1000 else 700, H_small=64, H_large=Hl, T=6 if Hl < 1000 else 3, tau=-1.0,
               start_model=1, d_min=1)
    wl = synth.Workload(cfg)
    ora = _oracle(cfg, wl)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        out = g.run(wl.h_small, wl.h_large, "run")
        again = g.run(wl.h_small, wl.h_large, "step")
    log = compare(out, ora, cfg.tau)
    assert log["cells"] == B * cfg.T and ora["used"].all()
    assert np.array_equal(out["tok"][-1], again["tok"][-1])


@pytest.mark.parametrize("B,V,temp", [(266, 36000, 0.0), (300, 36000, 0.9), (257, 1900, 0.0), (530, 21000, 0.0),
                                      (575, 21000, 1.3), (321, 3000, 0.0), (313, 35991, 0.0), (290, 35991, 1.1)])
def test_short_odd_row_block_rides_along_as_a_thin_block(B, V, temp):
    """Every row on the large head (hidden size 3072: two-block units).  266 / 300 / 257 rows: two
    blocks and a third of 10 / 44 / 1 rows, which the kernel multiplies with the operands swapped
    on tiles of 240 / 208 / 240 columns (whole rounds of tiles at the larger vocabularies, pieces
    only at 1900); 530 and 575 rows: five blocks, the last one a unit of its own beside two
    two-block units (575 sampled); 321: a 65-row third block is too long to ride along; 313 and
    290 rows on a vocabulary that is no multiple of 16: thin blocks of 57 rows (tiles of 192 columns,
    the second thin accumulator starting at tile row 64) and of 34 rows, sampled."""
    cfg = _cfg(B=B, V=V, H_small=64, H_large=3072, T=2, tau=-1.0, start_model=1, d_min=1)
    wl = synth.Workload(cfg)
    seed = 0xABCDEF12345
    ora = O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, w=cfg.w, d_min=cfg.d_min,
                tau=float(np.float32(cfg.tau)), start_model=1, temperature=temp, seed=seed)
    with GpuGate(cfg, wl.W_small, wl.W_large, temperature=temp, seed=seed) as g:
        out = g.run(wl.h_small, wl.h_large, "run")
        G = g.E.ead_launch_info(g.ctx)["ctas"]
        plan = g.E.ead_plan_units(G - 1, G, B, V, True)
    log = compare(out, ora, cfg.tau)
    assert log["cells"] == B * cfg.T and ora["used"].all()
    assert len(log["token_near_ties"]) <= 2
    last = B - (B - 1) // 128 * 128
    assert (plan["thin16"] > 0) == (last <= 64 and (B + 127) // 128 == 3)


def test_thin_block_on_the_small_head_with_the_large_head_idle():
    """The same unit on head 0: every row stays on a small head whose hidden size is long enough
    for two-block units (266 rows: two blocks and a thin one of 10), nothing on the large head."""
    cfg = _cfg(B=266, V=20000, H_small=3072, H_large=64, T=2, tau=99.0, d_min=1)
    wl = synth.Workload(cfg)
    ora = _oracle(cfg, wl)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        out = g.run(wl.h_small, wl.h_large, "run")
    log = compare(out, ora, cfg.tau)
    assert log["cells"] == cfg.B * cfg.T and not ora["used"].any()


def test_a_step_with_every_sequence_ended_computes_nothing_and_keeps_the_state():
    cfg = _cfg(B=150, V=900, T=6, tau=_mid_tau(900))
    wl = synth.Workload(cfg)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        g.run(wl.h_small[:3], wl.h_large[:3], "run")
        before = g.E.ead_get_state(g.ctx)
        g.E.ead_set_done(g.ctx, np.ones(cfg.B, dtype=np.uint8))
        out = g.run(wl.h_small[3:], wl.h_large[3:], "run")
        after = g.E.ead_get_state(g.ctx)
        assert g.E.ead_status(g.ctx) == 0
    assert (out["tok"] == -1).all() and np.isnan(out["H"]).all() and np.isnan(out["Hbar"]).all()
    assert np.array_equal(out["used"], out["next"])
    pad = (4 - cfg.B % 4) % 4
    done_at = 16 + cfg.B + pad
    # everything but the step count and the done mask is as before
    assert before[16:done_at] == after[16:done_at] and before[done_at + cfg.B + pad:] == after[done_at + cfg.B + pad:]
    assert after[done_at:done_at + cfg.B] == bytes([1]) * cfg.B


def test_maximum_batch_of_the_interface():
    """B = 4096, the largest batch ead_create takes: 32 row blocks over both heads, four or
    five CTAs per row block."""
    cfg = _cfg(B=4096, V=700, H_small=16, H_large=8, T=3, tau=_mid_tau(700), d_min=1, w=2)
    wl = synth.Workload(cfg)
    ora = _oracle(cfg, wl)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        out = g.run(wl.h_small, wl.h_large, "run")
    compare(out, ora, cfg.tau)
    assert 0 < ora["used"].mean() < 1


def test_vocabulary_of_thousands_of_tiles():
    """A vocabulary twice the size of the largest configuration's (narrow heads keep it cheap):
    every CTA walks many tiles, the last one ragged."""
    cfg = _cfg(B=2, V=300007, H_small=8, H_large=16, T=3, tau=_mid_tau(300007), d_min=1)
    wl = synth.Workload(cfg)
    ora = _oracle(cfg, wl)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        out = g.run(wl.h_small, wl.h_large, "run")
    compare(out, ora, cfg.tau)
    assert out["tok"].max() > 2 ** 17


def test_usage_counters_follow_the_trace_and_survive_a_checkpoint():
    cfg = _cfg(B=6, V=1500, T=40, tau=_mid_tau(1500))
    wl = synth.Workload(cfg)
    ora = _oracle(cfg, wl)
    want = [O.usage(ora["used"][:, b], ora["next"][:, b]) for b in range(cfg.B)]
    per_row = np.zeros((3, cfg.B), dtype=np.uint32)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        g.run(wl.h_small[:25], wl.h_large[:25], "run")
        blob = g.E.ead_get_state(g.ctx)
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        g.E.ead_set_state(g.ctx, blob)
        g.run(wl.h_small[25:], wl.h_large[25:], "run")
        tot = g.E.ead_usage(g.ctx, per_row)
        ratio = g.E.ead_parameter_ratio(tot["tokens_small"], tot["tokens_large"], 1.0, 3.0)
        g.E.ead_reset(g.ctx)
        assert g.E.ead_usage(g.ctx) == dict(tokens_small=0, tokens_large=0, switches=0)
    assert per_row.T.tolist() == [list(w) for w in want]
    assert tot == dict(tokens_small=sum(w[0] for w in want), tokens_large=sum(w[1] for w in want),
                       switches=sum(w[2] for w in want))
    assert tot["tokens_small"] + tot["tokens_large"] == cfg.B * cfg.T
    assert ratio == pytest.approx(O.parameter_ratio(ora["used"].mean(), 1.0, 3.0), rel=1e-12)


@pytest.mark.parametrize("B,V,Hs,Hl,temp", [(3, 1000, 64, 128, 1.0), (1, 4100, 256, 512, 0.7),
                                            (12, 2500, 128, 64, 1.5), (40, 3000, 64, 128, 1.0),
                                            (97, 1100, 64, 128, 1.2), (130, 1700, 64, 64, 0.8),
                                            (290, 800, 64, 3072, 1.1)])
def test_temperature_sampling_matches_the_oracle_draws(B, V, Hs, Hl, temp):
    """Algorithm 1's sampling lines: same Philox stream and Gumbel-max rule on both sides, so
    the drawn tokens must be identical (up to logged near-ties of the perturbed values);
    entropies and switches are those of the greedy run (entropy is taken before temperature)."""
    cfg = _cfg(B=B, V=V, H_small=Hs, H_large=Hl, tau=_mid_tau(V), T=16)
    wl = synth.Workload(cfg)
    seed = 0x1234567890ABCDEF
    ora = O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, w=cfg.w, d_min=cfg.d_min,
                tau=float(np.float32(cfg.tau)), temperature=temp, seed=seed)
    greedy = _oracle(cfg, wl)
    with GpuGate(cfg, wl.W_small, wl.W_large, temperature=temp, seed=seed) as g:
        out = g.run(wl.h_small, wl.h_large, "run")
        g.E.ead_reset(g.ctx)
        again = g.run(wl.h_small, wl.h_large, "step")
    log = compare(out, ora, cfg.tau)
    assert len(log["token_near_ties"]) <= 2
    assert np.array_equal(out["tok"], again["tok"])                # same stream after a reset
    assert (ora["tok"] != greedy["tok"]).mean() > 0.2              # the draws are not the arg max
    assert np.array_equal(out["used"], greedy["used"])
    assert out["tok"].min() >= 0 and out["tok"].max() < V


@pytest.mark.parametrize("B,V", [(6, 1200), (150, 900)])
def test_end_of_sequence_token_and_done_mask(B, V):
    cfg = _cfg(B=B, V=V, T=24, tau=_mid_tau(V))
    wl = synth.Workload(cfg)
    free = _oracle(cfg, wl)
    toks, counts = np.unique(free["tok"][4:12], return_counts=True)
    eos = int(toks[np.argmax(counts)])                      # ends at least one row mid-run
    ora = O.run(wl.W_small, wl.W_large, wl.h_small, wl.h_large, w=cfg.w, d_min=cfg.d_min,
                tau=float(np.float32(cfg.tau)), eos_token=eos)
    ended = np.isnan(ora["H"][-1])
    assert ended.any() and not ended.all()
    with GpuGate(cfg, wl.W_small, wl.W_large, eos_token=eos) as g:
        out = g.run(wl.h_small, wl.h_large, "run")
        assert np.array_equal(g.E.ead_get_done(g.ctx, B).astype(bool), ended)
        # usage counts generated tokens only: the steps after a row's end are in neither count
        per_row = np.zeros((3, B), dtype=np.uint32)
        tot = g.E.ead_usage(g.ctx, per_row)
        want = [O.usage(ora["used"][:, b], ora["next"][:, b], ora["tok"][:, b]) for b in range(B)]
        assert per_row.T.tolist() == [list(w) for w in want]
        assert tot["tokens_small"] + tot["tokens_large"] == int((ora["tok"] >= 0).sum()) < B * cfg.T
        blob = g.E.ead_get_state(g.ctx)
        # a row marked done by the caller stops as well; reset clears the mask
        g.E.ead_reset(g.ctx)
        assert not g.E.ead_get_done(g.ctx, B).any()
        mask = np.zeros(B, dtype=np.uint8)
        mask[1] = 1
        g.E.ead_set_done(g.ctx, mask)
        one = g.run(wl.h_small[:3], wl.h_large[:3], "run")
    compare(out, ora, cfg.tau)
    assert np.all(one["tok"][:, 1] == -1) and np.all(np.isnan(one["H"][:, 1]))
    assert np.array_equal(one["tok"][:, 0], free["tok"][:3, 0])
    assert len(blob) > 0


@pytest.mark.parametrize("B,Vs,Vl", [(3, 1000, 1700), (40, 2100, 900), (16, 257, 4100)])
def test_different_vocabularies_per_model(B, Vs, Vl):
    cfg = _cfg(B=B, V=Vs, T=20, tau=0.5 * (_mid_tau(Vs) + _mid_tau(Vl)))
    wl = synth.Workload(cfg)
    W_large = synth.lm_head(cfg.seed + 1, 1, Vl, cfg.H_large)
    ora = O.run(wl.W_small, W_large, wl.h_small, wl.h_large, w=cfg.w, d_min=cfg.d_min,
                tau=float(np.float32(cfg.tau)))
    with GpuGate(cfg, wl.W_small, W_large) as g:
        out = g.run(wl.h_small, wl.h_large, "run")
    compare(out, ora, cfg.tau)
    assert 0.02 < out["used"].mean() < 0.98
    assert out["tok"][out["used"] == 0].max() < Vs and out["tok"][out["used"] == 1].max() < Vl


def test_paper_threshold_grid_in_bits():
    """The paper's thresholds (bits, Table 1's tau column) on the tiny workload: usage grows as tau
    falls, tau = 99 never leaves the small model and tau = 0 leaves it after d_min tokens."""
    from workloads import configs
    cfg0 = configs.TINY.with_(unit=1)
    wl = synth.Workload(cfg0)
    shares = []
    for tau in (99.0, 1.0, 0.5, 0.25, 0.125, 0.0625, 0.03125, 0.0):
        cfg = cfg0.with_(tau=tau)
        with GpuGate(cfg, wl.W_small, wl.W_large) as g:
            out = g.run(wl.h_small, wl.h_large, "run")
            use = g.E.ead_usage(g.ctx)
        shares.append(use["tokens_large"] / (use["tokens_small"] + use["tokens_large"]))
        assert out["used"].mean() == pytest.approx(shares[-1])
    assert shares[0] == 0.0 and shares[-1] == pytest.approx((cfg0.T - 10) / cfg0.T)
    assert all(a <= b for a, b in zip(shares, shares[1:]))


def test_two_contexts_of_different_shape_interleaved_on_a_side_stream():
    """Contexts with different pipelines (stage counts, kernels) coexist and do not disturb each
    other; a non-default stream works."""
    import torch
    cfg_a = _cfg(B=3, V=1100, T=12, tau=_mid_tau(1100))
    cfg_b = _cfg(B=140, V=900, H_small=128, H_large=64, T=12, tau=_mid_tau(900), seed=9)
    wa, wb = synth.Workload(cfg_a), synth.Workload(cfg_b)
    oa, ob = _oracle(cfg_a, wa), _oracle(cfg_b, wb)
    side = torch.cuda.Stream()
    with GpuGate(cfg_b, wb.W_small, wb.W_large, stream=side) as gb, GpuGate(cfg_a, wa.W_small, wa.W_large) as ga:
        outs_a, outs_b = [], []
        for t0 in range(0, 12, 4):                       # alternate between the two contexts
            outs_a.append(ga.run(wa.h_small[t0:t0 + 4], wa.h_large[t0:t0 + 4], "run"))
            outs_b.append(gb.run(wb.h_small[t0:t0 + 4], wb.h_large[t0:t0 + 4], "run"))
    cat = lambda outs: {k: np.concatenate([o[k] for o in outs]) for k in outs[0]}
    compare(cat(outs_a), oa, cfg_a.tau)
    compare(cat(outs_b), ob, cfg_b.tau)


def test_host_entry_point_over_several_staging_chunks():
    """ead_run_host stages the hidden states in chunks (64 MB per buffer): a run longer than one
    chunk must give what the device-resident run gives."""
    cfg = _cfg(B=48, V=320, H_small=4096, H_large=4096, T=190, tau=_mid_tau(320), d_min=3)
    wl = synth.Workload(cfg)                             # 48 * 8192 * 2 B = 768 KB per step: 85 steps per chunk
    with GpuGate(cfg, wl.W_small, wl.W_large) as g:
        a = g.run(wl.h_small, wl.h_large, "run")
        g.E.ead_reset(g.ctx)
        b = g.run(wl.h_small, wl.h_large, "host")
    for k in ("tok", "H", "Hbar", "used", "next"):
        assert np.array_equal(a[k], b[k]), k
    ora = _oracle(cfg, wl, T=40)
    compare({k: v[:40] for k, v in a.items()}, ora, cfg.tau)
