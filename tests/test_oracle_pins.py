"""Pins of the CPU oracle against what the paper and the mathematics fix.

Nothing here calls the CUDA path.  Each test checks the oracle against a
closed form, a brute-force evaluation with different arithmetic, a library
routine on a special case, or a hand-worked trace, chosen so that a dropped
term, a wrong sign, index or comparison, or a transposed operand fails one.
"""
import math
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import ead_oracle as O
from workloads import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
LN2 = math.log(2.0)


# ---------------------------------------------------------------- Eq. 1-2
@pytest.mark.parametrize("V", [2, 7, 4096, 128256])
def test_uniform_logits_give_log_V(V):
    for level in (0.0, -3.25, 11.0):
        z = np.full(V, level)
        # plain left-to-right fp64 sums over V terms: error bound V * 2^-53 * ln V
        tol = max(1e-13, V * 2.0 ** -53 * math.log(V))
        assert O.entropy(z) == pytest.approx(math.log(V), abs=tol)
        assert O.entropy(z, unit=1) == pytest.approx(math.log2(V), abs=2 * tol)


@pytest.mark.parametrize("V", [2, 16, 4096])
def test_one_hot_logits_give_zero(V):
    z = np.zeros(V)
    z[V // 3] = 80.0
    assert 0.0 <= O.entropy(z) < 1e-28
    z = np.full(V, -1e300)          # exp underflows to exactly 0: 0 log 0 := 0
    z[V - 1] = 5.0
    assert O.entropy(z) == 0.0


def test_shift_invariance():
    rng = np.random.default_rng(11)
    z = rng.normal(0, 3, 1000)
    H0 = O.entropy(z)
    for c in (50.0, -50.0, 700.0):
        assert O.entropy(z + c) == pytest.approx(H0, abs=1e-11)


@pytest.mark.parametrize("V,a", [(2, 0.3), (10, 2.0), (4096, 6.0), (128256, -4.0)])
def test_two_level_closed_form(V, a):
    """z = (a, 0, ..., 0): p_1 = e^a / (e^a + V - 1), the rest share 1 - p_1."""
    z = np.zeros(V)
    z[0] = a
    p1 = math.exp(a) / (math.exp(a) + V - 1)
    q = (1.0 - p1) / (V - 1)
    H = -p1 * math.log(p1) - (V - 1) * q * math.log(q)
    tol = max(1e-13, V * 2.0 ** -53 * math.log(V))      # V-term plain fp64 sums
    assert O.entropy(z) == pytest.approx(H, abs=tol)
    assert O.entropy(z, unit=1) == pytest.approx(H / LN2, abs=2 * tol)


def test_brute_force_softmax_small_V():
    """Direct exp(l_i) / sum exp(l_j) in extended precision, no max subtraction."""
    rng = np.random.default_rng(5)
    for V in (2, 3, 5, 16):
        for _ in range(20):
            z = rng.normal(0, 2.5, V)
            e = np.exp(z.astype(np.longdouble))
            p = e / e.sum()
            H = float(-(p * np.log(p)).sum())
            Ho, po = O.entropy(z, return_p=True)
            assert Ho == pytest.approx(H, abs=1e-13)
            np.testing.assert_allclose(po, p.astype(np.float64), rtol=1e-13)
            assert abs(po.sum() - 1.0) < 1e-14


def test_matches_library_softmax_entropy():
    rng = np.random.default_rng(6)
    z = rng.normal(0, 3.0, 5000)
    p = scipy.special.softmax(z)
    assert O.entropy(z) == pytest.approx(scipy.stats.entropy(p), rel=1e-12)
    assert O.entropy(z, unit=1) == pytest.approx(scipy.stats.entropy(p, base=2), rel=1e-12)


def test_fused_identity_and_split_merge():
    """-sum p ln p = ln Z - E_p[z]; and partial (m, s, t) triples over any split
    of the vocabulary merge to the unsplit value (what a tiled evaluation relies on)."""
    rng = np.random.default_rng(7)
    z = rng.normal(0, 3.0, 3001)
    H, p = O.entropy(z, return_p=True)
    lnZ = math.log(np.exp(z - z.max()).sum()) + z.max()
    assert H == pytest.approx(lnZ - float((p * z).sum()), abs=1e-12)
    cuts = np.sort(rng.choice(np.arange(1, z.size), 9, replace=False))
    parts = np.split(z, cuts)
    ms = [q.max() for q in parts]
    M = max(ms)
    S = sum(np.exp(q - m).sum() * math.exp(m - M) for q, m in zip(parts, ms))
    Tt = sum((np.exp(q - m) * q).sum() * math.exp(m - M) for q, m in zip(parts, ms))
    assert H == pytest.approx(M + math.log(S) - Tt / S, abs=1e-12)


def test_non_finite_logits_give_nan():
    z = np.zeros(8)
    for bad in (np.nan, np.inf, -np.inf):
        z2 = z.copy()
        z2[3] = bad
        assert math.isnan(O.entropy(z2))
        assert O.greedy(z2)[0] == -1


# ---------------------------------------------------------------- greedy token
def test_greedy_lowest_index_on_ties_and_gap():
    z = np.array([0.0, 3.0, -1.0, 3.0, 2.5])
    tok, gap = O.greedy(z)
    assert tok == 1 and gap == 0.0
    z = np.array([0.0, 3.0, -1.0, 3.5, 2.5])
    tok, gap = O.greedy(z)
    assert tok == 3 and gap == pytest.approx(0.5)
    rng = np.random.default_rng(8)
    for _ in range(50):
        z = rng.integers(-3, 4, 12).astype(np.float64)
        best = max(range(12), key=lambda i: (z[i], -i))
        assert O.greedy(z)[0] == best


# ---------------------------------------------------------------- LM-head projection
def test_logits_exact_on_small_integers():
    """Integers up to 8 are exact in bf16 and their dot products exact in fp64:
    compare with Python integer arithmetic.  V != H and asymmetric data catch a
    transposed or mis-strided operand."""
    rng = np.random.default_rng(9)
    V, H = 37, 24
    Wi = rng.integers(-8, 9, (V, H))
    hi = rng.integers(-8, 9, H)
    Wb = synth.f32_to_bf16_bits(Wi.astype(np.float32))
    hb = synth.f32_to_bf16_bits(hi.astype(np.float32))
    z = O.logits(Wb, hb)
    want = [sum(int(Wi[i, j]) * int(hi[j]) for j in range(H)) for i in range(V)]
    assert z.tolist() == [float(x) for x in want]


def test_logits_match_library_matmul():
    rng = np.random.default_rng(10)
    V, H = 300, 136
    Wb = synth.f32_to_bf16_bits(rng.normal(0, 1, (V, H)).astype(np.float32))
    hb = synth.f32_to_bf16_bits(rng.normal(0, 1, H).astype(np.float32))
    want = synth.bf16_bits_to_f32(Wb).astype(np.float64) @ synth.bf16_bits_to_f32(hb).astype(np.float64)
    np.testing.assert_allclose(O.logits(Wb, hb), want, rtol=0, atol=1e-12)


def test_bf16_round_to_nearest_even():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -7, -2.5, 0.0],
                 dtype=np.float32)
    b = synth.f32_to_bf16_bits(x)
    back = synth.bf16_bits_to_f32(b)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: goes to the even mantissa (1.0);
    # 1 + 3*2^-8 is a tie between 1 + 2^-7 and 1 + 2^-6: goes to 1 + 2^-6.
    assert back.tolist() == [1.0, 1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7, -2.5, 0.0]


@pytest.mark.parametrize("V,H", [(4096, 256), (4096, 512)])
def test_hard_regime_entropy_level(V, H):
    """Logits that are nearly iid N(0, s^2) with small s have H close to
    ln V - s^2 / 2 (second-order expansion of ln sum exp): pins the whole
    chain weights -> logits -> softmax -> entropy on generated inputs."""
    s = 0.2
    W = synth.lm_head(123, 0, V, H)
    rng = np.random.default_rng(3)
    hb = synth.f32_to_bf16_bits((s * rng.normal(0, 1, H)).astype(np.float32))
    z = O.logits(W, hb)
    var = float(np.var(z))
    assert O.entropy(z) == pytest.approx(math.log(V) - var / 2.0, abs=2e-3)
    assert var == pytest.approx(s * s, rel=0.25)


# ---------------------------------------------------------------- window + switch
def _read_traces():
    traces, cur = [], None
    with open(os.path.join(GOLDEN, "gate_traces.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            if k == "trace":
                cur = dict(name=v[0], w=int(v[1]), d_min=int(v[2]), tau=float(v[3]))
                traces.append(cur)
            elif k in ("H", "Hbar"):
                cur[k] = [float(x) for x in v]
            else:
                cur[k] = [0 if x == "S" else 1 for x in v]
    return traces


@pytest.mark.parametrize("tr", _read_traces(), ids=lambda t: t["name"])
def test_hand_worked_switch_traces(tr):
    out = O.gate_trace(tr["H"], tr["w"], tr["d_min"], tr["tau"])
    np.testing.assert_allclose(out["Hbar"], tr["Hbar"], rtol=0, atol=1e-12)
    assert out["used"].tolist() == tr["used"]
    assert out["next"].tolist() == tr["next"]


@pytest.mark.parametrize("T", [64, 2048])
def test_threshold_below_every_entropy(T):
    """Paper defaults w = 5, d_min = 10: small for exactly d_min tokens, then large
    for ever; large share (T - 10) / T.  A threshold above every entropy never
    leaves the small model (the tau = 99 rows of Table 1: 0 % large usage)."""
    rng = np.random.default_rng(2)
    H = rng.uniform(3.0, 12.0, T)
    out = O.gate_trace(H, 5, 10, 2.0)
    assert out["used"].tolist() == [0] * 10 + [1] * (T - 10)
    assert out["used"].mean() == pytest.approx((T - 10) / T)
    out = O.gate_trace(H, 5, 10, 99.0)
    assert out["used"].sum() == 0 and out["next"].sum() == 0
    assert out["c_after"].tolist() == list(range(1, T + 1))


def test_rolling_mean_is_plain_window_mean():
    rng = np.random.default_rng(4)
    H = rng.uniform(0, 10, 40)
    for w in (1, 5, 20):
        out = O.gate_trace(H, w, 10, 5.0)
        want = [H[max(0, t + 1 - w): t + 1].mean() for t in range(40)]
        np.testing.assert_allclose(out["Hbar"], want, rtol=1e-14)


def test_dwell_never_shorter_than_d_min():
    rng = np.random.default_rng(12)
    H = rng.uniform(0, 2, 500)
    for d_min in (1, 3, 10):
        out = O.gate_trace(H, 2, d_min, 1.0)
        used = out["used"]
        runs = np.diff(np.flatnonzero(np.diff(used) != 0))
        assert runs.size > 0 and runs.min() >= d_min


def test_bits_convention_gives_same_switches():
    """Entropy in bits against tau / ln 2 decides exactly as nats against tau."""
    rng = np.random.default_rng(13)
    H = rng.uniform(0, 4, 300)
    a = O.gate_trace(H, 5, 10, 2.0)
    b = O.gate_trace(H / LN2, 5, 10, 2.0 / LN2)
    assert a["used"].tolist() == b["used"].tolist()


# ---------------------------------------------------------------- Algorithm 1 end to end
def _tiny_inputs(T=24, B=3, V=300, Hs=32, Hl=64, seed=77):
    r = synth.regimes(seed, T, B, 0.8, 0.8)
    hs = synth.hidden_states(seed, 0, r, Hs, 3.0, 0.2)
    hl = synth.hidden_states(seed, 1, r, Hl, 3.0, 0.2)
    Ws = synth.lm_head(seed, 0, V, Hs)
    Wl = synth.lm_head(seed, 1, V, Hl)
    return r, Ws, Wl, hs, hl


def test_run_composes_the_pinned_parts():
    """oracle_run = logits of the ACTIVE model only -> entropy -> greedy -> gate,
    per row independently, re-derived here cell by cell from the pinned pieces."""
    r, Ws, Wl, hs, hl = _tiny_inputs()
    T, B = r.shape
    tau = 4.6
    out = O.run(Ws, Wl, hs, hl, w=3, d_min=2, tau=tau)
    assert 0 < out["used"].mean() < 1          # both models really get used
    for b in range(B):
        model, Hs_ = 0, []
        for t in range(T):
            z = O.logits(Ws, hs[t, b]) if model == 0 else O.logits(Wl, hl[t, b])
            assert out["used"][t, b] == model
            assert out["H"][t, b] == O.entropy(z)
            assert out["tok"][t, b] == O.greedy(z)[0]
            Hs_.append(out["H"][t, b])
            g = O.gate_trace(Hs_, 3, 2, tau)
            assert out["Hbar"][t, b] == g["Hbar"][-1]
            model = int(g["next"][-1])
            assert out["next"][t, b] == model


def test_run_rows_are_independent_and_prefix_stable():
    r, Ws, Wl, hs, hl = _tiny_inputs()
    full = O.run(Ws, Wl, hs, hl, w=3, d_min=2, tau=4.6)
    sub = O.run(Ws, Wl, hs, hl, w=3, d_min=2, tau=4.6, rows=[2, 0], T=10)
    for k, b in enumerate([2, 0]):
        for key in ("tok", "H", "Hbar", "used", "next"):
            assert np.array_equal(sub[key][:, k], full[key][:10, b])


def test_run_literal_low_threshold_on_tiny_shapes():
    r, Ws, Wl, hs, hl = _tiny_inputs(T=16)
    out = O.run(Ws, Wl, hs, hl, w=5, d_min=10, tau=0.5)
    assert out["H"].min() > 0.5
    for b in range(r.shape[1]):
        assert out["used"][:, b].tolist() == [0] * 10 + [1] * 6


def test_generator_is_counter_based():
    a = synth.lm_head(5, 1, 5000, 16)
    b = synth.lm_head(5, 1, 2100, 16)
    assert np.array_equal(a[:2100], b)
    r = synth.regimes(5, 40, 6, 0.9, 0.9)
    h40 = synth.hidden_states(5, 0, r, 16, 3.0, 0.2)
    h20 = synth.hidden_states(5, 0, r[:20], 16, 3.0, 0.2)
    assert np.array_equal(h40[:20], h20)
    assert not np.array_equal(synth.lm_head(6, 1, 64, 16), a[:64])


# ---------------------------------------------------------------- usage / parameter ratio
def _read_table1():
    blocks, cur = [], None
    with open(os.path.join(GOLDEN, "table1.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            v = line.split()
            if v[0] == "pair":
                cur = dict(name=v[1], P_small=float(v[3]), P_large=float(v[5]), tol=float(v[7]), rows=[])
                blocks.append(cur)
            else:
                cur["rows"].append(tuple(float(x) for x in v))
    return blocks


@pytest.mark.parametrize("blk", _read_table1(), ids=lambda b: b["name"])
def test_parameter_ratio_reproduces_table_1(blk):
    """The printed parameter-ratio column follows from the printed usage column through the
    footnote's formula (to the rounding of the table; the tolerance per block is stated in the
    fixture).  A swapped alpha/beta or a normalisation by P_S fails every block."""
    assert len(blk["rows"]) == 8
    worst = 0.0
    for tau, usage_pct, _score, ratio_pct in blk["rows"]:
        got = 100.0 * O.parameter_ratio(usage_pct / 100.0, blk["P_small"], blk["P_large"])
        worst = max(worst, abs(got - ratio_pct))
        assert abs(got - ratio_pct) <= blk["tol"], (blk["name"], tau, got, ratio_pct)
    # end points are exact: all-small gives P_S / P_L, all-large gives 1
    assert O.parameter_ratio(0.0, blk["P_small"], blk["P_large"]) == blk["P_small"] / blk["P_large"]
    assert O.parameter_ratio(1.0, blk["P_small"], blk["P_large"]) == 1.0
    assert worst > 0.0 or blk["tol"] >= 0.0


def test_usage_counts_of_hand_traces():
    for tr in _read_traces():
        out = O.gate_trace(tr["H"], tr["w"], tr["d_min"], tr["tau"])
        s, l, sw = O.usage(out["used"], out["next"])
        assert s == tr["used"].count(0) and l == tr["used"].count(1)
        assert sw == sum(1 for u, n in zip(tr["used"], tr["next"]) if u != n)
    # trace D: used SLLLLLSSSSLL, next LLLLLSSSSLLL -> 5 small, 7 large, 3 switches
    tr = [t for t in _read_traces() if t["name"] == "D"][0]
    out = O.gate_trace(tr["H"], tr["w"], tr["d_min"], tr["tau"])
    assert O.usage(out["used"], out["next"]) == (5, 7, 3)


def test_usage_counts_only_generated_tokens():
    """Table 1's usage column is a share of generated tokens, and Algorithm 1 generates none once
    "while not done" has ended.  Hand trace: six steps, used SSLLLL, next SLLLLL, the fourth token
    is the last one (steps five and six report token -1): 2 small tokens, 2 large ones and the
    one switch; without the token trace all six steps count."""
    used, nxt = [0, 0, 1, 1, 1, 1], [0, 1, 1, 1, 1, 1]
    assert O.usage(used, nxt, [5, 7, 2, 9, -1, -1]) == (2, 2, 1)
    assert O.usage(used, nxt) == (2, 4, 1)
    # an ended row reports its frozen model as used = next, so only token counts can differ;
    # a step that produced nothing is no switch either (constructed: next differs on a dead step)
    assert O.usage([0, 0, 0], [0, 0, 1], [3, -1, -1]) == (1, 0, 0)


# ---------------------------------------------------------------- sampling (Algorithm 1, sampling lines)
def test_philox_known_answers():
    """Known-answer vectors of Philox4x32-10 published with the Random123 library."""
    assert O.philox4x32([0, 0, 0, 0], [0, 0]) == [0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8]
    assert O.philox4x32([0xffffffff] * 4, [0xffffffff] * 2) == [0x408f276d, 0x41c83b0e, 0xa20bc7c6,
                                                                 0x6d5451fd]
    assert O.philox4x32([0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344],
                        [0xa4093822, 0x299f31d0]) == [0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1]


def test_uniform_is_an_odd_multiple_of_2_pow_minus_24_and_flat():
    u = np.array([O.uniform(9, 3, 5, i) for i in range(20000)])
    k = u * 2 ** 24
    assert np.all(k == np.round(k)) and np.all(k.astype(np.int64) % 2 == 1)
    assert 0.0 < u.min() and u.max() < 1.0
    assert np.array_equal(u.astype(np.float32).astype(np.float64), u)      # exact in float32
    hist = np.histogram(u, bins=20, range=(0, 1))[0]
    chi2 = ((hist - 1000.0) ** 2 / 1000.0).sum()
    assert chi2 < 50.0                                                     # 19 d.o.f.: p ~ 1e-4
    # different (row, step) give different streams; blocks of 4 indices share one Philox call
    assert O.uniform(9, 3, 5, 0) != O.uniform(9, 3, 6, 0) != O.uniform(9, 4, 5, 0)
    w = O.philox4x32([1, 5, 3, 0], [9, 0])
    assert [O.uniform(9, 3, 5, 4 + j) for j in range(4)] == [(2 * (x >> 9) + 1) / 2 ** 24 for x in w]


def test_sampled_tokens_follow_softmax_of_logits_over_temperature():
    """Draws are distributed as p' = softmax(l / T) (chi-square against the exact p'), and an
    inverse-CDF sampler fed with independent uniforms agrees with that distribution too."""
    rng = np.random.default_rng(21)
    z = rng.normal(0, 1.5, 6)
    for T in (0.5, 1.0, 2.0):
        p = scipy.special.softmax(z / T)
        n = 20000
        counts = np.bincount([O.sample(z, T, 77, 0, step)[0] for step in range(n)], minlength=6)
        chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
        assert chi2 < 25.0, (T, counts, n * p)                            # 5 d.o.f.: p ~ 1e-4
        inv = np.searchsorted(np.cumsum(p), rng.random(n))
        chi2_inv = ((np.bincount(inv, minlength=6) - n * p) ** 2 / (n * p)).sum()
        assert chi2_inv < 25.0
    # temperature -> 0 approaches the arg max; a huge temperature approaches uniform
    cold = [O.sample(z, 1e-3, 5, 0, s)[0] for s in range(200)]
    assert set(cold) == {int(np.argmax(z))}
    hot = np.bincount([O.sample(z, 1e6, 5, 0, s)[0] for s in range(6000)], minlength=6)
    assert hot.min() > 800


def test_sample_is_argmax_of_perturbed_scaled_logits():
    rng = np.random.default_rng(22)
    z = rng.normal(0, 2, 50)
    for step in range(20):
        T = 0.7
        v = z / T - np.log(-np.log([O.uniform(3, 11, step, i) for i in range(50)]))
        tok, gap = O.sample(z, T, 3, 11, step)
        order = np.argsort(-v)
        assert tok == order[0] and gap == pytest.approx(v[order[0]] - v[order[1]], abs=1e-12)


def test_run_with_temperature_keeps_entropy_and_switches_of_the_greedy_run():
    """Entropy is taken before temperature scaling, and hidden states are inputs here, so only
    the token column changes when sampling is switched on."""
    r, Ws, Wl, hs, hl = _tiny_inputs()
    a = O.run(Ws, Wl, hs, hl, w=3, d_min=2, tau=4.6)
    b = O.run(Ws, Wl, hs, hl, w=3, d_min=2, tau=4.6, temperature=1.0, seed=5)
    for k in ("H", "Hbar", "used", "next"):
        assert np.array_equal(a[k], b[k])
    assert (a["tok"] != b["tok"]).mean() > 0.3
    T, B = r.shape
    for t in (0, 7, T - 1):
        for bb in range(B):
            z = O.logits(Ws, hs[t, bb]) if b["used"][t, bb] == 0 else O.logits(Wl, hl[t, bb])
            assert b["tok"][t, bb] == O.sample(z, 1.0, 5, bb, t)[0]


# ---------------------------------------------------------------- "while not done"
def test_end_of_sequence_token_stops_a_row_and_only_that_row():
    r, Ws, Wl, hs, hl = _tiny_inputs()
    full = O.run(Ws, Wl, hs, hl, w=3, d_min=2, tau=4.6)
    T, B = r.shape
    eos = int(full["tok"][6, 1])                      # row 1 emits this token at step 6
    first = [next((t for t in range(T) if full["tok"][t, b] == eos), None) for b in range(B)]
    assert first[1] is not None and first[1] <= 6
    out = O.run(Ws, Wl, hs, hl, w=3, d_min=2, tau=4.6, eos_token=eos)
    for b in range(B):
        stop = T if first[b] is None else first[b] + 1            # the step that emits it is complete
        for k in ("tok", "H", "Hbar", "used", "next", "c_after"):
            assert np.array_equal(out[k][:stop, b], full[k][:stop, b]), (k, b)
        assert np.all(out["tok"][stop:, b] == -1)
        assert np.all(np.isnan(out["H"][stop:, b])) and np.all(np.isnan(out["Hbar"][stop:, b]))
        if stop < T:
            assert np.all(out["used"][stop:, b] == full["next"][stop - 1, b])
            assert np.all(out["next"][stop:, b] == full["next"][stop - 1, b])
            assert np.all(out["c_after"][stop:, b] == full["c_after"][stop - 1, b])


# ---------------------------------------------------------------- two vocabularies
def test_run_with_different_vocabularies_per_model():
    """The models may be of different architectures: each step's logits, entropy and token
    live in the vocabulary of the model that produced them."""
    r, Ws, _, hs, hl = _tiny_inputs(V=300)
    Wl = synth.lm_head(78, 1, 520, hl.shape[2])
    out = O.run(Ws, Wl, hs, hl, w=3, d_min=2, tau=4.9)
    assert 0 < out["used"].mean() < 1
    T, B = r.shape
    for t in range(T):
        for b in range(B):
            if out["used"][t, b] == 0:
                z = O.logits(Ws, hs[t, b])
                assert z.size == 300
            else:
                z = O.logits(Wl, hl[t, b])
                assert z.size == 520
            assert out["H"][t, b] == O.entropy(z) and out["tok"][t, b] == O.greedy(z)[0]
    assert out["tok"][out["used"] == 1].max() >= 300       # tokens beyond the small vocabulary occur
