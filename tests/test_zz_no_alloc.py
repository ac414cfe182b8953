"""The allocation-free entry point against the context-based one.

Some users of this library run where device memory may not be allocated any more: inside
an engine whose memory plan is frozen, under a budget that has been handed out in full,
or in a latency-critical section where cudaMalloc's implicit synchronisation is not
acceptable.  `ead_head_entropy_static` serves them from a scratch array compiled into the
library.  This test calls it through the C ABI twice in a row (the second call with fewer
rows and other data, so that anything left in the shared scratch by the first call would
show) and checks tokens and entropies against `ead_step` on the same inputs and against the
CPU oracle, with the tolerance of the other parity tests; further cases run it at the limits
its scratch array is sized for.  It is collected last on purpose.
"""
import numpy as np
import pytest

from oracle import ead_oracle as O
from workloads import synth

pytestmark = pytest.mark.gpu

H_TOL_NATS = 2e-3
GAP_TIE = 1e-3


def _oracle_rows(Wb, hb):
    """Entropy (nats), greedy token and top-2 logit gap of every row by the CPU oracle."""
    out = []
    for row in hb:
        z = O.logits(Wb, row)
        tok, gap = O.greedy(z)
        out.append((O.entropy(z), tok, gap))
    return out


def _check_against_oracle(tok, Hh, want):
    tok, Hh = tok.cpu().numpy(), Hh.cpu().numpy()
    for b, (H_o, tok_o, gap) in enumerate(want):
        assert abs(float(Hh[b]) - H_o) <= H_TOL_NATS, (b, Hh[b], H_o)
        assert tok[b] == tok_o or gap < GAP_TIE, (b, tok[b], tok_o, gap)


def _bf16(bits):
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def test_static_entry_point_matches_ead_step_twice():
    import torch
    from paper_2502_06833_b200 import binding as E

    V, H, B1, B2 = 5000, 256, 5, 3            # ragged vocabulary tail, two batch sizes
    Wb = synth.lm_head(31, 0, V, H)
    rng = np.random.default_rng(31)
    h1 = synth.f32_to_bf16_bits((3.0 * rng.normal(0, 1, (B1, H))).astype(np.float32))
    h2 = synth.f32_to_bf16_bits((0.2 * rng.normal(0, 1, (B1, H))).astype(np.float32))
    W = _bf16(Wb)
    d1, d2 = _bf16(h1), _bf16(h2)
    stream = torch.cuda.current_stream().cuda_stream
    dev = torch.cuda.current_device()

    # existing entry point: a fresh context keeps every row on the small head for d_min steps
    ctx = E.ead_create(B=B1, V=V, H_small=H, H_large=H, w=5, d_min=10, tau=2.0, W_small=W,
                       W_large=W, device=dev, stream=stream)
    want = []
    for d in (d1, d2):
        tok = torch.full((B1,), -7, dtype=torch.int32, device="cuda")
        Hh = torch.full((B1,), -7.0, dtype=torch.float32, device="cuda")
        used = torch.full((B1,), 9, dtype=torch.uint8, device="cuda")
        E.ead_step(ctx, d, d, tok, Hh, None, used, None)
        E.ead_status(ctx)
        assert used.cpu().tolist() == [0] * B1
        want.append((tok.cpu().numpy(), Hh.cpu().numpy()))
    E.ead_destroy(ctx)

    # new entry point: outputs are allocated up front, then two calls in a row
    outs = [(torch.full((B,), -7, dtype=torch.int32, device="cuda"),
             torch.full((B,), -7.0, dtype=torch.float32, device="cuda"),
             torch.full((1,), 99, dtype=torch.int32, device="cuda")) for B in (B1, B2)]
    E.ead_head_entropy_static(W, d1, B1, V, H, outs[0][0], outs[0][1], outs[0][2], dev, stream)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    E.ead_head_entropy_static(W, d2, B2, V, H, outs[1][0], outs[1][1], outs[1][2], dev, stream)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before      # nothing was allocated by the call

    for (tok, Hh, st), (wtok, wH), B, hb in zip(outs, want, (B1, B2), (h1, h2)):
        assert st.item() == 0
        assert tok.cpu().numpy().tolist() == wtok[:B].tolist()
        np.testing.assert_allclose(Hh.cpu().numpy(), wH[:B], rtol=0, atol=H_TOL_NATS)
        _check_against_oracle(tok, Hh, _oracle_rows(Wb, hb[:B]))
    # the two calls saw different data: easy rows first, hard rows second
    assert want[0][1].max() < want[1][1].min()


@pytest.mark.parametrize("B,V,H", [
    (128, 3000, 256),      # the largest batch: every row of the padded operand is a real one
    (4, 2100, 8192),       # the longest hidden row: the staged rows fill the scratch array's width
    (128, 700, 8192),      # both at once: the scratch layout at its tightest
    (20, 40000, 200),      # full 256-column weight tiles and a hidden size that is no multiple of 64
])
def test_static_entry_point_at_its_limits_matches_the_oracle(B, V, H):
    """Two calls in a row at the sizes the built-in scratch is dimensioned for, the second on
    other data and fewer rows; both against the CPU oracle."""
    import torch
    from paper_2502_06833_b200 import binding as E

    Wb = synth.lm_head(77, 0, V, H)
    rng = np.random.default_rng(B * 1000003 + H)
    hA = synth.f32_to_bf16_bits((3.0 * rng.normal(0, 1, (B, H))).astype(np.float32))
    B2 = max(1, B - 3)
    hB = synth.f32_to_bf16_bits((1.0 * rng.normal(0, 1, (B2, H))).astype(np.float32))
    W = _bf16(Wb)
    stream = torch.cuda.current_stream().cuda_stream
    dev = torch.cuda.current_device()
    results = []
    for hb in (hA, hB):
        n = hb.shape[0]
        tok = torch.full((n,), -7, dtype=torch.int32, device="cuda")
        Hh = torch.full((n,), -7.0, dtype=torch.float32, device="cuda")
        st = torch.full((1,), 99, dtype=torch.int32, device="cuda")
        d = _bf16(hb)
        E.ead_head_entropy_static(W, d, n, V, H, tok, Hh, st, dev, stream)
        results.append((tok, Hh, st, hb, d))
    torch.cuda.synchronize()
    rows = np.unique(np.linspace(0, B2 - 1, 12).astype(int))           # a sample keeps the oracle quick
    for tok, Hh, st, hb, _ in results:
        assert st.item() == 0
        want = _oracle_rows(Wb, hb[rows])
        _check_against_oracle(tok[rows], Hh[rows], want)
        assert (Hh.cpu().numpy() >= 0).all() and (tok.cpu().numpy() >= 0).all() and tok.max().item() < V


def test_static_entry_point_rejects_sizes_beyond_its_scratch():
    import torch
    from paper_2502_06833_b200 import binding as E

    W = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    for B, H in ((E.EAD_STATIC_MAX_B + 1, 64), (4, E.EAD_STATIC_MAX_H + 8)):
        with pytest.raises(E.EadError) as err:
            E.ead_head_entropy_static(W, W, B, 64, H, None, None, None,
                                      torch.cuda.current_device(), 0)
        assert err.value.code == E.EAD_ELIMIT
