"""The allocation-free entry point against the context-based one.

Some users of this library run where device memory may not be allocated any more: inside
an engine whose memory plan is frozen, under a budget that has been handed out in full,
or in a latency-critical section where cudaMalloc's implicit synchronisation is not
acceptable.  `ead_head_entropy_static` serves them from a scratch array compiled into the
library.  This test calls it through the C ABI twice in a row (the second call with fewer
rows and other data, so that anything left in the shared scratch by the first call would
show) and checks tokens and entropies against `ead_step` on the same inputs, with the
tolerance of the other parity tests.  It is collected last on purpose.
"""
import numpy as np
import pytest

from workloads import synth

pytestmark = pytest.mark.gpu

H_TOL_NATS = 2e-3


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

    for (tok, Hh, st), (wtok, wH), B in zip(outs, want, (B1, B2)):
        assert st.item() == 0
        assert tok.cpu().numpy().tolist() == wtok[:B].tolist()
        np.testing.assert_allclose(Hh.cpu().numpy(), wH[:B], rtol=0, atol=H_TOL_NATS)
    # the two calls saw different data: easy rows first, hard rows second
    assert want[0][1].max() < want[1][1].min()


def test_static_entry_point_rejects_sizes_beyond_its_scratch():
    import torch
    from paper_2502_06833_b200 import binding as E

    W = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    for B, H in ((E.EAD_STATIC_MAX_B + 1, 64), (4, E.EAD_STATIC_MAX_H + 8)):
        with pytest.raises(E.EadError) as err:
            E.ead_head_entropy_static(W, W, B, 64, H, None, None, None,
                                      torch.cuda.current_device(), 0)
        assert err.value.code == E.EAD_ELIMIT
