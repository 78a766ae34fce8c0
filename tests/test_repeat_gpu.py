"""Repeated launches on the same inputs: no drift, no dependence on what the buffers held before.

Every case calls the forward and the backward 20 times.  Before each call the outputs AND the backward's
workspace are filled with NaN bit patterns, so a kernel that read an output or a workspace cell before
writing it, or skipped a row, shows up as a NaN or as a changed bit.  The forward has no atomics and must
repeat bit for bit (O and LSE); so must dK and dV (accumulated inside one CTA); dQ is summed by
floating-point reductions whose order changes from run to run, so it may move by rounding only.  The first
run of each case is compared with the float64 oracle on one head."""

import numpy as np
import pytest

from oracle.attention import attn_bwd_head, attn_fwd_head
from paper_2603_05451_b200 import inputs
from tests.gpu_util import GRAD_RTOL, LSE_TOL, O_TOL, to_dev, to_f64

pytestmark = pytest.mark.gpu

REPEATS = 20

# (B, H, Hkv, S, D, causal): both forward kernels (one tile per CTA / two tiles per CTA), both head
# dimensions, a ragged length, grouped heads
CASES = [(4, 8, 8, 512, 128, True), (2, 8, 2, 1664, 128, True), (2, 4, 4, 2048, 128, False), (2, 8, 8, 1000, 64, False),
         (1, 8, 4, 4224, 64, True)]


@pytest.mark.parametrize("B,H,Hkv,S,D,causal", CASES)
def test_twenty_repeats_agree(B, H, Hkv, S, D, causal):
    import torch

    from paper_2603_05451_b200 import binding

    t = inputs.make_qkv(9100 + S, B, H, Hkv, S, S, D, with_do=True, values=False)
    q, k, v, d_o = (to_dev(t[n][0]) for n in ("q", "k", "v", "do"))
    scale = D ** -0.5
    nan16 = torch.tensor(0x7FC1, dtype=torch.int32).to(torch.int16).item()

    def poison(x):
        x.view(torch.int16).fill_(nan16) if x.dtype != torch.float32 else x.fill_(float("nan"))

    o, dq, dk, dv = (torch.empty_like(x) for x in (q, q, k, v))
    lse = torch.empty(B, H, S, dtype=torch.float32, device=q.device)
    ws = torch.empty(binding.fa_bwd_workspace_bytes(B, H, Hkv, S, S, D), dtype=torch.uint8, device=q.device)
    first = None
    for rep in range(REPEATS):
        for x in (o, lse, dq, dk, dv):
            poison(x)
        ws.fill_(0xFF)  # every 4 bytes a NaN
        binding.fa_fwd(q, k, v, scale, causal, o=o, lse=lse)
        binding.fa_bwd(q, k, v, o, lse, d_o, scale, causal, dq=dq, dk=dk, dv=dv, workspace=ws)
        torch.cuda.synchronize()
        assert binding.fa_last_device_status() == 0
        got = [x.clone() for x in (o, lse, dq, dk, dv)]
        for x in got:
            assert torch.isfinite(x.float()).all(), rep
        if first is None:
            first = got
            continue
        assert torch.equal(got[0].view(torch.int16), first[0].view(torch.int16)), ("O changed", rep)
        assert torch.equal(got[1], first[1]), ("LSE changed", rep)
        assert torch.equal(got[3].view(torch.int16), first[3].view(torch.int16)), ("dK changed", rep)
        assert torch.equal(got[4].view(torch.int16), first[4].view(torch.int16)), ("dV changed", rep)
        drift = (got[2].float() - first[2].float()).abs().max().item()
        # reduction order only: a few units in the last place of bfloat16 at the largest |dQ|
        assert drift <= 2.0 ** -6 * first[2].float().abs().max().item(), ("dQ drifted", rep, drift)

    b, h = B - 1, H - 1
    g = h // (H // Hkv)
    f64 = inputs.bf16_bits_to_f64
    qh, kh, vh, doh = f64(t["q"][0][b, :, h, :]), f64(t["k"][0][b, :, g, :]), f64(t["v"][0][b, :, g, :]), f64(t["do"][0][b, :, h, :])
    o_ref, l_ref = attn_fwd_head(qh, kh, vh, scale, causal)
    assert np.abs(to_f64(first[0][b, :, h, :]) - o_ref).max() <= O_TOL
    assert np.abs(to_f64(first[1][b, h, :]) - l_ref).max() <= LSE_TOL
    if H == Hkv:  # dK and dV of a shared key/value head sum over its query heads; one head's oracle covers dQ only
        ref = attn_bwd_head(qh, kh, vh, doh, scale, causal)
        for name, x, want in zip(("dq", "dk", "dv"), (first[2], first[3], first[4]), ref):
            err = np.abs(to_f64(x[b, :, h if name == "dq" else g, :]) - want).max()
            assert err <= GRAD_RTOL * np.abs(want).max(), (name, err)
