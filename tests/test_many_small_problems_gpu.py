"""Large batches of short sequences: tens of thousands of thread blocks with one or two key blocks each
(forward and backward), a few (batch, head) slices against the float64 oracle."""

import numpy as np
import pytest

from oracle.attention import attn_bwd_head, attn_fwd_head
from paper_2603_05451_b200 import inputs
from tests.gpu_util import GRAD_RTOL, LSE_TOL, O_TOL, max_abs_err, to_dev, to_f64

pytestmark = pytest.mark.gpu

_f64 = inputs.bf16_bits_to_f64


@pytest.mark.parametrize("B,H,Hkv,S,D,causal", [(700, 12, 4, 150, 128, True), (1024, 16, 16, 64, 64, False),
                                                (333, 8, 8, 257, 64, True), (2000, 4, 1, 129, 128, False)])
def test_many_short_sequences(B, H, Hkv, S, D, causal):
    import torch

    from paper_2603_05451_b200 import binding

    t = inputs.make_qkv(7700 + S, B, H, Hkv, S, S, D, with_do=True, values=False)
    scale = D ** -0.5
    q, k, v, d_o = (to_dev(t[n][0]) for n in ("q", "k", "v", "do"))
    o, lse = binding.fa_fwd(q, k, v, scale, causal)
    dq, dk, dv = binding.fa_bwd(q, k, v, o, lse, d_o, scale, causal)
    torch.cuda.synchronize()
    assert binding.fa_last_device_status() == 0
    group = H // Hkv
    for b, g in ((0, 0), (B // 2, Hkv // 2), (B - 1, Hkv - 1)):
        kh, vh = _f64(t["k"][0][b, :, g, :]), _f64(t["v"][0][b, :, g, :])
        dk_ref, dv_ref = np.zeros_like(kh), np.zeros_like(vh)
        for h in range(g * group, (g + 1) * group):  # dK and dV of a key/value head sum over its query heads
            qh, doh = _f64(t["q"][0][b, :, h, :]), _f64(t["do"][0][b, :, h, :])
            o_ref, l_ref = attn_fwd_head(qh, kh, vh, scale, causal)
            assert max_abs_err(to_f64(o[b, :, h, :]), o_ref) <= O_TOL
            assert max_abs_err(to_f64(lse[b, h, :]), l_ref) <= LSE_TOL
            dq_ref, dk_h, dv_h = attn_bwd_head(qh, kh, vh, doh, scale, causal)
            dk_ref += dk_h
            dv_ref += dv_h
            assert np.abs(to_f64(dq[b, :, h, :]) - dq_ref).max() <= GRAD_RTOL * np.abs(dq_ref).max()
        assert np.abs(to_f64(dk[b, :, g, :]) - dk_ref).max() <= GRAD_RTOL * np.abs(dk_ref).max()
        assert np.abs(to_f64(dv[b, :, g, :]) - dv_ref).max() <= GRAD_RTOL * np.abs(dv_ref).max()
