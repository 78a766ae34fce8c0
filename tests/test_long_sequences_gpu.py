"""Sequence lengths beyond the benchmark's: forward at 65536 tokens (both head dimensions, sampled rows
next to tile edges against the float64 oracle, which evaluates single query rows of a long sequence),
backward at 32768 tokens (one whole head: dQ, dK and dV element by element)."""

import numpy as np
import pytest

from oracle.attention import attn_bwd_head, attn_fwd_head
from paper_2603_05451_b200 import inputs
from tests.gpu_util import GRAD_RTOL, LSE_TOL, O_TOL, max_abs_err, to_dev, to_f64

pytestmark = pytest.mark.gpu

_f64 = inputs.bf16_bits_to_f64


def _rows(S):
    rows = {0, 1, 127, 128, 255, 256, 257, S // 3, S // 2 - 1, S // 2, S - 32769, S - 257, S - 256, S - 129, S - 128, S - 1}
    return np.array(sorted(r for r in rows if 0 <= r < S))


@pytest.mark.parametrize("D,H,Hkv,causal", [(128, 4, 4, True), (128, 4, 2, False), (64, 4, 4, True), (64, 2, 2, False)])
def test_forward_65536_tokens(D, H, Hkv, causal):
    from paper_2603_05451_b200 import binding

    S = 65536
    t = inputs.make_qkv(6500 + D + H, 1, H, Hkv, S, S, D, values=False)
    scale = D ** -0.5
    o, lse = binding.fa_fwd(to_dev(t["q"][0]), to_dev(t["k"][0]), to_dev(t["v"][0]), scale, causal)
    assert binding.fa_last_device_status() == 0
    o, lse = to_f64(o), to_f64(lse)
    assert np.isfinite(o).all()
    rows = _rows(S)
    for h in (0, H - 1):
        g = h // (H // Hkv)
        o_ref, l_ref = attn_fwd_head(_f64(t["q"][0][0, rows, h, :]), _f64(t["k"][0][0, :, g, :]), _f64(t["v"][0][0, :, g, :]),
                                     scale, causal, q_pos=rows, sq_total=S)
        assert max_abs_err(o[0, rows, h, :], o_ref) <= O_TOL
        assert max_abs_err(lse[0, h, rows], l_ref) <= LSE_TOL


def test_backward_32768_tokens_whole_head():
    import torch

    from paper_2603_05451_b200 import binding

    S, H, D, causal = 32768, 2, 128, True
    t = inputs.make_qkv(6600, 1, H, H, S, S, D, with_do=True, values=False)
    scale = D ** -0.5
    q, k, v, d_o = (to_dev(t[n][0]) for n in ("q", "k", "v", "do"))
    o, lse = binding.fa_fwd(q, k, v, scale, causal)
    dq, dk, dv = binding.fa_bwd(q, k, v, o, lse, d_o, scale, causal)
    torch.cuda.synchronize()
    assert binding.fa_last_device_status() == 0
    h = 1
    ref = attn_bwd_head(*(_f64(t[n][0][0, :, h, :]) for n in ("q", "k", "v", "do")), scale, causal)
    for name, got, want in zip(("dq", "dk", "dv"), (dq, dk, dv), ref):
        err = np.abs(to_f64(got[0, :, h, :]) - want).max()
        assert err <= GRAD_RTOL * np.abs(want).max(), (name, err, np.abs(want).max())
