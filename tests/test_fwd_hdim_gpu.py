"""Forward parity for head dimensions (192, 128) (Section 5's second forward workload): O and LSE
from fa_fwd_hdim through the C ABI against the float64 oracle, element by element."""

import numpy as np
import pytest

from oracle.attention import attn_fwd, attn_fwd_head
from paper_2603_05451_b200 import inputs
from tests.gpu_util import LSE_TOL, O_TOL, max_abs_err, to_dev, to_f64

pytestmark = pytest.mark.gpu

DQK, DV = 192, 128


def _tensors(seed, B, H, Hkv, Sq, Sk, mult=1.0):
    return {
        "q": inputs.make_tensor(seed, "q", (B, Sq, H, DQK), mult),
        "k": inputs.make_tensor(seed, "k", (B, Sk, Hkv, DQK), mult),
        "v": inputs.make_tensor(seed, "v", (B, Sk, Hkv, DV), 1.0),
    }


def _run(t, causal, scale):
    import torch

    from paper_2603_05451_b200 import binding

    q, k, v = (to_dev(t[n][0]) for n in ("q", "k", "v"))
    o, lse = binding.fa_fwd_hdim(q, k, v, scale, causal)
    torch.cuda.synchronize()
    assert binding.fa_last_device_status() == 0
    return o, lse


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("B,H,Hkv,Sq,Sk", [(1, 1, 1, 128, 128), (1, 2, 1, 256, 256), (2, 2, 2, 333, 333),
                                           (1, 3, 3, 300, 77), (1, 2, 2, 77, 700), (1, 2, 1, 1024, 1024),
                                           (1, 1, 1, 1, 1), (1, 4, 2, 640, 513)])
def test_small_shapes_element_by_element(B, H, Hkv, Sq, Sk, causal):
    t = _tensors(9100 + Sq + Sk, B, H, Hkv, Sq, Sk)
    scale = DQK ** -0.5
    o, lse = _run(t, causal, scale)
    o_ref, lse_ref = attn_fwd(t["q"][1], t["k"][1], t["v"][1], scale, causal)
    assert max_abs_err(to_f64(o), o_ref) <= O_TOL
    assert max_abs_err(to_f64(lse), lse_ref) <= LSE_TOL


def test_wide_scores_many_rescales():
    """Q, K x3: the running maximum moves a lot, the correction path runs often."""
    t = _tensors(9300, 1, 2, 2, 1024, 1024, mult=3.0)
    scale = DQK ** -0.5
    o, lse = _run(t, True, scale)
    o_ref, lse_ref = attn_fwd(t["q"][1], t["k"][1], t["v"][1], scale, True)
    assert np.abs(to_f64(o) - o_ref).max() <= O_TOL
    assert np.abs(to_f64(lse) - lse_ref).max() <= LSE_TOL


@pytest.mark.parametrize("S", [16384])
def test_paper_shape_causal_sampled_rows(S):
    """16 heads, 16384 tokens, causal (the shape the paper times): sampled rows of sampled heads."""
    B, H = 16384 // S, 16
    t = {
        "q": inputs.make_tensor(9400, "q", (B, S, H, DQK), 1.0, values=False),
        "k": inputs.make_tensor(9400, "k", (B, S, H, DQK), 1.0, values=False),
        "v": inputs.make_tensor(9400, "v", (B, S, H, DV), 1.0, values=False),
    }
    scale = DQK ** -0.5
    o, lse = _run(t, True, scale)
    o_np, lse_np = to_f64(o), to_f64(lse)
    rows = np.array([0, 1, 127, 128, 255, 256, 4095, 4096, 8191, S - 129, S - 128, S - 2, S - 1])
    for h in (0, 7, 15):
        q = inputs.bf16_bits_to_f64(t["q"][0][0, rows, h, :])
        k = inputs.bf16_bits_to_f64(t["k"][0][0, :, h, :])
        v = inputs.bf16_bits_to_f64(t["v"][0][0, :, h, :])
        o_ref, lse_ref = attn_fwd_head(q, k, v, scale, True, q_pos=rows, sq_total=S)
        assert np.abs(o_np[0, rows, h, :] - o_ref).max() <= O_TOL
        assert np.abs(lse_np[0, h, rows] - lse_ref).max() <= LSE_TOL


def test_unsupported_pairs_are_refused():
    import torch

    from paper_2603_05451_b200 import binding

    q = torch.zeros((1, 128, 1, 96), dtype=torch.bfloat16, device="cuda")
    v = torch.zeros((1, 128, 1, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.FaError):
        binding.fa_fwd_hdim(q, q.clone(), v)
