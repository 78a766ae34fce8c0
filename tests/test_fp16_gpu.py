"""FP16 inputs (fa_fwd_f16, fa_bwd_f16): forward and backward parity against the float64 oracle
on inputs rounded to half precision."""

import numpy as np
import pytest

from oracle.attention import attn_bwd, attn_fwd
from paper_2603_05451_b200 import inputs
from tests.gpu_util import GRAD_RTOL, LSE_TOL, O_TOL, max_abs_err

pytestmark = pytest.mark.gpu


def _half(seed, name, shape, mult=1.0):
    """(float16 array, the same values as float64) from the seeded normal generator."""
    x = inputs.normal_f64(seed, inputs.TENSOR_IDS[name], int(np.prod(shape))) * mult
    h = x.astype(np.float16).reshape(shape)
    return h, h.astype(np.float64)


def _dev(h):
    import torch

    return torch.from_numpy(h).cuda()


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D", [(1, 2, 1, 384, 384, 128), (2, 2, 2, 333, 333, 64), (1, 3, 3, 300, 77, 128),
                                             (1, 2, 2, 1024, 1024, 128), (1, 4, 2, 200, 640, 64)])
def test_forward(B, H, Hkv, Sq, Sk, D, causal):
    import torch

    from paper_2603_05451_b200 import binding

    q, k, v = _half(6100, "q", (B, Sq, H, D)), _half(6100, "k", (B, Sk, Hkv, D)), _half(6100, "v", (B, Sk, Hkv, D))
    scale = D ** -0.5
    o, lse = binding.fa_fwd(_dev(q[0]), _dev(k[0]), _dev(v[0]), scale, causal)
    torch.cuda.synchronize()
    assert binding.fa_last_device_status() == 0 and o.dtype == torch.float16
    o_ref, lse_ref = attn_fwd(q[1], k[1], v[1], scale, causal)
    assert max_abs_err(o.float().cpu().numpy().astype(np.float64), o_ref) <= O_TOL
    assert max_abs_err(lse.cpu().numpy().astype(np.float64), lse_ref) <= LSE_TOL


def test_forward_wide_scores():
    import torch

    from paper_2603_05451_b200 import binding

    B, H, S, D = 1, 2, 1024, 128
    q, k, v = _half(6200, "q", (B, S, H, D), 3.0), _half(6200, "k", (B, S, H, D), 3.0), _half(6200, "v", (B, S, H, D))
    scale = D ** -0.5
    o, lse = binding.fa_fwd(_dev(q[0]), _dev(k[0]), _dev(v[0]), scale, True)
    torch.cuda.synchronize()
    o_ref, lse_ref = attn_fwd(q[1], k[1], v[1], scale, True)
    assert max_abs_err(o.float().cpu().numpy().astype(np.float64), o_ref) <= O_TOL
    assert max_abs_err(lse.cpu().numpy().astype(np.float64), lse_ref) <= LSE_TOL


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D", [(1, 2, 1, 384, 384, 128), (2, 2, 2, 333, 333, 128), (1, 3, 3, 300, 77, 128),
                                             (1, 2, 2, 1024, 1024, 128), (1, 4, 2, 384, 384, 64), (2, 2, 2, 333, 200, 64)])
def test_backward(B, H, Hkv, Sq, Sk, D, causal):
    import torch

    from paper_2603_05451_b200 import binding

    q, k, v = _half(6300, "q", (B, Sq, H, D)), _half(6300, "k", (B, Sk, Hkv, D)), _half(6300, "v", (B, Sk, Hkv, D))
    d_o = _half(6300, "do", (B, Sq, H, D))
    scale = D ** -0.5
    qd, kd, vd, dod = (_dev(t[0]) for t in (q, k, v, d_o))
    o, lse = binding.fa_fwd(qd, kd, vd, scale, causal)
    grads = binding.fa_bwd(qd, kd, vd, o, lse, dod, scale, causal)
    torch.cuda.synchronize()
    assert binding.fa_last_device_status() == 0
    ref = attn_bwd(q[1], k[1], v[1], d_o[1], scale, causal)
    floor = 0.1 * max(np.abs(r).max() for r in ref)
    for name, got, want in zip(("dq", "dk", "dv"), grads, ref):
        g = got.float().cpu().numpy().astype(np.float64)
        assert got.dtype == torch.float16 and np.isfinite(g).all(), name
        assert np.abs(g - want).max() <= GRAD_RTOL * max(np.abs(want).max(), floor), name


@pytest.mark.parametrize("D", [64, 128])
def test_backward_deterministic(D):
    """fa_bwd_deterministic_f16: bit-identical across runs and within tolerance of the oracle."""
    import torch

    from paper_2603_05451_b200 import binding

    B, H, Hkv, Sq, Sk = 1, 4, 2, 700, 520
    q, k, v = _half(6400, "q", (B, Sq, H, D)), _half(6400, "k", (B, Sk, Hkv, D)), _half(6400, "v", (B, Sk, Hkv, D))
    d_o = _half(6400, "do", (B, Sq, H, D))
    scale = D ** -0.5
    qd, kd, vd, dod = (_dev(t[0]) for t in (q, k, v, d_o))
    o, lse = binding.fa_fwd(qd, kd, vd, scale, True)
    runs = [tuple(t.clone() for t in binding.fa_bwd(qd, kd, vd, o, lse, dod, scale, True, deterministic=True))
            for _ in range(3)]
    torch.cuda.synchronize()
    assert binding.fa_last_device_status() == 0
    for r in runs[1:]:
        for a, b in zip(runs[0], r):
            assert torch.equal(a, b)
    ref = attn_bwd(q[1], k[1], v[1], d_o[1], scale, True)
    floor = 0.1 * max(np.abs(r).max() for r in ref)
    for name, got, want in zip(("dq", "dk", "dv"), runs[0], ref):
        g = got.float().cpu().numpy().astype(np.float64)
        assert got.dtype == torch.float16 and np.isfinite(g).all(), name
        assert np.abs(g - want).max() <= GRAD_RTOL * max(np.abs(want).max(), floor), name


@pytest.mark.parametrize("D,H,S,B,causal", [(128, 16, 4096, 4, True), (64, 32, 8192, 2, False)])
def test_benchmark_sized_launch_whole_heads(D, H, S, B, causal):
    """FP16 at a benchmark-sized launch (16384 tokens, hidden size 2048): whole heads of O, LSE, dQ, dK, dV."""
    import torch

    from oracle.attention import attn_bwd_head, attn_fwd_head
    from paper_2603_05451_b200 import binding

    shape = (B, S, H, D)
    q, k, v, d_o = (_half(6400 + D, n, shape) for n in ("q", "k", "v", "do"))
    scale = D ** -0.5
    qd, kd, vd, dod = (_dev(x[0]) for x in (q, k, v, d_o))
    o, lse = binding.fa_fwd(qd, kd, vd, scale, causal)
    dq, dk, dv = binding.fa_bwd(qd, kd, vd, o, lse, dod, scale, causal)
    torch.cuda.synchronize()
    assert binding.fa_last_device_status() == 0 and o.dtype == torch.float16 and dq.dtype == torch.float16
    f64 = lambda x: x.float().cpu().numpy().astype(np.float64)
    for b, h in ((0, 0), (B - 1, H - 1)):
        qh, kh, vh, doh = (x[1][b, :, h, :] for x in (q, k, v, d_o))
        o_ref, l_ref = attn_fwd_head(qh, kh, vh, scale, causal)
        assert max_abs_err(f64(o[b, :, h, :]), o_ref) <= O_TOL
        assert max_abs_err(f64(lse[b, h, :]), l_ref) <= LSE_TOL
        for name, got, want in zip(("dq", "dk", "dv"), (dq, dk, dv), attn_bwd_head(qh, kh, vh, doh, scale, causal)):
            err = np.abs(f64(got[b, :, h, :]) - want).max()
            assert err <= GRAD_RTOL * np.abs(want).max(), (name, err)
