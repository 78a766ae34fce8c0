"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

Every case launches the full-size problem and compares WHOLE (batch, head) slices with the float64
oracle, element by element, at the literal tolerances (O 2e-2, LSE 1e-3, gradients 5e-2 of the
largest oracle gradient of the tensor).  A head costs the oracle one to fifteen seconds at these
lengths, so a few heads per case are compared whole; on three more heads the rows next to every
tile edge are compared as well."""

import numpy as np
import pytest

from oracle.attention import attn_bwd_head, attn_fwd_head
from paper_2603_05451_b200 import inputs
from tests.gpu_util import GRAD_RTOL, LSE_TOL, O_TOL, max_abs_err, to_dev, to_f64

pytestmark = pytest.mark.gpu

_cache = {}


def _tensors(seed, B, H, Hkv, S, D, mult=1.0, v_mult=None, with_do=False):
    key = (seed, B, H, Hkv, S, D, mult, v_mult, with_do)
    if key not in _cache:
        _cache.clear()  # one full-size set at a time (each is ~0.5 GB on the host)
        _cache[key] = inputs.make_qkv(seed, B, H, Hkv, S, S, D, multiplier=mult, v_multiplier=v_mult, with_do=with_do,
                                      values=False)
    return _cache[key]


def _edge_rows(S):
    """Rows next to tile edges (0, 127, 128, 255, 256, ...) at both ends plus a few in the middle."""
    rows = {0, 1, 127, 128, 129, 255, 256, S // 2 - 1, S // 2, S // 2 + 127, S - 257, S - 256, S - 129, S - 128, S - 2,
            S - 1}
    return np.array(sorted(r for r in rows if 0 <= r < S))


def _f64(bits):
    return inputs.bf16_bits_to_f64(bits)


def _whole_heads(B, H, n):
    """`n` distinct (batch, head) pairs spread over the batch and the heads (first and last included)."""
    picks = [(0, 0), (B - 1, H - 1), (B // 2, H // 3), ((B - 1) // 2, (2 * H) // 3)]
    out = []
    for bh in picks:
        if bh not in out:
            out.append(bh)
    return out[:n]


def _check_forward(seed, B, H, Hkv, S, D, causal, mult=1.0, v_mult=None, n_whole=2, o_rel=0.0):
    """Compares `n_whole` whole heads and the tile-edge rows of three more with the oracle.

    Bound per element of O: O_TOL + o_rel * |oracle O| (o_rel = 0: the literal tolerance)."""
    from paper_2603_05451_b200 import binding

    t = _tensors(seed, B, H, Hkv, S, D, mult, v_mult)
    scale = D ** -0.5
    o, lse = binding.fa_fwd(to_dev(t["q"][0]), to_dev(t["k"][0]), to_dev(t["v"][0]), scale, causal)
    assert binding.fa_last_device_status() == 0
    o = to_f64(o)
    lse = to_f64(lse)
    assert np.isfinite(o).all()
    group = H // Hkv
    worst = {"o": 0.0, "lse": 0.0}

    def compare(b, h, rows):
        g = h // group
        q = _f64(t["q"][0][b, :, h, :] if rows is None else t["q"][0][b, rows, h, :])
        o_ref, l_ref = attn_fwd_head(q, _f64(t["k"][0][b, :, g, :]), _f64(t["v"][0][b, :, g, :]), scale, causal,
                                     q_pos=rows, sq_total=S)
        got_o = o[b, :, h, :] if rows is None else o[b, rows, h, :]
        got_l = lse[b, h, :] if rows is None else lse[b, h, rows]
        excess = np.abs(got_o - o_ref) - o_rel * np.abs(o_ref)
        worst["o"] = max(worst["o"], float(excess.max()))
        worst["lse"] = max(worst["lse"], max_abs_err(got_l, l_ref))

    whole = _whole_heads(B, H, n_whole)
    for b, h in whole:
        compare(b, h, None)
    rows = _edge_rows(S)
    for b, h in [(0, H - 1), (B - 1, 0), (B // 2, H // 2)]:
        if (b, h) not in whole:
            compare(b, h, rows)
    assert worst["o"] <= O_TOL and worst["lse"] <= LSE_TOL, worst
    return worst


@pytest.mark.parametrize("S", [1024, 2048, 4096, 8192, 16384])
def test_config2_forward_noncausal(S):
    _check_forward(2000 + S, 16384 // S, 16, 16, S, 128, False, n_whole=4 if S <= 4096 else 2)


@pytest.mark.parametrize("S", [1024, 2048, 4096, 8192, 16384, 32768])
def test_config3_forward_causal(S):
    n = 4 if S <= 4096 else (2 if S <= 16384 else 1)
    _check_forward(3000 + S, max(1, 16384 // S), 16, 16, S, 128, True, n_whole=n)


@pytest.mark.parametrize("S", [1024, 8192])
def test_config3_forward_causal_gqa(S):
    _check_forward(3500 + S, 16384 // S, 32, 8, S, 128, True, n_whole=3)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("D,H", [(64, 32), (128, 16)])
def test_config4_head_dim_sweep_wide_scores(D, H, causal):
    # Q, K scaled by 3 (row maxima move a lot between blocks, most rows put their weight on one key);
    # V unscaled: four whole heads at the literal tolerances
    _check_forward(4000 + D, 2, H, H, 8192, D, causal, mult=3.0, v_mult=1.0, n_whole=4)
    # Q, K and V scaled by 3: |O| reaches 8..16, where the spacing of bfloat16 is 0.0625, so the output
    # format alone misses 2e-2; half a unit in the last place of the exact value (<= 2^-8 |O|) is allowed
    # on top of the literal tolerance
    _check_forward(4100 + D, 2, H, H, 8192, D, causal, mult=3.0, n_whole=4, o_rel=2.0 ** -8)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("S", [1024, 2048, 4096, 8192, 16384])
def test_config5_backward(S, causal):
    """dQ, dK and dV of whole heads, element by element, O and LSE taken from the GPU forward."""
    import torch

    from paper_2603_05451_b200 import binding

    B, H, D = 16384 // S, 16, 128
    t = _tensors(5000 + S, B, H, H, S, D, with_do=True)
    scale = D ** -0.5
    q, k, v, d_o = (to_dev(t[n][0]) for n in ("q", "k", "v", "do"))
    o, lse = binding.fa_fwd(q, k, v, scale, causal)
    dq, dk, dv = binding.fa_bwd(q, k, v, o, lse, d_o, scale, causal)
    torch.cuda.synchronize()
    assert binding.fa_last_device_status() == 0
    for x in (dq, dk, dv):
        assert torch.isfinite(x.float()).all()
    for b, h in _whole_heads(B, H, 3 if S <= 2048 else (2 if S <= 8192 else 1)):
        qh, kh, vh, doh = (_f64(t[n][0][b, :, h, :]) for n in ("q", "k", "v", "do"))
        ref = attn_bwd_head(qh, kh, vh, doh, scale, causal)
        for name, got, want in zip(("dq", "dk", "dv"), (dq, dk, dv), ref):
            err = np.abs(to_f64(got[b, :, h, :]) - want).max()
            assert err <= GRAD_RTOL * np.abs(want).max(), (name, b, h, err, np.abs(want).max())


@pytest.mark.parametrize("causal", [False, True])
def test_backward_head_dim_64_full_size(causal):
    """The D = 64 shape of the head-dim sweep (32 heads, 8192 tokens, batch 2) through the backward pass:
    whole heads of dQ, dK and dV against the oracle."""
    import torch

    from paper_2603_05451_b200 import binding

    B, H, S, D = 2, 32, 8192, 64
    t = _tensors(6000, B, H, H, S, D, with_do=True)
    scale = D ** -0.5
    q, k, v, d_o = (to_dev(t[n][0]) for n in ("q", "k", "v", "do"))
    o, lse = binding.fa_fwd(q, k, v, scale, causal)
    dq, dk, dv = binding.fa_bwd(q, k, v, o, lse, d_o, scale, causal)
    torch.cuda.synchronize()
    assert binding.fa_last_device_status() == 0
    for b, h in _whole_heads(B, H, 2):
        qh, kh, vh, doh = (_f64(t[n][0][b, :, h, :]) for n in ("q", "k", "v", "do"))
        ref = attn_bwd_head(qh, kh, vh, doh, scale, causal)
        for name, got, want in zip(("dq", "dk", "dv"), (dq, dk, dv), ref):
            err = np.abs(to_f64(got[b, :, h, :]) - want).max()
            assert err <= GRAD_RTOL * np.abs(want).max(), (name, b, h, err, np.abs(want).max())
