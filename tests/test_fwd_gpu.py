"""Forward parity: the CUDA path (through the C ABI) against the float64 oracle."""

import numpy as np
import pytest

from oracle.attention import attn_fwd, attn_fwd_head
from paper_2603_05451_b200 import inputs
from tests.gpu_util import LSE_TOL, O_TOL, max_abs_err, to_dev, to_f64

pytestmark = pytest.mark.gpu


def _fwd_case(B, H, Hkv, Sq, Sk, D, causal, seed, mult=1.0, v_mult=None, scale=None, o_rel=0.0):
    """Returns (max over elements of |O - oracle| - o_rel * |oracle|, max |LSE - oracle|)."""
    from paper_2603_05451_b200 import binding

    t = inputs.make_qkv(seed, B, H, Hkv, Sq, Sk, D, multiplier=mult, v_multiplier=v_mult)
    scale = D ** -0.5 if scale is None else scale
    o, lse = binding.fa_fwd(to_dev(t["q"][0]), to_dev(t["k"][0]), to_dev(t["v"][0]), scale, causal)
    assert binding.fa_last_device_status() == 0
    o_ref, lse_ref = attn_fwd(t["q"][1], t["k"][1], t["v"][1], scale, causal)
    o = to_f64(o)
    assert not np.isnan(o).any()
    return float((np.abs(o - o_ref) - o_rel * np.abs(o_ref)).max()), max_abs_err(to_f64(lse), lse_ref)


def test_config1_tiny_forward():
    eo, el = _fwd_case(1, 1, 1, 128, 128, 64, False, seed=1000)
    assert eo <= O_TOL and el <= LSE_TOL, (eo, el)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("S", [1, 127, 128, 129, 200, 256, 333, 512, 1024])
def test_square_sizes_with_ragged_tails(S, causal, D):
    eo, el = _fwd_case(2, 2, 2, S, S, D, causal, seed=11 + S)
    assert eo <= O_TOL and el <= LSE_TOL, (eo, el)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("Sq,Sk", [(64, 512), (300, 77), (129, 640), (512, 128), (1, 1000), (700, 1)])
def test_rectangular_and_empty_rows(Sq, Sk, causal, D):
    eo, el = _fwd_case(1, 3, 3, Sq, Sk, D, causal, seed=500 + Sq + Sk)
    assert eo <= O_TOL and el <= LSE_TOL, (eo, el)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("H,Hkv", [(8, 2), (4, 1), (32, 8)])
def test_grouped_query_heads(H, Hkv, causal):
    eo, el = _fwd_case(2, H, Hkv, 384, 384, 128, causal, seed=70 + H)
    assert eo <= O_TOL and el <= LSE_TOL, (eo, el)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("causal", [False, True])
def test_wide_scores_exercise_conditional_rescaling(causal, D):
    # Q and K scaled by 3: scores ~ N(0, 81), row maxima move a lot between blocks and most rows put
    # nearly all their weight on one key; V unscaled: the literal tolerances
    eo, el = _fwd_case(1, 4, 4, 1536, 1536, D, causal, seed=4000, mult=3.0, v_mult=1.0)
    assert eo <= O_TOL and el <= LSE_TOL, (eo, el)
    # V scaled as well: |O| reaches 8..16 where bfloat16's spacing is 0.0625, so half a unit in the last
    # place of the exact value (<= 2^-8 |O|) is allowed on top of the literal tolerance
    eo, el = _fwd_case(1, 4, 4, 1536, 1536, D, causal, seed=4001, mult=3.0, o_rel=2.0 ** -8)
    assert eo <= O_TOL and el <= LSE_TOL, (eo, el)


def test_other_scales():
    for scale in (1.0, 0.01):
        eo, el = _fwd_case(1, 2, 2, 256, 256, 64, False, seed=81, scale=scale)
        assert eo <= O_TOL and el <= LSE_TOL, (scale, eo, el)


def test_forward_is_bit_reproducible():
    from paper_2603_05451_b200 import binding

    t = inputs.make_qkv(9, 2, 4, 2, 640, 640, 128)
    q, k, v = (to_dev(t[n][0]) for n in ("q", "k", "v"))
    o1, l1 = binding.fa_fwd(q, k, v, None, True)
    o2, l2 = binding.fa_fwd(q, k, v, None, True)
    import torch

    torch.cuda.synchronize()
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16)) and torch.equal(l1, l2)


def test_closed_forms_on_gpu():
    """Identical keys -> running mean of V; a single key -> V itself."""
    import torch

    from paper_2603_05451_b200 import binding

    S, D = 300, 128
    t = inputs.make_qkv(5, 1, 1, 1, S, S, D)
    kbits = np.broadcast_to(t["k"][0][:, :1], t["k"][0].shape).copy()
    o, lse = binding.fa_fwd(to_dev(t["q"][0]), to_dev(kbits), to_dev(t["v"][0]), None, True)
    v = t["v"][1][0, :, 0, :]
    ref = np.cumsum(v, axis=0) / np.arange(1, S + 1)[:, None]
    assert max_abs_err(to_f64(o)[0, :, 0, :], ref) <= O_TOL
    o1, _ = binding.fa_fwd(to_dev(t["q"][0]), to_dev(t["k"][0][:, :1]), to_dev(t["v"][0][:, :1]), None, False)
    torch.cuda.synchronize()
    assert max_abs_err(to_f64(o1), np.broadcast_to(t["v"][1][:, :1], o1.shape)) == 0.0


def test_software_exp2_matches_cpu_model():
    import torch

    from oracle import exp2_emulation as em
    from paper_2603_05451_b200 import binding

    rng = np.random.default_rng(3)
    x = np.concatenate([rng.random(1 << 20), rng.uniform(-126, 8, 1 << 20), np.arange(-126, 9)]).astype(np.float32)
    y = binding.fa_exp2_emulated(torch.from_numpy(x).cuda()).cpu().numpy()
    # the kernel's constants come from its own Remez fit, the model's from a linear program: compare to 2^x
    ref = np.exp2(x.astype(np.float64))
    rel = np.abs(y.astype(np.float64) / ref - 1.0)
    assert rel.max() < 1e-4
    model = em.exp2_emulated(x, em.minimax_coefficients(3)).astype(np.float64)
    assert np.abs(y / model - 1.0).max() < 2e-6
    assert (y[-135:] == np.exp2(np.arange(-126, 9, dtype=np.float32))).all()


_TAU_SCRIPT = r"""
import sys, numpy as np, torch
sys.path.insert(0, sys.argv[1])
from paper_2603_05451_b200 import binding, inputs
t = inputs.make_qkv(4242, 1, 4, 4, 1536, 1536, 128, multiplier=3.0, v_multiplier=1.0, values=False)
dev = lambda b: torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16)
o, lse = binding.fa_fwd(dev(t["q"][0]), dev(t["k"][0]), dev(t["v"][0]), None, bool(int(sys.argv[3])))
assert binding.fa_last_device_status() == 0
np.savez(sys.argv[2], o=o.float().cpu().numpy(), lse=lse.cpu().numpy())
"""


@pytest.mark.parametrize("causal", [0, 1])
def test_result_does_not_depend_on_the_rescale_threshold(causal, tmp_path):
    """Eq. 6: skipping rescales below tau changes nothing after the final normalisation.  The
    threshold is read from FA_TAU once per process, so each setting runs in a process of its own."""
    import os
    import subprocess
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    outs = {}
    for tau in ("0", "8", "1e9"):
        path = str(tmp_path / f"tau_{tau}.npz")
        env = dict(os.environ, FA_TAU=tau)
        subprocess.run([sys.executable, "-c", _TAU_SCRIPT, root, path, str(causal)], check=True, env=env, timeout=300)
        outs[tau] = np.load(path)
    t = inputs.make_qkv(4242, 1, 4, 4, 1536, 1536, 128, multiplier=3.0, v_multiplier=1.0)
    o_ref, lse_ref = attn_fwd(t["q"][1], t["k"][1], t["v"][1], 128 ** -0.5, bool(causal))
    for tau in ("0", "8", "1e9"):
        # every threshold gives the same exact quantity along a different rounding path: each stays
        # within the literal tolerances of the oracle
        assert max_abs_err(outs[tau]["o"], o_ref) <= O_TOL, tau
        assert max_abs_err(outs[tau]["lse"], lse_ref) <= LSE_TOL, tau
    for tau in ("0", "1e9"):
        assert np.abs(outs[tau]["lse"] - outs["8"]["lse"]).max() <= 1e-4


def test_a_wait_that_cannot_be_satisfied_ends_with_a_status_not_a_hang():
    """Every device-side wait is bounded: the kernel gives up, the host reads FA_ERR_DEVICE_TIMEOUT once,
    and the context keeps working."""
    import torch

    from paper_2603_05451_b200 import binding

    assert binding.fa_last_device_status() == 0
    binding.fa_selftest_unsatisfied_wait()
    assert binding.fa_last_device_status() == 5      # FA_ERR_DEVICE_TIMEOUT, cleared by the read
    assert binding.fa_last_device_status() == 0
    eo, el = _fwd_case(1, 2, 2, 256, 256, 128, True, seed=77)
    assert eo <= O_TOL and el <= LSE_TOL, (eo, el)
    torch.cuda.synchronize()


def test_calls_after_an_unread_timeout_still_compute():
    """A recorded timeout belongs to the launch that caused it: a forward and a backward call made
    BEFORE the host has read the status word run normally and match the oracle; the word still
    reports the earlier timeout afterwards."""
    import torch

    from oracle.attention import attn_bwd
    from paper_2603_05451_b200 import binding
    from tests.gpu_util import GRAD_RTOL

    assert binding.fa_last_device_status() == 0
    binding.fa_selftest_unsatisfied_wait()
    torch.cuda.synchronize()                         # the timeout is recorded, and not read
    t = inputs.make_qkv(78, 1, 2, 2, 640, 640, 128, with_do=True)
    q, k, v, d_o = (to_dev(t[n][0]) for n in ("q", "k", "v", "do"))
    scale = 128 ** -0.5
    o, lse = binding.fa_fwd(q, k, v, scale, True)
    dq, dk, dv = binding.fa_bwd(q, k, v, o, lse, d_o, scale, True)
    torch.cuda.synchronize()
    o_ref, lse_ref = attn_fwd(t["q"][1], t["k"][1], t["v"][1], scale, True)
    assert max_abs_err(to_f64(o), o_ref) <= O_TOL and max_abs_err(to_f64(lse), lse_ref) <= LSE_TOL
    for got, want in zip((dq, dk, dv), attn_bwd(t["q"][1], t["k"][1], t["v"][1], t["do"][1], scale, True)):
        assert np.abs(to_f64(got) - want).max() <= GRAD_RTOL * np.abs(want).max()
    assert binding.fa_last_device_status() == 5      # still the first failure, now cleared
    assert binding.fa_last_device_status() == 0
