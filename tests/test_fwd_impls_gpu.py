"""Forward parity for every kernel variant that an environment switch selects.

The switches are read once per process, so each setting runs in a child interpreter that evaluates a
list of shapes (several key blocks, ragged tails, causal, grouped heads, more queries than keys so
that some rows see no key at all, both head dimensions, the x3 inputs that keep the conditional
rescale busy) and prints its errors against the float64 oracle; the parent asserts the literal
tolerances.

  FA_EMU_PER8 = 1, 2, 3    that many of every 8 exponentials on the FMA pipe (Section 3.1.3)
  FA_FWD_SECTION_MB = 0, 1  all heads in one launch section / sections of one key-value head (Section 3.3)
  FA_FWD_TILE = 0, 1        the pipelined kernel (256 rows per CTA) / the one-tile kernel (128 rows per CTA,
                            two CTAs per SM) for every dense shape, whatever its length
"""

import json
import os
import subprocess
import sys

import pytest

from tests.gpu_util import LSE_TOL, O_TOL

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import json, sys
sys.path.insert(0, %(root)r)
from tests.test_fwd_gpu import _fwd_case
# (B, H, Hkv, Sq, Sk, D, causal, multiplier of Q and K)
cases = [(1, 1, 1, 128, 128, 64, False, 1.0), (2, 2, 2, 333, 333, 128, True, 1.0), (1, 3, 3, 300, 77, 128, True, 1.0),
         (1, 2, 2, 1024, 1024, 128, False, 1.0), (1, 2, 2, 1024, 1024, 64, True, 1.0), (2, 8, 2, 640, 640, 128, True, 1.0),
         (1, 4, 1, 200, 1100, 64, True, 1.0), (1, 2, 2, 1, 700, 128, False, 1.0), (1, 2, 2, 1536, 1536, 128, True, 3.0),
         (1, 2, 2, 1536, 1536, 64, False, 3.0), (4, 4, 4, 2048, 2048, 128, True, 1.0), (3, 2, 1, 129, 257, 128, False, 1.0),
         (2, 3, 3, 255, 255, 64, True, 1.0), (1, 2, 2, 2, 1, 128, True, 1.0), (8, 16, 4, 512, 512, 128, True, 1.0)]
out = []
for idx, c in enumerate(cases):
    eo, el = _fwd_case(*c[:7], seed=8100 + idx, mult=c[7], v_mult=1.0)
    out.append([list(c), eo, el])
print("RESULT " + json.dumps(out))
"""


@pytest.mark.parametrize("name,value", [("FA_EMU_PER8", "1"), ("FA_EMU_PER8", "2"), ("FA_EMU_PER8", "3"),
                                        ("FA_FWD_SECTION_MB", "0"), ("FA_FWD_SECTION_MB", "1"),
                                        ("FA_FWD_TILE", "0"), ("FA_FWD_TILE", "1"),
                                        ("FA_FWD_TILE+FA_EMU_PER8", "1+2")])
def test_forward_variants_match_the_oracle(name, value):
    env = dict(os.environ)
    for n, v in zip(name.split("+"), value.split("+")):
        env[n] = v
    res = subprocess.run([sys.executable, "-c", CHILD % {"root": ROOT}], env=env, capture_output=True, text=True,
                         timeout=900, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    line = [l for l in res.stdout.splitlines() if l.startswith("RESULT ")][-1]
    for case, eo, el in json.loads(line[len("RESULT "):]):
        assert eo <= O_TOL and el <= LSE_TOL, (name, value, case, eo, el)


def test_fa_log_names_the_wait_that_gave_up():
    """FA_LOG=1: reading a recorded timeout prints the code and the source line of the wait."""
    code = ("import sys; sys.path.insert(0, %r)\n"
            "from paper_2603_05451_b200 import binding\n"
            "binding.fa_selftest_unsatisfied_wait()\n"
            "assert binding.fa_last_device_status() == 5\n") % ROOT
    res = subprocess.run([sys.executable, "-c", code], env=dict(os.environ, FA_LOG="1"), capture_output=True, text=True,
                         timeout=300, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    assert "device-side wait expired (code 5, site" in res.stderr


@pytest.mark.parametrize("emu", ["1", "3"])
def test_emulated_exponentials_hold_the_tolerance_on_the_wide_score_configuration(emu):
    """Config 4 at full size (Q and K scaled by 3: most rows put their weight on one key, so the rounding of
    the largest probability shows in O) with part of the exponentials on the FMA pipe: the row-sum
    compensation has to round the value that was actually stored, whichever unit produced it."""
    res = subprocess.run([sys.executable, "-m", "pytest", "tests/test_full_size_gpu.py", "-x", "-q", "-m", "gpu", "-k",
                          "config4"], env=dict(os.environ, FA_EMU_PER8=emu), capture_output=True, text=True,
                         timeout=1800, cwd=ROOT)
    assert res.returncode == 0, res.stdout[-3000:]


@pytest.mark.parametrize("tile", ["0", "1"])
def test_packed_batches_through_either_forward_kernel(tile):
    """The packed-batch tests (per-sequence oracle parity, ragged ends, grouped heads, longest-first order) with
    every call forced through the pipelined kernel (0) or the one-tile kernel (1)."""
    res = subprocess.run([sys.executable, "-m", "pytest", "tests/test_fwd_varlen_gpu.py", "-x", "-q", "-m", "gpu"],
                         env=dict(os.environ, FA_FWD_TILE=tile), capture_output=True, text=True, timeout=1800, cwd=ROOT)
    assert res.returncode == 0, res.stdout[-3000:]


@pytest.mark.parametrize("tile", ["0", "1"])
def test_random_shapes_through_either_forward_kernel(tile):
    """The seeded random problem shapes (odd head counts, unequal lengths around the tile size) with every dense
    forward call forced through one kernel: by default most of them are short enough for the one-tile kernel."""
    res = subprocess.run([sys.executable, "-m", "pytest", "tests/test_random_shapes_gpu.py", "-x", "-q", "-m", "gpu", "-k",
                          "forward"], env=dict(os.environ, FA_FWD_TILE=tile), capture_output=True, text=True,
                         timeout=1800, cwd=ROOT)
    assert res.returncode == 0, res.stdout[-3000:]
