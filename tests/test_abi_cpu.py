"""CPU checks of the C-ABI library: it loads, exports every declared symbol, and rejects bad
arguments without launching anything."""

import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2603_05451_b200 import binding as b
    from paper_2603_05451_b200 import build

    build.build()
    return b


def test_every_declared_symbol_is_exported(binding):
    header = open(os.path.join(ROOT, "include", "fa.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = re.findall(r"\b(fa_[a-z0-9_]+)\s*\(", header)
    assert set(names) >= {"fa_fwd", "fa_bwd", "fa_bwd_workspace_bytes", "fa_status_string", "fa_last_device_status"}
    lib = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings(binding):
    assert binding.status_string(0) == "ok"
    seen = {binding.status_string(i) for i in range(6)}
    assert len(seen) == 6
    assert binding.status_string(99) == "unknown status"


@pytest.mark.parametrize("kwargs,expected", [
    (dict(B=0), 1), (dict(Sq=0), 1), (dict(Sk=-3), 1), (dict(H=3, Hkv=2), 1),
    (dict(scale=0.0), 1), (dict(scale=float("nan")), 1), (dict(scale=float("inf")), 1), (dict(scale=-1.0), 1),
    (dict(D=96), 2), (dict(D=256), 2),
    (dict(q=0), 1), (dict(k=8), 1), (dict(o=0x1004), 1), (dict(lse=0), 1), (dict(lse=0x1002), 1),
])
def test_forward_rejects_bad_arguments(binding, kwargs, expected):
    a = dict(q=0x1000, k=0x2000, v=0x3000, o=0x4000, lse=0x5000, B=1, H=2, Hkv=2, Sq=128, Sk=128, D=128,
             scale=0.1, causal=0)
    a.update(kwargs)
    st = binding.fa_fwd_raw(a["q"], a["k"], a["v"], a["o"], a["lse"], a["B"], a["H"], a["Hkv"], a["Sq"], a["Sk"],
                            a["D"], a["scale"], a["causal"])
    assert st == expected


def test_workspace_query_and_backward_argument_checks(binding):
    n = binding.fa_bwd_workspace_bytes(2, 4, 2, 300, 200, 128)
    assert n >= 2 * 300 * 4 * 128 * 4 + 2 * 2 * 4 * 300 * 4 and n % 256 == 0
    assert binding.fa_bwd_workspace_bytes(2, 4, 2, 300, 200, 96) == 0
    assert binding.fa_bwd_workspace_bytes(2, 4, 3, 300, 200, 128) == 0
    lib = binding.lib()
    ptrs = [0x1000 * (i + 1) for i in range(9)]
    args = ptrs + [2, 4, 2, 300, 200, 128, 0.1, 0]
    assert lib.fa_bwd(*args, 0, n, None) == 4                   # null workspace
    assert lib.fa_bwd(*args, 0x100010, n, None) == 4            # misaligned workspace
    assert lib.fa_bwd(*args, 0x100000, n - 1, None) == 4        # too small
    bad = list(args)
    bad[5] = 0
    assert lib.fa_bwd(*bad, 0x100000, n, None) == 1             # null d_o


def test_no_gpu_means_an_error_not_a_fallback(binding):
    import torch

    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    st = binding.fa_fwd_raw(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 1, 2, 2, 128, 128, 128, 0.1, 0)
    assert st in (2, 3)


def test_per_device_bookkeeping_is_independent_per_ordinal(binding):
    """Function attributes and the architecture check are cached per device ordinal; the host-only
    self-test walks two ordinals and the out-of-range cases."""
    assert binding.lib().fa_selftest_per_device_flags() == 0
