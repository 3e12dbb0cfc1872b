"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, builds the same H_m as the oracle, and rejects bad arguments with status codes."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2504_13989_b200 import binding, build as gbs_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    gbs_build.build()
    return binding.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "gbs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gbs_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings(lib):
    for code in (0, -1, -2, -3, -4, -5):
        s = binding.status_string(code)
        assert s.startswith("GBS_")
    assert "unknown" in binding.status_string(-99)


@pytest.mark.parametrize("m", [1, 12, 20, 24, 28, 44, 48, 60, 68, 72, 80, 84, 104, 108])
def test_library_and_oracle_build_the_same_small_hadamard(m, lib):
    """Two independently written constructions (Euler criterion / discrete logs in the library,
    exhaustive squaring in the oracle) must give one canonical matrix (Algorithm 2)."""
    H = binding.gbs_hadamard_m(m).numpy().astype(np.int64)
    assert np.array_equal(H, oracle.hadamard_m(m))
    assert np.array_equal(H @ H.T, m * np.eye(m, dtype=np.int64))


def test_hadamard_m_rejects_unsupported_orders(lib):
    buf = (ctypes.c_int8 * 4096)()
    for m in (2, 3, 6, 16, 36, 52, 112):
        assert lib.gbs_hadamard_m(m, buf) == binding.GBS_ERR_UNSUPPORTED
    assert lib.gbs_hadamard_m(0, buf) == binding.GBS_ERR_INVALID_ARG
    assert lib.gbs_hadamard_m(12, None) == binding.GBS_ERR_INVALID_ARG


BAD_PLANS = [
    # d, d_pad, m, bits, group, alpha, expected
    (0, 128, 1, 4, 0, 1.0, binding.GBS_ERR_INVALID_ARG),       # d < 1
    (129, 128, 1, 4, 0, 1.0, binding.GBS_ERR_INVALID_ARG),     # d > d'
    (128, 128, 1, 5, 0, 1.0, binding.GBS_ERR_INVALID_ARG),     # bits
    (128, 128, 1, 2, 0, 1.0, binding.GBS_ERR_INVALID_ARG),
    (128, 128, 1, 4, 0, 0.0, binding.GBS_ERR_INVALID_ARG),     # alpha
    (128, 128, 1, 4, 0, 1.5, binding.GBS_ERR_INVALID_ARG),
    (128, 128, 1, 4, 0, float("nan"), binding.GBS_ERR_INVALID_ARG),
    (100, 100, 1, 4, 0, 1.0, binding.GBS_ERR_INVALID_ARG),     # not m * 2^k
    (4, 4, 1, 4, 0, 1.0, binding.GBS_ERR_INVALID_ARG),         # 2^k < 8
    (48, 48, 12, 4, 0, 1.0, binding.GBS_ERR_INVALID_ARG),      # 2^k = 4 < 8
    (128, 128, 1, 4, 12, 1.0, binding.GBS_ERR_INVALID_ARG),    # group not a power of two
    (128, 128, 1, 4, 4, 1.0, binding.GBS_ERR_INVALID_ARG),     # group < 8
    (128, 128, 1, 4, 256, 1.0, binding.GBS_ERR_INVALID_ARG),   # group > 2^k
    (3584, 3584, 28, 3, 256, 1.0, binding.GBS_ERR_INVALID_ARG),  # group straddles blocks of H_28
    (128, 128, 16, 4, 0, 1.0, binding.GBS_ERR_UNSUPPORTED),    # no construction for m = 16
    (416, 416, 52, 4, 0, 1.0, binding.GBS_ERR_UNSUPPORTED),    # 51 is not prime: no construction for m = 52
    (65536, 65536, 1, 4, 0, 1.0, binding.GBS_ERR_UNSUPPORTED),  # d' too large
]


@pytest.mark.parametrize("d,d_pad,m,bits,group,alpha,want", BAD_PLANS)
def test_plan_create_rejects_bad_arguments_on_the_host(lib, d, d_pad, m, bits, group, alpha, want):
    h = ctypes.c_void_p()
    assert lib.gbs_plan_create(ctypes.byref(h), d, d_pad, m, bits, group, alpha) == want
    assert h.value is None


def test_null_arguments(lib):
    assert lib.gbs_plan_create(None, 128, 128, 1, 4, 0, 1.0) == binding.GBS_ERR_INVALID_ARG
    assert lib.gbs_plan_destroy(None) == binding.GBS_OK
    info = binding.PlanInfo()
    assert lib.gbs_plan_info(None, ctypes.byref(info)) == binding.GBS_ERR_INVALID_ARG
    assert lib.gbs_rotate_quantize(None, None, 0, 1, 128, None, None, None, None) == binding.GBS_ERR_INVALID_ARG
    assert lib.gbs_dequantize(None, None, None, 1, None, 0, 0, None) == binding.GBS_ERR_INVALID_ARG
    assert lib.gbs_clip_error(None, None, 0, 1, 128, None, 1, None, None, None) == binding.GBS_ERR_INVALID_ARG


def test_binding_refuses_cpu_tensors(lib):
    import torch
    with pytest.raises(ValueError):
        binding._rows_view(torch.zeros(4, 128), 128)
