"""The asymmetric KV quantizer (GBS_PLAN_ASYMMETRIC; Section 5.1 names it, textbook definition) on the
d' = 128 row kernel, against the oracle: scales and zero points within 1e-6 relative, codes identical
except at rounding ties, dequantized values exact given the kernel's own codes and scales."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2504_13989_b200 import Plan, binding, synth
from paper_2504_13989_b200 import build as gbs_build
from parity_util import TOL_CODE_FRAC, TOL_SCALE

DEV = "cuda:0"


def test_asymmetric_plans_outside_the_row_family_are_refused_on_the_host():
    gbs_build.build()
    L = binding.lib()
    h = ctypes.c_void_p()
    A = binding.GBS_PLAN_ASYMMETRIC
    assert L.gbs_plan_create_ex(ctypes.byref(h), 4096, 4096, 1, 3, 0, 0.9, A) == binding.GBS_ERR_UNSUPPORTED
    assert L.gbs_plan_create_ex(ctypes.byref(h), 128, 128, 1, 3, 16, 0.9, A) == binding.GBS_ERR_UNSUPPORTED
    assert L.gbs_plan_create_ex(ctypes.byref(h), 96, 96, 12, 3, 0, 0.9, A) == binding.GBS_ERR_UNSUPPORTED
    assert L.gbs_plan_create_ex(ctypes.byref(h), 128, 128, 1, 3, 0, 0.9, 2) == binding.GBS_ERR_INVALID_ARG
    assert h.value is None


CASES = [
    # d, bits, group, alpha, rows
    (128, 3, 128, 1.0, 1000),
    (128, 4, 0, 0.9, 129),
    (128, 3, 32, 0.8, 4099),
    (128, 4, 64, 1.0, 77),
    (96, 3, 0, 0.95, 300),
]


@pytest.mark.gpu
@pytest.mark.parametrize("d,bits,group,alpha,rows", CASES)
def test_asymmetric_row_quantizer_parity(d, bits, group, alpha, rows):
    gbs_build.build()
    rng = np.random.Generator(np.random.PCG64(d + bits * 7 + group + rows))
    xs = rng.standard_t(3, size=(rows, d)) + 0.3
    xs[:, rng.integers(0, d, 2)] *= 30
    if rows > 2:
        xs[2, :] = 0.0
    x = torch.from_numpy(xs.astype(np.float32)).to(torch.bfloat16)
    ref = oracle.rotate_quantize_asym_rows(synth.to_oracle_array(x), d, 128, 1, bits, group, alpha)
    g = group or 128
    with Plan(d, 128, 1, bits, group, alpha, asymmetric=True) as plan:
        assert plan.info.asymmetric == 1 and plan.info.variant == 2
        assert plan.info.scale_floats_per_row == 2 * plan.info.scales_per_row
        codes, scales, y = plan.rotate_quantize(x.to(DEV), want_y=True)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        # rotated values: the same rotation as the symmetric path
        yg = y.cpu().double().numpy()
        den = np.linalg.norm(ref["y"], axis=1)
        num = np.linalg.norm(yg - ref["y"], axis=1)
        assert np.all(num <= 1e-5 * den + 1e-30)
        sc = scales.cpu().double().numpy().reshape(rows, -1, 2)
        dref, zref = ref["delta"], ref["zero"]
        assert np.all(np.abs(sc[:, :, 0] - dref) <= TOL_SCALE * np.abs(dref))
        # the zero point is alpha*min: compare relative to the group's range (it may be near zero itself)
        span = np.maximum(np.abs(zref), dref * (2 ** bits - 1))
        assert np.all(np.abs(sc[:, :, 1] - zref) <= TOL_SCALE * span)
        q = oracle.unpack(codes.cpu().numpy().ravel(), rows * 128, bits).reshape(rows, 128) & (2 ** bits - 1)
        diff = q != ref["q"]
        assert diff.mean() <= TOL_CODE_FRAC
        if diff.any():
            assert np.abs(q - ref["q"])[diff].max() <= 1
            t = (ref["y"] - np.repeat(zref, g, axis=1))[diff] / np.repeat(dref, g, axis=1)[diff]
            assert np.all(np.abs(np.abs(t - np.floor(t)) - 0.5) < 2e-4), "a mismatching code is not at a rounding tie"
        if rows > 2:
            assert int(codes[2].max()) == 0 and float(scales[2].abs().max()) == 0.0
        # dequantize the kernel's own codes: q * Delta + lo, exactly
        yhat = plan.dequantize(codes, scales)
        want = oracle.dequantize_asym_rows(codes.cpu().numpy(), sc[:, :, 0], sc[:, :, 1], 128, bits, group)
        np.testing.assert_allclose(yhat.cpu().double().numpy(), want, rtol=3e-7, atol=1e-30)
        # and through the inverse rotation back to width d
        xhat = plan.dequantize(codes, scales, inverse=True).cpu().double().numpy()
        H = oracle.hadamard_full(1, 7).astype(np.float64)
        wantx = (want @ H / np.sqrt(128.0))[:, :d]
        assert np.all(np.linalg.norm(xhat - wantx, axis=1) <= 1e-5 * np.linalg.norm(wantx, axis=1) + 1e-30)
        # scoring clip ratios is not defined for the asymmetric quantizer here
        with pytest.raises(binding.GbsError) as ei:
            plan.clip_error(x.to(DEV), [0.9])
        assert ei.value.status == binding.GBS_ERR_UNSUPPORTED
