"""Pins of the oracle's asymmetric quantizer (KV entries, Section 5.1; textbook definition): hand-worked
examples, code range, both range ends reproduced at alpha = 1, half-step error bound, constant groups,
and the pack / dequantize round trip."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "asym_quantizer_examples.txt")


def test_hand_worked_examples():
    n = 0
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        bits, alpha, y, delta, zero, codes = [f.strip() for f in line.split("|")]
        y = np.array([float(v) for v in y.split()])
        q, d, z = oracle.quantize_asym(y, int(bits), 0, float(alpha))
        assert d[0] == float(delta) and z[0] == float(zero)
        assert list(q) == [int(v) for v in codes.split()]
        n += 1
    assert n == 3


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("group", [0, 32])
@pytest.mark.parametrize("alpha", [1.0, 0.8])
def test_properties(bits, group, alpha):
    rng = np.random.Generator(np.random.PCG64(bits * 10 + group))
    y = rng.standard_t(3, size=128) + 0.7
    q, delta, zero = oracle.quantize_asym(y, bits, group, alpha)
    L = 2 ** bits - 1
    g = group or 128
    assert q.min() >= 0 and q.max() <= L
    yhat = q * np.repeat(delta, g) + np.repeat(zero, g)
    for i in range(128 // g):
        seg, sh = y[i * g:(i + 1) * g], yhat[i * g:(i + 1) * g]
        lo, hi = alpha * seg.min(), alpha * seg.max()
        inside = (seg >= lo) & (seg <= hi)
        assert np.all(np.abs(seg - sh)[inside] <= delta[i] / 2 * (1 + 1e-12))
        assert np.all(sh[seg > hi] == pytest.approx(hi)) and np.all(sh[seg < lo] == pytest.approx(lo))
        if alpha == 1.0:                                   # both ends of the range are reproduced
            assert sh[seg.argmin()] == seg.min() and sh[seg.argmax()] == pytest.approx(seg.max(), rel=1e-15)
            assert q[i * g + seg.argmin()] == 0 and q[i * g + seg.argmax()] == L


def test_constant_group_and_round_trip_through_packing():
    q, delta, zero = oracle.quantize_asym(np.full(16, 2.5), 4, 8, 1.0)
    assert not q.any() and not delta.any() and np.all(zero == 2.5)
    rng = np.random.Generator(np.random.PCG64(3))
    x = rng.standard_normal((5, 128)).astype(np.float32)
    for bits in (3, 4):
        ref = oracle.rotate_quantize_asym_rows(x, 128, 128, 1, bits, 64, 0.9)
        assert ref["packed"].shape == (5, 128 * bits // 8)
        back = oracle.dequantize_asym_rows(ref["packed"], ref["delta"], ref["zero"], 128, bits, 64)
        want = ref["q"] * np.repeat(ref["delta"], 64, axis=1) + np.repeat(ref["zero"], 64, axis=1)
        np.testing.assert_allclose(back, want, rtol=0, atol=0)
        # quantization shrinks towards the clipped range but stays within half a step inside it
        inside = (ref["y"] >= np.repeat(ref["zero"], 64, axis=1)) & \
                 (ref["y"] <= np.repeat(ref["zero"] + 15 * ref["delta"] if bits == 4 else ref["zero"] + 7 * ref["delta"], 64, axis=1))
        assert np.all(np.abs(ref["y"] - back)[inside] <= np.repeat(ref["delta"], 64, axis=1)[inside] / 2 * (1 + 1e-9))
