"""The full Paley order (Section 5.2.2): width 1536 expanded by 8 to d' = m = 1544 = 1543 + 1, the rotation being
Algorithm 2's matrix itself, run as a dense tensor-core contraction; against the oracle's dense definition."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_13989_b200 import Plan, binding, synth
from paper_2504_13989_b200 import build as gbs_build
from parity_util import compare_rotate_quantize, unpack_codes

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
D, M = 1536, 1544


def _rows(n, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    x = 0.5 * rng.standard_t(3.0, size=(n, D))
    x[:, rng.choice(D, 8, replace=False)] *= 50.0
    x[rng.choice(n, max(1, n // 100), replace=False)] *= 20.0
    return torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16)


@pytest.mark.parametrize("bits,rows,alpha", [(3, 130, 0.9), (4, 1, 1.0)])
def test_full_paley_1544_against_the_dense_definition(bits, rows, alpha):
    gbs_build.build()
    x = _rows(rows, 40 + rows)
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(x), D, M, M, bits, 0, alpha, dense=True)
    with Plan(D, M, M, bits, 0, alpha) as plan:
        assert plan.info.variant == 4 and plan.info.k == 0 and plan.info.code_bytes_per_row == M * bits // 8
        codes, scales, y = plan.rotate_quantize(x.to(DEV), want_y=True)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        compare_rotate_quantize(x, ref, codes, scales, y, bits, 0, M, alpha)
        # rotated-domain dequantize of these codes
        yhat = plan.dequantize(codes, scales)
        q = unpack_codes(codes.cpu().numpy(), M, bits)
        np.testing.assert_allclose(yhat.cpu().double().numpy(), q * scales.cpu().double().numpy(), rtol=2e-7, atol=0)
        # back to the input domain: xhat = (H^T yhat / sqrt(m))[0:d] against the oracle on the GPU's own codes and scales
        want = oracle.dequantize_rows(codes.cpu().numpy(), scales.cpu().double().numpy(), D, M, M, bits, 0, inverse=True)
        for dtype, tol in ((torch.float32, 2e-7), (torch.bfloat16, 2.0 ** -8)):
            xhat = torch.full((rows + 1, D), float("nan"), dtype=dtype, device=DEV)
            plan.dequantize(codes, scales, inverse=True, out=xhat[:rows])
            torch.cuda.synchronize()
            assert plan.device_status() == 0 and bool(torch.isnan(xhat[rows]).all())
            got = xhat[:rows].cpu().double().numpy()
            err = np.linalg.norm(got - want, axis=1) / np.maximum(np.linalg.norm(want, axis=1), 1e-300)
            assert err.max() <= tol, err.max()
        # what this family does not serve is refused, not faulted
        with pytest.raises(binding.GbsError) as e:
            plan.clip_error(x.to(DEV), [0.5, 1.0])
        assert e.value.status == binding.GBS_ERR_UNSUPPORTED


@pytest.mark.parametrize("d,m,bits,rows", [(256, 264, 3, 300), (120, 128, 4, 77), (368, 368, 4, 129)])
def test_other_full_orders_against_the_dense_definition(d, m, bits, rows):
    """Smaller full orders (263, 127 and 367 are primes = 3 mod 4): a last block of 8 coordinates, a single block, an
    order without expansion; every row against the oracle's dense definition."""
    gbs_build.build()
    rng = np.random.Generator(np.random.PCG64(d + m))
    x = torch.from_numpy((0.5 * rng.standard_t(3.0, size=(rows, d))).astype(np.float32)).to(torch.bfloat16)
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(x), d, m, m, bits, 0, 0.9, dense=True)
    with Plan(d, m, m, bits, 0, 0.9) as plan:
        assert plan.info.variant == 4
        codes, scales, y = plan.rotate_quantize(x.to(DEV), want_y=True)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        compare_rotate_quantize(x, ref, codes, scales, y, bits, 0, m, 0.9)
        # and back: widths that are not a multiple of the kernel's 256-coordinate output blocks
        want = oracle.dequantize_rows(codes.cpu().numpy(), scales.cpu().double().numpy(), d, m, m, bits, 0, inverse=True)
        got = plan.dequantize(codes, scales, inverse=True).cpu().double().numpy()
        assert got.shape == (rows, d) and plan.device_status() == 0
        err = np.linalg.norm(got - want, axis=1) / np.maximum(np.linalg.norm(want, axis=1), 1e-300)
        assert err.max() <= 2e-7, err.max()


def test_full_paley_1544_with_256_token_tiles_sampled_rows():
    """A batch large enough for the kernel's 256-token tiles (two sub-tiles sharing each chunk of H), with a ragged last
    tile; sampled rows (first, last, across sub-tile and tile borders) against the oracle's dense definition."""
    gbs_build.build()
    rows, bits, alpha = 19000 + 37, 3, 0.9
    x = _rows(rows, 7)
    idx = np.unique(np.concatenate([np.arange(0, 6), np.arange(125, 131), np.arange(253, 259), np.arange(9000, 9004),
                                    np.arange(rows - 40, rows)]))
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(x[idx]), D, M, M, bits, 0, alpha, dense=True)
    with Plan(D, M, M, bits, 0, alpha) as plan:
        codes = torch.full((rows + 1, M * bits // 8), 0xEE, dtype=torch.uint8, device=DEV)
        scales = torch.full((rows + 1, 1), -1.0, dtype=torch.float32, device=DEV)
        y = torch.empty((rows, M), dtype=torch.float32, device=DEV)
        binding.gbs_rotate_quantize(plan.handle, x.to(DEV), codes[:rows], scales[:rows], y)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        assert bool((codes[rows] == 0xEE).all()) and float(scales[rows, 0]) == -1.0, "wrote past the last row"
        t = torch.from_numpy(idx).to(DEV)
        compare_rotate_quantize(x[idx], ref, codes[t], scales[t], y[t], bits, 0, M, alpha)


def test_full_order_plans_are_validated_on_the_host():
    gbs_build.build()
    lib = binding.lib()
    import ctypes
    h = ctypes.c_void_p()
    # 1545 - 1 is not a prime = 3 mod 4; 1544 with a group; fp32 rows
    assert lib.gbs_plan_create(ctypes.byref(h), 1536, 1545, 1545, 3, 0, 0.9) in (binding.GBS_ERR_INVALID_ARG, binding.GBS_ERR_UNSUPPORTED)
    assert lib.gbs_plan_create(ctypes.byref(h), 1536, 1544, 1544, 3, 8, 0.9) == binding.GBS_ERR_INVALID_ARG
    with Plan(D, M, M, 3, 0, 0.9) as plan:
        x = torch.zeros((4, D), dtype=torch.float32, device=DEV)
        with pytest.raises(binding.GbsError) as e:
            plan.rotate_quantize(x)
        assert e.value.status == binding.GBS_ERR_UNSUPPORTED
    hm = binding.gbs_hadamard_m(M).to(torch.int64)
    assert torch.equal(hm @ hm.T, M * torch.eye(M, dtype=torch.int64))
