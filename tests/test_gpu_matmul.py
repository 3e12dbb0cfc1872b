"""The consumer of the packed codes (Section 4.2, Eq. (2)): gbs_weight_rotate_quantize and gbs_quantized_matmul
against the oracle -- the weight rows through the oracle's rotate/quantize, and the product of the two DEQUANTIZED
rotated operands as a float64 matmul."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_13989_b200 import Plan, binding, synth
from paper_2504_13989_b200 import build as gbs_build
from parity_util import compare_rotate_quantize, unpack_codes

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
# the int32 sums are exact; the output is fp32(sum) * fp32(Delta_x * Delta_w): two roundings of 2^-24 each
TOL_MATMUL = 2.5e-7


def _weights(n_out, d, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    w = rng.standard_normal((n_out, d)) / np.sqrt(d)
    w[:, rng.choice(d, 3, replace=False)] *= 8.0
    return torch.from_numpy(w.astype(np.float32)).to(torch.bfloat16)


CASES = [
    # workload, tokens, outputs, bits_x, bits_w   (ragged in both directions: tiles are 128 x 256)
    ("llama4096", 300, 520, 3, 3),
    ("llama4096", 129, 257, 4, 4),
    ("llama4096", 64, 1024, 3, 4),
    ("llama4096", 128, 256, 4, 3),
    ("mlp18944", 40, 264, 4, 4),
]


@pytest.mark.parametrize("name,n_tok,n_out,bx,bw", CASES)
def test_quantized_matmul_against_the_dequantized_float64_product(name, n_tok, n_out, bx, bw):
    gbs_build.build()
    w = synth.WORKLOADS[name]
    x = synth.make_host(name, n_tok, seed=21)
    wt = _weights(n_out, w.d, 22)
    alpha_w = 1.0
    ref_x = oracle.rotate_quantize_rows(synth.to_oracle_array(x), w.d, w.d_pad, w.m, bx, 0, w.alpha)
    ref_w = oracle.rotate_quantize_rows(synth.to_oracle_array(wt), w.d, w.d_pad, w.m, bw, 0, alpha_w)
    with Plan(w.d, w.d_pad, w.m, bx, 0, w.alpha) as px, Plan(w.d, w.d_pad, w.m, bw, 0, alpha_w) as pw:
        cx, sx, _ = px.rotate_quantize(x.to(DEV))
        cw, sw = pw.weight_rotate_quantize(wt.to(DEV))
        torch.cuda.synchronize()
        # the weight side is the same path: its codes and scales against the oracle's
        compare_rotate_quantize(wt, ref_w, cw, sw, None, bw, 0, w.d_pad)
        for dtype in (torch.float32, torch.bfloat16):
            pad = 8 + (-n_out) % 8                                                # strided rows (16-byte multiple) + guard
            out = torch.full((n_tok + 1, n_out + pad), float("nan"), dtype=dtype, device=DEV)
            view = out[:n_tok, :n_out]
            px.quantized_matmul(cx, sx, pw, cw, sw, out=view)
            torch.cuda.synchronize()
            assert px.device_status() == 0
            assert bool(torch.isnan(out[n_tok:]).all()) and bool(torch.isnan(out[:, n_out:]).all()), "wrote outside the tile"
            # expected value from what the GPU itself produced (its codes and scales), in float64
            qx = unpack_codes(cx.cpu().numpy(), w.d_pad, bx).astype(np.float64)
            qw = unpack_codes(cw.cpu().numpy(), w.d_pad, bw).astype(np.float64)
            want = (qx @ qw.T) * sx.cpu().double().numpy() * sw.cpu().double().numpy().T
            got = view.cpu().double().numpy()
            tol = TOL_MATMUL if dtype == torch.float32 else 2.0 ** -8
            np.testing.assert_allclose(got, want, rtol=tol, atol=0)
        # the activation side against the oracle too: with both sides' codes and scales at parity (identical except at
        # rounding ties) and the product exact given the codes, the product is at parity up to those ties; where no
        # code of a token row and an output row differs, the all-oracle product must agree to the fp32 tolerance
        compare_rotate_quantize(x, ref_x, cx, sx, None, bx, 0, w.d_pad)
        oracle_out = (ref_x["q"].astype(np.float64) @ ref_w["q"].astype(np.float64).T) * ref_x["delta"] * ref_w["delta"].T
        got32 = px.quantized_matmul(cx, sx, pw, cw, sw).cpu().double().numpy()
        clean_t = (unpack_codes(cx.cpu().numpy(), w.d_pad, bx) == ref_x["q"]).all(axis=1)
        clean_o = (unpack_codes(cw.cpu().numpy(), w.d_pad, bw) == ref_w["q"]).all(axis=1)
        sub_g, sub_o = got32[np.ix_(clean_t, clean_o)], oracle_out[np.ix_(clean_t, clean_o)]
        assert clean_t.mean() > 0.9 and clean_o.mean() > 0.9
        # scales agree to 1e-6 each, the two fp32 roundings add 2.5e-7
        np.testing.assert_allclose(sub_g, sub_o, rtol=2.5e-6, atol=0)
        # Eq. (2): the quantized product approximates x w^T itself (rotation and padding cancel)
        exact = x.double().numpy() @ wt.double().numpy().T
        rel = np.linalg.norm(got32 - exact) / np.linalg.norm(exact)
        assert rel < (0.7 if min(bx, bw) == 3 else 0.35), rel          # quantization error of both sides, nothing more


def test_quantized_matmul_refuses_what_it_cannot_serve():
    gbs_build.build()
    with Plan(4096, 4096, 1, 3, 0, 0.9) as px, Plan(4096, 4096, 1, 3, 128, 0.9) as pg, Plan(3584, 3584, 28, 3, 0, 0.9) as p2:
        cx = torch.zeros((4, 1536), dtype=torch.uint8, device=DEV)
        sx = torch.zeros((4, 1), dtype=torch.float32, device=DEV)
        sg = torch.zeros((4, 32), dtype=torch.float32, device=DEV)
        out = torch.zeros((4, 4), dtype=torch.float32, device=DEV)
        with pytest.raises(binding.GbsError) as e:
            binding.gbs_quantized_matmul(px.handle, cx, sx, pg.handle, cx, sg, out)           # per-group weight scales
        assert e.value.status == binding.GBS_ERR_UNSUPPORTED
        c2 = torch.zeros((4, 1344), dtype=torch.uint8, device=DEV)
        with pytest.raises(binding.GbsError) as e:
            binding.gbs_quantized_matmul(px.handle, cx, sx, p2.handle, c2, sx, out)           # different rotations
        assert e.value.status == binding.GBS_ERR_INVALID_ARG
        binding.gbs_quantized_matmul(px.handle, cx[:0], sx[:0], px.handle, cx, sx, out[:0])     # no tokens: no-op
