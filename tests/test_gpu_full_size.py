"""GPU parity at the full workload sizes, in the launch configuration the benchmark times (the plans the
benchmark builds, whole batches, no optional rotated output): every row where the oracle finishes in
seconds, sampled rows where the tensor is too large, plus properties that hold at any size."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_13989_b200 import Plan, synth
from paper_2504_13989_b200 import build as gbs_build
from parity_util import TOL_CLIP, TOL_SCALE, compare_rotate_quantize, oracle_rq, unpack_codes

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _lib():
    gbs_build.build()


@pytest.mark.parametrize("name", ["llama4096", "qwen3584", "mlp18944"])
def test_full_batch_every_row(name):
    w = synth.WORKLOADS[name]
    x = synth.make_host(name)
    xd = x.to(DEV)
    for bits in w.bits:
        ref = oracle_rq(x, w, bits)
        with Plan(w.d, w.d_pad, w.m, bits, w.group, w.alpha) as plan:
            codes, scales, _ = plan.rotate_quantize(xd)
            torch.cuda.synchronize()
            assert plan.device_status() == 0
            stats = compare_rotate_quantize(x, ref, codes, scales, None, bits, w.group, w.d_pad)
            print(name, bits, stats)


def test_kv_tensor_sampled_rows_and_code_range():
    """Both KV tensors' worth of rows (2 097 152 x 128) in one launch; the oracle checks the first and
    last tiles and every 257th row; every code of every row must lie in [-D, D]."""
    w = synth.WORKLOADS["kv128"]
    x = synth.make_device("kv128", device=DEV)
    n = x.shape[0]
    with Plan(w.d, w.d_pad, w.m, 3, w.group, w.alpha) as plan:
        assert plan.info.variant == 2
        codes, scales, _ = plan.rotate_quantize(x)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        idx = torch.unique(torch.cat([torch.arange(0, 256), torch.arange(n - 300, n), torch.arange(0, n, 257)]))
        xs = x[idx.to(DEV)].cpu()
        ref = oracle_rq(xs, w, 3)
        compare_rotate_quantize(xs, ref, codes[idx.to(DEV)], scales[idx.to(DEV)], None, 3, w.group, w.d_pad)
        # any size: 3-bit fields never hold the pattern 100 (= -4), i.e. codes stay in [-3, 3]
        c = codes.view(-1, 3).to(torch.int32)
        word = c[:, 0] | (c[:, 1] << 8) | (c[:, 2] << 16)
        bad = torch.zeros((), dtype=torch.bool, device=DEV)
        for e in range(8):
            bad |= (((word >> (3 * e)) & 7) == 4).any()
        assert not bool(bad)
        # alpha = 1: each row's largest code magnitude is D wherever the row is not all zero
        assert bool((scales >= 0).all())


@pytest.mark.parametrize("layer", [0, 31])
def test_calibration_layer_clip_error_sampled_rows(layer):
    """One whole calibration layer (128 sequences x 2048 tokens = 262 144 rows of d = 4096, seed 5 + layer) in
    ONE scoring call at K = 32, the launch configuration the benchmark times; per-row errors of sampled rows
    against the oracle, and the fp64 totals against the sum of the kernel's own rows."""
    w = synth.WORKLOADS["calib4096"]
    n = w.n_rows
    assert n == 128 * 2048
    x = synth.make_device("calib4096", n, seed=w.seed + layer, device=DEV)
    alphas = np.linspace(0.5, 1.0, 32)
    with Plan(w.d, w.d_pad, w.m, 3, w.group, w.alpha) as plan:
        err, rows = plan.clip_error(x, alphas, want_rows=True)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        idx = torch.arange(0, n, 1021)
        xs = x[idx.to(DEV)].cpu()
        eref, rref = oracle.clip_error_rows(synth.to_oracle_array(xs), w.d, w.d_pad, w.m, 3, w.group, alphas,
                                            want_rows=True)
        np.testing.assert_allclose(rows[idx.to(DEV)].cpu().double().numpy(), rref, rtol=1e-4, atol=1e-12)
        np.testing.assert_allclose(err.cpu().numpy(), rows.double().sum(dim=0).cpu().numpy(), rtol=TOL_CLIP)
        # the sampled rows' totals agree with the oracle's totals to the tolerance of the sums
        np.testing.assert_allclose(rows[idx.to(DEV)].double().sum(dim=0).cpu().numpy(), eref, rtol=TOL_CLIP)


@pytest.mark.parametrize("name,rows,bits,asym,dtype", [
    ("llama4096", 20000, 3, False, torch.bfloat16),      # large enough for the shared-memory-staged form, ragged tile
    ("llama4096", 20000, 4, False, torch.float32),
    ("kv128", 300001, 3, True, torch.bfloat16),          # 128-wide rows (an item spans two rows), odd row count
    ("qwen3584", 9000, 3, False, torch.bfloat16),        # per-group scales, width not a power of two
    ("llama4096", 300, 3, False, torch.bfloat16),        # small launch: the direct form
])
def test_rotated_domain_dequantize_at_launch_sizes_of_both_forms(name, rows, bits, asym, dtype):
    """gbs_dequantize without inverse rotation, yhat = q * Delta (+ lo), at sizes that take the staged form and the
    direct form of the streaming kernel: every element against the codes and scales unpacked independently."""
    w = synth.WORKLOADS[name]
    x = synth.make_device(name, rows, device=DEV)
    group = 128 if asym else w.group
    with Plan(w.d, w.d_pad, w.m, bits, group, w.alpha, asymmetric=asym) as plan:
        codes, scales, _ = plan.rotate_quantize(x)
        out = torch.full((rows + 1, w.d_pad), float("nan"), dtype=dtype, device=DEV)
        plan.dequantize(codes, scales, out=out[:rows])
        torch.cuda.synchronize()
        assert bool(torch.isnan(out[rows]).all()), "wrote past the last row"
        g = group or w.d_pad
        step = 7 if rows > 1000 else 1                      # every seventh row, plus the last rows (the ragged tail)
        idx = torch.unique(torch.cat([torch.arange(0, rows, step), torch.arange(max(0, rows - 70), rows)])).to(DEV)
        cb = codes[idx].cpu().numpy()
        bitsarr = np.unpackbits(cb, axis=1, bitorder="little")[:, : w.d_pad * bits].reshape(len(idx), w.d_pad, bits)
        f = (bitsarr.astype(np.int32) * (1 << np.arange(bits))).sum(axis=2)
        sc = scales[idx].cpu().double().numpy()
        if asym:
            sc = sc.reshape(len(idx), -1, 2)
            want = f * np.repeat(sc[:, :, 0], g, axis=1) + np.repeat(sc[:, :, 1], g, axis=1)
        else:
            q = np.where(f >= (1 << (bits - 1)), f - (1 << bits), f)
            want = q * np.repeat(sc, g, axis=1)
        got = out[idx].cpu().double().numpy()
        tol = 2e-7 if dtype == torch.float32 else 2.0 ** -8
        np.testing.assert_allclose(got, want, rtol=tol, atol=1e-30 if not asym else 1e-6 * np.abs(want).max())


@pytest.mark.parametrize("bits,group", [(3, 0), (4, 128)])
def test_mlp_width_long_batch_sampled_rows(bits, group):
    """Sixteen batches' worth of MLP rows (65 536 x 18944 -> 20480) in one launch: every block of the wide kernel walks
    several hundred tokens, so every ring, stage and barrier index wraps many times; the oracle checks the first and last
    rows and a random sample, and every code of every row must lie in [-D, D]."""
    w = synth.WORKLOADS["mlp18944"]
    rows = 65536
    x = synth.make_device("mlp18944", rows, device=DEV)
    pick = np.unique(np.concatenate([np.arange(3), np.arange(rows - 3, rows),
                                     np.random.Generator(np.random.PCG64(bits + group)).integers(0, rows, 26)]))
    xs = x[torch.from_numpy(pick).to(DEV)].cpu()
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(xs), w.d, w.d_pad, w.m, bits, group, w.alpha)
    with Plan(w.d, w.d_pad, w.m, bits, group, w.alpha) as plan:
        codes, scales, _ = plan.rotate_quantize(x)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        idx = torch.from_numpy(pick).to(DEV)
        print(compare_rotate_quantize(xs, ref, codes[idx], scales[idx], None, bits, group, w.d_pad, alpha=w.alpha))
        # the code range over the whole tensor, on the device: no field of any row outside [-D, D]
        D = (1 << (bits - 1)) - 1
        flat = codes.view(-1)
        if bits == 4:
            lo, hi = (flat & 15).to(torch.int16), (flat >> 4).to(torch.int16)
            for f in (lo, hi):
                q = torch.where(f >= 8, f - 16, f)
                assert int(q.min()) >= -D and int(q.max()) <= D
        else:
            sample = codes[:: 97].cpu().numpy()
            q = unpack_codes(sample.reshape(sample.shape[0], -1), w.d_pad, bits)
            assert q.min() >= -D and q.max() <= D
