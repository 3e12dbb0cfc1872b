"""GPU parity: the CUDA path, called through the C ABI, against the float64 CPU oracle on the same
seeded inputs, element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_13989_b200 import Plan, binding, synth
from paper_2504_13989_b200 import build as gbs_build
from parity_util import (TOL_CLIP, TOL_ROT_L2, compare_rotate_quantize, oracle_rq, unpack_codes)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _lib():
    gbs_build.build()
    binding.lib()


def _guarded(n_bytes, dtype, device=DEV, guard=256):
    """Buffer with sentinel guard bands on both sides; returns (view, checker)."""
    item = torch.empty((), dtype=dtype).element_size()
    total = n_bytes + 2 * guard
    raw = torch.full((total,), 0xA5, dtype=torch.uint8, device=device)
    view = raw[guard:guard + n_bytes].view(dtype) if n_bytes else raw[guard:guard].view(dtype)

    def check():
        r = raw.cpu()
        assert bool((r[:guard] == 0xA5).all()) and bool((r[guard + n_bytes:] == 0xA5).all()), "guard band overwritten"
    return view, check, item


def _run_rq(plan: Plan, x_dev, n_rows, want_y=True):
    info = plan.info
    codes, c1, _ = _guarded(n_rows * info.code_bytes_per_row, torch.uint8)
    scales, c2, _ = _guarded(n_rows * info.scales_per_row * 4, torch.float32)
    y, c3, _ = _guarded(n_rows * info.d_pad * 4, torch.float32)
    binding.gbs_rotate_quantize(plan.handle, x_dev, codes, scales, y if want_y else None)
    torch.cuda.synchronize()
    c1(); c2(); c3()
    return (codes.view(n_rows, -1) if n_rows else codes, scales.view(n_rows, -1) if n_rows else scales,
            y.view(n_rows, info.d_pad) if (want_y and n_rows) else None)


# ------------------------------------------------------------------------------------------
# the tiny configuration, fully, with the dense-definition oracle
# ------------------------------------------------------------------------------------------
def test_tiny_config_rotate_quantize_dequantize_clip_error():
    w = synth.WORKLOADS["tiny"]
    x = synth.make_host("tiny")
    ref = oracle_rq(x, w, 4, dense=True)
    with Plan(w.d, w.d_pad, w.m, 4, w.group, w.alpha) as plan:
        codes, scales, y = _run_rq(plan, x.to(DEV), w.n_rows)
        compare_rotate_quantize(x, ref, codes, scales, y, 4, w.group, w.d_pad)
        # dequantize (rotated domain) and inverse rotation
        yhat = plan.dequantize(codes, scales)
        want = oracle.dequantize_rows(codes.cpu().numpy(), scales.cpu().double().numpy(), w.d, w.d_pad, w.m, 4, w.group)
        np.testing.assert_allclose(yhat.cpu().double().numpy(), want, rtol=2e-7, atol=0)
        xhat = plan.dequantize(codes, scales, inverse=True)
        wantx = oracle.dequantize_rows(codes.cpu().numpy(), scales.cpu().double().numpy(), w.d, w.d_pad, w.m, 4,
                                       w.group, inverse=True)
        rel = np.linalg.norm(xhat.cpu().double().numpy() - wantx, axis=1) / np.linalg.norm(wantx, axis=1)
        assert rel.max() <= TOL_ROT_L2
        # clip-error sweep, K = 8 alphas in [0.5, 1]
        alphas = np.linspace(0.5, 1.0, 8)
        err, rows = plan.clip_error(x.to(DEV), alphas, want_rows=True)
        torch.cuda.synchronize()
        eref, rref = oracle.clip_error_rows(synth.to_oracle_array(x), w.d, w.d_pad, w.m, 4, w.group, alphas,
                                            want_rows=True)
        np.testing.assert_allclose(err.cpu().numpy(), eref, rtol=TOL_CLIP)
        np.testing.assert_allclose(rows.cpu().double().numpy(), rref, rtol=1e-4)
        # accumulation semantics: a second call adds to err_sum
        plan.clip_error(x.to(DEV), alphas, err_sum=err)
        torch.cuda.synchronize()
        np.testing.assert_allclose(err.cpu().numpy(), 2 * eref, rtol=TOL_CLIP)


def test_literal_formula_at_b3_is_the_4bit_plan():
    """Delta = max|X| / (2^b - 1) exactly as printed (Section 2.1) at b = 3 is D = 7: the bits = 4 plan."""
    w = synth.WORKLOADS["tiny"]
    x = synth.make_host("tiny")
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(x), w.d, w.d_pad, w.m, 3, 0, 1.0, literal=True, dense=True)
    with Plan(w.d, w.d_pad, 1, 4, 0, 1.0) as plan:
        codes, scales, y = _run_rq(plan, x.to(DEV), w.n_rows)
        compare_rotate_quantize(x, ref, codes, scales, y, 4, 0, w.d_pad)


# ------------------------------------------------------------------------------------------
# reduced-size versions of every workload: several tiles and a ragged tail
# ------------------------------------------------------------------------------------------
CASES = [
    # name, rows, bits
    ("llama4096", 301, 3), ("llama4096", 301, 4),
    ("qwen3584", 203, 3),
    ("mlp18944", 37, 4),
    ("kv128", 4099, 3),
    ("calib4096", 150, 3),
]


@pytest.mark.parametrize("name,rows,bits", CASES)
def test_workload_parity_reduced(name, rows, bits):
    w = synth.WORKLOADS[name]
    x = synth.make_host(name, rows)
    ref = oracle_rq(x, w, bits)
    with Plan(w.d, w.d_pad, w.m, bits, w.group, w.alpha) as plan:
        codes, scales, y = _run_rq(plan, x.to(DEV), rows)
        stats = compare_rotate_quantize(x, ref, codes, scales, y, bits, w.group, w.d_pad)
        print(name, bits, stats)
        # same call without the optional rotated output must give identical codes and scales
        codes2, scales2, _ = _run_rq(plan, x.to(DEV), rows, want_y=False)
        assert torch.equal(codes, codes2) and torch.equal(scales, scales2)
        # dequantize of the GPU's own codes against the oracle's dequantize of the same bytes
        sc64 = scales.cpu().double().numpy()
        yhat = plan.dequantize(codes, scales)
        want = oracle.dequantize_rows(codes.cpu().numpy(), sc64, w.d, w.d_pad, w.m, bits, w.group)
        np.testing.assert_allclose(yhat.cpu().double().numpy(), want, rtol=2e-7, atol=0)
        yhat16 = plan.dequantize(codes, scales, dtype=torch.bfloat16)
        np.testing.assert_allclose(yhat16.cpu().double().numpy(), want, rtol=2 ** -8, atol=0)
        xhat = plan.dequantize(codes, scales, inverse=True)
        wantx = oracle.dequantize_rows(codes.cpu().numpy(), sc64, w.d, w.d_pad, w.m, bits, w.group, inverse=True)
        num = np.linalg.norm(xhat.cpu().double().numpy() - wantx, axis=1)
        den = np.linalg.norm(wantx, axis=1)
        assert np.all(num <= TOL_ROT_L2 * den + 1e-30)
        # clip error
        K = 5
        alphas = np.linspace(0.5, 1.0, K)
        err, erows = plan.clip_error(x.to(DEV), alphas, want_rows=True)
        torch.cuda.synchronize()
        eref, rref = oracle.clip_error_rows(synth.to_oracle_array(x), w.d, w.d_pad, w.m, bits, w.group, alphas,
                                            want_rows=True)
        np.testing.assert_allclose(err.cpu().numpy(), eref, rtol=TOL_CLIP)
        np.testing.assert_allclose(erows.cpu().double().numpy(), rref, rtol=1e-4, atol=1e-12)


# ------------------------------------------------------------------------------------------
# the tensor-core family (bf16, d' = U*32 with U = m*2^j <= 128): row counts around the 4-token
# tile, the 148-CTA grid and the 4-stage pipeline; strides; zero padding; every m; per-token and
# per-group scales; and the generic family forced
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("rows", [1, 2, 3, 4, 5, 7, 148 * 4 - 1, 148 * 4 + 1, 148 * 4 * 4 + 3, 5003])
@pytest.mark.parametrize("bits", [3, 4])
def test_tensor_core_family_row_counts(rows, bits):
    w = synth.WORKLOADS["llama4096"]
    x = synth.make_host("llama4096", rows, seed=1000 + rows)
    ref = oracle_rq(x, w, bits)
    with Plan(w.d, w.d_pad, 1, bits, 0, w.alpha) as plan:
        assert plan.info.variant == 1, "the tensor-core family must be the one that runs for this plan"
        codes, scales, y = _run_rq(plan, x.to(DEV), rows)
        assert plan.device_status() == 0
        stats = compare_rotate_quantize(x, ref, codes, scales, y, bits, 0, w.d_pad)
        print(rows, bits, stats)


@pytest.mark.parametrize("d,stride", [(4096, 4096 + 64), (4000, 4000), (4064, 4096), (32, 32), (2048, 8192)])
def test_tensor_core_family_padding_and_stride(d, stride):
    rng = np.random.Generator(np.random.PCG64(d + stride))
    rows = 37
    xs = torch.from_numpy(rng.standard_t(3, size=(rows, stride)).astype(np.float32)).to(torch.bfloat16)
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(xs), d, 4096, 1, 3, 0, 0.9)
    with Plan(d, 4096, 1, 3, 0, 0.9) as plan:
        assert plan.info.variant == 1
        xd = xs.to(DEV)[:, :d]
        codes, scales, y = _run_rq(plan, xd, rows)
        assert plan.device_status() == 0
        compare_rotate_quantize(xs[:, :d], ref, codes, scales, y, 3, 0, 4096)


def test_generic_family_forced_matches_too(monkeypatch):
    monkeypatch.setenv("GBS_FORCE_GENERIC", "1")
    w = synth.WORKLOADS["llama4096"]
    x = synth.make_host("llama4096", 77)
    ref = oracle_rq(x, w, 3)
    with Plan(w.d, w.d_pad, 1, 3, 0, w.alpha) as plan:
        assert plan.info.variant == 0
        codes, scales, y = _run_rq(plan, x.to(DEV), 77)
        compare_rotate_quantize(x, ref, codes, scales, y, 3, 0, w.d_pad)


UV_SHAPES = [
    # d, d_pad, m, bits, group, alpha, rows
    (512, 512, 1, 4, 0, 0.9, 41),
    (512, 512, 1, 3, 32, 0.9, 41),
    (1024, 1024, 1, 3, 1024, 0.8, 150),
    (1000 // 32 * 32, 1024, 1, 4, 64, 1.0, 33),
    (2048, 2048, 1, 3, 0, 0.9, 599),
    (2048, 2048, 1, 4, 256, 0.7, 64),
    (1536, 1536, 12, 3, 128, 0.9, 77),
    (1536, 1536, 24, 4, 64, 0.9, 77),
    (1536, 1536, 24, 3, 0, 0.9, 5),
    (2560, 2560, 20, 3, 0, 0.95, 90),
    (2560, 2560, 20, 4, 32, 0.95, 90),
    (2400, 2560, 20, 4, 128, 0.85, 19),
    (3584, 3584, 28, 3, 128, 0.85, 601),
    (3584, 3584, 28, 4, 0, 0.85, 148 * 4 + 2),
    (3584, 3584, 28, 3, 64, 0.5, 9),
    (3520, 3584, 28, 3, 32, 1.0, 21),
    (4096, 4096, 1, 3, 1024, 0.9, 50),
    (4096, 4096, 1, 4, 128, 0.9, 50),
    # orders beyond 28, and factors U = m 2^j that are not multiples of the MMA's K = 16 (zero-padded)
    (768, 768, 12, 4, 0, 0.9, 33),
    (1408, 1408, 44, 3, 32, 0.9, 41),
    (2816, 2816, 44, 4, 0, 0.9, 77),
    (3072, 3072, 48, 4, 64, 0.9, 30),
    (1920, 1920, 60, 3, 0, 0.9, 150),
    (3840, 3840, 60, 4, 64, 0.8, 35),
    (2176, 2176, 68, 3, 0, 1.0, 20),
    (2304, 2304, 72, 4, 32, 0.9, 20),
    (2560, 2560, 80, 3, 32, 0.9, 20),
    (2688, 2688, 84, 3, 0, 0.9, 149),
    (3328, 3328, 104, 4, 0, 0.9, 20),
    (3456, 3456, 108, 4, 32, 0.85, 75),
    (3296, 3456, 108, 3, 0, 0.9, 9),
]


@pytest.mark.parametrize("d,d_pad,m,bits,group,alpha,rows", UV_SHAPES)
def test_tensor_core_family_shapes(d, d_pad, m, bits, group, alpha, rows):
    rng = np.random.Generator(np.random.PCG64(d * 11 + m * 5 + bits + group))
    xs = rng.standard_t(3, size=(rows, d))
    xs[:, rng.integers(0, d, 3)] *= 40
    if rows > 2:
        xs[2, :] = 0.0
    x = torch.from_numpy(xs.astype(np.float32)).to(torch.bfloat16)
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(x), d, d_pad, m, bits, group, alpha,
                                      dense=(d_pad <= 2048))
    with Plan(d, d_pad, m, bits, group, alpha) as plan:
        assert plan.info.variant == 1, "the tensor-core family must be the one that runs for this plan"
        codes, scales, y = _run_rq(plan, x.to(DEV), rows)
        assert plan.device_status() == 0
        stats = compare_rotate_quantize(x, ref, codes, scales, y, bits, group, d_pad)
        print(stats)
        if rows > 2:
            assert int(codes[2].max()) == 0 and float(scales[2].abs().max()) == 0.0
        codes2, scales2, _ = _run_rq(plan, x.to(DEV), rows, want_y=False)
        assert torch.equal(codes, codes2) and torch.equal(scales, scales2)
        # clip-ratio scoring on the same front end, K not a multiple of the 8-candidate sweep and K = 64
        K = (3, 8, 11, 33, 64)[(d + bits + group) % 5]
        alphas = np.linspace(0.3, 1.0, K)
        err, erows = plan.clip_error(x.to(DEV), alphas, want_rows=True)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        eref, rref = oracle.clip_error_rows(synth.to_oracle_array(x), d, d_pad, m, bits, group, alphas, want_rows=True)
        np.testing.assert_allclose(err.cpu().numpy(), eref, rtol=TOL_CLIP)
        np.testing.assert_allclose(erows.cpu().double().numpy(), rref, rtol=1e-4, atol=1e-12)


UVM_SHAPES = [
    # d, d_pad, m, bits, alpha, rows, group
    (8192, 8192, 1, 3, 0.9, 149, 0),
    (8192 - 64, 8192, 1, 4, 0.9, 1, 0),
    (16384, 16384, 1, 4, 0.8, 37, 0),
    (16000, 16384, 1, 3, 1.0, 150, 0),
    (12288, 12288, 12, 3, 0.9, 75, 0),
    (18944, 20480, 20, 4, 0.95, 301, 0),
    (20480, 20480, 20, 3, 0.9, 4, 0),
    (24576, 24576, 24, 4, 0.9, 33, 0),
    (28672, 28672, 28, 3, 0.85, 150, 0),
    (32768, 32768, 1, 4, 0.9, 31, 0),
    # per-group scales: a group is part of a lane's chunks, one lane, or several lanes of a warp
    (8192, 8192, 1, 3, 0.9, 149, 32),
    (8192, 8192, 1, 4, 0.9, 30, 64),
    (8192 - 64, 8192, 1, 3, 0.8, 151, 128),
    (8192, 8192, 1, 4, 1.0, 17, 2048),
    (8192, 8192, 1, 3, 0.9, 40, 4096),
    (12288, 12288, 12, 4, 0.9, 75, 64),
    (12288, 12288, 12, 3, 0.9, 150, 128),
    (16384, 16384, 1, 3, 0.9, 37, 256),
    (18944, 20480, 20, 4, 0.95, 301, 128),
    (18944, 20480, 20, 3, 0.9, 149, 32),
    (18944, 20480, 20, 3, 0.9, 33, 256),
    (20480, 20480, 20, 4, 0.85, 150, 512),
    (18944, 20480, 20, 4, 0.9, 9, 1024),
    (16000, 16384, 1, 3, 1.0, 150, 4096),
    (28672, 28672, 28, 4, 0.9, 50, 128),
    (32768, 32768, 1, 3, 0.9, 31, 8192),
    # orders beyond 28 (11008 -> 11264 = 44 * 256 and 13824 = 108 * 128 are MLP widths of 7B / 13B models)
    (11008, 11264, 44, 4, 0.9, 75, 0),
    (11008, 11264, 44, 3, 0.9, 40, 128),
    (13824, 13824, 108, 4, 0.9, 33, 0),
    (13824, 13824, 108, 3, 0.85, 33, 128),
    (7680, 7680, 60, 3, 0.9, 50, 0),
    (8704, 8704, 68, 4, 0.9, 21, 64),
]


@pytest.mark.parametrize("d,d_pad,m,bits,alpha,rows,group", UVM_SHAPES)
def test_wide_family_shapes(d, d_pad, m, bits, alpha, rows, group):
    """4096 < d' <= 32768: tensor cores for H_m (x) H_{2^j}, two register sweeps over TMEM for the rest."""
    rng = np.random.Generator(np.random.PCG64(d * 3 + m + bits + rows + group))
    xs = rng.standard_t(3, size=(rows, d))
    xs[:, rng.integers(0, d, 3)] *= 40
    if rows > 2:
        xs[2, :] = 0.0
    x = torch.from_numpy(xs.astype(np.float32)).to(torch.bfloat16)
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(x), d, d_pad, m, bits, group, alpha)
    with Plan(d, d_pad, m, bits, group, alpha) as plan:
        assert plan.info.variant in (3, 5), "a wide tensor-core family must be the one that runs for this plan"
        codes, scales, y = _run_rq(plan, x.to(DEV), rows)
        assert plan.device_status() == 0
        stats = compare_rotate_quantize(x, ref, codes, scales, y, bits, group, d_pad)
        print(stats)
        if rows > 2:
            assert int(codes[2].max()) == 0 and float(scales[2].abs().max()) == 0.0
        codes2, scales2, _ = _run_rq(plan, x.to(DEV), rows, want_y=False)
        assert torch.equal(codes, codes2) and torch.equal(scales, scales2)
        # clip-ratio scoring on the same front end (a third sweep that scores instead of packing)
        K = (3, 8, 11, 33, 64)[(d + bits + group + rows) % 5]
        alphas = np.linspace(0.3, 1.0, K)
        nc = min(rows, 40)
        xc = x[:nc].contiguous()
        for _ in range(2):
            err, erows = plan.clip_error(xc.to(DEV), alphas, want_rows=True)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        eref, rref = oracle.clip_error_rows(synth.to_oracle_array(xc), d, d_pad, m, bits, group, alphas, want_rows=True)
        np.testing.assert_allclose(err.cpu().numpy(), eref, rtol=TOL_CLIP)
        np.testing.assert_allclose(erows.cpu().double().numpy(), rref, rtol=1e-4, atol=1e-12)


@pytest.mark.parametrize("d,d_pad,m,bits,group", [
    (16384, 16384, 1, 3, 0), (12288, 12288, 12, 4, 128), (14336, 14336, 28, 3, 0), (24576, 24576, 24, 4, 0),
    (28672, 28672, 28, 3, 512), (32768, 32768, 1, 4, 0), (18944, 20480, 20, 3, 1024),
])
def test_wide_family_many_tokens_per_block(d, d_pad, m, bits, group):
    """A batch that gives every block a dozen tokens and more (the accumulator stages, the shared-memory ring and
    the rendezvous slots of the register-resident kernel all wrap several times): sampled rows against the oracle,
    and the whole batch against a second run."""
    rows = 148 * 13 + 5
    g = torch.Generator().manual_seed(d + m + bits + group)
    x = (torch.randn((rows, d), generator=g) * torch.rand((rows, 1), generator=g) * 3).to(torch.bfloat16)
    x[7, :] = 0
    pick = np.unique(np.concatenate([np.arange(4), np.arange(rows - 4, rows),
                                     np.random.Generator(np.random.PCG64(rows + d)).integers(0, rows, 24), [7, 148, 149, 295, 296]]))
    xs = x[pick].contiguous()
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(xs), d, d_pad, m, bits, group, 0.9)
    with Plan(d, d_pad, m, bits, group, 0.9) as plan:
        assert plan.info.variant in (3, 5)
        codes, scales, y = _run_rq(plan, x.to(DEV), rows)
        assert plan.device_status() == 0
        idx = torch.from_numpy(pick).to(DEV)
        print(compare_rotate_quantize(xs, ref, codes[idx], scales[idx], y[idx], bits, group, d_pad))
        codes2, scales2, _ = _run_rq(plan, x.to(DEV), rows, want_y=False)
        assert torch.equal(codes, codes2) and torch.equal(scales, scales2)
        assert plan.device_status() == 0


@pytest.mark.parametrize("d,d_pad,m,bits,group,rows", [
    (16384, 16384, 1, 3, 0, 151), (18944, 20480, 20, 4, 0, 300), (12288, 12288, 12, 4, 128, 75), (28672, 28672, 28, 3, 512, 40),
])
def test_three_sweep_kernel_where_the_register_kernel_would_run(d, d_pad, m, bits, group, rows, monkeypatch):
    """GBS_NO_UVR=1 at plan creation keeps a wide plan on the three-sweep kernel (it still serves clip scoring, groups
    above 4096 and widths the register-resident kernel does not take): its rotate-quantize stays covered."""
    monkeypatch.setenv("GBS_NO_UVR", "1")
    rng = np.random.Generator(np.random.PCG64(d + 7 * m + bits + rows))
    xs = rng.standard_t(3, size=(rows, d))
    xs[:, rng.integers(0, d, 3)] *= 40
    x = torch.from_numpy(xs.astype(np.float32)).to(torch.bfloat16)
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(x), d, d_pad, m, bits, group, 0.9)
    with Plan(d, d_pad, m, bits, group, 0.9) as plan:
        assert plan.info.variant == 3
        codes, scales, y = _run_rq(plan, x.to(DEV), rows)
        assert plan.device_status() == 0
        print(compare_rotate_quantize(x, ref, codes, scales, y, bits, group, d_pad))
    monkeypatch.delenv("GBS_NO_UVR")
    with Plan(d, d_pad, m, bits, group, 0.9) as plan:
        assert plan.info.variant == 5


ROW_SHAPES = [
    # d, bits, group, alpha, rows, stride
    (128, 3, 0, 1.0, 1, 128),
    (128, 4, 0, 0.9, 127, 128),
    (128, 3, 0, 1.0, 129, 128),
    (128, 3, 32, 0.8, 148 * 128 + 5, 128),
    (128, 4, 64, 0.9, 1000, 256),
    (128, 3, 128, 0.7, 70001, 128),
    (96, 4, 0, 0.9, 300, 96),
    (64, 3, 32, 1.0, 300, 72),
    (40, 3, 0, 0.9, 515, 40),
    (8, 4, 64, 0.9, 33, 8),
]


@pytest.mark.parametrize("d,bits,group,alpha,rows,stride", ROW_SHAPES)
def test_row_family_shapes(d, bits, group, alpha, rows, stride):
    """d' = 128 rows (KV entries): one tensor-core contraction per 128-row tile, one thread per row."""
    rng = np.random.Generator(np.random.PCG64(d * 13 + bits + group + rows))
    xs = rng.standard_t(3, size=(rows, stride))
    xs[:, rng.integers(0, d, 2)] *= 40
    if rows > 2:
        xs[2, :] = 0.0
    xb = torch.from_numpy(xs.astype(np.float32)).to(torch.bfloat16)
    x = xb[:, :d]
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(x.contiguous()), d, 128, 1, bits, group, alpha, dense=True)
    with Plan(d, 128, 1, bits, group, alpha) as plan:
        assert plan.info.variant == 2, "the row tensor-core family must be the one that runs for this plan"
        xd = xb.to(DEV)[:, :d]
        codes, scales, y = _run_rq(plan, xd, rows)
        assert plan.device_status() == 0
        stats = compare_rotate_quantize(x, ref, codes, scales, y, bits, group, 128)
        print(stats)
        if rows > 2:
            assert int(codes[2].max()) == 0 and float(scales[2].abs().max()) == 0.0
        codes2, scales2, _ = _run_rq(plan, xd, rows, want_y=False)
        assert torch.equal(codes, codes2) and torch.equal(scales, scales2)
        # clip-ratio scoring from the thread-owned row
        K = (3, 8, 11, 33, 64)[(d + bits + group + rows) % 5]
        alphas = np.linspace(0.3, 1.0, K)
        err, erows = plan.clip_error(xd, alphas, want_rows=True)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        eref, rref = oracle.clip_error_rows(synth.to_oracle_array(x.contiguous()), d, 128, 1, bits, group, alphas,
                                            want_rows=True)
        np.testing.assert_allclose(err.cpu().numpy(), eref, rtol=TOL_CLIP)
        np.testing.assert_allclose(erows.cpu().double().numpy(), rref, rtol=1e-4, atol=1e-12)


def test_back_to_back_launches_on_one_stream():
    """Consecutive launches overlap their set-up with the predecessor's tail (programmatic dependent
    launch); a launch that reads what the previous one on the stream wrote must still see it."""
    w = synth.WORKLOADS["llama4096"]
    rows = 600
    x = synth.make_host("llama4096", rows).to(DEV)
    ref = oracle_rq(x.cpu(), w, 3)
    with Plan(w.d, w.d_pad, 1, 3, 0, w.alpha) as plan:
        buf = torch.zeros_like(x)
        outs = [plan.alloc_outputs(rows, DEV) for _ in range(6)]
        for i in range(6):
            buf.copy_(x if i % 2 == 0 else torch.flip(x, dims=(0,)))      # a writer between the launches
            plan.rotate_quantize(buf, out=outs[i])
        for i in range(3):                                                # launches chained directly
            plan.rotate_quantize(x, out=outs[i])
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        for i in (0, 1, 2):
            compare_rotate_quantize(x.cpu(), ref, outs[i][0], outs[i][1], None, 3, 0, w.d_pad)
        assert torch.equal(outs[3][0], torch.flip(outs[0][0], dims=(0,)))
        assert torch.equal(outs[4][0], outs[0][0])


# ------------------------------------------------------------------------------------------
# shapes: every supported m, small and large k, groups, padding, strides
# ------------------------------------------------------------------------------------------
SHAPES = [
    # d, d_pad, m, bits, group, alpha, rows, dtype
    (8, 8, 1, 3, 0, 1.0, 5, torch.float32),
    (8, 8, 1, 4, 8, 0.7, 300, torch.bfloat16),
    (13, 16, 1, 3, 0, 0.9, 33, torch.bfloat16),
    (16, 16, 1, 4, 8, 1.0, 257, torch.float32),
    (32, 32, 1, 3, 16, 0.8, 149, torch.bfloat16),
    (64, 64, 1, 4, 0, 0.95, 147, torch.float32),
    (96, 96, 12, 3, 0, 0.9, 21, torch.bfloat16),
    (90, 96, 12, 4, 8, 0.9, 22, torch.float32),
    (160, 160, 20, 3, 8, 1.0, 13, torch.bfloat16),
    (192, 192, 24, 4, 0, 0.85, 17, torch.bfloat16),
    (224, 224, 28, 3, 8, 0.6, 19, torch.float32),
    (300, 384, 12, 3, 32, 0.9, 9, torch.bfloat16),
    (256, 256, 1, 3, 256, 0.9, 64, torch.bfloat16),
    (1024, 1024, 1, 4, 64, 0.5, 31, torch.bfloat16),
    (1000, 1024, 1, 3, 0, 0.3, 31, torch.float32),
    (2048, 2048, 1, 3, 512, 0.9, 12, torch.bfloat16),
    (1536, 1536, 24, 4, 64, 0.9, 40, torch.bfloat16),
    (1536, 1536, 12, 3, 128, 0.9, 40, torch.bfloat16),
    (3584, 3584, 28, 4, 0, 0.9, 10, torch.float32),
    (8192, 8192, 1, 3, 0, 0.9, 7, torch.bfloat16),
    (30000, 32768, 1, 4, 1024, 0.9, 3, torch.bfloat16),
    (32768, 32768, 1, 3, 0, 1.0, 2, torch.float32),
    (20480, 20480, 20, 3, 1024, 0.9, 3, torch.bfloat16),
    (28672, 28672, 28, 4, 0, 0.9, 2, torch.bfloat16),
    # orders beyond 28 on the generic family
    (352, 352, 44, 4, 8, 0.9, 21, torch.float32),
    (384, 384, 48, 3, 0, 0.9, 21, torch.bfloat16),
    (480, 480, 60, 3, 8, 1.0, 11, torch.bfloat16),
    (544, 544, 68, 4, 0, 0.9, 11, torch.float32),
    (570, 576, 72, 3, 8, 0.9, 11, torch.float32),
    (640, 640, 80, 4, 0, 0.9, 11, torch.bfloat16),
    (672, 672, 84, 3, 0, 0.7, 11, torch.float32),
    (832, 832, 104, 4, 8, 0.9, 5, torch.float32),
    (864, 864, 108, 3, 0, 0.9, 9, torch.float32),
    (13824, 13824, 108, 4, 128, 0.9, 3, torch.float32),
]


@pytest.mark.parametrize("d,d_pad,m,bits,group,alpha,rows,dtype", SHAPES)
def test_shape_sweep(d, d_pad, m, bits, group, alpha, rows, dtype):
    rng = np.random.Generator(np.random.PCG64(d * 7 + m * 3 + bits))
    xs = rng.standard_t(3, size=(rows, d))
    xs[:, rng.integers(0, d, 2)] *= 30
    if rows > 2:
        xs[1, :] = 0.0                      # an all-zero row: codes 0, scale 0
    x = torch.from_numpy(xs.astype(np.float32)).to(dtype)
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(x), d, d_pad, m, bits, group, alpha,
                                      dense=(d_pad <= 2048))
    # rows must start on 16-byte boundaries: place them in a buffer whose stride is a multiple of 8
    stride = (d + 7) // 8 * 8
    xd = torch.zeros((rows, stride), dtype=dtype, device=DEV)
    xd[:, :d] = x.to(DEV)
    xd = xd[:, :d]
    with Plan(d, d_pad, m, bits, group, alpha) as plan:
        codes, scales, y = _run_rq(plan, xd, rows)
        compare_rotate_quantize(x, ref, codes, scales, y, bits, group, d_pad)
        if rows > 2:
            assert int(codes[1].max()) == 0 and float(scales[1].abs().max()) == 0.0
        alphas = [1.0, 0.8, 0.45]
        err = plan.clip_error(xd, alphas)
        torch.cuda.synchronize()
        eref = oracle.clip_error_rows(synth.to_oracle_array(x), d, d_pad, m, bits, group, np.array(alphas))
        np.testing.assert_allclose(err.cpu().numpy(), eref, rtol=TOL_CLIP)
        xhat = plan.dequantize(codes, scales, inverse=True)
        wantx = oracle.dequantize_rows(codes.cpu().numpy(), scales.cpu().double().numpy(), d, d_pad, m, bits,
                                       group, inverse=True)
        num = np.linalg.norm(xhat.cpu().double().numpy() - wantx, axis=1)
        den = np.linalg.norm(wantx, axis=1)
        assert np.all(num <= TOL_ROT_L2 * den + 1e-30)


def test_strided_rows_and_leading_dims():
    """x_row_stride > d (a slice of a wider buffer) and KV-style [batch, heads, seq, 128] views."""
    rng = np.random.Generator(np.random.PCG64(99))
    big = torch.from_numpy(rng.standard_normal((50, 512)).astype(np.float32)).to(torch.bfloat16)
    x = big[:, :256]
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(big), 256, 256, 1, 4, 0, 0.9)
    with Plan(256, 256, 1, 4, 0, 0.9) as plan:
        xd = big.to(DEV)[:, :256]
        assert xd.stride(0) == 512
        codes, scales, y = _run_rq(plan, xd, 50)
        compare_rotate_quantize(x, ref, codes, scales, y, 4, 0, 256)
    kv = torch.from_numpy(rng.standard_t(3, size=(2, 3, 17, 128)).astype(np.float32)).to(torch.bfloat16)
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(kv.reshape(-1, 128)), 128, 128, 1, 3, 0, 1.0)
    with Plan(128, 128, 1, 3, 0, 1.0) as plan:
        codes, scales, y = _run_rq(plan, kv.to(DEV), 2 * 3 * 17)
        compare_rotate_quantize(kv.reshape(-1, 128), ref, codes, scales, y, 3, 0, 128)


def test_empty_and_error_paths_on_device():
    with Plan(128, 128, 1, 4, 0, 1.0) as plan:
        x = torch.zeros((0, 128), dtype=torch.bfloat16, device=DEV)
        codes, scales, _ = plan.alloc_outputs(0, DEV)
        binding.gbs_rotate_quantize(plan.handle, x, codes, scales)          # n_rows = 0: no-op
        L = binding.lib()
        xb = torch.zeros((4, 136), dtype=torch.bfloat16, device=DEV)
        c, s, _ = plan.alloc_outputs(4, DEV)
        h = plan.handle
        import ctypes
        vp = ctypes.c_void_p
        # misaligned base pointer / stride not a multiple of 16 bytes / stride < d / bad dtype / bad K
        assert L.gbs_rotate_quantize(vp(h), xb.data_ptr() + 2, 1, 4, 136, c.data_ptr(), s.data_ptr(), None, None) == binding.GBS_ERR_ALIGNMENT
        assert L.gbs_rotate_quantize(vp(h), xb.data_ptr(), 1, 4, 130, c.data_ptr(), s.data_ptr(), None, None) == binding.GBS_ERR_ALIGNMENT
        assert L.gbs_rotate_quantize(vp(h), xb.data_ptr(), 1, 4, 64, c.data_ptr(), s.data_ptr(), None, None) == binding.GBS_ERR_INVALID_ARG
        assert L.gbs_rotate_quantize(vp(h), xb.data_ptr(), 7, 4, 136, c.data_ptr(), s.data_ptr(), None, None) == binding.GBS_ERR_INVALID_ARG
        assert L.gbs_rotate_quantize(vp(h), xb.data_ptr(), 1, -1, 136, c.data_ptr(), s.data_ptr(), None, None) == binding.GBS_ERR_INVALID_ARG
        assert L.gbs_rotate_quantize(vp(h), xb.data_ptr(), 1, 4, 136, None, s.data_ptr(), None, None) == binding.GBS_ERR_INVALID_ARG
        err = torch.zeros(4, dtype=torch.float64, device=DEV)
        a = (ctypes.c_float * 3)(0.5, 1.2, 0.9)
        assert L.gbs_clip_error(vp(h), xb.data_ptr(), 1, 4, 136, a, 3, err.data_ptr(), None, None) == binding.GBS_ERR_INVALID_ARG
        assert L.gbs_clip_error(vp(h), xb.data_ptr(), 1, 4, 136, a, 0, err.data_ptr(), None, None) == binding.GBS_ERR_INVALID_ARG
        assert L.gbs_clip_error(vp(h), xb.data_ptr(), 1, 4, 136, a, 65, err.data_ptr(), None, None) == binding.GBS_ERR_INVALID_ARG
        assert L.gbs_dequantize(vp(h), c.data_ptr(), s.data_ptr(), 4, xb.data_ptr(), 0, 2, None) == binding.GBS_ERR_INVALID_ARG
        torch.cuda.synchronize()            # the context is still healthy
        assert float(err.sum()) == 0.0


def test_quantizer_invariants_on_device():
    """Properties that hold at any size: alpha = 1 reproduces the max (Section 2.1); the norm is preserved
    (Section 2.3.1); Lemma 1 for a single spike."""
    n, d = 64, 4096
    x = synth.make_host("llama4096", n)
    with Plan(d, d, 1, 4, 0, 1.0) as plan:
        codes, scales, y = _run_rq(plan, x.to(DEV), n)
        yn = y.double().norm(dim=1).cpu()
        xn = x.double().norm(dim=1)
        assert torch.all((yn - xn).abs() <= 1e-5 * xn)
        q = unpack_codes(codes.cpu().numpy(), d, 4)
        assert np.all(np.abs(q).max(axis=1) == 7)
        amax = y.abs().max(dim=1).values.cpu().double()
        np.testing.assert_allclose((scales[:, 0].cpu().double() * 7).numpy(), amax.numpy(), rtol=3e-7)
        spike = torch.zeros((3, d), dtype=torch.float32)
        spike[0, 0] = 200.0; spike[1, 1777] = 200.0; spike[2, d - 1] = -200.0
        _, _, ys = _run_rq(plan, spike.to(DEV), 3)
        np.testing.assert_allclose(ys.abs().cpu().numpy(), 200.0 / 64.0, rtol=1e-6)


@pytest.mark.parametrize("d,d_pad,m", [(3584, 3584, 28), (18944, 20480, 20), (4000, 4096, 1), (96, 128, 1)])
def test_expansion_identity_of_eq_2_through_the_library(d, d_pad, m):
    """Eq. (2): with activations and weight rows both zero-padded to d' and rotated by the same
    normalised Hadamard, (X_pad H^T)(H W_pad^T) = X W^T.  Rotating the rows of W^T is the weight-side
    half of the expansion; both halves go through gbs_rotate_quantize's rotated output here."""
    rng = np.random.Generator(np.random.PCG64(d + m))
    x = torch.from_numpy(rng.standard_normal((24, d)).astype(np.float32)).to(torch.bfloat16)
    wt = torch.from_numpy((rng.standard_normal((40, d)) / np.sqrt(d)).astype(np.float32)).to(torch.bfloat16)
    with Plan(d, d_pad, m, 4, 0, 1.0) as plan:
        _, _, yx = _run_rq(plan, x.to(DEV), 24)
        _, _, yw = _run_rq(plan, wt.to(DEV), 40)
    got = (yx.double() @ yw.double().T).cpu().numpy()
    want = x.double().numpy() @ wt.double().numpy().T
    np.testing.assert_allclose(got, want, rtol=0, atol=2e-5 * np.abs(want).max() + 1e-6)


@pytest.mark.parametrize("rows,chunks", [(1000, 4), (3, 8), (257, 1), (0, 4)])
def test_host_pipeline_equals_the_one_shot_call(rows, chunks):
    """Pinned host rows through two plans in overlapping chunks: byte-identical to device-resident calls."""
    from paper_2504_13989_b200 import HostPipeline
    d = 512
    rng = np.random.Generator(np.random.PCG64(rows + chunks))
    x = torch.from_numpy(rng.standard_t(3, size=(rows, d)).astype(np.float32)).to(torch.bfloat16).pin_memory()
    with Plan(d, d, 1, 3, 0, 0.9) as p3, Plan(d, d, 1, 4, 64, 0.8) as p4:
        plans = [p3, p4]
        outs = [(torch.zeros((rows, p.info.code_bytes_per_row), dtype=torch.uint8).pin_memory(),
                 torch.zeros((rows, p.info.scales_per_row), dtype=torch.float32).pin_memory()) for p in plans]
        pipe = HostPipeline(plans, rows, device=DEV, chunks=chunks)
        st = torch.cuda.Stream()
        for _ in range(2):                      # twice: the staging buffers are reused
            pipe.run(x, outs, stream=st)
        st.synchronize()
        for p, (ch, sh) in zip(plans, outs):
            if rows == 0:
                continue
            c, s, _ = _run_rq(p, x.to(DEV), rows, want_y=False)
            assert torch.equal(ch, c.cpu()) and torch.equal(sh, s.cpu())


INV_SHAPES = [
    # d, d_pad, m, bits, rows
    (4096, 4096, 1, 4, 4096 // 8 + 3),
    (4096, 4096, 1, 3, 149),
    (4000 // 32 * 32, 4096, 1, 4, 5),
    (512, 512, 1, 3, 1),
    (2560, 2560, 20, 4, 148 * 4 + 1),
    (3584, 3584, 28, 3, 77),
    (3456, 3456, 108, 4, 33),          # U = 108: the contraction is padded to 112
    (1408, 1408, 44, 3, 9),
]


@pytest.mark.parametrize("d,d_pad,m,bits,rows", INV_SHAPES)
def test_inverse_dequantize_on_the_tensor_cores(d, d_pad, m, bits, rows, monkeypatch):
    """gbs_dequantize with GBS_INVERSE_ROTATE for per-token plans of the tensor-core family:
    xhat = (H^T (q Delta) / sqrt(d'))[0:d] against the oracle, in fp32 and bf16, and against the generic kernel."""
    rng = np.random.Generator(np.random.PCG64(d + m * 7 + bits + rows))
    x = torch.from_numpy(rng.standard_t(3, size=(rows, d)).astype(np.float32)).to(torch.bfloat16)
    with Plan(d, d_pad, m, bits, 0, 0.9) as plan:
        assert plan.info.variant == 1
        codes, scales, _ = _run_rq(plan, x.to(DEV), rows, want_y=False)
        want = oracle.dequantize_rows(codes.cpu().numpy(), scales.cpu().double().numpy(), d, d_pad, m, bits, 0,
                                      inverse=True)
        for _ in range(2):                                     # twice: pipeline state does not leak between launches
            got32 = plan.dequantize(codes, scales, inverse=True, dtype=torch.float32)
        got16 = plan.dequantize(codes, scales, inverse=True, dtype=torch.bfloat16)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
    assert got32.shape == (rows, d) and got16.shape == (rows, d)
    g = got32.cpu().double().numpy()
    num = np.linalg.norm(g - want, axis=1)
    den = np.linalg.norm(want, axis=1)
    assert np.all(num <= 2e-7 * den + 1e-30), float((num / np.maximum(den, 1e-30)).max())   # exact rotation, one rounding
    g16 = got16.cpu().double().numpy()
    assert np.all(np.abs(g16 - want) <= 2.0 ** -8 * np.abs(want) + 1e-30)
    monkeypatch.setenv("GBS_FORCE_GENERIC", "1")
    with Plan(d, d_pad, m, bits, 0, 0.9) as gen:
        assert gen.info.variant == 0
        ref32 = gen.dequantize(codes, scales, inverse=True, dtype=torch.float32)
        torch.cuda.synchronize()
    num = np.linalg.norm(g - ref32.cpu().double().numpy(), axis=1)
    assert np.all(num <= TOL_ROT_L2 * den + 1e-30)


@pytest.mark.parametrize("d,bits,group,asym,rows", [
    (128, 3, 0, False, 1), (128, 4, 128, False, 127), (128, 3, 0, False, 148 * 128 * 4 + 129),
    (96, 4, 0, False, 300), (64, 3, 128, False, 129), (32, 4, 0, False, 77),
    (128, 3, 128, True, 1000), (128, 4, 0, True, 129), (96, 3, 128, True, 515), (64, 4, 0, True, 5),
])
def test_inverse_dequantize_of_kv_rows_on_the_tensor_cores(d, bits, group, asym, rows):
    """d' = 128 rows with one scale (pair) per row: xhat = (H_128 yhat / sqrt(128))[0:d] with
    yhat = q Delta (Section 2.1) or code Delta + lo (Section 5.1), against the dense definition."""
    rng = np.random.Generator(np.random.PCG64(d + bits * 3 + group + rows + int(asym)))
    xs = rng.standard_t(3, size=(rows, d)) + (0.7 if asym else 0.0)
    if rows > 4:
        xs[3, :] = 0.0
        xs[4, :] = 1.5                                    # constant row: after rotation one non-zero coordinate
    x = torch.from_numpy(xs.astype(np.float32)).to(torch.bfloat16)
    with Plan(d, 128, 1, bits, group, 0.9, asymmetric=asym) as plan:
        assert plan.info.variant == 2
        codes, scales, _ = plan.rotate_quantize(x.to(DEV))
        for _ in range(2):
            got32 = plan.dequantize(codes, scales, inverse=True, dtype=torch.float32)
        got16 = plan.dequantize(codes, scales, inverse=True, dtype=torch.bfloat16)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
    sc = scales.cpu().double().numpy()
    if asym:
        sc = sc.reshape(rows, -1, 2)
        yhat = oracle.dequantize_asym_rows(codes.cpu().numpy(), sc[:, :, 0], sc[:, :, 1], 128, bits, group)
    else:
        yhat = oracle.dequantize_rows(codes.cpu().numpy(), sc.reshape(rows, -1), 128, 128, 1, bits, group)
    H = oracle.hadamard_full(1, 7).astype(np.float64)
    want = (yhat @ H / np.sqrt(128.0))[:, :d]
    g = got32.cpu().double().numpy()
    assert g.shape == (rows, d)
    scale_of_row = np.abs(yhat).max(axis=1, keepdims=True) * np.sqrt(128.0) + 1e-30
    assert np.all(np.abs(g - want) <= 3e-7 * scale_of_row)
    assert np.all(np.abs(got16.cpu().double().numpy() - want) <= 2.0 ** -8 * np.abs(want) + 3e-7 * scale_of_row)


def _random_plans(n_cases: int, seed: int):
    """Seeded draw of valid (d, d', m, bits, group, alpha, rows, dtype) over every order and kernel family."""
    rng = np.random.Generator(np.random.PCG64(seed))
    orders = [1, 1, 1, 12, 20, 24, 28, 44, 48, 60, 68, 72, 80, 84, 104, 108]
    cases = []
    while len(cases) < n_cases:
        m = int(rng.choice(orders))
        k = int(rng.integers(3, 14))
        d_pad = m << k
        if d_pad > 32768:
            continue
        bits = int(rng.choice([3, 4]))
        if rng.random() < 0.5:
            group = 0
        else:
            group = 1 << int(rng.integers(3, k + 1))
        # widths: full, a multiple of 32 below d', or an arbitrary multiple of 8
        r = rng.random()
        if r < 0.4:
            d = d_pad
        elif r < 0.7 and d_pad >= 64:
            d = int(rng.integers(1, d_pad // 32 + 1)) * 32
        else:
            d = int(rng.integers(1, d_pad // 8 + 1)) * 8
        rows = int(rng.choice([1, 3, 4, 5, 33, 130, 149, 600])) if d_pad <= 8192 else int(rng.choice([1, 2, 5, 9]))
        dtype = torch.bfloat16 if rng.random() < 0.75 else torch.float32
        alpha = float(rng.choice([1.0, 0.9, 0.75, 0.5]))
        cases.append((d, d_pad, m, bits, group, alpha, rows, dtype))
    return cases


@pytest.mark.parametrize("d,d_pad,m,bits,group,alpha,rows,dtype", _random_plans(60, 20250413))
def test_random_plans_against_the_oracle(d, d_pad, m, bits, group, alpha, rows, dtype):
    """Whatever family the plan picks: rotated values, scales and codes against the oracle, then the inverse
    dequantize of the kernel's own codes."""
    rng = np.random.Generator(np.random.PCG64(d * 31 + d_pad + m + bits + group + rows))
    xs = rng.standard_t(3, size=(rows, d))
    xs[:, rng.integers(0, d, 2)] *= 25
    x = torch.from_numpy(xs.astype(np.float32)).to(dtype)
    ref = oracle.rotate_quantize_rows(synth.to_oracle_array(x), d, d_pad, m, bits, group, alpha, dense=(d_pad <= 1024))
    with Plan(d, d_pad, m, bits, group, alpha) as plan:
        codes, scales, y = _run_rq(plan, x.to(DEV), rows)
        assert plan.device_status() == 0
        compare_rotate_quantize(x, ref, codes, scales, y, bits, group, d_pad)
        xhat = plan.dequantize(codes, scales, inverse=True)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
    wantx = oracle.dequantize_rows(codes.cpu().numpy(), scales.cpu().double().numpy(), d, d_pad, m, bits, group,
                                   inverse=True)
    num = np.linalg.norm(xhat.cpu().double().numpy() - wantx, axis=1)
    den = np.linalg.norm(wantx, axis=1)
    assert np.all(num <= TOL_ROT_L2 * den + 1e-30)


@pytest.mark.parametrize("d,d_pad,m,rows", [(4096, 4096, 1, 4096), (128, 128, 1, 70000), (2560, 2560, 20, 601)])
def test_producer_consumer_chain_without_host_synchronisation(d, d_pad, m, rows):
    """quantize -> dequantize with inverse rotation -> quantize the result -> ... on one stream, each kernel
    reading what the kernel before it is still writing when it becomes resident (programmatic dependent
    launch; the quantizer also prefetches its first tile into L2 before its dependency wait).  The chain must
    give bit-identical results with and without a host synchronisation between the calls."""
    rng = np.random.Generator(np.random.PCG64(d + rows))
    x0 = torch.from_numpy(rng.standard_t(3, size=(rows, d)).astype(np.float32)).to(torch.bfloat16).to(DEV)
    with Plan(d, d_pad, m, 4, 0, 0.9) as plan:
        def chain(sync: bool):
            xa = x0.clone()
            xb = torch.empty_like(xa)
            outs = [plan.alloc_outputs(rows, DEV) for _ in range(2)]
            torch.cuda.synchronize()
            trace = []
            for i in range(12):
                o = outs[i & 1]
                plan.rotate_quantize(xa, out=o)
                if sync:
                    torch.cuda.synchronize()
                plan.dequantize(o[0], o[1], inverse=True, dtype=torch.bfloat16, out=xb)
                if sync:
                    torch.cuda.synchronize()
                xa, xb = xb, xa
                if i in (0, 5, 11):
                    trace.append((o[0].clone(), o[1].clone()))
            torch.cuda.synchronize()
            return trace, xa.clone()
        t_sync, x_sync = chain(True)
        for _ in range(3):
            t_free, x_free = chain(False)
            assert torch.equal(x_sync, x_free)
            for (c1, s1), (c2, s2) in zip(t_sync, t_free):
                assert torch.equal(c1, c2) and torch.equal(s1, s2)
        assert plan.device_status() == 0


def test_one_plan_from_several_streams_and_host_threads():
    """A plan is immutable: launches from different streams and host threads at once give the same bytes."""
    import threading
    d, rows = 4096, 1500
    rng = np.random.Generator(np.random.PCG64(99))
    xs = [torch.from_numpy(rng.standard_t(3, size=(rows, d)).astype(np.float32)).to(torch.bfloat16).to(DEV)
          for _ in range(4)]
    with Plan(d, d, 1, 3, 0, 0.9) as plan:
        refs = [plan.rotate_quantize(x) for x in xs]
        torch.cuda.synchronize()
        results = [None] * 4
        errors = []

        def worker(i):
            try:
                st = torch.cuda.Stream(device=DEV)
                out = None
                with torch.cuda.stream(st):           # allocations of this thread belong to its stream
                    for _ in range(25):
                        out = plan.rotate_quantize(xs[i], stream=st)
                        plan.clip_error(xs[i], [0.8, 1.0], stream=st)
                st.synchronize()
                results[i] = out
            except Exception as exc:      # surfaced below: an assertion in a thread would be lost
                errors.append(exc)
        threads = [threading.Thread(target=worker, args=(i,)) for i in range(4)]
        for t in threads:
            t.start()
        for t in threads:
            t.join()
        assert not errors, errors
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        for (c, s, _), (cr, sr, _) in zip(results, refs):
            assert torch.equal(c, cr) and torch.equal(s, sr)


@pytest.mark.gpu
def test_a_bounded_wait_that_runs_out_returns_its_code_and_leaves_the_context_usable():
    """The tensor-core kernels bound every barrier wait.  gbs_selftest_wait_expiry makes one such wait run out
    (a barrier nothing arrives at, limit 1 ms): it must come back with the wait's code and raised abort flag
    after about the limit, and a normal launch afterwards must still match the oracle."""
    code, abort, waited_us = binding.gbs_selftest_wait_expiry(1000)
    assert code == 7 and abort == 1
    assert 1000 <= waited_us <= 5000, waited_us
    w = synth.WORKLOADS["llama4096"]
    x = synth.make_host("llama4096", 64, seed=3)
    ref = oracle_rq(x, w, 3)
    with Plan(w.d, w.d_pad, w.m, 3, w.group, w.alpha) as plan:
        codes, scales, y = plan.rotate_quantize(x.to(DEV), want_y=True)
        torch.cuda.synchronize()
        compare_rotate_quantize(x, ref, codes, scales, y, 3, w.group, w.d_pad)
        assert plan.device_status() == 0
