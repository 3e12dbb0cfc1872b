"""gbs_rotate_quantize_static: the plan-free entry point for callers that cannot allocate device
memory (a process whose pool already owns the whole GPU, or one that may not take the device-wide
synchronisation of cudaMalloc).  It runs the same fused kernel with its table in a fixed array inside
the library, so its output must equal the plan-based call's, call after call, also when the array has
to be rewritten between calls.  This file is collected last on purpose: a run that stops at the first
failure has then already been through every other test."""
import ctypes

import pytest
import torch

from paper_2504_13989_b200 import Plan, binding, synth
from paper_2504_13989_b200 import build as gbs_build

DEV = "cuda:0"


@pytest.fixture(scope="module")
def lib():
    gbs_build.build()
    return binding.lib()


def test_static_entry_point_rejects_bad_and_oversized_requests_on_the_host(lib):
    """Argument checks come before any CUDA call, so they can be exercised without a device."""
    f = lib.gbs_rotate_quantize_static
    buf = ctypes.create_string_buffer(64)
    p = ctypes.addressof(buf)
    assert f(4096, 4096, 1, 5, 0, 0.9, p, 1, 4096, p, p, None) == binding.GBS_ERR_INVALID_ARG      # bits
    assert f(4096, 4096, 1, 3, 0, 1.5, p, 1, 4096, p, p, None) == binding.GBS_ERR_INVALID_ARG      # alpha
    assert f(4096, 4097, 1, 3, 0, 0.9, p, 1, 4096, p, p, None) == binding.GBS_ERR_INVALID_ARG      # d_pad not 2^k
    assert f(4096, 4096, 1, 3, 0, 0.9, p, -1, 4096, p, p, None) == binding.GBS_ERR_INVALID_ARG     # n_rows
    # beyond the fixed array's maximum, or outside the kernel it serves: a clear refusal, not a fault
    assert f(8192, 8192, 1, 3, 0, 0.9, p, 1, 8192, p, p, None) == binding.GBS_ERR_UNSUPPORTED
    assert f(18944, 20480, 20, 4, 0, 0.95, p, 1, 18944, p, p, None) == binding.GBS_ERR_UNSUPPORTED
    assert f(128, 128, 1, 3, 0, 1.0, p, 1, 128, p, p, None) == binding.GBS_ERR_UNSUPPORTED
    assert f(4096, 4096, 1, 3, 8, 0.9, p, 1, 4096, p, p, None) == binding.GBS_ERR_UNSUPPORTED
    assert f(3584, 3584, 44, 3, 0, 0.9, p, 1, 3584, p, p, None) in (binding.GBS_ERR_UNSUPPORTED,
                                                                     binding.GBS_ERR_INVALID_ARG)
    assert f(4096, 4096, 1, 3, 0, 0.9, p, 0, 4096, None, None, None) == binding.GBS_OK               # empty: no-op
    assert "UNSUPPORTED" in binding.status_string(binding.GBS_ERR_UNSUPPORTED)


@pytest.mark.gpu
def test_static_entry_point_matches_the_plan_based_call_twice_in_a_row():
    """Two calls in a row, then a change of (d_pad, m) that forces the array to be rewritten, then
    back again: every result must equal the plan-based entry point's bytes and scales exactly."""
    gbs_build.build()
    sequence = [("llama4096", 3, 613), ("llama4096", 3, 613), ("qwen3584", 3, 407), ("qwen3584", 3, 407),
                ("llama4096", 4, 5), ("qwen3584", 3, 1)]
    for name, bits, rows in sequence:
        w = synth.WORKLOADS[name]
        x = synth.make_host(name, rows, seed=77 + rows + bits).to(DEV)
        with Plan(w.d, w.d_pad, w.m, bits, w.group, w.alpha) as plan:
            codes_ref, scales_ref, _ = plan.rotate_quantize(x)
            codes = torch.full_like(codes_ref, 0xEE)
            scales = torch.full_like(scales_ref, -1.0)
            binding.gbs_rotate_quantize_static(w.d, w.d_pad, w.m, bits, w.group, w.alpha, x, codes, scales)
            torch.cuda.synchronize()
            assert torch.equal(codes, codes_ref), (name, bits, rows)
            assert torch.equal(scales, scales_ref), (name, bits, rows)
            assert plan.device_status() == 0
            assert binding.gbs_static_device_status() == 0          # the plan-free call's own status word


@pytest.mark.gpu
def test_static_entry_point_from_two_streams_with_the_same_table_after_a_change():
    """Callers on different streams that use the same (d_pad, m) may overlap: the shared table is rewritten on
    the stream of every call that is not ordered behind the last write, and all of them write the same bytes.
    A change of (d_pad, m) in between (serialised, as the header asks) must not leave either stream with a
    stale table."""
    gbs_build.build()
    s1, s2 = torch.cuda.Stream(DEV), torch.cuda.Stream(DEV)
    cases = []
    for name, bits, rows in (("llama4096", 3, 2048), ("qwen3584", 3, 1024)):
        w = synth.WORKLOADS[name]
        x = synth.make_host(name, rows, seed=5 + bits).to(DEV)
        with Plan(w.d, w.d_pad, w.m, bits, w.group, w.alpha) as plan:
            ref = plan.rotate_quantize(x)
            torch.cuda.synchronize()
        cases.append((w, bits, x, ref))
    for rounds in range(3):
        for w, bits, x, (codes_ref, scales_ref, _) in cases:
            outs = []
            for s in (s1, s2, s1, s2):                      # same table on both streams, back to back, no host sync
                codes = torch.full_like(codes_ref, 0xEE)
                scales = torch.full_like(scales_ref, -1.0)
                binding.gbs_rotate_quantize_static(w.d, w.d_pad, w.m, bits, w.group, w.alpha, x, codes, scales, stream=s)
                outs.append((codes, scales))
            torch.cuda.synchronize()                        # the change of table that follows is serialised
            for codes, scales in outs:
                assert torch.equal(codes, codes_ref) and torch.equal(scales, scales_ref), (w.name, rounds)
    assert binding.gbs_static_device_status() == 0


@pytest.mark.gpu
def test_static_entry_point_inside_a_captured_graph_and_eagerly_afterwards():
    """A captured call carries its own rewrite of the table, so a replay is right whatever ran in between,
    and eager calls made after a replay rewrite too."""
    gbs_build.build()
    wa, wb = synth.WORKLOADS["llama4096"], synth.WORKLOADS["qwen3584"]
    xa = synth.make_host("llama4096", 512, seed=11).to(DEV)
    xb = synth.make_host("qwen3584", 512, seed=12).to(DEV)
    with Plan(wa.d, wa.d_pad, wa.m, 4, wa.group, wa.alpha) as pa, Plan(wb.d, wb.d_pad, wb.m, 3, wb.group, wb.alpha) as pb:
        ca_ref, sa_ref, _ = pa.rotate_quantize(xa)
        cb_ref, sb_ref, _ = pb.rotate_quantize(xb)
        ca, sa = torch.zeros_like(ca_ref), torch.zeros_like(sa_ref)
        cb, sb = torch.zeros_like(cb_ref), torch.zeros_like(sb_ref)
        st = torch.cuda.Stream(DEV)
        binding.gbs_rotate_quantize_static(wa.d, wa.d_pad, wa.m, 4, wa.group, wa.alpha, xa, ca, sa, stream=st)   # set-up before capture
        st.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            binding.gbs_rotate_quantize_static(wa.d, wa.d_pad, wa.m, 4, wa.group, wa.alpha, xa, ca, sa, stream=st)
        for _ in range(2):
            binding.gbs_rotate_quantize_static(wb.d, wb.d_pad, wb.m, 3, wb.group, wb.alpha, xb, cb, sb, stream=st)  # other table, eager
            st.synchronize()
            assert torch.equal(cb, cb_ref) and torch.equal(sb, sb_ref)
            ca.zero_(); sa.zero_()
            torch.cuda.synchronize()
            g.replay()
            torch.cuda.synchronize()
            assert torch.equal(ca, ca_ref) and torch.equal(sa, sa_ref)
        assert binding.gbs_static_device_status() == 0
