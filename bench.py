#!/usr/bin/env python
"""Benchmark of the fused rotate-and-quantize hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One STEP = one pass of the fused path over one batch of the headline workload: the 4096-token x
d=4096 bf16 activation batch, quantized at b=3 and at b=4 (two launches of the fused kernel, as the
workload names both bit-widths).  Inputs are synthetic, resident in HBM before the timed region; the
launches rotate over NSETS distinct buffer sets whose footprint exceeds 4x the L2 so every launch
reads from HBM.  The K steps are replayed from CUDA graphs, bracketed by a barrier and a device
synchronise, timed with CUDA events on the launching stream, max over ranks; they are repeated whole
times until the timed region lasts --min-ms (50 ms by default; `steps_timed` says how many ran).

Prints ONE JSON line.  `value` is GB/s of algorithmic bytes (row in, packed codes + scales out).
Extra keys: `roofline` (d=4096) and `roofline_d3584` (the metric's second width, its own timed loop), each
with the size-matched plain copy beside the measured peak, `cpu_baseline`, `e2e`, `clocks`, `gpu_launches`,
and `also` (every other workload and entry point, timed outside the K steps, for context).

The path does not shard: with --gpus N every rank runs an independent replica on its own GPU.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "rotate+quantize GB/s and Mtokens/s at d=4096/3584, % of B200 HBM peak"
HEADLINE = "llama4096"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the fused kernel on the headline
# workload, from the ncu capture summarised under profiles/ (None until a capture exists).
NCU_TRAFFIC_BYTES_PER_LAUNCH = 33_624_064   # dram reads 33.62 MB + writes 0 (codes still in L2 at kernel end); profiles/uv_rq_llama4096.md
NCU_TRAFFIC_BYTES_PER_LAUNCH_D3584 = 59_470_592   # 58.79 MB read + 0.68 MB written; profiles/uv_rq_qwen3584.md


def algorithmic_bytes(n_rows: int, d: int, d_pad: int, bits: int, group: int, in_bytes: int) -> int:
    """Bytes the method must move per launch: the row in, packed codes and scales out."""
    spr = d_pad // group if group else 1
    return n_rows * (d * in_bytes + d_pad * bits // 8 + 4 * spr)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measured_bf16_tflops():
    """Dense bf16 tensor throughput measured on this machine (burst figure: for a kernel timed alone)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    except Exception:
        return 1590.0, "fallback"


def aggregate(local_ms: float, local_units: float, dist_ok: bool, device=None):
    """Whole-job figures: time = max over ranks, units = sum over ranks (replicas are independent)."""
    if not dist_ok:
        return local_ms, local_units
    import torch.distributed as dist
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the benchmark runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.timed = [], []
        self.in_timed = False
        self._stop_evt = threading.Event()
        self.max_mhz = None
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if vis:
                ids = [v for v in vis.split(",") if v.strip() != ""]
                if index < len(ids) and ids[index].strip().isdigit():
                    phys = int(ids[index])
            self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self._stop_evt.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                util = nv.nvmlDeviceGetUtilizationRates(self.h).gpu
                rec = (mhz, int(reasons), util)
                self.samples.append(rec)
                if self.in_timed:
                    self.timed.append(rec)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()

    def mark(self) -> int:
        return len(self.samples)

    def median_mhz_since(self, mark: int):
        """Median SM clock of the samples taken since mark() while the GPU was busy (None without samples)."""
        pool = [s[0] for s in self.samples[mark:] if s[2] > 0] or [s[0] for s in self.samples[mark:]]
        return statistics.median(pool) if pool else None

    def summary(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        nv = self.nv
        pool = self.timed if len(self.timed) >= 3 else [s for s in self.samples if s[2] > 0] or self.samples
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        seen = [n for n, bit in names.items() if any(s[1] & bit for s in pool)]
        return {"sm_mhz": statistics.median(s[0] for s in pool), "sm_max_mhz": self.max_mhz,
                "reasons": seen, "samples": len(pool),
                "window": "timed" if pool is self.timed else "under_load"}


def time_oracle(x_host, w, bits_list, min_seconds: float, nthreads: int = 0):
    """Time the float64 CPU oracle (as it stands) on whole-batch steps for about min_seconds."""
    import oracle
    from paper_2504_13989_b200 import synth
    xa = synth.to_oracle_array(x_host)
    steps, t0 = 0, time.perf_counter()
    while True:
        for b in bits_list:
            oracle.rotate_quantize_rows(xa, w.d, w.d_pad, w.m, b, w.group, w.alpha, dense=False,
                                        want_y=False, want_q=False, want_packed=True, nthreads=nthreads)
        steps += 1
        el = time.perf_counter() - t0
        if el >= min_seconds:
            return steps, el


def run_reference(args, rank: int):
    """Reference arm: the CPU oracle, as it stands, on the host cores (rank 0 only).

    Each step is a bounded sample of the headline batch: the first `rows` token rows, quantized at
    b=3 and b=4.  `rows` is sized from a short calibration so that K + W steps end within about two
    minutes; the reported rate does not depend on it.
    """
    if rank != 0:
        return
    import oracle
    from paper_2504_13989_b200 import synth
    w = synth.WORKLOADS[HEADLINE]
    cores = oracle.max_threads()
    x_full = synth.make_host(HEADLINE, 1024)

    def one_step(xa):
        for b in w.bits:
            oracle.rotate_quantize_rows(xa, w.d, w.d_pad, w.m, b, w.group, w.alpha,
                                        dense=False, want_y=False, want_q=False, want_packed=True)
    probe = synth.to_oracle_array(x_full[:128])
    one_step(probe)
    t0 = time.perf_counter()
    one_step(probe)
    per_row = (time.perf_counter() - t0) / 128
    budget = 120.0
    rows = int(budget / ((args.steps + args.warmup) * per_row))
    rows = max(8, min(1024, rows))
    xa = synth.to_oracle_array(x_full[:rows])
    step_bytes = sum(algorithmic_bytes(rows, w.d, w.d_pad, b, w.group, 2) for b in w.bits)
    for _ in range(args.warmup):
        one_step(xa)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one_step(xa)
    el = time.perf_counter() - t0
    ms = el * 1e3 / args.steps
    gbs = step_bytes / (ms * 1e-3) / 1e9
    sample = "first %d of %d rows of the batch per step, b=3 and b=4, butterfly rotation, OpenMP over rows" % (
        rows, w.n_rows)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s: %d of %d tokens x d=%d bf16, b=3 and b=4, per-token, alpha=%.2f" %
                   (HEADLINE, rows, w.n_rows, w.d, w.alpha)},
        "mtokens_per_s": len(w.bits) * rows / (ms * 1e-3) / 1e6,
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def build_sets(plan_list, x_base, nsets, device):
    """NSETS distinct input/output buffer sets (inputs are row-rolled copies of the same batch)."""
    sets = []
    for i in range(nsets):
        x = torch.roll(x_base, shifts=i * 17, dims=0).contiguous().to(device)
        outs = [pl.alloc_outputs(x.shape[0], device) for pl in plan_list]
        sets.append((x, outs))
    return sets


def run_step(plan_list, sets, i):
    """One step: every plan's launch over one batch.  Launch j of step i reads the batch copy of buffer set
    i + j * nsets / len(plans), so that no launch finds its input in L2 from the launch before it."""
    nsets = len(sets)
    for j, pl in enumerate(plan_list):
        x = sets[(i + j * (nsets // len(plan_list))) % nsets][0]
        pl.rotate_quantize(x, out=sets[i % nsets][1][j])


def capture(plan_list, sets, idx_list, stream):
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for i in idx_list:
            run_step(plan_list, sets, i)
    return g


MIN_TIMED_MS = 50.0      # a timed region shorter than this is repeated (whole multiples of the K steps)


def timed_graph_loop(plan_list, sets, steps, warmup, stream, dist_ok, sampler=None, min_ms=MIN_TIMED_MS):
    """Time `steps` steps replayed from CUDA graphs, repeated R >= 1 times so that the timed region lasts at
    least min_ms; returns (local milliseconds, steps actually timed = R * steps)."""
    nsets = len(sets)
    with torch.cuda.stream(stream):
        for i in range(max(warmup, 3)):
            run_step(plan_list, sets, i % nsets)
    stream.synchronize()
    g_all = capture(plan_list, sets, list(range(nsets)), stream)
    rem = steps % nsets
    g_rem = capture(plan_list, sets, list(range(rem)), stream) if rem else None

    def k_steps():
        for _ in range(steps // nsets):
            g_all.replay()
        if g_rem is not None:
            g_rem.replay()

    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        g_all.replay()
        start.record(stream)
        g_all.replay()
        end.record(stream)
    stream.synchronize()
    est_ms = start.elapsed_time(end) / nsets * steps             # one pass over the K steps
    reps = max(1, int(np.ceil(min_ms / max(est_ms, 1e-6))))
    if dist_ok:
        r = torch.tensor([reps], dtype=torch.int64, device=sets[0][0].device)
        torch.distributed.all_reduce(r, op=torch.distributed.ReduceOp.MAX)
        reps = int(r.item())
    if dist_ok:
        torch.distributed.barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.in_timed = True
    with torch.cuda.stream(stream):
        start.record(stream)
        for _ in range(reps):
            k_steps()
        end.record(stream)
    if dist_ok:
        torch.distributed.barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.in_timed = False
    return start.elapsed_time(end), steps * reps


def plain_traffic(stream, device, read_bytes, write_bytes, min_ms=20.0):
    """Size-matched denominators under the same protocol (graph replay, buffers rotating through > 4x L2):
    a plain device copy that moves read_bytes + write_bytes in total (half of it read, half written), and a
    plain fill of write_bytes.  Returns (copy GB/s of bytes read + written, fill GB/s)."""
    out = []
    for kind, nbytes in (("copy", (read_bytes + write_bytes) // 2), ("fill", write_bytes)):
        nbytes = max(1024, nbytes // 16 * 16)
        nsets = max(2, min(32, int(4 * 126e6 / nbytes) + 1))
        src = [torch.empty(nbytes, dtype=torch.uint8, device=device).fill_(i) for i in range(nsets)] if kind == "copy" else None
        dst = [torch.empty(nbytes, dtype=torch.uint8, device=device) for _ in range(nsets)]
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            for i in range(min(3, nsets)):
                dst[i].copy_(src[i]) if kind == "copy" else dst[i].fill_(7)
        stream.synchronize()
        with torch.cuda.graph(g, stream=stream):
            for i in range(nsets):
                dst[i].copy_(src[(i + nsets // 2) % nsets]) if kind == "copy" else dst[i].fill_(7)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            g.replay()
            a.record(stream)
            g.replay()
            b.record(stream)
        stream.synchronize()
        reps = max(1, int(np.ceil(min_ms / max(a.elapsed_time(b), 1e-6))))
        with torch.cuda.stream(stream):
            a.record(stream)
            for _ in range(reps):
                g.replay()
            b.record(stream)
        stream.synchronize()
        ms = a.elapsed_time(b) / (reps * nsets)
        moved = 2 * nbytes if kind == "copy" else nbytes
        out.append(moved / ms / 1e6)
        del src, dst, g
        torch.cuda.empty_cache()
    return out[0], out[1]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--nsets", type=int, default=16)
    ap.add_argument("--e2e-chunks", type=int, default=4, help="row chunks of the host-buffer pipeline (copies overlap)")
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--no-extras", action="store_true", help="skip the context legs under `also`")
    ap.add_argument("--min-ms", type=float, default=MIN_TIMED_MS,
                    help="the K steps are repeated until the timed region lasts this long (0: exactly K steps)")
    ap.add_argument("--profile", default=None, metavar="WORKLOAD[:ROWS]",
                    help="launch one workload's kernel a few times and exit (for ncu captures), e.g. kv128:262144, llama4096-inverse:4096, "
                         "clip:8192")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the product path has no CPU fallback")
    if args.gpus > 1 and world != args.gpus:
        raise SystemExit("bench.py: --gpus %d must be launched with torch.distributed.run (WORLD_SIZE=%d)" %
                         (args.gpus, world))
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    dist_ok = world > 1
    if dist_ok:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    from paper_2504_13989_b200 import HostPipeline, Plan, synth
    from paper_2504_13989_b200 import build as gbs_build
    gbs_build.build()

    if args.profile:
        run_profile(args.profile, device)
        return

    sampler = ClockSampler(local_rank, period_s=0.005)
    sampler.start()

    w = synth.WORKLOADS[HEADLINE]
    x_base = synth.make_host(HEADLINE)                       # seeded; every rank draws the same batch
    plans = [Plan(w.d, w.d_pad, w.m, b, w.group, w.alpha) for b in w.bits]
    sets = build_sets(plans, x_base, args.nsets, device)
    stream = torch.cuda.Stream(device)
    step_bytes = sum(algorithmic_bytes(w.n_rows, w.d, w.d_pad, b, w.group, 2) for b in w.bits)
    step_tokens = len(w.bits) * w.n_rows
    launches_per_step = len(w.bits)

    local_ms, steps_timed = timed_graph_loop(plans, sets, args.steps, args.warmup, stream, dist_ok, sampler,
                                             min_ms=args.min_ms)
    total_ms, total_bytes = aggregate(local_ms, step_bytes * steps_timed, dist_ok, device)
    _, total_tokens = aggregate(local_ms, step_tokens * steps_timed, dist_ok, device)
    ms_per_step = total_ms / steps_timed
    value = total_bytes / (total_ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak()

    # roofline of the fused kernel on this rank: algorithmic bytes per launch / mean launch duration
    launch_ms = local_ms / (steps_timed * launches_per_step)
    achieved = (step_bytes / launches_per_step) / (launch_ms * 1e-3) / 1e9
    del sets
    torch.cuda.empty_cache()
    copy_gbs, _ = plain_traffic(stream, device, w.n_rows * w.d * 2, step_bytes // launches_per_step - w.n_rows * w.d * 2)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH, "peak_kind": "of " + peak_kind,
                "kernel": "fused rotate-quantize at d=4096, mean of the b=3 and b=4 launches",
                "frac_of_8000_nominal": achieved / 8000.0,
                "copy_same_size_gbs": copy_gbs,
                "copy_same_size_note": "plain device copy moving the same %.1f MB per launch (read + written), same "
                                       "graph-replay protocol; context beside `peak`, not a replacement" %
                                       (step_bytes / launches_per_step / 1e6)}

    # the metric's second width, d = 3584 (H_28 (x) H_128, groups of 128): its own timed loop and roofline object
    w2 = synth.WORKLOADS["qwen3584"]
    plans2 = [Plan(w2.d, w2.d_pad, w2.m, b, w2.group, w2.alpha) for b in w2.bits]
    bytes2 = sum(algorithmic_bytes(w2.n_rows, w2.d, w2.d_pad, b, w2.group, 2) for b in w2.bits)
    sets2 = build_sets(plans2, synth.make_host("qwen3584"), 8, device)
    steps2 = max(8, args.steps // 2 // 8 * 8)
    ms2, timed2 = timed_graph_loop(plans2, sets2, steps2, 3, stream, False, min_ms=args.min_ms)
    del sets2
    torch.cuda.empty_cache()
    ach2 = bytes2 / (ms2 / timed2 * 1e-3) / 1e9
    copy2, _ = plain_traffic(stream, device, w2.n_rows * w2.d * 2, bytes2 - w2.n_rows * w2.d * 2)
    roofline_d3584 = {"bound": "hbm", "achieved": ach2, "peak": peak, "unit": "GB/s", "frac": ach2 / peak,
                      "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH_D3584, "peak_kind": "of " + peak_kind,
                      "kernel": "fused rotate-quantize at d=3584 (8192 tokens, b=3, groups of 128)",
                      "us_per_launch": ms2 / timed2 * 1e3, "steps_timed": timed2,
                      "mtokens_per_s": w2.n_rows / (ms2 / timed2) / 1e3,
                      "frac_of_8000_nominal": ach2 / 8000.0, "copy_same_size_gbs": copy2}

    # ---- end to end through the public API with host buffers (copies inside the timed region)
    x_pin = x_base.pin_memory()
    host_outs = []
    for pl in plans:
        host_outs.append((torch.empty((w.n_rows, pl.info.code_bytes_per_row), dtype=torch.uint8).pin_memory(),
                          torch.empty((w.n_rows, pl.info.scales_per_row), dtype=torch.float32).pin_memory()))
    e2e_steps = max(3, min(args.steps, 60))

    pipe = HostPipeline(plans, w.n_rows, device=device, chunks=args.e2e_chunks)

    def e2e_step():
        pipe.run(x_pin, host_outs, stream=stream)
    for _ in range(3):
        e2e_step()
    stream.synchronize()
    if dist_ok:
        torch.distributed.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    stream.synchronize()
    e2e_ms_local = e0.elapsed_time(e1)
    e2e_ms, e2e_bytes = aggregate(e2e_ms_local, step_bytes * e2e_steps, dist_ok, device)
    h2d = x_pin.numel() * x_pin.element_size()
    d2h = sum(c.numel() + 4 * s.numel() for c, s in host_outs)
    e2e = {"value": e2e_bytes / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps}

    # ---- context legs (outside the K timed steps)
    also = {}
    if not args.no_extras and rank == 0:
        also = extras(device, stream, args, peak, sampler)

    sampler.stop()
    clocks = sampler.summary()

    # ---- the oracle timed beside it, rank 0 at N=1 only
    cpu_baseline = None
    if rank == 0 and world == 1 and args.cpu_seconds > 0:
        import oracle
        n_steps, el = time_oracle(x_base, w, w.bits, args.cpu_seconds)
        cpu_baseline = {"value": step_bytes * n_steps / el / 1e9, "unit": "GB/s", "cores": oracle.max_threads(),
                        "kind": "oracle", "mtokens_per_s": step_tokens * n_steps / el / 1e6,
                        "sample": "%d whole-batch steps (4096 rows, b=3 and b=4) in %.1f s, butterfly rotation, "
                                  "OpenMP over rows" % (n_steps, el)}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "steps_timed": steps_timed,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "%s: %d tokens x d=%d bf16, H_%d, b=3 and b=4 (one launch each per step), "
                                   "per-token scales, alpha=%.2f" % (HEADLINE, w.n_rows, w.d, w.d_pad, w.alpha),
                       "replicas": world, "l2": "inputs rotate over %d buffer sets (%.0f MB > 4x L2); the b=3 and b=4 launches of a step read "
                       "different copies" %
                       (args.nsets, args.nsets * (step_bytes + w.n_rows * w.d * 2) / 1e6),
                       "launch": "CUDA graph replay", "levels": "D=2^(b-1)-1",
                       "timed_region": "the K steps repeated %d time(s): at least %.0f ms on the device" %
                                       (steps_timed // args.steps, args.min_ms)},
            "mtokens_per_s": total_tokens / (total_ms * 1e-3) / 1e6,
            "hbm_frac_of_measured": value / world / peak, "hbm_frac_of_8000": value / world / 8000.0,
            "roofline": roofline, "roofline_d3584": roofline_d3584, "cpu_baseline": cpu_baseline, "e2e": e2e, "clocks": clocks,
            "gpu_launches": steps_timed * launches_per_step, "also": also,
        }
        print(json.dumps(line))
    if dist_ok:
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()


def run_profile(spec, device):
    """A few launches of one kernel on a small case, for an ncu capture (prints nothing a result line would)."""
    from paper_2504_13989_b200 import Plan, synth
    name, _, rows = spec.partition(":")
    if name in ("matmul", "dense1544"):
        n = int(rows) if rows else 4096
        if name == "matmul":          # the consumer: 4-bit codes x 4-bit codes, n tokens x n output channels x 4096
            px, pw = Plan(4096, 4096, 1, 4, 0, 0.9), Plan(4096, 4096, 1, 4, 0, 1.0)
            xq = synth.make_device("llama4096", n, device=str(device))
            wq = (torch.randn((n, 4096), device=device) / 64).to(torch.bfloat16)
            cx, sx, _ = px.rotate_quantize(xq)
            cw, sw = pw.weight_rotate_quantize(wq)
            out = torch.empty((n, n), dtype=torch.bfloat16, device=device)
            for _ in range(4):
                px.quantized_matmul(cx, sx, pw, cw, sw, out=out)
            torch.cuda.synchronize()
            print(json.dumps({"profile": spec, "rows": n, "status": px.device_status()}))
        else:                         # the full Paley order: width 1536 -> d' = m = 1544
            pl = Plan(1536, 1544, 1544, 3, 0, 0.9)
            xq = (torch.randn((n, 1536), device=device) * 0.5).to(torch.bfloat16)
            outs = pl.alloc_outputs(n, device)
            for _ in range(4):
                pl.rotate_quantize(xq, out=outs)
            torch.cuda.synchronize()
            print(json.dumps({"profile": spec, "rows": n, "kernel_family": pl.info.variant, "status": pl.device_status()}))
        return
    clip = name == "clip"
    inverse = name.endswith("-inverse")               # e.g. llama4096-inverse: gbs_dequantize with inverse rotation
    if inverse:
        name = name[:-len("-inverse")]
    plain_dq = name.endswith("-dequantize")           # e.g. llama4096-dequantize: gbs_dequantize, rotated domain
    if plain_dq:
        name = name[:-len("-dequantize")]
    w = synth.WORKLOADS["calib4096" if clip else name]
    n = int(rows) if rows else min(w.n_rows, 8192)
    bits = w.bits[0]
    x = synth.make_device(w.name, n, device=str(device))
    pl = Plan(w.d, w.d_pad, w.m, bits, w.group, w.alpha)
    outs = pl.alloc_outputs(n, device)
    err = torch.zeros(32, dtype=torch.float64, device=device)
    xhat = torch.empty((n, w.d), dtype=torch.bfloat16, device=device) if inverse else None
    yhat = torch.empty((n, w.d_pad), dtype=torch.bfloat16, device=device) if plain_dq else None
    for _ in range(6):
        if clip:
            pl.clip_error(x, np.linspace(0.5, 1.0, 32), err_sum=err)
        else:
            pl.rotate_quantize(x, out=outs)
            if inverse:
                pl.dequantize(outs[0], outs[1], inverse=True, out=xhat)
            if plain_dq:
                pl.dequantize(outs[0], outs[1], out=yhat)
    torch.cuda.synchronize()
    print(json.dumps({"profile": spec, "rows": n, "kernel_family": pl.info.variant, "status": pl.device_status()}))


def extras(device, stream, args, peak, sampler=None):
    """Context figures for the other workloads / entry points (not part of the K timed steps)."""
    from paper_2504_13989_b200 import Plan, synth
    out = {}

    def time_loop(fn, iters, min_ms=20.0):
        """Mean milliseconds per call of fn(i), i < iters, replayed from a CUDA graph (no host launch cost in
        the figure) for at least min_ms."""
        with torch.cuda.stream(stream):
            for _ in range(3):
                fn(0)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(iters):
                fn(i)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            g.replay()
            a.record(stream)
            g.replay()
            b.record(stream)
        stream.synchronize()
        reps = max(1, int(np.ceil(min_ms / max(a.elapsed_time(b), 1e-6))))
        with torch.cuda.stream(stream):
            a.record(stream)
            for _ in range(reps):
                g.replay()
            b.record(stream)
        stream.synchronize()
        return a.elapsed_time(b) / (iters * reps)

    def rq_leg(name, bits, n_rows=None, xb=None, min_ms=20.0):
        """One rotate-quantize workload: graph replay over buffer sets > 4x L2, at least min_ms timed."""
        w = synth.WORKLOADS[name]
        if xb is None:
            xb = synth.make_host(name) if name != "kv128" else synth.make_device(name, device=str(device))
        n = xb.shape[0]
        pl = Plan(w.d, w.d_pad, w.m, bits, w.group, w.alpha)
        nbytes = algorithmic_bytes(n, w.d, w.d_pad, bits, w.group, 2)
        nsets = max(2, min(16, int(4 * 126e6 / (nbytes + 1)) + 1))
        sets = build_sets([pl], xb, nsets, device)
        ms, timed = timed_graph_loop([pl], sets, nsets, 3, stream, False, min_ms=min_ms)
        ms /= timed
        rec = {"us_per_launch": ms * 1e3, "gbs": nbytes / ms / 1e6, "frac_of_measured": nbytes / ms / 1e6 / peak,
               "frac_of_8000": nbytes / ms / 1e6 / 8000.0, "mrows_per_s": n / ms / 1e3,
               "kernel_family": pl.info.variant, "launches_timed": timed}
        del sets, pl
        torch.cuda.empty_cache()
        return rec

    # per-bit figures of every rotate-quantize workload
    for name in ("llama4096", "qwen3584", "mlp18944", "kv128"):
        w = synth.WORKLOADS[name]
        xb = synth.make_host(name) if name != "kv128" else synth.make_device(name, device=str(device))
        for b in w.bits:
            out["%s_b%d" % (name, b)] = rq_leg(name, b, xb=xb)
        del xb
        torch.cuda.empty_cache()
    # the asymmetric KV quantizer (group 128 = one row) on the same KV tensor
    w = synth.WORKLOADS["kv128"]
    xb = synth.make_device("kv128", device=str(device))
    pl = Plan(w.d, w.d_pad, w.m, 3, 128, 1.0, asymmetric=True)
    nbytes = w.n_rows * (w.d * 2 + w.d_pad * 3 // 8 + 8)
    sets = build_sets([pl], xb, 2, device)
    ms, timed = timed_graph_loop([pl], sets, 2, 3, stream, False, min_ms=20.0)
    ms /= timed
    out["kv128_b3_asymmetric_group128"] = {"us_per_launch": ms * 1e3, "gbs": nbytes / ms / 1e6,
                                           "frac_of_measured": nbytes / ms / 1e6 / peak}
    del sets, pl, xb
    torch.cuda.empty_cache()
    # steady state of the two widths of the metric: 65536 tokens per launch (the batch tiled)
    for name, reps in (("llama4096", 16), ("qwen3584", 8)):
        xb = synth.make_host(name).repeat(reps, 1)
        out["%s_b3_65536rows" % name] = rq_leg(name, 3, xb=xb)
        del xb
    # the wide kernel away from the launch boundaries: four MLP batches tiled into one launch
    xb = synth.make_host("mlp18944").repeat(4, 1)
    out["mlp18944_b4_16384rows"] = rq_leg("mlp18944", 4, xb=xb)
    del xb
    # dequantize on the headline workload, with the plain fill of the same output bytes beside it
    w = synth.WORKLOADS["llama4096"]
    x = synth.make_host("llama4096").to(device)
    pl = Plan(w.d, w.d_pad, w.m, 3, w.group, w.alpha)
    codes, scales, _ = pl.rotate_quantize(x)
    yhat = [torch.empty((w.n_rows, w.d_pad), dtype=torch.bfloat16, device=device) for _ in range(16)]
    ms = time_loop(lambda i: pl.dequantize(codes, scales, out=yhat[i % 16], stream=stream), 48)
    dq_in, dq_out = w.n_rows * (w.d_pad * 3 // 8 + 4), w.n_rows * w.d_pad * 2
    copy_gbs, fill_gbs = plain_traffic(stream, device, dq_in, dq_out)
    fill_us = dq_out / fill_gbs / 1e3
    out["dequantize_b3_bf16"] = {"us_per_launch": ms * 1e3, "gbs": (dq_in + dq_out) / ms / 1e6,
                                 "frac_of_measured": (dq_in + dq_out) / ms / 1e6 / peak,
                                 "fill_same_output_bytes_us": fill_us, "fill_same_output_bytes_gbs": fill_gbs,
                                 "copy_same_size_gbs": copy_gbs,
                                 "note": "write-bound: %.1f of its %.1f MB are output; a plain fill of that output alone "
                                         "takes the time beside it" % (dq_out / 1e6, (dq_in + dq_out) / 1e6)}
    xhat = yhat
    ms = time_loop(lambda i: pl.dequantize(codes, scales, inverse=True, out=xhat[i % 16], stream=stream), 48)
    out["dequantize_inverse_rotate_b3_bf16"] = {"us_per_launch": ms * 1e3,
                                                "gbs": w.n_rows * (w.d_pad * 3 // 8 + 4 + w.d * 2) / ms / 1e6}
    del xhat, x, codes, scales, yhat
    torch.cuda.empty_cache()
    # the consumer of the codes: the layer's output from the packed codes of activations and weights (int8 x int8
    # -> int32 on the tensor cores), 4096 tokens x 4096 output channels x d' = 4096
    bf16_tf, bf16_kind = measured_bf16_tflops()
    i8_peak = 2.0 * bf16_tf                      # nominal dense int8 : bf16 ratio of the part (4.5 : 2.25 PFLOP/s)
    xq = synth.make_host("llama4096").to(device)
    wq = (torch.randn((4096, w.d), generator=torch.Generator().manual_seed(7)) / 64.0).to(torch.bfloat16).to(device)
    for bx, bw in ((4, 4), (3, 3)):
        px, pw = Plan(w.d, w.d_pad, w.m, bx, 0, w.alpha), Plan(w.d, w.d_pad, w.m, bw, 0, 1.0)
        cx, sx, _ = px.rotate_quantize(xq)
        cw, sw = pw.weight_rotate_quantize(wq)
        outm = torch.empty((xq.shape[0], wq.shape[0]), dtype=torch.bfloat16, device=device)
        ms = time_loop(lambda i: px.quantized_matmul(cx, sx, pw, cw, sw, out=outm, stream=stream), 8)
        tops = 2.0 * xq.shape[0] * wq.shape[0] * w.d_pad / ms / 1e9
        out["quantized_matmul_x%d_w%d_4096x4096x4096" % (bx, bw)] = {
            "us_per_launch": ms * 1e3, "tops": tops,
            "roofline": {"bound": "tensor", "unit": "TOP/s", "achieved": tops, "peak": i8_peak, "frac": tops / i8_peak,
                         "note": "int8 peak = 2 x the %s bf16 figure (nominal int8 : bf16 ratio); the kernel is bound by "
                                 "unpacking the codes to int8, not by the tensor pipe" % bf16_kind}}
        del px, pw, cx, sx, cw, sw, outm
    ms = time_loop(lambda i: torch.matmul(xq, wq.t()), 8)
    out["bf16_matmul_of_the_unquantized_operands_4096x4096x4096"] = {"us_per_launch": ms * 1e3,
                                                                     "note": "library GEMM, context only"}
    del xq, wq
    torch.cuda.empty_cache()
    # the full Paley order (width 1536 -> d' = m = 1544): the rotation is a dense contraction with H_m, forward in
    # two sweeps (max|.|, then quantize: 2 x 2 m^2 flops per token), inverse in one (2 m d flops per token)
    pd = Plan(1536, 1544, 1544, 3, 0, 0.9)
    for n_d in (4096, 65536):
        xd = (torch.randn((n_d, 1536), generator=torch.Generator().manual_seed(11)) * 0.5).to(torch.bfloat16).to(device)
        od = pd.alloc_outputs(n_d, device)
        ms = time_loop(lambda i: pd.rotate_quantize(xd, out=od, stream=stream), 4)
        tf = 2.0 * 2.0 * n_d * 1544.0 * 1544.0 / ms / 1e9
        out["paley1544_b3_%d_rows" % n_d] = {
            "us_per_launch": ms * 1e3, "mrows_per_s": n_d / ms / 1e3, "kernel_family": pd.info.variant,
            "roofline": {"bound": "tensor", "unit": "TFLOP/s", "achieved": tf, "peak": bf16_tf, "frac": tf / bf16_tf,
                         "note": "two dense sweeps with H_1544 per token; peak = the %s bf16 figure" % bf16_kind}}
        if True:
            xh = torch.empty((n_d, 1536), dtype=torch.bfloat16, device=device)
            ms = time_loop(lambda i: pd.dequantize(od[0], od[1], inverse=True, out=xh, stream=stream), 4)
            tf = 2.0 * n_d * 1544.0 * 1536.0 / ms / 1e9
            out["paley1544_b3_inverse_dequantize_%d_rows" % n_d] = {
                "us_per_launch": ms * 1e3,
                "roofline": {"bound": "tensor", "unit": "TFLOP/s", "achieved": tf, "peak": bf16_tf, "frac": tf / bf16_tf,
                             "note": "codes unpacked to bf16 in the CTA, one dense contraction with H_1544"}}
            del xh
        del xd, od
    del pd
    torch.cuda.empty_cache()
    # clip-ratio scoring at the calibration size: K = 32 candidates over one full layer of 128 sequences x 2048
    # tokens x d = 4096 per launch, for each of 32 layers (its own seeded tensor each: seed 5 + layer)
    wc = synth.WORKLOADS["calib4096"]
    alphas = np.linspace(0.5, 1.0, 32)
    layer_ms = []
    mark = sampler.mark() if sampler else 0
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for layer in range(32):
        xc = synth.make_device("calib4096", wc.n_rows, seed=wc.seed + layer, device=str(device))
        err = torch.zeros(32, dtype=torch.float64, device=device)
        if layer == 0:
            pl.clip_error(xc[:4096], alphas, err_sum=err, stream=stream)          # warm-up launch
            err.zero_()
        stream.synchronize()
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            a.record(stream)
            pl.clip_error(xc, alphas, err_sum=err, stream=stream)
            b.record(stream)
        stream.synchronize()
        layer_ms.append(a.elapsed_time(b))
        if layer == 31:
            t0 = time.perf_counter()
            res = pl.search_clip_ratio(xc, 1.0 / 64, stream=stream)
            dt = time.perf_counter() - t0
        del xc, err
    sm_mhz = (sampler.median_mhz_since(mark) if sampler else None) or 1965.0
    ms = statistics.median(layer_ms)
    evals = wc.n_rows * wc.d_pad * 32
    alu_peak = 148 * 128 * sm_mhz * 1e6                   # fp32 lanes x sampled SM clock: lane-operations per second
    out["clip_error_K32"] = {"ms_per_layer_262144_tokens": ms, "ms_32_layers": sum(layer_ms),
                             "ms_per_layer_min_max": [min(layer_ms), max(layer_ms)],
                             "gevals_per_s": evals / ms / 1e6, "mtokens_per_s": wc.n_rows / ms / 1e3,
                             "hbm_gbs": wc.n_rows * wc.d * 2 / ms / 1e6,
                             "roofline": {"bound": "alu", "unit": "Glane-op/s", "achieved": 5 * evals / ms / 1e6,
                                          "peak": alu_peak / 1e9, "frac": 5 * evals / ms / 1e6 / (alu_peak / 1e9),
                                          "sm_mhz_sampled": sm_mhz,
                                          "note": "5 fp32 operations per value and candidate; peak = 148 SMs x 128 "
                                                  "lanes x the SM clock sampled during these launches"}}
    # Algorithm 1's bracket search on the last layer's tensor (eps = 1/64): rounds of <= 31 probes, blocking
    out["search_clip_ratio_eps_1_64"] = {"alpha": res.alpha, "iterations": res.iterations, "rounds": res.rounds,
                                         "evaluations": res.evaluations, "wall_ms_per_layer_262144_tokens": dt * 1e3}
    return out


if __name__ == "__main__":
    main()
