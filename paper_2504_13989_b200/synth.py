"""Seeded synthetic inputs shaped like the paper's workloads.

The paper measures on activations and KV entries of Llama / Mistral / Qwen models
(Section 5.1); neither weights nor text are available here, so these tensors stand in
for them: heavy-tailed entries, a few outlier channels and a few massive-activation
tokens (the outlier structure of Section 2.2), at the widths the paper names (4096,
3584, the 18944-wide MLP).

This module holds input generation only -- none of the method's arithmetic -- and is
the one piece shared by the CPU oracle's tests and the CUDA path's tests/benchmark.
"""
from __future__ import annotations

import dataclasses

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    n_rows: int
    d: int
    d_pad: int
    m: int
    bits: tuple
    group: int
    alpha: float
    dtype: str          # "f32" | "bf16"
    dist: str           # "normal" | "student_t3" | "silu_gate"
    outlier_channels: int
    outlier_scale: float
    token_frac: float   # fraction of rows scaled by token_scale
    token_scale: float
    seed: int


WORKLOADS = {
    # tiny power-of-2 case the oracle finishes instantly
    "tiny": Workload("tiny", 64, 128, 128, 1, (4,), 0, 1.0, "f32", "normal", 2, 40.0, 0.0, 1.0, 0),
    # Llama/Mistral-like hidden activations
    "llama4096": Workload("llama4096", 4096, 4096, 4096, 1, (3, 4), 0, 0.9, "bf16", "student_t3",
                          16, 50.0, 0.01, 20.0, 1),
    # Qwen-like non-power-of-2 width, H_28 (x) H_128, per-group scales
    "qwen3584": Workload("qwen3584", 8192, 3584, 3584, 28, (3,), 128, 0.85, "bf16", "student_t3",
                         12, 60.0, 0.01, 20.0, 2),
    # MLP down_proj input with dimension expansion, H_20 (x) H_1024
    "mlp18944": Workload("mlp18944", 4096, 18944, 20480, 20, (4,), 0, 0.95, "bf16", "silu_gate",
                         32, 100.0, 0.0, 1.0, 3),
    # KV cache rows: (batch 16 x heads 32 x seq 4096) rows of head_dim 128
    "kv128": Workload("kv128", 16 * 32 * 4096, 128, 128, 1, (3,), 0, 1.0, "bf16", "student_t3",
                      4, 50.0, 0.0, 1.0, 4),
    # calibration activations for clip-ratio scoring (per layer; seed + layer)
    "calib4096": Workload("calib4096", 128 * 2048, 4096, 4096, 1, (3,), 0, 0.9, "bf16", "student_t3",
                          0, 1.0, 0.0, 1.0, 5),
}

TINY_OUTLIER_CHANNELS = (7, 93)   # the two fixed outlier channels of the tiny case


def _base_numpy(w: Workload, n_rows: int, rng: np.random.Generator) -> np.ndarray:
    if w.dist == "normal":
        x = rng.standard_normal((n_rows, w.d))
    elif w.dist == "student_t3":
        x = 0.5 * rng.standard_t(3.0, size=(n_rows, w.d))
    elif w.dist == "silu_gate":
        g = rng.standard_normal((n_rows, w.d))
        u = rng.standard_normal((n_rows, w.d))
        x = (g / (1.0 + np.exp(-g))) * u          # SiLU(gate) * up
    else:
        raise ValueError(w.dist)
    return x


def make_host(name: str, n_rows: int | None = None, seed: int | None = None) -> torch.Tensor:
    """CPU tensor [n_rows, d] in the workload's storage dtype (numpy PCG64, float64 then one cast)."""
    w = WORKLOADS[name]
    n = w.n_rows if n_rows is None else n_rows
    rng = np.random.Generator(np.random.PCG64(w.seed if seed is None else seed))
    x = _base_numpy(w, n, rng)
    if w.outlier_channels:
        if name == "tiny":
            ch = np.array(TINY_OUTLIER_CHANNELS)
        else:
            ch = rng.choice(w.d, size=w.outlier_channels, replace=False)
        x[:, ch] *= w.outlier_scale
    if w.token_frac > 0.0 and n > 0:
        n_tok = max(1, int(round(w.token_frac * n)))
        rows = rng.choice(n, size=n_tok, replace=False)
        x[rows, :] *= w.token_scale
    t = torch.from_numpy(x.astype(np.float32))
    return t if w.dtype == "f32" else t.to(torch.bfloat16)


def make_device(name: str, n_rows: int | None = None, seed: int | None = None,
                device: str = "cuda:0") -> torch.Tensor:
    """Same recipe drawn on the device (torch.Generator), for tensors too large to draw on the host.

    The stream differs from make_host; tests copy back the rows they check.
    """
    w = WORKLOADS[name]
    n = w.n_rows if n_rows is None else n_rows
    gen = torch.Generator(device=device)
    gen.manual_seed(w.seed if seed is None else seed)
    dt = torch.float32
    if w.dist == "normal":
        x = torch.randn((n, w.d), generator=gen, device=device, dtype=dt)
    elif w.dist == "student_t3":
        # t_3 = z / sqrt(chi2_3 / 3), chi2_3 as a sum of three squared normals
        x = torch.randn((n, w.d), generator=gen, device=device, dtype=dt)
        c = torch.zeros_like(x)
        for _ in range(3):
            c.addcmul_(*(2 * [torch.randn((n, w.d), generator=gen, device=device, dtype=dt)]))
        x.div_(c.div_(3.0).sqrt_()).mul_(0.5)
        del c
    elif w.dist == "silu_gate":
        g = torch.randn((n, w.d), generator=gen, device=device, dtype=dt)
        u = torch.randn((n, w.d), generator=gen, device=device, dtype=dt)
        x = torch.nn.functional.silu(g) * u
        del g, u
    else:
        raise ValueError(w.dist)
    if w.outlier_channels:
        ch = torch.randperm(w.d, generator=gen, device=device)[: w.outlier_channels]
        x[:, ch] *= w.outlier_scale
    if w.token_frac > 0.0 and n > 0:
        n_tok = max(1, int(round(w.token_frac * n)))
        rows = torch.randperm(n, generator=gen, device=device)[:n_tok]
        x[rows, :] *= w.token_scale
    return x if w.dtype == "f32" else x.to(torch.bfloat16)


def to_oracle_array(t: torch.Tensor) -> np.ndarray:
    """CPU view the oracle accepts: float32 array, or uint16 array of bf16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.float32:
        return t.numpy()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    raise ValueError("unsupported dtype %s" % t.dtype)


def to_float64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()
