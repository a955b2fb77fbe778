"""Shared pieces of the GPU parity tests: seeded problems, error metrics, tolerances.

Tolerances are the benchmark contract's: bf16 inputs with fp32 accumulation -> max abs error <= 2e-2
and mean abs error <= 2e-3 on outputs and gradients; fp32 -> max abs error <= 1e-4.
"""
from __future__ import annotations

import numpy as np
import torch

from mka_inputs import approx_normal

BF16_MAX, BF16_MEAN, F32_MAX = 2e-2, 2e-3, 1e-4


def problem(seed, B, H, T, d, N, D, dtype, device="cuda", router_std=0.05, with_dO=False):
    """Seeded tensors in `dtype` on `device` (values already rounded to the storage dtype)."""
    def mk(tid, shape, std=1.0, dt=dtype):
        n = int(np.prod(shape))
        return approx_normal(seed, tid, 0, n, std, "cpu", dt).view(shape).to(device)
    out = {
        "X": mk(0, (B, T, D)), "W_r": mk(1, (D, 3), router_std, torch.float32),
        "Q": mk(2, (B, H, T, d)),
        "K": [mk(3 + 2 * l, (B, H, N[l], d)) for l in range(3)],
        "V": [mk(4 + 2 * l, (B, H, N[l], d)) for l in range(3)],
    }
    if with_dO:
        out["dO"] = mk(9, (B, H, T, d))
    return out


def err(gpu: torch.Tensor, ref: np.ndarray):
    g = gpu.detach().double().cpu().numpy()
    e = np.abs(g - ref)
    return float(e.max()) if e.size else 0.0, float(e.mean()) if e.size else 0.0


def check(gpu, ref, dtype, what=""):
    mx, mean = err(gpu, ref)
    if dtype == torch.bfloat16:
        assert mx <= BF16_MAX and mean <= BF16_MEAN, f"{what}: max {mx:.3e} mean {mean:.3e}"
    else:
        assert mx <= F32_MAX, f"{what}: max {mx:.3e}"
    return mx, mean


def np64(t):
    return t.detach().double().cpu().numpy()
