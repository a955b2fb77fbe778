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


def poison_unused_pool_rows(P, cfg, rows):
    """NaN into every pool row that no sequence owns: the rows after a sequence's last row inside its last page, and
    every page that no table entry in use points to (a serving engine's recycled or never-written pages)."""
    for l in range(3):
        pk, pv, tab = P["pools_k"][l], P["pools_v"][l], P["tables"][l].cpu().numpy()
        used = np.zeros((pk.shape[0], cfg.page_rows), dtype=bool)
        for b in range(cfg.B):
            n = int(rows[l][b])
            r = np.arange(n)
            used[tab[b, r // cfg.page_rows], r % cfg.page_rows] = True
        dead = torch.from_numpy(~used).to(pk.device)
        assert bool(dead.any())
        pk.permute(0, 2, 1, 3)[dead] = float("nan")
        pv.permute(0, 2, 1, 3)[dead] = float("nan")
