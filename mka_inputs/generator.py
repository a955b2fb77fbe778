"""Counter-based synthetic input generator (no attention arithmetic here).

Every element of every tensor is a pure function of (seed, tensor id, flat
index), so any slice can be regenerated on its own, on the host or on the GPU,
with bit-identical values: the hash uses only wrapping 64-bit integer
operations, and the final integer -> float32 conversion and single float32
multiply are exactly rounded on both.

Distribution: the sum of eight independent 16-bit uniform integers, centred and
scaled to the requested standard deviation (an Irwin-Hall approximation of a
normal law, support +-4.9 sigma).  Values destined for a bf16 configuration are
rounded to bf16 (round to nearest even) by the final dtype cast, before anybody
reads them.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, Tuple

import torch

_MASK64 = (1 << 64) - 1


def _signed(x: int) -> int:
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLD = 0x9E3779B97F4A7C15
_M1 = _signed(0xBF58476D1CE4E5B9)
_M2 = _signed(0x94D049BB133111EB)


def _mix64_int(x: int) -> int:
    x &= _MASK64
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _MASK64
    return x ^ (x >> 31)


def _lsr(x: torch.Tensor, k: int) -> torch.Tensor:
    return (x >> k) & ((1 << (64 - k)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lsr(x, 30)) * _M1
    x = (x ^ _lsr(x, 27)) * _M2
    return x ^ _lsr(x, 31)


def _field_sum(h: torch.Tensor) -> torch.Tensor:
    return (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + _lsr(h, 48)


_UNIT_STD = 2.0 * math.sqrt(8.0 * (65536.0 ** 2 - 1.0) / 12.0)  # std of (2*sum - 8*65535)


def approx_normal(seed: int, tensor_id: int, start: int, count: int, std: float,
                  device="cpu", dtype=torch.float32, chunk: int = 1 << 24) -> torch.Tensor:
    """`count` values of stream (seed, tensor_id) beginning at flat index `start`."""
    key = _mix64_int(seed * _GOLD + tensor_id * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D)
    gold = _signed(_GOLD)
    scale = torch.tensor(std / _UNIT_STD, dtype=torch.float32, device=device)
    out = torch.empty(count, dtype=dtype, device=device)
    for c0 in range(0, count, chunk):
        n = min(chunk, count - c0)
        i = torch.arange(start + c0, start + c0 + n, dtype=torch.int64, device=device)
        ctr = i * 2
        h1 = _mix64((ctr + 1) * gold + _signed(key))
        h2 = _mix64((ctr + 2) * gold + _signed(key))
        s = _field_sum(h1) + _field_sum(h2)            # 0 .. 8*65535
        centred = (2 * s - 8 * 65535).to(torch.float32)  # exact: |.| < 2^24
        out[c0:c0 + n] = (centred * scale).to(dtype)
    return out


TENSOR_IDS: Dict[str, int] = {
    "X": 0, "W_r": 1, "Q": 2, "K1": 3, "V1": 4, "K2": 5, "V2": 6, "K3": 7, "V3": 8, "dO": 9,
}


@dataclass(frozen=True)
class WorkloadConfig:
    """One benchmark configuration: shapes follow the paper's notation.

    B batch, H heads, d head width, D model width, T query tokens, W the L1
    window, N = rows of the three level sources.  `decode` marks the
    single-token form where every cached row is visible.
    """
    name: str
    seed: int
    dtype: str          # "bf16" | "f32"
    B: int
    H: int
    d: int
    D: int
    T: int
    W: int
    N: Tuple[int, int, int]
    decode: bool = False
    router_std: float = 0.02
    extra: dict = field(default_factory=dict)

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def q_offset(self) -> int:
        return 0

    def shape_of(self, name: str) -> Tuple[int, ...]:
        if name == "X":
            return (self.B, self.T, self.D)
        if name == "W_r":
            return (self.D, 3)
        if name in ("Q", "dO"):
            return (self.B, self.H, self.T, self.d)
        lvl = int(name[1]) - 1
        return (self.B, self.H, self.N[lvl], self.d)

    def visible_pairs_per_head(self) -> int:
        """Number of (query, key) pairs the masks leave visible, per (b, h)."""
        if self.decode:
            return sum(self.N)
        T, W = self.T, min(self.W, self.T)
        return (T * W - W * (W - 1) // 2) + T * (T + 1) // 2 + T * self.N[2]


CONFIGS: Dict[str, WorkloadConfig] = {
    "c1": WorkloadConfig("c1", 0, "f32", 1, 4, 64, 256, 256, 64, (256, 256, 128)),
    "c2": WorkloadConfig("c2", 1, "bf16", 8, 16, 64, 1024, 2048, 512, (2048, 2048, 1024)),
    "c3": WorkloadConfig("c3", 2, "bf16", 1, 32, 128, 4096, 32768, 4096, (32768, 32768, 8192)),
    "c4": WorkloadConfig("c4", 3, "bf16", 32, 32, 128, 4096, 1, 4096, (4096, 32768, 8192), decode=True),
    "c5": WorkloadConfig("c5", 4, "bf16", 4, 16, 128, 2048, 8192, 1024, (8192, 8192, 2048)),
    # route-fusion / cache write of Alg. 2 (levels token-aligned): c3's geometry with N_3 = T, and a profiler-sized variant
    "f3": WorkloadConfig("f3", 5, "bf16", 1, 32, 128, 4096, 32768, 4096, (32768, 32768, 32768)),
    "f3p": WorkloadConfig("f3p", 5, "bf16", 1, 8, 128, 4096, 32768, 4096, (32768, 32768, 32768)),
    # L2 session summary (a scan over the router input X of c3), and a profiler-sized variant
    "s3": WorkloadConfig("s3", 6, "bf16", 1, 32, 128, 4096, 32768, 4096, (32768, 32768, 8192)),
    "s3p": WorkloadConfig("s3p", 6, "bf16", 1, 32, 128, 4096, 12288, 4096, (12288, 12288, 8192)),
    # profiler-sized variants (same per-head geometry, fewer heads / sequences) for ncu captures
    "c3p": WorkloadConfig("c3p", 2, "bf16", 1, 8, 128, 4096, 32768, 4096, (32768, 32768, 8192)),
    "c4p": WorkloadConfig("c4p", 3, "bf16", 2, 32, 128, 4096, 1, 4096, (4096, 32768, 8192), decode=True),
    "c5p": WorkloadConfig("c5p", 4, "bf16", 1, 16, 128, 2048, 8192, 1024, (8192, 8192, 2048)),
}


def make_tensor(cfg: WorkloadConfig, name: str, device="cpu", flat_start: int = 0,
                flat_count: int | None = None, std: float | None = None) -> torch.Tensor:
    """Tensor `name` of configuration `cfg` (or a flat slice of it), in the
    configuration's storage dtype; W_r is always float32."""
    shape = cfg.shape_of(name)
    total = 1
    for s in shape:
        total *= s
    if std is None:
        std = cfg.router_std if name == "W_r" else 1.0
    dtype = torch.float32 if name == "W_r" else cfg.torch_dtype
    if flat_count is None:
        return approx_normal(cfg.seed, TENSOR_IDS[name], 0, total, std, device, dtype).view(shape)
    assert 0 <= flat_start and flat_start + flat_count <= total
    return approx_normal(cfg.seed, TENSOR_IDS[name], flat_start, flat_count, std, device, dtype)


# ---- paged levels (serving layout): page pools plus per-sequence page tables -------------------------------------------

@dataclass(frozen=True)
class PagedConfig:
    """A paged, grouped-query decode workload: B sequences, H query heads sharing H_kv KV heads of width d, levels of
    N rows at most, kept in pages of page_rows rows.  `rows_frac[b % len]` scales every level's rows for sequence b
    (a mix of lengths); `spare` extra pages per pool are never referenced."""
    name: str
    seed: int
    B: int
    H: int
    H_kv: int
    d: int
    N: Tuple[int, int, int]
    page_rows: int
    rows_frac: Tuple[float, ...] = (1.0,)
    spare: int = 3


PAGED_CONFIGS: Dict[str, PagedConfig] = {
    # Qwen2.5-7B-like head geometry (28 query heads on 4 KV heads), a 128K-token session level
    "g4": PagedConfig("g4", 7, 4, 28, 4, 128, (4096, 131072, 8192), 16),
    "g4p": PagedConfig("g4p", 7, 1, 28, 4, 128, (4096, 131072, 8192), 16),
    "g1": PagedConfig("g1", 8, 3, 12, 4, 64, (100, 700, 333), 16, rows_frac=(1.0, 0.37, 0.0)),
}


def paged_rows(cfg: PagedConfig):
    """int32 [3][B]: valid rows of every sequence on every level."""
    out = []
    for l in range(3):
        out.append(torch.tensor([int(cfg.N[l] * cfg.rows_frac[b % len(cfg.rows_frac)]) for b in range(cfg.B)],
                                dtype=torch.int32))
    return out


def paged_tables(cfg: PagedConfig):
    """Page tables int32 [3][B, pages] and pool sizes: the pages a sequence needs are dealt from a seeded shuffle of the
    pool, so consecutive logical pages are scattered; table entries past a sequence's last page are 0."""
    rows = paged_rows(cfg)
    tables, pool_pages = [], []
    for l in range(3):
        per_seq = [-(-int(r) // cfg.page_rows) for r in rows[l]]
        width = max(1, -(-cfg.N[l] // cfg.page_rows))
        P = sum(per_seq) + cfg.spare
        gen = torch.Generator().manual_seed(cfg.seed * 1000 + l)
        order = torch.randperm(P, generator=gen).to(torch.int32)
        tab = torch.zeros(cfg.B, width, dtype=torch.int32)
        nxt = 0
        for b in range(cfg.B):
            tab[b, :per_seq[b]] = order[nxt:nxt + per_seq[b]]
            nxt += per_seq[b]
        tables.append(tab)
        pool_pages.append(P)
    return tables, pool_pages


def make_paged(cfg: PagedConfig, device="cpu"):
    """q [B, H, d], pools_k / pools_v [3][P_l, H_kv, page_rows, d] (bf16), tables, rows, gate logits source X-free:
    the gate itself is drawn as three positive numbers per sequence, normalised by the caller."""
    tables, pool_pages = paged_tables(cfg)
    q = approx_normal(cfg.seed, 20, 0, cfg.B * cfg.H * cfg.d, 1.0, device, torch.bfloat16).view(cfg.B, cfg.H, cfg.d)
    pk, pv = [], []
    for l in range(3):
        shape = (pool_pages[l], cfg.H_kv, cfg.page_rows, cfg.d)
        cnt = shape[0] * shape[1] * shape[2] * shape[3]
        pk.append(approx_normal(cfg.seed, 21 + 2 * l, 0, cnt, 1.0, device, torch.bfloat16).view(shape))
        pv.append(approx_normal(cfg.seed, 22 + 2 * l, 0, cnt, 1.0, device, torch.bfloat16).view(shape))
    g = approx_normal(cfg.seed, 27, 0, cfg.B * 3, 1.0, device, torch.float32).view(cfg.B, 3).abs() + 0.05
    return {"q": q, "pools_k": pk, "pools_v": pv, "tables": [t.to(device) for t in tables],
            "rows": [r.to(device) for r in paged_rows(cfg)], "gate_raw": g}


# ---- L3 recall: a long-term bank of chunks (pages) per sequence ----------------------------------------------------------

@dataclass(frozen=True)
class RecallConfig:
    """B sequences whose long-term memory holds `bank` chunks (pages of page_rows rows) each; H query heads on H_kv KV
    heads of width d; `bits`-bit codes; R chunks recalled per (sequence, KV head).  `len_frac[b % len]` scales how much
    of the bank sequence b uses."""
    name: str
    seed: int
    B: int
    H: int
    H_kv: int
    d: int
    bank: int
    page_rows: int
    bits: int
    R: int
    len_frac: Tuple[float, ...] = (1.0,)


RECALL_CONFIGS: Dict[str, RecallConfig] = {
    # 128K tokens of long-term memory per sequence in 16-row chunks, top-8 recall (the passkey table's R)
    "r3": RecallConfig("r3", 9, 4, 28, 4, 128, 8192, 16, 64, 8),
    "r3p": RecallConfig("r3p", 9, 1, 28, 4, 128, 8192, 16, 64, 8),
    "r1": RecallConfig("r1", 10, 3, 12, 4, 64, 37, 8, 32, 8, len_frac=(1.0, 0.1, 0.0)),
}


def make_recall(cfg: RecallConfig, device="cpu"):
    """q [B, H, d] bf16; pools_k / pools_v [B * bank + 1, H_kv, page_rows, d] bf16; proj [bits, d] f32; bank int32
    [B, bank]: the pool pages of every sequence's chunks, dealt from a seeded shuffle; bank_len int32 [B]."""
    P = cfg.B * cfg.bank + 1
    shape = (P, cfg.H_kv, cfg.page_rows, cfg.d)
    cnt = shape[0] * shape[1] * shape[2] * shape[3]
    out = {"q": approx_normal(cfg.seed, 30, 0, cfg.B * cfg.H * cfg.d, 1.0, device, torch.bfloat16).view(cfg.B, cfg.H, cfg.d),
           "pool_k": approx_normal(cfg.seed, 31, 0, cnt, 1.0, device, torch.bfloat16).view(shape),
           "pool_v": approx_normal(cfg.seed, 32, 0, cnt, 1.0, device, torch.bfloat16).view(shape),
           "proj": approx_normal(cfg.seed, 33, 0, cfg.bits * cfg.d, 1.0, device, torch.float32).view(cfg.bits, cfg.d)}
    gen = torch.Generator().manual_seed(cfg.seed * 1000 + 7)
    order = torch.randperm(P, generator=gen).to(torch.int32)
    out["bank"] = order[:cfg.B * cfg.bank].view(cfg.B, cfg.bank).contiguous().to(device)
    out["bank_len"] = torch.tensor([int(cfg.bank * cfg.len_frac[b % len(cfg.len_frac)]) for b in range(cfg.B)],
                                   dtype=torch.int32, device=device)
    return out
