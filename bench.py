#!/usr/bin/env python
"""Benchmark of the FastMKA hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3|c2|c5|c4] [--legs c4,c5]
                    [--impl ours|reference] [--no-e2e] [--no-cpu-baseline]

One JSON line on stdout (rank 0).  A "step" is one pass of the path over one batch of seeded synthetic
input of the named configuration:
    c2 / c3 (prefill)   mka_router -> mka_fwd
    c5      (training)  mka_router -> mka_fwd -> mka_bwd
    c4      (decode)    mka_router -> mka_decode
The headline `value` is the primary workload's algorithmic throughput (visible query-key pairs only) with
inputs resident in HBM; `legs` holds the same measurement for the other configurations, each with its own
roofline entry.  `e2e` repeats the primary workload with pinned HOST buffers: host->device copies of every
input and the device->host read of the result are inside the timed region.  `--impl reference` times the
CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from mka_inputs import CONFIGS, PAGED_CONFIGS, RECALL_CONFIGS, make_paged, make_recall, make_tensor  # noqa: E402

DATASHEET = {"bf16_tflops": 2250.0, "hbm_gbs": 8000.0}
FALLBACK = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"bf16_tflops": float(d["bf16_tflops"]), "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return dict(FALLBACK, source="fallback")


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch, from the ncu captures summarised under
# profiles/.  The captures run the profiler-sized workloads (c3p, c4p, c5p, ...: the same per-head geometry with fewer
# heads / sequences); traffic grows in proportion to the number of units (batch x head pairs, sequences, KV heads), so
# a full launch is the captured figure times the ratio below.  Every entry carries a digest of the kernel's source file
# as it was when the counters were taken: when the file has changed since, the figure is reported as null ("stale").
NCU_TRAFFIC = {
    # kernel@workload: (bytes in the capture, units of the capture, summary file under profiles/, source file, its digest)
    "fwd_tc_kernel@c3": (376.523776e6 + 61.946368e6, 1 * 8, "fwd_tc_kernel_c3p.md", "fwd_tc.cu", "58f08d0c47e4"),
    "fwd_tc_kernel64@c2": (204.546304e6 + 28.208640e6, 8 * 16, "fwd_tc_kernel64_c2.md", "fwd_tc.cu", "58f08d0c47e4"),   # the whole configuration
    "decode_partial_kernel@c4": (1.476476e9 + 5.132288e6, 2 * 32, "decode_partial_kernel_c4p.md", "decode.cu", "ed9d09920f1b"),
    "bwd_dq_tc_kernel@c5": (220.275200e6 + 27.056128e6, 1 * 16, "bwd_tc_kernels_c5p.md", "bwd_tc.cu", "5b543af267de"),
    "bwd_dkv_tc_kernel@c5": (220.271872e6 + 114.367232e6, 1 * 16, "bwd_tc_kernels_c5p.md", "bwd_tc.cu", "5b543af267de"),
    "l2_summary_seg_kernel@s3": (101.000704e6 + 55.384064e6, 12288.0 / 32768.0, "l2_summary_seg_kernel_s3p.md", "summary_seg.cu", "6e2dcc00fbde"),   # 12288 of the 32768 tokens
    "fuse_kv_kernel@f3": (403.137024e6 + 83.414784e6, 1 * 8, "fuse_kv_kernel_f3p.md", "fuse_kv.cu", "3becacc721a4"),
    "decode_paged_kernel@g4": (293.682688e6 + 3.988480e6, 1 * 4, "decode_paged_kernel_g4p.md", "decode_paged.cu", "712e1e791061"),   # one of the four sequences (g4p)
    "l3_index_kernel@r3": (134.301696e6 + 3.607552e6, 1, "l3_index_kernel_r3p.md", "l3.cu", "6e05d1bc7821"),            # one of the four sequences (r3p)
}


def _source_digest(name):
    import hashlib
    path = os.path.join(ROOT, "paper_2603_20586_b200", "csrc", name)
    try:
        with open(path, "rb") as f:
            return hashlib.sha256(f.read()).hexdigest()[:12]
    except OSError:
        return None


def ncu_traffic(key, cfg):
    """(bytes per full launch, where the figure comes from), or (None, why not)."""
    ent = NCU_TRAFFIC.get(key)
    if ent is None:
        return None, None
    if _source_digest(ent[3]) != ent[4]:
        return None, f"stale: {ent[3]} has changed since the capture in profiles/{ent[2]}"
    if key.startswith("l3_index"):
        units = cfg.B                                                      # one sequence's bank
    elif key.startswith("decode_paged"):
        units = cfg.B * cfg.H_kv                                           # one KV head of one sequence
    else:
        units = cfg.B if key.startswith("l2_summary") else cfg.B * cfg.H     # the summary's unit is a whole sequence
    ratio = units / ent[1]
    return ent[0] * ratio, f"profiles/{ent[2]}, scaled x{ratio:.4g}"


def sig(x, n=5):
    """Rounds floats (recursively) to n significant digits: keeps the JSON line short."""
    if isinstance(x, float):
        return float(f"{x:.{n}g}") if x == x and abs(x) != float("inf") else x
    if isinstance(x, dict):
        return {k: sig(v, n) for k, v in x.items()}
    if isinstance(x, (list, tuple)):
        return [sig(v, n) for v in x]
    return x


def algorithmic_work(cfg):
    """Flops / bytes the method itself must do (visible pairs only)."""
    pairs = cfg.visible_pairs_per_head() * cfg.B * cfg.H
    return {"pairs": pairs, "fwd_flops": 4.0 * cfg.d * pairs, "bwd_flops": 10.0 * cfg.d * pairs,
            "decode_bytes": 2.0 * 2.0 * cfg.d * sum(cfg.N) * cfg.B * cfg.H,
            # route-fusion: K and V of three levels read, one fused K and V written (2 bytes each), plus the gate
            # L2 summary: X read once, M2 written once
            "summary_bytes": 2.0 * 2.0 * cfg.D * cfg.T * cfg.B,
            "fuse_bytes": 2.0 * (3 + 1) * 2.0 * cfg.d * cfg.T * cfg.B * cfg.H + 12.0 * cfg.B * cfg.T}


class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(power),
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------ ours
class Leg:
    """One configuration resident on the device plus the calls of its step."""

    def __init__(self, name, device, seed_shift=0):
        import paper_2603_20586_b200 as mka
        self.mka, self.name, self.dev = mka, name, device
        if name in PAGED_CONFIGS:
            self._init_paged(PAGED_CONFIGS[name], device, seed_shift)
            return
        if name in RECALL_CONFIGS:
            self._init_recall(RECALL_CONFIGS[name], device, seed_shift)
            return
        cfg = CONFIGS[name]
        if seed_shift:
            cfg = type(cfg)(**{**cfg.__dict__, "seed": cfg.seed + 1000 * seed_shift})
        self.cfg = cfg
        self.work = algorithmic_work(cfg)
        self.kind = {"c4": "decode", "c5": "train", "f3": "fuse", "s3": "summary"}.get(name[:2], "prefill")
        names = ["X", "W_r", "Q", "K1", "V1", "K2", "V2", "K3", "V3"] + (["dO"] if self.kind == "train" else [])
        if self.kind == "fuse":
            names.remove("Q")
        if self.kind == "summary":
            names = ["X"]
        self.t = {n: make_tensor(cfg, n, device) for n in names}
        B, H, T, d, D = cfg.B, cfg.H, cfg.T, cfg.d, cfg.D
        if self.kind == "summary":
            self.M2 = torch.empty_like(self.t["X"])
            self.state = torch.zeros(B, D, device=device)
            self.ws = mka.mka_l2_summary_workspace(self.t["X"]).zero_()
            self.launches_per_step = 1
            self.work = dict(self.work)
            self.ev = []
            return
        self.K = [self.t["K1"], self.t["K2"], self.t["K3"]]
        self.V = [self.t["V1"], self.t["V2"], self.t["V3"]]
        self.shape = mka.make_shape(B, H, T, d, D, cfg.W, 0)
        self.gate = torch.empty(B, T, 3, device=device)
        self.O = torch.empty_like(self.t["Q"]) if "Q" in self.t else None
        self.LSE = torch.empty(B, H, T, device=device)
        which = {"decode": mka.MKA_WS_DECODE, "train": mka.MKA_WS_BWD}.get(self.kind, mka.MKA_WS_FWD)
        self.ws = mka.alloc_workspace(self.shape, cfg.N, which, device)
        self.launches = 0
        if self.kind == "fuse":
            self.cache_k, self.cache_v = torch.empty_like(self.K[0]), torch.empty_like(self.V[0])
            self.ws.zero_()                         # no kernel of this leg writes the status word
            self.launches_per_step = 2              # router, fuse_kv
        elif self.kind == "decode":
            self.q = self.t["Q"].view(B, H, d)
            self.Od = torch.empty_like(self.q)
            self.gate_d = self.gate.view(B, 3)
            self.LSEd = self.LSE.view(B, H)
            self.launches_per_step = 1 + 2          # router, decode partial, decode combine
        elif self.kind == "train":
            self.grads = {"dQ": torch.empty_like(self.t["Q"]), "dK": [torch.empty_like(k) for k in self.K],
                          "dV": [torch.empty_like(v) for v in self.V], "dG": torch.empty(B, T, 3, device=device),
                          "dW_r": torch.empty(D, 3, device=device), "db_r": torch.empty(3, device=device)}
            self.launches_per_step = 1 + 1 + (1 + 1 + 1 + 1) + 3   # router, fwd, bwd(prep,dq,dkv,dgate), router bwd
            self.bwd_executed_ratio = 1.4           # the two-pass backward runs 14 d flops per pair for the method's 10 d
        else:
            self.launches_per_step = 2              # router, fwd
        self.ev = []

    def _init_paged(self, cfg, device, seed_shift):
        """Paged, grouped-query decode: pools, page tables and the gate are resident; one step = partial + combine."""
        import dataclasses
        mka = self.mka
        if seed_shift:
            cfg = dataclasses.replace(cfg, seed=cfg.seed + 1000 * seed_shift)
        self.cfg, self.kind = cfg, "paged"
        P = make_paged(cfg, device)
        self.t = {"q": P["q"]}
        for l in range(3):
            self.t[f"pk{l}"], self.t[f"pv{l}"] = P["pools_k"][l], P["pools_v"][l]
        self.tables, self.rows = P["tables"], P["rows"]
        self.gate_d = (P["gate_raw"] / P["gate_raw"].sum(1, keepdim=True)).contiguous()
        self.shape = mka.make_shape(cfg.B, cfg.H, 1, cfg.d, 32)
        self.Od = torch.empty_like(P["q"])
        self.LSEd = torch.empty(cfg.B, cfg.H, device=device)
        self.ws = torch.zeros(mka.mka_decode_paged_workspace_bytes(self.shape, cfg.H_kv, list(cfg.N)), dtype=torch.uint8,
                              device=device)
        rows_total = float(sum(int(r.sum()) for r in self.rows))
        # every valid cached row of every KV head once: K and V, 2 bytes per element
        self.work = {"decode_bytes": 2.0 * 2.0 * cfg.d * rows_total * cfg.H_kv}
        self.launches_per_step = 2
        self.ev = []

    def _init_recall(self, cfg, device, seed_shift):
        """L3 recall: index the long-term key pool, recall R chunks per (sequence, KV head), decode over them."""
        import dataclasses
        mka = self.mka
        if seed_shift:
            cfg = dataclasses.replace(cfg, seed=cfg.seed + 1000 * seed_shift)
        self.cfg, self.kind = cfg, "recall"
        P = make_recall(cfg, device)
        self.t = {"q": P["q"], "pool_k": P["pool_k"], "pool_v": P["pool_v"]}
        self.proj, self.bank, self.bank_len = P["proj"], P["bank"], P["bank_len"]
        self.codes = torch.empty(P["pool_k"].shape[0], cfg.H_kv, cfg.bits // 32, dtype=torch.int32, device=device)
        self.table = torch.empty(cfg.B, cfg.H_kv, cfg.R, dtype=torch.int32, device=device)
        self.n_sel = torch.empty(cfg.B, dtype=torch.int32, device=device)
        self.rows3 = torch.empty(cfg.B, dtype=torch.int32, device=device)
        self.gate_d = torch.tensor([[0.0, 0.0, 1.0]] * cfg.B, device=device)
        self.shape = mka.make_shape(cfg.B, cfg.H, 1, cfg.d, 32)
        self.n3 = cfg.R * cfg.page_rows
        self.Od = torch.empty_like(P["q"])
        self.LSEd = torch.empty(cfg.B, cfg.H, device=device)
        self.ws = torch.zeros(mka.mka_decode_paged_workspace_bytes(self.shape, cfg.H_kv, [0, 0, self.n3]), dtype=torch.uint8,
                              device=device)
        k = P["pool_k"]
        # the index kernel reads every key of the pool once and writes bits/8 bytes per (page, KV head)
        self.work = {"index_bytes": float(k.numel() * 2 + self.codes.numel() * 4)}
        self.launches_per_step = 4              # index, retrieve, decode partial, decode combine
        self.ev = []

    def step(self, record=False):
        mka, t = self.mka, self.t
        if self.kind == "recall":
            cfg = self.cfg
            e = [torch.cuda.Event(enable_timing=True) for _ in range(4)] if record else None
            if record:
                e[0].record(); e[1].record()
            mka.mka_l3_index(t["pool_k"], self.proj, codes=self.codes)
            if record:
                e[2].record()
            mka.mka_l3_retrieve(t["q"], cfg.H_kv, self.proj, self.codes, self.bank, self.bank_len, cfg.R, cfg.page_rows,
                                table=self.table, n_sel=self.n_sel, rows=self.rows3)
            mka.mka_decode_paged(self.shape, cfg.H_kv, t["q"], [None, None, t["pool_k"]], [None, None, t["pool_v"]],
                                 [None, None, self.table], [0, 0, self.n3], self.gate_d, rows=[None, None, self.rows3],
                                 O=self.Od, LSE=self.LSEd, ws=self.ws)
            if record:
                e[3].record()
                self.ev.append(e)
            return
        if self.kind == "paged":
            e = [torch.cuda.Event(enable_timing=True) for _ in range(4)] if record else None
            if record:
                e[0].record(); e[1].record()
            cfg = self.cfg
            mka.mka_decode_paged(self.shape, cfg.H_kv, t["q"], [t["pk0"], t["pk1"], t["pk2"]], [t["pv0"], t["pv1"], t["pv2"]],
                                 self.tables, list(cfg.N), self.gate_d, rows=self.rows, O=self.Od, LSE=self.LSEd, ws=self.ws)
            if record:
                e[2].record(); e[3].record()
                self.ev.append(e)
            return
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)] if record else None
        if record:
            e[0].record()
        if self.kind == "summary":
            if record:
                e[1].record()
            mka.mka_l2_summary(t["X"], mka.MKA_SUMMARY_MEAN, state=self.state, n_prev=0, M2=self.M2, ws=self.ws)
            if record:
                e[2].record(); e[3].record()
                self.ev.append(e)
            return
        mka.mka_router(t["X"], t["W_r"], None, gate=self.gate)
        if record:
            e[1].record()
        if self.kind == "fuse":
            mka.mka_fuse_kv(self.K, self.V, self.gate, out_k=self.cache_k, out_v=self.cache_v)
        elif self.kind == "decode":
            mka.mka_decode(self.shape, self.q, self.K, self.V, self.gate_d, O=self.Od, LSE=self.LSEd, ws=self.ws)
        else:
            mka.mka_fwd(self.shape, t["Q"], self.K, self.V, self.gate, O=self.O, LSE=self.LSE, ws=self.ws)
        if record:
            e[2].record()
        if self.kind == "train":
            g = self.grads
            mka.mka_bwd(self.shape, t["Q"], self.K, self.V, self.gate, self.O, self.LSE, t["dO"], R=t["X"], dQ=g["dQ"],
                        dK=g["dK"], dV=g["dV"], dG=g["dG"], dW_r=g["dW_r"], db_r=g["db_r"], ws=self.ws)
        if record:
            e[3].record()
            self.ev.append(e)

    def rebind(self, t):
        """Makes `t` (a dict with the same names and shapes) the step's input tensors."""
        self.t = t
        if self.kind in ("paged", "recall", "summary"):
            return
        self.K = [t["K1"], t["K2"], t["K3"]]
        self.V = [t["V1"], t["V2"], t["V3"]]
        if self.kind == "decode":
            self.q = t["Q"].view(self.cfg.B, self.cfg.H, self.cfg.d)

    def result_tensor(self):
        if self.kind in ("paged", "recall"):
            return self.Od
        if self.kind == "summary":
            return self.M2
        if self.kind == "fuse":
            return self.cache_k
        return self.Od if self.kind == "decode" else (self.grads["dQ"] if self.kind == "train" else self.O)

    def kernel_ms(self):
        """Average device time of (router, main kernel, backward) over the recorded steps."""
        r = [statistics.mean(a[i].elapsed_time(a[i + 1]) for a in self.ev) for i in range(3)]
        return {"router": r[0], "main": r[1], "bwd": r[2]}

    def step_stats(self):
        """Median and best device time of one whole step, and of its main kernel, over the recorded steps."""
        whole = [a[0].elapsed_time(a[3]) for a in self.ev]
        main = [a[1].elapsed_time(a[2]) for a in self.ev]
        return {"n": len(whole), "step_median": statistics.median(whole), "step_best": min(whole),
                "main_median": statistics.median(main), "main_best": min(main)}


def timed_steps(leg, steps, warmup, dist=None):
    for _ in range(warmup):
        leg.step()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    leg.ev = []
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        leg.step(record=True)
    t1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    from paper_2603_20586_b200 import shard
    ms = shard.max_over_ranks(t0.elapsed_time(t1), dist, leg.dev)
    if leg.mka.mka_device_status(leg.ws) != 0:
        raise RuntimeError("device status word reports a timed-out wait")
    return ms / steps


def _hbm_roof(kernel, achieved, peaks, traffic):
    t, src = traffic
    roof = {"kernel": kernel, "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": achieved / peaks["hbm_gbs"], "frac_datasheet": achieved / DATASHEET["hbm_gbs"], "traffic": t,
            "traffic_source": src}
    if roof["frac"] > 1.0:
        roof["note"] = "peak is a measured COPY rate (read + write); a read-mostly stream can exceed it"
    return roof


def _tensor_roof(kernel, achieved, peaks, traffic):
    t, src = traffic
    return {"kernel": kernel, "bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
            "frac": achieved / peaks["bf16_tflops"], "frac_sustained_peak": achieved / peaks["bf16_tflops_sustained"],
            "frac_datasheet": achieved / DATASHEET["bf16_tflops"], "traffic": t, "traffic_source": src}


def leg_report(leg, ms_per_step, n_gpus, peaks):
    cfg, w, k = leg.cfg, leg.work, leg.kernel_ms()
    none = (None, None)
    tag = leg.name[:2]
    if leg.kind == "recall":
        # main = the index kernel; "bwd" holds the recall-list kernel plus the decode over the recalled chunks
        work, unit, metric = w["index_bytes"], "GB/s", "l3_recall_hbm_gbs"
        roof = _hbm_roof("l3_index_kernel", work / (k["main"] * 1e-3) / 1e9, peaks,
                         ncu_traffic("l3_index_kernel@r3", cfg) if tag == "r3" else none)
    elif leg.kind == "paged":
        work, unit, metric = w["decode_bytes"], "GB/s", "decode_paged_hbm_gbs"
        roof = _hbm_roof("decode_paged_tma_kernel+decode_combine_kernel", work / (k["main"] * 1e-3) / 1e9, peaks,
                         ncu_traffic("decode_paged_kernel@g4", cfg) if tag == "g4" else none)
    elif leg.kind == "summary":
        work, unit, metric = w["summary_bytes"], "GB/s", "l2_summary_hbm_gbs"
        roof = _hbm_roof("l2_summary_seg_kernel", work / (k["main"] * 1e-3) / 1e9, peaks,
                         ncu_traffic("l2_summary_seg_kernel@s3", cfg) if tag == "s3" else none)
    elif leg.kind == "fuse":
        work, unit, metric = w["fuse_bytes"], "GB/s", "route_fuse_hbm_gbs"
        roof = _hbm_roof("fuse_kv_kernel", work / (k["main"] * 1e-3) / 1e9, peaks,
                         ncu_traffic("fuse_kv_kernel@f3", cfg) if tag == "f3" else none)
    elif leg.kind == "decode":
        work, unit, metric = w["decode_bytes"], "GB/s", "decode_hbm_gbs"
        roof = _hbm_roof("decode_partial_kernel+decode_combine_kernel", work / (k["main"] * 1e-3) / 1e9, peaks,
                         ncu_traffic("decode_partial_kernel@c4", cfg) if tag == "c4" else none)
    else:
        work = w["fwd_flops"] + (w["bwd_flops"] if leg.kind == "train" else 0.0)
        unit, metric = "TFLOP/s", ("fwd_bwd_tflops" if leg.kind == "train" else "prefill_fwd_tflops")
        roof = _tensor_roof("fwd_tc_kernel", w["fwd_flops"] / (k["main"] * 1e-3) / 1e12, peaks,
                            ncu_traffic("fwd_tc_kernel@c3", cfg) if tag == "c3" else
                            (ncu_traffic("fwd_tc_kernel64@c2", cfg) if leg.name == "c2" else none))
    scale = 1e9 if unit == "GB/s" else 1e12
    value = n_gpus * work / (ms_per_step * 1e-3) / scale
    st = leg.step_stats()
    rep = {"workload": leg.name, "metric": metric, "value": value, "unit": unit, "ms_per_step": ms_per_step,
           "steps": st["n"], "value_median": work / (st["step_median"] * 1e-3) / scale,
           "value_best": work / (st["step_best"] * 1e-3) / scale, "kernel_ms": k, "roofline": roof}
    if leg.kind == "train":
        # the backward as a whole (prep, dQ kernel, dK/dV kernel, gate and router reductions) against the same peak;
        # "achieved" counts the 10*d flops per visible pair the method needs, not the 14*d the two-kernel form executes
        ach = w["bwd_flops"] / (k["bwd"] * 1e-3) / 1e12
        rep["bwd_tflops"] = ach
        tq, sq = ncu_traffic("bwd_dq_tc_kernel@c5", cfg)
        tkv, _ = ncu_traffic("bwd_dkv_tc_kernel@c5", cfg)
        both = tq is not None and tkv is not None and tag == "c5"
        rep["roofline_bwd"] = _tensor_roof("bwd_dq_tc_kernel+bwd_dkv_tc_kernel", ach, peaks,
                                           ((tq + tkv), sq) if both else ((None, sq) if tag == "c5" else none))
        rep["roofline_bwd"]["executed_tflops"] = ach * leg.bwd_executed_ratio
    return rep


def e2e_run(leg, steps, warmup):
    """The same step fed from pinned HOST buffers, through the public binding: every step's inputs are copied host to
    device and its result device to host inside the timed region.  Two device buffer sets: the copy of step i + 1's
    inputs (on a second stream) overlaps the kernels of step i, as a serving or training loop would pipeline it.  The
    timed region starts with an empty pipeline (the first copy overlaps nothing) and ends when the last result is on
    the host."""
    names = list(leg.t.keys())
    host = {n: torch.empty(leg.t[n].shape, dtype=leg.t[n].dtype, pin_memory=True).copy_(leg.t[n]) for n in names}
    sets = [leg.t, {n: torch.empty_like(leg.t[n]) for n in names}]
    res = leg.result_tensor()
    host_out = torch.empty(res.shape, dtype=res.dtype, pin_memory=True)
    h2d = sum(h.numel() * h.element_size() for h in host.values())
    d2h = host_out.numel() * host_out.element_size()
    cur, cp = torch.cuda.current_stream(), torch.cuda.Stream()
    landed = [torch.cuda.Event() for _ in range(2)]       # the inputs of set k are on the device
    freed = [torch.cuda.Event() for _ in range(2)]        # the kernels that read set k have finished

    def upload(k):
        cp.wait_event(freed[k])
        with torch.cuda.stream(cp):
            for n in names:
                sets[k][n].copy_(host[n], non_blocking=True)
            landed[k].record(cp)

    def run(k):
        cur.wait_event(landed[k])
        leg.rebind(sets[k])
        leg.step()
        freed[k].record(cur)
        host_out.copy_(leg.result_tensor(), non_blocking=True)

    def loop(n):
        for k in range(2):
            freed[k].record(cur)
        upload(0)
        for i in range(n):
            if i + 1 < n:
                upload((i + 1) & 1)
            run(i & 1)

    loop(max(2, warmup))
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    loop(steps)
    t1.record()
    torch.cuda.synchronize()
    leg.rebind(sets[0])
    return t0.elapsed_time(t1) / steps, h2d, d2h


# ------------------------------------------------------------------------------------------------ oracle arm
_ROUTER_INPUTS = {}


def _router_inputs(cfg):
    """Router input and weights of a configuration (generated once per process; not part of any timing)."""
    if cfg.name not in _ROUTER_INPUTS:
        _ROUTER_INPUTS[cfg.name] = (make_tensor(cfg, "X").double().numpy(), make_tensor(cfg, "W_r").double().numpy())
    return _ROUTER_INPUTS[cfg.name]


def oracle_sample_paged(name):
    """The oracle's paged decode on sequence 0 of the configuration (all heads, all rows)."""
    import dataclasses
    from oracle import mka_oracle as orc
    cfg = dataclasses.replace(PAGED_CONFIGS[name], B=1)
    P = make_paged(cfg, "cpu")
    f = lambda t: t.double().numpy()
    gate = f(P["gate_raw"] / P["gate_raw"].sum(1, keepdim=True))
    rows = [r.numpy().astype(np.int64) for r in P["rows"]]
    t0 = time.perf_counter()
    orc.decode_paged(f(P["q"]), [f(k) for k in P["pools_k"]], [f(v) for v in P["pools_v"]],
                     [t.numpy().astype(np.int64) for t in P["tables"]], rows, cfg.page_rows, gate)
    dt = time.perf_counter() - t0
    bytes_ = 2.0 * 2.0 * cfg.d * float(sum(int(r.sum()) for r in rows)) * cfg.H_kv
    return {"value": bytes_ / dt / 1e9, "unit": "GB/s", "cores": orc.num_threads(), "kind": "oracle", "seconds": dt,
            "sample": f"one sequence of the configuration's {PAGED_CONFIGS[name].B}: all {cfg.H} heads, all {int(sum(int(r.sum()) for r in rows))} cached rows"}


def oracle_sample_recall(name):
    """The oracle index + recall lists on one sequence of the configuration."""
    import dataclasses
    from oracle import mka_oracle as orc
    full = RECALL_CONFIGS[name]
    cfg = dataclasses.replace(full, B=1)
    P = make_recall(cfg, "cpu")
    pool, proj = P["pool_k"].float().numpy(), P["proj"].numpy()
    t0 = time.perf_counter()
    codes = orc.l3_index(pool, proj)
    orc.l3_retrieve(P["q"].float().numpy(), proj, codes, P["bank"].numpy(), P["bank_len"].numpy(), cfg.R, cfg.H_kv)
    dt = time.perf_counter() - t0
    bytes_ = float(pool.size * 2 + codes.size * 4)
    return {"value": bytes_ / dt / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle", "seconds": dt,
            "sample": f"index and recall lists of {cfg.bank} of sequence 0's {full.bank} chunks (one thread)"}


def oracle_sample(name, budget_rows=None):
    """Times the CPU oracle, as it stands, on a bounded seeded sample of workload `name`."""
    if name in PAGED_CONFIGS:
        return oracle_sample_paged(name)
    if name in RECALL_CONFIGS:
        return oracle_sample_recall(name)
    from oracle import mka_oracle as orc
    orc.build()
    cfg = CONFIGS[name]
    rng = np.random.default_rng(1234 + cfg.seed)
    cores = orc.num_threads()
    d, W = cfg.d, cfg.W
    if name[:2] == "c4":
        heads = [(int(rng.integers(cfg.B)), int(rng.integers(cfg.H))) for _ in range(64)]
        per = cfg.H * 1
        X, Wr = _router_inputs(cfg)
        gate, _ = orc.router(X, Wr)
        dt = 0.0
        for (b, h) in heads:
            def sl(nm, n):
                off = ((b * cfg.H + h) * n) * d
                return make_tensor(cfg, nm, flat_start=off, flat_count=n * d).double().numpy().reshape(1, 1, n, d)
            K = [sl(f"K{l + 1}", cfg.N[l]) for l in range(3)]
            V = [sl(f"V{l + 1}", cfg.N[l]) for l in range(3)]
            q = make_tensor(cfg, "Q", flat_start=(b * cfg.H + h) * d, flat_count=d).double().numpy().reshape(1, 1, 1, d)
            t0 = time.perf_counter()
            orc.fwd(q, K, V, gate[b:b + 1], 1, decode=True)
            dt += time.perf_counter() - t0
        bytes_ = 2.0 * 2.0 * d * sum(cfg.N) * len(heads)
        return {"value": bytes_ / dt / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle", "seconds": dt,
                "sample": f"{len(heads)} of {cfg.B * cfg.H} (batch, head) pairs, all {sum(cfg.N)} cached rows each"}
    if name[:2] == "s3":
        rows = min(cfg.T, 4096)
        X = make_tensor(cfg, "X", flat_start=0, flat_count=rows * cfg.D).double().numpy().reshape(1, rows, cfg.D)
        t0 = time.perf_counter()
        orc.l2_summary(X, orc.SUMMARY_MEAN)
        dt = time.perf_counter() - t0
        return {"value": 2.0 * 2.0 * cfg.D * rows / dt / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle", "seconds": dt,
                "sample": f"the first {rows} of {cfg.T} tokens of one sequence (numpy, one thread)"}
    if name[:2] == "f3":
        X, Wr = _router_inputs(cfg)
        t0 = time.perf_counter()
        gate, _ = orc.router(X, Wr)
        dt = time.perf_counter() - t0
        heads = [(int(rng.integers(cfg.B)), int(rng.integers(cfg.H))) for _ in range(4)]
        for (b, h) in heads:
            def sl(nm):
                off = ((b * cfg.H + h) * cfg.T) * d
                return make_tensor(cfg, nm, flat_start=off, flat_count=cfg.T * d).double().numpy().reshape(1, 1, cfg.T, d)
            K = [sl(f"K{l + 1}") for l in range(3)]
            V = [sl(f"V{l + 1}") for l in range(3)]
            t0 = time.perf_counter()
            orc.route_fuse(K, gate[b:b + 1])
            orc.route_fuse(V, gate[b:b + 1])
            dt += time.perf_counter() - t0
        bytes_ = 2.0 * 4 * 2.0 * d * cfg.T * len(heads)
        return {"value": bytes_ / dt / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle", "seconds": dt,
                "sample": f"{len(heads)} of {cfg.B * cfg.H} (batch, head) pairs, all {cfg.T} rows each (numpy, one thread); router on all tokens"}
    # prefill / training: a few heads, a seeded sample of query rows
    n_heads = 2 if budget_rows else 8          # the default sample is sized for roughly 15 s of host work
    n_rows = budget_rows or 4096
    n_rows = min(n_rows, cfg.T)
    heads = [(int(rng.integers(cfg.B)), int(rng.integers(cfg.H))) for _ in range(n_heads)]
    rows = np.sort(rng.choice(cfg.T, size=n_rows, replace=False))
    X, Wr = _router_inputs(cfg)
    t_all, pairs = 0.0, 0
    t0 = time.perf_counter()
    gate, _ = orc.router(X, Wr)
    t_all += time.perf_counter() - t0
    for (b, h) in heads:
        def sl(nm, n):
            off = ((b * cfg.H + h) * n) * d
            return make_tensor(cfg, nm, flat_start=off, flat_count=n * d).double().numpy().reshape(1, 1, n, d)
        Q = sl("Q", cfg.T)
        K = [sl(f"K{l + 1}", cfg.N[l]) for l in range(3)]
        V = [sl(f"V{l + 1}", cfg.N[l]) for l in range(3)]
        t0 = time.perf_counter()
        orc.fwd(Q, K, V, gate[b:b + 1], W, rows=rows)
        if name[:2] == "c5":
            dO = sl("dO", cfg.T)
            orc.bwd(Q, K, V, gate[b:b + 1], dO, W, rows=rows, want_kv=False)
        t_all += time.perf_counter() - t0
        for t in rows:
            pairs += min(t + 1, W) + (t + 1) + cfg.N[2]
    flops = (4.0 if name[:2] != "c5" else 14.0) * d * pairs
    return {"value": flops / t_all / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "seconds": t_all,
            "sample": f"{n_heads} (batch, head) pairs x {n_rows} seeded query rows of {cfg.T}"
                      + (" (forward + dQ/dG backward rows)" if name[:2] == "c5" else "") + "; router on all tokens"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c3", choices=["c2", "c3", "c4", "c5", "f3", "s3", "g4", "r3", "c3p", "c4p", "c5p", "f3p", "s3p", "g4p", "r3p"])
    ap.add_argument("--legs", default="c4,c5,c2,f3,s3,g4,r3", help="other configurations measured after the primary one ('' = none)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--source-digests", action="store_true", help="print the digests of the kernel sources (for NCU_TRAFFIC) and exit")
    args = ap.parse_args()
    if args.source_digests:
        for name in sorted({e[3] for e in NCU_TRAFFIC.values()}):
            print(name, _source_digest(name))
        return
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    wk = args.workload[:2]
    paged = args.workload in PAGED_CONFIGS or args.workload in RECALL_CONFIGS
    cfg = PAGED_CONFIGS.get(args.workload) or RECALL_CONFIGS.get(args.workload) or CONFIGS[args.workload]
    metric_name = {"c4": "decode_hbm_gbs", "c5": "fwd_bwd_tflops", "f3": "route_fuse_hbm_gbs", "s3": "l2_summary_hbm_gbs",
                   "g4": "decode_paged_hbm_gbs", "r3": "l3_recall_hbm_gbs"}.get(wk, "prefill_fwd_tflops")
    describe = (f"{args.workload}: B={cfg.B} H={cfg.H} H_kv={cfg.H_kv} d={cfg.d} bank={cfg.bank} chunks x {cfg.page_rows} rows, {cfg.bits}-bit codes, R={cfg.R} seed={cfg.seed}"
                if args.workload in RECALL_CONFIGS else
                f"{args.workload}: B={cfg.B} H={cfg.H} H_kv={cfg.H_kv} d={cfg.d} N={list(cfg.N)} page_rows={cfg.page_rows} seed={cfg.seed}"
                if paged else
                f"{args.workload}: B={cfg.B} H={cfg.H} d={cfg.d} D={cfg.D} T={cfg.T} W={cfg.W} N={list(cfg.N)} seed={cfg.seed}")
    base = {"metric": f"FastMKA {metric_name} (algorithmic, visible pairs only)", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "data": "synthetic",
            "dtype": "bf16" if (paged or cfg.dtype == "bf16") else "f32",
            "config": {"workload": describe,
                       "l2": "inputs larger than L2 (no flush needed)" if args.workload != "c2" else "inputs ~235 MB, larger than the 126 MB L2",
                       "per_gpu": "each rank runs the whole configuration on its own seeded batch (no collective on the data path)"}}

    if args.impl == "reference":
        if rank != 0:
            return
        vals = []
        for _ in range(args.warmup):
            oracle_sample(args.workload, budget_rows=64)
        t0 = time.perf_counter()
        for _ in range(args.steps):
            vals.append(oracle_sample(args.workload, budget_rows=256 if wk != "c4" else None))
        dt = (time.perf_counter() - t0) / max(1, args.steps)
        v = statistics.mean(x["value"] for x in vals)
        cb = dict(vals[-1], value=v)
        out = dict(base, impl="reference", value=v, unit=cb["unit"], ms_per_step=dt * 1e3, dtype="f64", cpu_baseline=cb,
                   e2e={"value": v, "unit": cb["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, gpu_launches=0,
                   n_gpus=args.gpus)
        print(json.dumps(out))
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod
    peaks = load_peaks()
    sampler = ClockSampler(local)
    leg = Leg(args.workload, dev, seed_shift=rank)
    sampler.start()
    ms = timed_steps(leg, args.steps, args.warmup, dist)
    clocks = sampler.stop()
    rep = leg_report(leg, ms, world, peaks)
    launches = leg.launches_per_step * args.steps
    out = dict(base, value=rep["value"], unit=rep["unit"], ms_per_step=ms, value_median=rep["value_median"] * world,
               value_best=rep["value_best"] * world, roofline=rep["roofline"], kernel_ms=rep["kernel_ms"],
               clocks=clocks, gpu_launches=launches, n_gpus=world)
    out["roofline"]["peak_source"] = peaks["source"]
    if "bwd_tflops" in rep:
        out["bwd_tflops"] = rep["bwd_tflops"]
        out["roofline_bwd"] = rep["roofline_bwd"]
    if not args.no_e2e:
        e_ms, h2d, d2h = e2e_run(leg, max(4, min(args.steps, 10)), 2)
        w = leg.work
        if wk == "r3":
            ev = world * w["index_bytes"] / (e_ms * 1e-3) / 1e9
        elif wk in ("c4", "g4"):
            ev = world * w["decode_bytes"] / (e_ms * 1e-3) / 1e9
        elif wk == "f3":
            ev = world * w["fuse_bytes"] / (e_ms * 1e-3) / 1e9
        elif wk == "s3":
            ev = world * w["summary_bytes"] / (e_ms * 1e-3) / 1e9
        else:
            ev = world * (w["fwd_flops"] + (w["bwd_flops"] if wk == "c5" else 0.0)) / (e_ms * 1e-3) / 1e12
        out["e2e"] = {"value": ev, "unit": rep["unit"], "ms_per_step": e_ms, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                      "pipelined": "two device buffer sets: the host-to-device copy of step i + 1 overlaps the kernels of step i"}
    del leg
    torch.cuda.empty_cache()
    if rank == 0 and not args.no_cpu_baseline and world == 1:
        out["cpu_baseline"] = oracle_sample(args.workload)
    # The other configurations, each for --steps timed steps.  The two the headline metric names besides prefill --
    # training (c5) and decode (c4) -- come last, so that they end the line.
    legs = []
    if world == 1:
        wanted = [x for x in args.legs.split(",") if x and x != args.workload]
        order = {n: i for i, n in enumerate(["r3", "g4", "s3", "f3", "c2", "c5", "c4"])}
        wanted.sort(key=lambda n: order.get(n[:2], -1))
        for name in wanted:
            l2 = Leg(name, dev)
            ms2 = timed_steps(l2, max(3, args.steps), max(3, args.warmup))
            legs.append(leg_report(l2, ms2, 1, peaks))
            del l2
            torch.cuda.empty_cache()
    out["legs"] = legs
    if rank == 0:
        print(json.dumps(sig(out)))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
