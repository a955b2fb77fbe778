"""Parity at the benchmark's full sizes (configurations c1-c5), in the launch configuration bench.py times.

c1 is compared in full.  For c2, c3, c5 the GPU computes everything and the oracle evaluates a seeded
sample of query rows of every head exactly (each output row depends only on its own query row); for c5
dK/dV are compared in full for two (batch, head) pairs; for c4 the oracle evaluates 64 sampled
(batch, head) pairs.  Inputs come from the seeded generator, on the device, already rounded to bf16.
"""
import numpy as np
import pytest
import torch

from gpu_helpers import BF16_MAX, BF16_MEAN, F32_MAX, np64
from mka_inputs import CONFIGS, make_tensor

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mka():
    import paper_2603_20586_b200 as m
    assert torch.cuda.is_available()
    return m


def _load(cfg, names):
    return {n: make_tensor(cfg, n, "cuda") for n in names}


def _sample_rows(cfg, n_random, rng):
    fixed = {0, 1, cfg.W - 1, cfg.W, cfg.T // 2, cfg.T - 1}
    fixed = {r for r in fixed if 0 <= r < cfg.T}
    extra = set(int(x) for x in rng.choice(cfg.T, size=n_random, replace=False))
    return np.array(sorted(fixed | extra), dtype=np.int64)


def _bf16_ok(gpu_rows, ref_rows, what):
    e = np.abs(gpu_rows - ref_rows)
    assert e.max() <= BF16_MAX and e.mean() <= BF16_MEAN, f"{what}: max {e.max():.3e} mean {e.mean():.3e}"


def test_c1_full_fp32_fast_full_and_backward(mka, orc):
    cfg = CONFIGS["c1"]
    t = _load(cfg, ["X", "W_r", "Q", "K1", "V1", "K2", "V2", "K3", "V3"])
    K, V = [t["K1"], t["K2"], t["K3"]], [t["V1"], t["V2"], t["V3"]]
    gate = mka.mka_router(t["X"], t["W_r"], None)
    rg, _ = orc.router(np64(t["X"]), np64(t["W_r"]))
    assert np.abs(np64(gate) - rg).max() <= 2e-6
    shape = mka.make_shape(cfg.B, cfg.H, cfg.T, cfg.d, cfg.D, cfg.W, dtype=mka.MKA_F32)
    O, LSE = mka.mka_fwd(shape, t["Q"], K, V, gate)
    Or, Lr = orc.fwd(t["Q"], K, V, rg, cfg.W)
    assert np.abs(np64(O) - Or).max() <= F32_MAX and np.abs(np64(LSE) - Lr).max() <= F32_MAX
    shape_full = mka.make_shape(cfg.B, cfg.H, cfg.T, cfg.d, cfg.D, cfg.W, dtype=mka.MKA_F32, mode=mka.MKA_MODE_FULL)
    Of, _ = mka.mka_fwd(shape_full, t["Q"], K, V, gate)
    Ofr, _ = orc.fwd(t["Q"], K, V, rg, cfg.W, mode="full")
    assert np.abs(np64(Of) - Ofr).max() <= F32_MAX
    dO = make_tensor(cfg, "dO", "cuda")
    g = mka.mka_bwd(shape, t["Q"], K, V, gate, O, LSE, dO, R=t["X"])
    ref = orc.bwd(t["Q"], K, V, rg, dO, cfg.W)
    assert np.abs(np64(g["dQ"]) - ref["dQ"]).max() <= F32_MAX
    for l in range(3):
        assert np.abs(np64(g["dK"][l]) - ref["dK"][l]).max() <= F32_MAX
        assert np.abs(np64(g["dV"][l]) - ref["dV"][l]).max() <= F32_MAX
    assert np.abs(np64(g["dG"]) - ref["dG"]).max() <= F32_MAX
    dW, db = orc.router_bwd(np64(t["X"]), ref["dG"])
    assert np.abs(np64(g["dW_r"]) - dW).max() <= 2e-4 * max(1.0, np.abs(dW).max())


def _prefill_check(mka, orc, name, n_random, peaky=False):
    cfg = CONFIGS[name]
    t = _load(cfg, ["X", "W_r", "Q", "K1", "V1", "K2", "V2", "K3", "V3"])
    if peaky:                                # extra coverage: a router with large logits (peaky gates)
        t["W_r"] = make_tensor(cfg, "W_r", "cuda", std=1.0)
    K, V = [t["K1"], t["K2"], t["K3"]], [t["V1"], t["V2"], t["V3"]]
    gate = mka.mka_router(t["X"], t["W_r"], None)
    shape = mka.make_shape(cfg.B, cfg.H, cfg.T, cfg.d, cfg.D, cfg.W)
    assert mka.mka_fwd_kernel_kind(shape, K, V) == 1
    ws = mka.alloc_workspace(shape, cfg.N, mka.MKA_WS_FWD, "cuda")
    O, LSE = mka.mka_fwd(shape, t["Q"], K, V, gate, ws=ws)
    assert mka.mka_device_status(ws) == 0
    assert torch.isfinite(O.float()).all() and torch.isfinite(LSE).all()
    rg, _ = orc.router(np64(t["X"]), np64(t["W_r"]))
    assert np.abs(np64(gate) - rg).max() <= 5e-6
    rng = np.random.default_rng(100 + cfg.seed)
    rows = _sample_rows(cfg, n_random, rng)
    ridx = torch.from_numpy(rows).cuda()
    errs = []
    for b in range(cfg.B):
        for h in range(cfg.H):
            sl = lambda x: x[b:b + 1, h:h + 1]
            Or, Lr = orc.fwd(sl(t["Q"]), [sl(k) for k in K], [sl(v) for v in V], rg[b:b + 1], cfg.W, rows=rows)
            e = np.abs(np64(O[b, h, ridx]) - Or[0, 0])
            errs.append(e)
            assert np.abs(np64(LSE[b, h, ridx]) - Lr[0, 0]).max() <= 2e-3
    e = np.concatenate([x.ravel() for x in errs])
    assert e.max() <= BF16_MAX and e.mean() <= BF16_MEAN, f"{name}: max {e.max():.3e} mean {e.mean():.3e}"
    return t, K, V, gate, rg, O, LSE, shape


def test_c2_training_shape_forward(mka, orc):
    _prefill_check(mka, orc, "c2", 26)


def test_c2_peaky_gates(mka, orc):
    _prefill_check(mka, orc, "c2", 10, peaky=True)


def test_c3_long_context_prefill(mka, orc):
    _prefill_check(mka, orc, "c3", 250)


def test_c4_decode(mka, orc):
    cfg = CONFIGS["c4"]
    t = _load(cfg, ["X", "W_r", "Q", "K1", "V1", "K2", "V2", "K3", "V3"])
    K, V = [t["K1"], t["K2"], t["K3"]], [t["V1"], t["V2"], t["V3"]]
    B, H, d = cfg.B, cfg.H, cfg.d
    gate = mka.mka_router(t["X"], t["W_r"], None).view(B, 3)
    rg, _ = orc.router(np64(t["X"]), np64(t["W_r"]))
    q = t["Q"].view(B, H, d)
    shape = mka.make_shape(B, H, 1, d, cfg.D)
    chunk, n_chunks, total = mka.mka_decode_plan(cfg.N, B, H, d)
    assert chunk == 1024 and n_chunks == [4, 32, 8] and total == 44          # the split table bench.py runs
    O, LSE = mka.mka_decode(shape, q, K, V, gate)
    assert torch.isfinite(O.float()).all()
    rng = np.random.default_rng(103)
    pairs = sorted({(int(rng.integers(B)), int(rng.integers(H))) for _ in range(64)})
    errs = []
    for b, h in pairs:
        sl = lambda x: x[b:b + 1, h:h + 1]
        Or, Lr = orc.fwd(sl(t["Q"]), [sl(k) for k in K], [sl(v) for v in V], rg[b:b + 1], 1, decode=True)
        errs.append(np.abs(np64(O[b, h]) - Or[0, 0, 0]))
        assert abs(float(LSE[b, h]) - Lr[0, 0, 0]) <= 2e-3
    e = np.concatenate(errs)
    assert e.max() <= BF16_MAX and e.mean() <= BF16_MEAN, f"c4: max {e.max():.3e} mean {e.mean():.3e}"
    # regenerating a sampled head on the host from the counter-based generator gives the same bits
    b, h = pairs[0]
    off = ((b * H + h) * cfg.N[1]) * d
    host = make_tensor(cfg, "K2", flat_start=off, flat_count=cfg.N[1] * d).view(cfg.N[1], d)
    assert torch.equal(host, t["K2"][b, h].cpu())


def test_c5_training_forward_backward(mka, orc):
    cfg = CONFIGS["c5"]
    t, K, V, gate, rg, O, LSE, shape = _prefill_check(mka, orc, "c5", 100)
    dO = make_tensor(cfg, "dO", "cuda")
    ws = mka.alloc_workspace(shape, cfg.N, mka.MKA_WS_BWD, "cuda")
    g = mka.mka_bwd(shape, t["Q"], K, V, gate, O, LSE, dO, R=t["X"], ws=ws)
    assert mka.mka_device_status(ws) == 0
    rng = np.random.default_rng(104)
    rows = _sample_rows(cfg, 26, rng)
    ridx = torch.from_numpy(rows).cuda()
    dQ_err = []
    dG_ref = np.zeros((cfg.B, len(rows), 3))
    for b in range(cfg.B):
        for h in range(cfg.H):
            sl = lambda x: x[b:b + 1, h:h + 1]
            r = orc.bwd(sl(t["Q"]), [sl(k) for k in K], [sl(v) for v in V], rg[b:b + 1], sl(dO), cfg.W, rows=rows,
                        want_kv=False)
            dQ_err.append(np.abs(np64(g["dQ"][b, h, ridx]) - r["dQ"][0, 0]))
            dG_ref[b] += r["G"][0, 0]
    e = np.concatenate([x.ravel() for x in dQ_err])
    assert e.max() <= BF16_MAX and e.mean() <= BF16_MEAN, f"dQ: max {e.max():.3e} mean {e.mean():.3e}"
    eg = np.abs(np64(g["dG"][:, ridx]) - dG_ref)
    assert eg.max() <= BF16_MAX and eg.mean() <= BF16_MEAN, f"dG: max {eg.max():.3e}"
    # dW_r = X^T dG, db_r = sum dG: checked in fp64 from the GPU's own dG (the product is a plain contraction)
    dW, db = orc.router_bwd(np64(t["X"]), np64(g["dG"]))
    assert np.abs(np64(g["dW_r"]) - dW).max() <= 1e-3 * max(1.0, np.abs(dW).max())
    assert np.abs(np64(g["db_r"]) - db).max() <= 1e-3 * max(1.0, np.abs(db).max())
    # dK, dV in full for two (batch, head) pairs
    for b, h in [(0, 3), (cfg.B - 1, cfg.H - 1)]:
        sl = lambda x: x[b:b + 1, h:h + 1]
        r = orc.bwd(sl(t["Q"]), [sl(k) for k in K], [sl(v) for v in V], rg[b:b + 1], sl(dO), cfg.W)
        for l in range(3):
            _bf16_ok(np64(g["dK"][l][b, h]), r["dK"][l][0, 0], f"dK{l}[{b},{h}]")
            _bf16_ok(np64(g["dV"][l][b, h]), r["dV"][l][0, 0], f"dV{l}[{b},{h}]")


def test_g4_paged_grouped_query_decode_full_size(mka, orc):
    """Workload g4 as bench.py launches it; the oracle evaluates sequence 0 (all 28 heads, all 143360 cached rows)."""
    from mka_inputs import PAGED_CONFIGS, make_paged
    cfg = PAGED_CONFIGS["g4"]
    P = make_paged(cfg, "cuda")
    gate = (P["gate_raw"] / P["gate_raw"].sum(1, keepdim=True)).contiguous()
    shape = mka.make_shape(cfg.B, cfg.H, 1, cfg.d, 32)
    O, LSE = mka.mka_decode_paged(shape, cfg.H_kv, P["q"], P["pools_k"], P["pools_v"], P["tables"], list(cfg.N), gate,
                                  rows=P["rows"])
    i64 = lambda t: t.cpu().numpy().astype(np.int64)
    Or, Lr = orc.decode_paged(np64(P["q"][:1]), [np64(k) for k in P["pools_k"]], [np64(v) for v in P["pools_v"]],
                              [i64(t[:1]) for t in P["tables"]], [i64(r[:1]) for r in P["rows"]], cfg.page_rows, np64(gate[:1]))
    _bf16_ok(np64(O[:1]), Or, "g4 O")
    assert np.abs(np64(LSE[:1]) - Lr).max() <= 2e-3
    assert torch.isfinite(O.float()).all() and torch.isfinite(LSE).all()


def test_r3_recall_full_size_is_bit_exact(mka, orc):
    """Workload r3: codes of the whole pool and the recall lists of every (sequence, KV head) against the oracle."""
    from mka_inputs import RECALL_CONFIGS, make_recall
    cfg = RECALL_CONFIGS["r3"]
    P = make_recall(cfg, "cuda")
    codes = mka.mka_l3_index(P["pool_k"], P["proj"])
    proj = P["proj"].cpu().numpy()
    want = orc.l3_index(P["pool_k"].float().cpu().numpy(), proj)
    assert np.array_equal(codes.cpu().numpy().view(np.uint32), want)
    table, n_sel, rows = mka.mka_l3_retrieve(P["q"], cfg.H_kv, P["proj"], codes, P["bank"], P["bank_len"], cfg.R, cfg.page_rows)
    t_ref, n_ref = orc.l3_retrieve(P["q"].float().cpu().numpy(), proj, want, P["bank"].cpu().numpy(), P["bank_len"].cpu().numpy(),
                                   cfg.R, cfg.H_kv)
    assert np.array_equal(table.cpu().numpy(), t_ref) and np.array_equal(n_sel.cpu().numpy(), n_ref)
