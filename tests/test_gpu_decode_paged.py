"""GPU parity of the paged, grouped-query decode against the oracle, through the C ABI."""
import dataclasses

import numpy as np
import pytest
import torch

from gpu_helpers import check, np64, poison_unused_pool_rows
from mka_inputs import PAGED_CONFIGS, PagedConfig, make_paged

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mka():
    import paper_2603_20586_b200 as m
    assert torch.cuda.is_available()
    return m


def _run(mka, cfg, P, gate, rows=True, **kw):
    shape = mka.make_shape(cfg.B, cfg.H, 1, cfg.d, 32)
    return mka.mka_decode_paged(shape, cfg.H_kv, P["q"], P["pools_k"], P["pools_v"], P["tables"], list(cfg.N), gate,
                                rows=P["rows"] if rows else None, **kw)


def _oracle(orc, cfg, P, gate, rows=None):
    rows = [np64(r).astype(np.int64) for r in (rows if rows is not None else P["rows"])]
    opt = lambda t: None if t is None else np64(t)
    return orc.decode_paged(np64(P["q"]), [opt(k) for k in P["pools_k"]], [opt(v) for v in P["pools_v"]],
                            [np64(t).astype(np.int64) for t in P["tables"]], rows, cfg.page_rows, np64(gate))


def _gate(P):
    g = P["gate_raw"]
    return (g / g.sum(1, keepdim=True)).contiguous()


CASES = [
    PAGED_CONFIGS["g1"],                                                                 # G = 3, d = 64, ragged, one empty sequence
    PagedConfig("t_mha", 11, 2, 4, 4, 128, (70, 300, 129), 16, rows_frac=(1.0, 0.5)),    # G = 1
    PagedConfig("t_g7", 12, 2, 28, 4, 128, (257, 2100, 64), 16, rows_frac=(1.0, 0.71)),  # Qwen-like 28 / 4
    PagedConfig("t_g16", 13, 1, 16, 1, 64, (64, 1500, 40), 32),                          # the widest group
    PagedConfig("t_p1", 14, 2, 8, 2, 64, (33, 90, 17), 1, rows_frac=(1.0, 0.6)),         # one row per page
    PagedConfig("t_p256", 15, 2, 8, 4, 128, (300, 5000, 1000), 256, rows_frac=(0.9, 1.0)),
    PagedConfig("t_l2only", 16, 2, 6, 2, 128, (0, 1300, 0), 16),                         # absent levels
    # many (sequence, KV head) groups make the split table pick chunks of more than 1024 rows; with one row per page a
    # chunk then spans more table entries than the kernel keeps in shared memory (it looks them up in place)
    PagedConfig("t_longchunk", 22, 8, 8, 8, 64, (0, 40000, 0), 1, rows_frac=(1.0, 0.93)),
]


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
def test_paged_decode_matches_oracle(mka, orc, cfg):
    P = make_paged(cfg, "cuda")
    gate = _gate(P)
    O, LSE = _run(mka, cfg, P, gate)
    Or, Lr = _oracle(orc, cfg, P, gate)
    live = np.isfinite(Lr)                                   # a sequence with no rows at all: O = 0, LSE = -inf
    check(O, np.where(live[..., None], Or, 0.0), torch.bfloat16, "paged decode O")
    assert np.array_equal(np.isfinite(np64(LSE)), live)
    assert np.abs(np64(LSE)[live] - Lr[live]).max() <= 2e-3


def test_rows_pointer_null_means_every_sequence_is_full(mka, orc):
    cfg = PagedConfig("t_full", 17, 2, 8, 2, 128, (128, 640, 96), 16)
    P = make_paged(cfg, "cuda")
    gate = _gate(P)
    O, _ = _run(mka, cfg, P, gate, rows=False)
    O2, _ = _run(mka, cfg, P, gate, rows=True)
    assert torch.equal(O, O2)
    Or, _ = _oracle(orc, cfg, P, gate)
    check(O, Or, torch.bfloat16, "paged decode, rows = NULL")


def test_zero_gate_level_is_not_read(mka, orc):
    cfg = PagedConfig("t_skip", 18, 2, 8, 2, 128, (100, 900, 200), 16)
    P = make_paged(cfg, "cuda")
    gate = _gate(P)
    gate[:, 1] = 0.0
    gate = (gate / gate.sum(1, keepdim=True)).contiguous()
    P["pools_k"][1].fill_(float("nan"))                      # whatever is there must not matter
    P["pools_v"][1].fill_(float("nan"))
    O, LSE = _run(mka, cfg, P, gate)
    assert torch.isfinite(O.float()).all() and torch.isfinite(LSE).all()
    off = dataclasses.replace(cfg, N=(cfg.N[0], 0, cfg.N[2]))
    rows = [P["rows"][0], torch.zeros_like(P["rows"][1]), P["rows"][2]]
    Or, Lr = _oracle(orc, off, {**P, "pools_k": [P["pools_k"][0], None, P["pools_k"][2]],
                                "pools_v": [P["pools_v"][0], None, P["pools_v"][2]]}, gate, rows=rows)
    check(O, Or, torch.bfloat16, "paged decode, gated-off level")


def test_dense_decode_skips_a_gated_off_level_too(mka, orc):
    B, H, d = 2, 4, 128
    K = [torch.randn(B, H, n, d, device="cuda").bfloat16() for n in (64, 500, 100)]
    V = [torch.randn(B, H, n, d, device="cuda").bfloat16() for n in (64, 500, 100)]
    q = torch.randn(B, H, d, device="cuda").bfloat16()
    gate = torch.tensor([[0.4, 0.0, 0.6], [1.0, 0.0, 0.0]], device="cuda")
    K[1].fill_(float("nan")); V[1].fill_(float("nan"))
    O, LSE = mka.mka_decode(mka.make_shape(B, H, 1, d, 32), q, K, V, gate)
    assert torch.isfinite(O.float()).all() and torch.isfinite(LSE).all()
    Kz = [K[0], torch.zeros(B, H, 0, d, device="cuda").bfloat16(), K[2]]
    Vz = [V[0], torch.zeros(B, H, 0, d, device="cuda").bfloat16(), V[2]]
    Or, _ = orc.fwd(np64(q)[:, :, None, :], [np64(k) for k in Kz], [np64(v) for v in Vz], np64(gate).reshape(B, 1, 3), 1,
                    decode=True)
    check(O.view(B, H, 1, d), Or, torch.bfloat16, "dense decode, gated-off level")


def test_pool_layout_with_rows_outermost(mka, orc):
    """Pools stored [pages, page_rows, H_kv, d] (heads interleaved inside a row) reach the same result through strides."""
    cfg = PagedConfig("t_layout", 19, 2, 12, 4, 64, (50, 800, 70), 16, rows_frac=(1.0, 0.8))
    P = make_paged(cfg, "cuda")
    gate = _gate(P)
    O1, _ = _run(mka, cfg, P, gate)
    P2 = dict(P)
    P2["pools_k"] = [k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) for k in P["pools_k"]]
    P2["pools_v"] = [v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) for v in P["pools_v"]]
    assert P2["pools_k"][1].stride() != P["pools_k"][1].stride()
    O2, _ = _run(mka, cfg, P2, gate)
    assert torch.equal(O1, O2)


def test_paged_equals_dense_on_the_gathered_levels(mka):
    cfg = PagedConfig("t_same", 20, 2, 8, 8, 128, (256, 2048, 512), 16)      # G = 1, every sequence full
    P = make_paged(cfg, "cuda")
    gate = _gate(P)
    O, LSE = _run(mka, cfg, P, gate)
    K, V = [], []
    for l in range(3):
        idx = P["tables"][l].long()                                            # [B, pages]
        K.append(P["pools_k"][l][idx].permute(0, 2, 1, 3, 4).reshape(cfg.B, cfg.H, -1, cfg.d)[:, :, :cfg.N[l]].contiguous())
        V.append(P["pools_v"][l][idx].permute(0, 2, 1, 3, 4).reshape(cfg.B, cfg.H, -1, cfg.d)[:, :, :cfg.N[l]].contiguous())
    Od, Ld = mka.mka_decode(mka.make_shape(cfg.B, cfg.H, 1, cfg.d, 32), P["q"], K, V, gate)
    assert (O.float() - Od.float()).abs().max() <= 1e-2 and (LSE - Ld).abs().max() <= 1e-3


def test_paged_decode_rejects_bad_arguments(mka):
    cfg = PagedConfig("t_bad", 21, 1, 8, 2, 128, (32, 64, 32), 16)
    P = make_paged(cfg, "cuda")
    gate = _gate(P)
    shape = mka.make_shape(1, 8, 1, 128, 32)
    with pytest.raises(mka.MkaError) as e:                                     # 8 heads do not split over 3 KV heads
        mka.mka_decode_paged(shape, 3, P["q"], P["pools_k"], P["pools_v"], P["tables"], list(cfg.N), gate)
    assert e.value.code == 2
    with pytest.raises(mka.MkaError) as e:                                     # page table too narrow for n
        mka.mka_decode_paged(shape, 2, P["q"], P["pools_k"], P["pools_v"], P["tables"], [32, 6400, 32], gate)
    assert e.value.code == 2
    bad = [k[:, :, :12] for k in P["pools_k"]]                                 # 12 rows per page: not a power of two
    with pytest.raises(mka.MkaError) as e:
        mka.mka_decode_paged(shape, 2, P["q"], bad, [v[:, :, :12] for v in P["pools_v"]], P["tables"], list(cfg.N), gate)
    assert e.value.code == 2
    with pytest.raises(mka.MkaError) as e:                                     # workspace too small
        mka.mka_decode_paged(shape, 2, P["q"], P["pools_k"], P["pools_v"], P["tables"], list(cfg.N), gate,
                             ws=torch.empty(64, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 4


@pytest.mark.parametrize("cfg", [
    PagedConfig("t_nan16", 23, 2, 8, 2, 128, (300, 2500, 90), 16, rows_frac=(1.0, 0.73)),      # the copy-engine kernel
    PagedConfig("t_nan256", 24, 2, 6, 2, 64, (700, 3000, 300), 256, rows_frac=(0.9, 1.0)),     # pages longer than a tile
    PagedConfig("t_nan4", 25, 2, 4, 2, 64, (70, 500, 30), 4, rows_frac=(1.0, 0.6)),            # small pages: the cp.async kernel
], ids=lambda c: c.name)
def test_paged_decode_ignores_rows_after_a_sequence_end(mka, orc, cfg):
    """Pool rows that no sequence owns (the rest of a partly filled last page, unused pages) hold NaN: their weights are
    zero and they must not reach the output through 0 x NaN in the value product."""
    P = make_paged(cfg, "cuda")
    gate = _gate(P)
    rows = [r.cpu().numpy() for r in P["rows"]]
    poison_unused_pool_rows(P, cfg, rows)
    O, LSE = _run(mka, cfg, P, gate)
    assert bool(torch.isfinite(O.float()).all()) and bool(torch.isfinite(LSE).all())
    clean = {**P, "pools_k": [torch.nan_to_num(k, nan=0.0) for k in P["pools_k"]],
             "pools_v": [torch.nan_to_num(v, nan=0.0) for v in P["pools_v"]]}       # the oracle never gathers those rows either
    Or, Lr = _oracle(orc, cfg, clean, gate)
    check(O, Or, torch.bfloat16, "paged decode, poisoned tails")
    assert np.abs(np64(LSE) - Lr).max() <= 2e-3
