"""GPU parity of the fused forward over paged levels (grouped-query heads) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from gpu_helpers import check, np64, poison_unused_pool_rows
from mka_inputs import PagedConfig, approx_normal, make_paged

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mka():
    import paper_2603_20586_b200 as m
    assert torch.cuda.is_available()
    return m


def _inputs(cfg, T, seed):
    P = make_paged(cfg, "cuda")
    Q = approx_normal(seed, 60, 0, cfg.B * cfg.H * T * cfg.d, 1.0, "cpu", torch.bfloat16).view(cfg.B, cfg.H, T, cfg.d).cuda()
    g = approx_normal(seed, 61, 0, cfg.B * T * 3, 1.0, "cpu", torch.float32).view(cfg.B, T, 3).cuda()
    return P, Q, torch.softmax(g, -1).contiguous()


# (config, T, window, q_offset): the levels hold q_offset + T rows where the visibility is causal
CASES = [
    (PagedConfig("f_16", 51, 2, 4, 2, 128, (300, 300, 90), 16), 300, 70, 0),
    (PagedConfig("f_8", 52, 1, 8, 2, 64, (520, 520, 200), 8), 400, 129, 120),        # a later chunk of a prefill
    (PagedConfig("f_128", 53, 2, 2, 2, 128, (384, 384, 256), 128), 384, 384, 0),       # page = tile, one group per head
    (PagedConfig("f_256", 54, 1, 6, 1, 64, (700, 700, 300), 256), 700, 100, 0),       # pages longer than a tile, 6 heads on 1
    (PagedConfig("f_l12", 55, 2, 4, 4, 128, (260, 260, 0), 32), 260, 64, 0),          # no long-term level
]


@pytest.mark.parametrize("cfg,T,W,q_off", CASES, ids=lambda c: c.name if isinstance(c, PagedConfig) else None)
def test_paged_forward_matches_oracle(mka, orc, cfg, T, W, q_off):
    P, Q, gate = _inputs(cfg, T, cfg.seed)
    shape = mka.make_shape(cfg.B, cfg.H, T, cfg.d, 32, W, q_off)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    O, LSE = mka.mka_fwd_paged(shape, cfg.H_kv, Q, P["pools_k"], P["pools_v"], P["tables"], list(cfg.N), gate, ws=ws)
    assert mka.mka_device_status(ws) == 0
    opt = lambda t: None if t is None else np64(t)
    Or, Lr = orc.fwd_paged(np64(Q), [opt(k) for k in P["pools_k"]], [opt(v) for v in P["pools_v"]],
                           [t.cpu().numpy().astype(np.int64) for t in P["tables"]], list(cfg.N), cfg.page_rows, np64(gate), W,
                           q_offset=q_off)
    check(O, Or, torch.bfloat16, "paged fwd O")
    live = np.isfinite(Lr)
    assert np.array_equal(np.isfinite(np64(LSE)), live) and np.abs(np64(LSE)[live] - Lr[live]).max() <= 2e-3


def test_paged_forward_with_a_length_per_sequence(mka, orc):
    cfg, T, W = PagedConfig("f_ragged", 58, 3, 4, 2, 128, (400, 400, 150), 16, rows_frac=(1.0, 0.55, 0.0)), 400, 90
    P, Q, gate = _inputs(cfg, T, cfg.seed)
    O, LSE = mka.mka_fwd_paged(mka.make_shape(cfg.B, cfg.H, T, cfg.d, 32, W), cfg.H_kv, Q, P["pools_k"], P["pools_v"], P["tables"],
                               list(cfg.N), gate, rows=P["rows"])
    Or, Lr = orc.fwd_paged(np64(Q), [np64(k) for k in P["pools_k"]], [np64(v) for v in P["pools_v"]],
                           [t.cpu().numpy().astype(np.int64) for t in P["tables"]], [r.cpu().numpy() for r in P["rows"]],
                           cfg.page_rows, np64(gate), W)
    live = np.isfinite(Lr)                                    # the empty sequence sees nothing: O = 0, LSE = -inf
    assert live[:2].all() and not live[2].any()
    check(O, np.where(live[..., None], Or, 0.0), torch.bfloat16, "paged fwd, ragged")
    assert np.array_equal(np.isfinite(np64(LSE)), live) and np.abs(np64(LSE)[live] - Lr[live]).max() <= 2e-3


@pytest.mark.parametrize("cfg,T,W", [
    (PagedConfig("f_nan16", 59, 2, 4, 2, 128, (300, 300, 90), 16, rows_frac=(1.0, 0.7)), 300, 70),
    (PagedConfig("f_nan256", 60, 2, 6, 1, 64, (700, 700, 300), 256, rows_frac=(0.9, 1.0)), 700, 100),
], ids=lambda c: c.name if isinstance(c, PagedConfig) else None)
def test_paged_forward_ignores_rows_after_a_sequence_end(mka, orc, cfg, T, W):
    """Rows of a partly filled page after the sequence's last row hold NaN here; their weights are zero and must not
    reach the output through 0 x NaN in the value product."""
    P, Q, gate = _inputs(cfg, T, cfg.seed)
    rows = [r.cpu().numpy() for r in P["rows"]]
    poison_unused_pool_rows(P, cfg, rows)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    O, LSE = mka.mka_fwd_paged(mka.make_shape(cfg.B, cfg.H, T, cfg.d, 32, W), cfg.H_kv, Q, P["pools_k"], P["pools_v"], P["tables"],
                               list(cfg.N), gate, rows=P["rows"], ws=ws)
    assert mka.mka_device_status(ws) == 0
    assert bool(torch.isfinite(O.float()).all())
    clean = lambda t: np.nan_to_num(np64(t), nan=0.0)          # the oracle never gathers those rows either
    Or, Lr = orc.fwd_paged(np64(Q), [clean(k) for k in P["pools_k"]], [clean(v) for v in P["pools_v"]],
                           [t.cpu().numpy().astype(np.int64) for t in P["tables"]], rows, cfg.page_rows, np64(gate), W)
    live = np.isfinite(Lr)
    check(O, np.where(live[..., None], Or, 0.0), torch.bfloat16, "paged fwd, poisoned tails")
    assert np.array_equal(np.isfinite(np64(LSE)), live) and np.abs(np64(LSE)[live] - Lr[live]).max() <= 2e-3


def test_paged_forward_equals_dense_forward_on_gathered_levels(mka):
    cfg, T, W = PagedConfig("f_same", 56, 2, 4, 2, 128, (512, 512, 128), 16), 512, 200
    P, Q, gate = _inputs(cfg, T, cfg.seed)
    O, LSE = mka.mka_fwd_paged(mka.make_shape(cfg.B, cfg.H, T, cfg.d, 32, W), cfg.H_kv, Q, P["pools_k"], P["pools_v"], P["tables"],
                               list(cfg.N), gate)
    K, V = [], []
    for l in range(3):
        idx = P["tables"][l].long()
        K.append(P["pools_k"][l][idx].permute(0, 2, 1, 3, 4).reshape(cfg.B, cfg.H_kv, -1, cfg.d)[:, :, :cfg.N[l]].contiguous())
        V.append(P["pools_v"][l][idx].permute(0, 2, 1, 3, 4).reshape(cfg.B, cfg.H_kv, -1, cfg.d)[:, :, :cfg.N[l]].contiguous())
    Od, Ld = mka.mka_fwd(mka.make_shape(cfg.B, cfg.H, T, cfg.d, 32, W, kv_heads=cfg.H_kv), Q, K, V, gate)
    assert torch.equal(O, Od) and torch.equal(LSE, Ld)       # same tiles, same order of operations


def test_paged_forward_rejects_what_it_does_not_do(mka):
    cfg, T = PagedConfig("f_bad", 57, 1, 4, 2, 128, (128, 128, 64), 16), 128
    P, Q, gate = _inputs(cfg, T, cfg.seed)
    with pytest.raises(mka.MkaError) as e:                    # four rows per page: below the 8-row swizzle atom
        mka.mka_fwd_paged(mka.make_shape(1, 4, T, 128, 32, 32), 2, Q, [k[:, :, :4] for k in P["pools_k"]],
                          [v[:, :, :4] for v in P["pools_v"]], P["tables"], [16, 16, 16], gate)
    assert e.value.code == 2
    with pytest.raises(mka.MkaError) as e:                    # the CUDA-core kernel has no paged form
        mka.mka_fwd_paged(mka.make_shape(1, 4, T, 128, 32, 32, flags=1), 2, Q, P["pools_k"], P["pools_v"], P["tables"],
                          list(cfg.N), gate)
    assert e.value.code == 5
