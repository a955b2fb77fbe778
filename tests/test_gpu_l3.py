"""GPU parity of the L3 recall (codes, recall lists: bit-exact) and of the decode over the recalled chunks."""
import numpy as np
import pytest
import torch

from gpu_helpers import check, np64
from mka_inputs import RECALL_CONFIGS, RecallConfig, approx_normal, make_recall

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mka():
    import paper_2603_20586_b200 as m
    assert torch.cuda.is_available()
    return m


def _u32(t):
    return t.cpu().numpy().view(np.uint32)


CASES = [
    RECALL_CONFIGS["r1"],                                                         # d = 64, 32 bits, short and empty banks
    RecallConfig("t_64", 31, 2, 8, 2, 128, 300, 16, 64, 8, len_frac=(1.0, 0.5)),
    RecallConfig("t_128", 32, 1, 16, 1, 128, 129, 4, 128, 5),
    RecallConfig("t_256", 33, 2, 4, 4, 64, 70, 32, 256, 64, len_frac=(1.0, 0.9)),   # R = 64 = most of the bank
    RecallConfig("t_g7", 34, 2, 28, 4, 128, 2000, 16, 64, 8),
    # a 16 KB chunk (64 rows of 128), and 128-bit codes over many batches with a partly used and an empty bank
    RecallConfig("t_p64", 37, 1, 4, 2, 128, 300, 64, 64, 8),
    RecallConfig("t_b128", 38, 3, 8, 2, 128, 333, 8, 128, 8, len_frac=(1.0, 0.3, 0.0)),
]


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
def test_index_and_recall_lists_are_bit_exact(mka, orc, cfg):
    P = make_recall(cfg, "cuda")
    codes = mka.mka_l3_index(P["pool_k"], P["proj"])
    want = orc.l3_index(P["pool_k"].float().cpu().numpy(), P["proj"].cpu().numpy())
    assert np.array_equal(_u32(codes), want)
    table, n_sel, rows = mka.mka_l3_retrieve(P["q"], cfg.H_kv, P["proj"], codes, P["bank"], P["bank_len"], cfg.R, cfg.page_rows)
    t_ref, n_ref = orc.l3_retrieve(P["q"].float().cpu().numpy(), P["proj"].cpu().numpy(), want, P["bank"].cpu().numpy(),
                                   P["bank_len"].cpu().numpy(), cfg.R, cfg.H_kv)
    assert np.array_equal(table.cpu().numpy(), t_ref)
    assert np.array_equal(n_sel.cpu().numpy(), n_ref)
    assert np.array_equal(rows.cpu().numpy(), n_ref * cfg.page_rows)


def test_index_reads_a_strided_pool(mka):
    cfg = RecallConfig("t_str", 35, 1, 8, 4, 64, 50, 8, 64, 4)
    P = make_recall(cfg, "cuda")
    a = mka.mka_l3_index(P["pool_k"], P["proj"])
    strided = P["pool_k"].permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)       # rows outermost inside a page
    assert strided.stride() != P["pool_k"].stride()
    assert torch.equal(a, mka.mka_l3_index(strided, P["proj"]))


def test_planted_chunk_is_recalled_and_dominates_the_decode(mka, orc):
    cfg = RecallConfig("t_plant", 36, 2, 8, 2, 128, 500, 16, 64, 8)
    P = make_recall(cfg, "cuda")
    G = cfg.H // cfg.H_kv
    planted = []
    for b in range(cfg.B):                                                          # one chunk per (sequence, KV head)
        for h in range(cfg.H_kv):
            page = int(P["bank"][b, 100 + 17 * h + b])
            qsum = P["q"][b, h * G:(h + 1) * G].float().sum(0)
            P["pool_k"][page, h] = (qsum / 4).bfloat16()[None, :]                  # keys along the summed query
            planted.append((b, h, page))
    codes = mka.mka_l3_index(P["pool_k"], P["proj"])
    table, n_sel, rows = mka.mka_l3_retrieve(P["q"], cfg.H_kv, P["proj"], codes, P["bank"], P["bank_len"], cfg.R, cfg.page_rows)
    for b, h, page in planted:
        assert page in table[b, h].tolist()
    # decode over the recalled chunks alone (L3 only), per-head recall lists
    gate = torch.tensor([[0.0, 0.0, 1.0]] * cfg.B, device="cuda")
    shape = mka.make_shape(cfg.B, cfg.H, 1, cfg.d, 32)
    n3 = cfg.R * cfg.page_rows
    O, LSE = mka.mka_decode_paged(shape, cfg.H_kv, P["q"], [None, None, P["pool_k"]], [None, None, P["pool_v"]],
                                  [None, None, table], [0, 0, n3], gate, rows=[None, None, rows])
    Or, Lr = orc.decode_paged(np64(P["q"]), [None, None, np64(P["pool_k"])], [None, None, np64(P["pool_v"])],
                              [None, None, table.cpu().numpy().astype(np.int64)],
                              [np.zeros(cfg.B, int), np.zeros(cfg.B, int), rows.cpu().numpy().astype(np.int64)],
                              cfg.page_rows, np64(gate))
    check(O, Or, torch.bfloat16, "decode over recalled chunks")
    assert np.abs(np64(LSE) - Lr).max() <= 2e-3


def test_l3_rejects_bad_arguments(mka):
    cfg = RecallConfig("t_bad", 37, 1, 8, 2, 64, 20, 8, 64, 4)
    P = make_recall(cfg, "cuda")
    with pytest.raises(mka.MkaError) as e:
        mka.mka_l3_index(P["pool_k"], P["proj"][:48].contiguous())                   # 48 bits
    assert e.value.code == 2
    codes = mka.mka_l3_index(P["pool_k"], P["proj"])
    with pytest.raises(mka.MkaError) as e:
        mka.mka_l3_retrieve(P["q"], 3, P["proj"], codes, P["bank"], P["bank_len"], 4, 8)   # 8 heads on 3 KV heads
    assert e.value.code == 2
    with pytest.raises(mka.MkaError) as e:
        mka.mka_l3_retrieve(P["q"], 2, P["proj"], codes, P["bank"], P["bank_len"], 65, 8)  # R too large
    assert e.value.code == 2


def test_recall_over_a_bank_of_70000_chunks(mka, orc):
    """A bank longer than 65536 chunks (scores beyond 128 KB of shared memory); codes are planted by hand."""
    B, H, H_kv, d, bits, R, n = 1, 2, 1, 64, 64, 8, 70000
    g = torch.Generator().manual_seed(5)
    codes = torch.randint(-2**31, 2**31 - 1, (n + 5, H_kv, bits // 32), generator=g, dtype=torch.int64).int().cuda()
    proj = approx_normal(38, 1, 0, bits * d, 1.0, "cpu", torch.float32).view(bits, d).cuda()
    q = approx_normal(38, 2, 0, B * H * d, 1.0, "cpu", torch.bfloat16).view(B, H, d).cuda()
    bank = torch.randperm(n + 5, generator=g)[:n].int().view(1, n).cuda()
    bank_len = torch.tensor([n], dtype=torch.int32, device="cuda")
    table, n_sel, rows = mka.mka_l3_retrieve(q, H_kv, proj, codes, bank, bank_len, R, 16)
    t_ref, n_ref = orc.l3_retrieve(q.float().cpu().numpy(), proj.cpu().numpy(), codes.cpu().numpy().view(np.uint32),
                                   bank.cpu().numpy(), bank_len.cpu().numpy(), R, H_kv)
    assert np.array_equal(table.cpu().numpy(), t_ref) and int(n_sel[0]) == R
