"""Pins of the oracle's paged, grouped-query decode: the gather against a hand-written page walk, the whole function
against Eq. 5 written out for one row, and its reduction to the dense decode."""
import numpy as np
import pytest


def _case(rng, B, H, H_kv, d, page_rows, rows, extra_pages=3):
    """Pools whose pages are handed out in a shuffled order; unused tail rows and unused pages hold huge values."""
    pools_k, pools_v, tables = [], [], []
    for l in range(3):
        pages_per_seq = [-(-int(r) // page_rows) for r in rows[l]]
        P = sum(pages_per_seq) + extra_pages
        order = rng.permutation(P)
        pk = np.full((P, H_kv, page_rows, d), 1e4)
        pv = np.full((P, H_kv, page_rows, d), -1e4)
        tab = np.zeros((B, max(pages_per_seq + [1])), dtype=np.int32)
        nxt = 0
        for b in range(B):
            for i in range(pages_per_seq[b]):
                pg = int(order[nxt]); nxt += 1
                tab[b, i] = pg
                valid = min(page_rows, int(rows[l][b]) - i * page_rows)
                pk[pg, :, :valid] = rng.normal(size=(H_kv, valid, d))
                pv[pg, :, :valid] = rng.normal(size=(H_kv, valid, d))
        pools_k.append(pk); pools_v.append(pv); tables.append(tab)
    q = rng.normal(size=(B, H, d))
    g = rng.random((B, 3)) + 0.05
    return q, pools_k, pools_v, tables, g / g.sum(1, keepdims=True)


def test_gather_walks_the_page_table(orc):
    pool = np.arange(5 * 2 * 4 * 3, dtype=np.float64).reshape(5, 2, 4, 3)
    got = orc.gather_pages(pool, [3, 0, 4], 10, 4)
    assert got.shape == (2, 10, 3)
    # row 0..3 = page 3, rows 4..7 = page 0, rows 8, 9 = the first two rows of page 4
    want = np.concatenate([pool[3], pool[0], pool[4][:, :2]], axis=1)
    assert np.array_equal(got, want)


def test_paged_decode_equals_eq5_written_out(orc):
    rng = np.random.default_rng(5)
    B, H, H_kv, d, pr = 2, 6, 2, 8, 4
    rows = [np.array([5, 9]), np.array([13, 2]), np.array([7, 0])]
    q, pk, pv, tab, g = _case(rng, B, H, H_kv, d, pr, rows)
    O, LSE = orc.decode_paged(q, pk, pv, tab, rows, pr, g)
    tau = 1.0 / np.sqrt(d)
    for b in range(B):
        for h in range(H):
            kvh = h // 3                                  # heads 0-2 share KV head 0, heads 3-5 KV head 1
            num, Z = np.zeros(d), 0.0
            for l in range(3):
                for r in range(int(rows[l][b])):
                    page, off = tab[l][b, r // pr], r % pr
                    w = g[b, l] * np.exp(tau * q[b, h] @ pk[l][page, kvh, off])
                    num += w * pv[l][page, kvh, off]
                    Z += w
            assert np.allclose(O[b, h], num / Z, rtol=1e-12, atol=1e-12)
            assert np.isclose(LSE[b, h], np.log(Z), rtol=1e-12)


def test_identity_table_one_group_is_the_dense_decode(orc):
    rng = np.random.default_rng(6)
    B, H, d, pr, n = 2, 3, 8, 4, 12
    K = [rng.normal(size=(B, H, n, d)) for _ in range(3)]
    V = [rng.normal(size=(B, H, n, d)) for _ in range(3)]
    q = rng.normal(size=(B, H, d))
    g = np.full((B, 3), 1.0 / 3)
    # pool page (b * n/pr + i) holds rows [i*pr, (i+1)*pr) of sequence b
    pk = [k.reshape(B, H, n // pr, pr, d).transpose(0, 2, 1, 3, 4).reshape(B * n // pr, H, pr, d) for k in K]
    pv = [v.reshape(B, H, n // pr, pr, d).transpose(0, 2, 1, 3, 4).reshape(B * n // pr, H, pr, d) for v in V]
    tab = [np.arange(B * n // pr, dtype=np.int32).reshape(B, n // pr)] * 3
    rows = [np.full(B, n)] * 3
    O, LSE = orc.decode_paged(q, pk, pv, tab, rows, pr, g)
    Od, Ld = orc.fwd(q[:, :, None, :], K, V, g.reshape(B, 1, 3), 1, decode=True)
    assert np.array_equal(O, Od[:, :, 0]) and np.array_equal(LSE, Ld[:, :, 0])


def test_result_does_not_depend_on_where_the_pages_live(orc):
    rng = np.random.default_rng(7)
    B, H, H_kv, d, pr = 1, 4, 2, 8, 4
    rows = [np.array([6]), np.array([11]), np.array([8])]
    q, pk, pv, tab, g = _case(rng, B, H, H_kv, d, pr, rows)
    O1, L1 = orc.decode_paged(q, pk, pv, tab, rows, pr, g)
    pk2, pv2, tab2 = [], [], []
    for l in range(3):
        perm = rng.permutation(pk[l].shape[0])            # new home of every page
        inv = np.empty_like(perm); inv[perm] = np.arange(perm.size)
        pk2.append(pk[l][inv]); pv2.append(pv[l][inv])    # page j of the old pool now sits at perm[j]
        tab2.append(perm[tab[l]].astype(np.int32))
    O2, L2 = orc.decode_paged(q, pk2, pv2, tab2, rows, pr, g)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)


def test_per_head_tables_that_agree_equal_the_shared_table(orc):
    rng = np.random.default_rng(8)
    B, H, H_kv, d, pr = 2, 4, 2, 8, 4
    rows = [np.array([6, 3]), np.array([9, 12]), np.array([8, 8])]
    q, pk, pv, tab, g = _case(rng, B, H, H_kv, d, pr, rows)
    O1, L1 = orc.decode_paged(q, pk, pv, tab, rows, pr, g)
    per_head = [np.repeat(t[:, None, :], H_kv, axis=1) for t in tab]
    O2, L2 = orc.decode_paged(q, pk, pv, per_head, rows, pr, g)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)
    # and a table that differs between the heads moves only the heads of that KV head
    per_head[1][0, 1] = per_head[1][0, 1][::-1].copy()
    O3, _ = orc.decode_paged(q, pk, pv, per_head, rows, pr, g)
    assert np.array_equal(O3[0, :2], O1[0, :2]) and not np.array_equal(O3[0, 2:], O1[0, 2:])
    assert np.array_equal(O3[1], O1[1])


def test_paged_forward_with_identity_tables_is_the_dense_forward(orc):
    rng = np.random.default_rng(9)
    B, H, T, d, pr, n, W = 2, 2, 10, 8, 4, 12, 5
    K = [rng.normal(size=(B, H, n, d)) for _ in range(3)]
    V = [rng.normal(size=(B, H, n, d)) for _ in range(3)]
    Q = rng.normal(size=(B, H, T, d))
    g = rng.random((B, T, 3)) + 0.1
    g /= g.sum(-1, keepdims=True)
    pk = [k.reshape(B, H, n // pr, pr, d).transpose(0, 2, 1, 3, 4).reshape(B * n // pr, H, pr, d) for k in K]
    pv = [v.reshape(B, H, n // pr, pr, d).transpose(0, 2, 1, 3, 4).reshape(B * n // pr, H, pr, d) for v in V]
    tab = [np.arange(B * n // pr, dtype=np.int32).reshape(B, n // pr)] * 3
    O, L = orc.fwd_paged(Q, pk, pv, tab, [n, n, n], pr, g, W, q_offset=2)
    Od, Ld = orc.fwd(Q, K, V, g, W, q_offset=2)
    assert np.array_equal(O, Od) and np.array_equal(L, Ld)


def test_paged_forward_equals_eq5_written_out_through_the_tables(orc):
    """Grouped heads, shuffled pools, a level with one page table per KV head, per-sequence row counts with one empty
    sequence, a window shorter than the sequence and a query offset: every output row against Eq. 5 written out with
    its own page walk and its own visibility rules."""
    rng = np.random.default_rng(10)
    B, H, H_kv, T, d, pr, W, q_off = 2, 6, 2, 7, 8, 4, 3, 2
    rows = [np.array([9, 6]), np.array([8, 0]), np.array([9, 14])]       # level 2 of sequence 1 is empty
    _, pk, pv, tab, _ = _case(rng, B, H, H_kv, d, pr, rows)
    # long-term level: one table per KV head, the second head walks the same pages in reverse order
    per_head = np.repeat(tab[2][:, None, :], H_kv, axis=1)
    for b in range(B):
        used = -(-int(rows[2][b]) // pr)
        full = int(rows[2][b]) // pr                                       # only whole pages can swap places
        per_head[b, 1, :full] = per_head[b, 1, :full][::-1].copy()
        assert used > full >= 2
    tables = [tab[0], tab[1], per_head]
    Q = rng.normal(size=(B, H, T, d))
    g = rng.random((B, T, 3)) + 0.05
    g /= g.sum(-1, keepdims=True)
    O, LSE = orc.fwd_paged(Q, pk, pv, tables, rows, pr, g, W, q_offset=q_off)
    tau = 1.0 / np.sqrt(d)
    for b in range(B):
        for h in range(H):
            kvh = h // 3                                  # heads 0-2 share KV head 0, heads 3-5 KV head 1
            for t in range(T):
                p = t + q_off
                num, Z = np.zeros(d), 0.0
                for l in range(3):
                    for r in range(int(rows[l][b])):
                        if l == 0 and not (p - W < r <= p):
                            continue
                        if l == 1 and not r <= p:
                            continue
                        page = tables[l][b, kvh, r // pr] if l == 2 else tables[l][b, r // pr]
                        w = g[b, t, l] * np.exp(tau * Q[b, h, t] @ pk[l][page, kvh, r % pr])
                        num += w * pv[l][page, kvh, r % pr]
                        Z += w
                assert Z > 0
                assert np.allclose(O[b, h, t], num / Z, rtol=1e-12, atol=1e-12)
                assert np.isclose(LSE[b, h, t], np.log(Z), rtol=1e-12)
    # a table entry of KV head 1 that points somewhere else must change the heads of that KV head only
    other = per_head.copy()
    other[0, 1, 0] = per_head[1, 0, 0]                     # a full page of the other sequence: valid, different data
    O2, _ = orc.fwd_paged(Q, pk, pv, [tab[0], tab[1], other], rows, pr, g, W, q_offset=q_off)
    assert np.array_equal(O2[0, :3], O[0, :3]) and not np.array_equal(O2[0, 3:], O[0, 3:])
    assert np.array_equal(O2[1], O[1])
