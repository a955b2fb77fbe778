"""Pins of the oracle's L3 recall (sign-random-projection codes, Hamming top-R): closed forms and brute force."""
import numpy as np


def _bits(code, bits):
    return [(int(code[j // 32]) >> (j % 32)) & 1 for j in range(bits)]


def test_code_under_identity_projection_is_the_sign_pattern(orc):
    d = 32
    x = np.arange(d, dtype=np.float32) - 11.0            # negative for i < 11, zero at 11, positive after
    code = orc.srp_code(x, np.eye(d, dtype=np.float32))
    assert _bits(code, d) == [0 if v < 0 else 1 for v in x]
    # bit j looks at row j of the projection, column i at x[i]: a single off-diagonal entry moves one bit only
    P = np.eye(d, dtype=np.float32); P[3, 20] = 10.0      # row 3: x[3] + 10 x[20] = -8 + 90 > 0
    assert _bits(orc.srp_code(x, P), d) == [1 if (j == 3 or x[j] >= 0) else 0 for j in range(d)]


def test_code_matches_integer_arithmetic_and_scaling(orc):
    rng = np.random.default_rng(0)
    d, bits = 24, 64
    x = rng.integers(-9, 10, size=d).astype(np.float32)
    P = rng.integers(-5, 6, size=(bits, d)).astype(np.float32)
    want = [1 if int(np.dot(P[j].astype(np.int64), x.astype(np.int64))) >= 0 else 0 for j in range(bits)]
    assert _bits(orc.srp_code(x, P), bits) == want       # all partial sums are small integers: fp32 is exact
    assert np.array_equal(orc.srp_code(4.0 * x, P), orc.srp_code(x, P))
    flipped = _bits(orc.srp_code(-x, P), bits)
    dots = P.astype(np.int64) @ x.astype(np.int64)
    assert all(f == 1 - w for f, w, t in zip(flipped, want, dots) if t != 0)


def test_row_sums_run_in_fp32_row_order(orc):
    x = np.array([[2.0 ** 24], [1.0], [1.0], [-(2.0 ** 24)]], dtype=np.float32)
    assert orc.sum_rows_f32(x)[0] == 0.0                  # 2^24 + 1 rounds back to 2^24 twice; exact maths would say 2
    assert orc.sum_rows_f32(x[[1, 2, 0, 3]])[0] == 2.0    # 1 + 1 first survives


def test_index_is_the_code_of_each_pages_key_sum(orc):
    rng = np.random.default_rng(1)
    pool = rng.integers(-3, 4, size=(5, 2, 4, 16)).astype(np.float32)
    P = rng.integers(-4, 5, size=(32, 16)).astype(np.float32)
    codes = orc.l3_index(pool, P)
    assert codes.shape == (5, 2, 1)
    for pg in range(5):
        for h in range(2):
            t = P.astype(np.int64) @ pool[pg, h].astype(np.int64).sum(0)
            assert _bits(codes[pg, h], 32) == [1 if v >= 0 else 0 for v in t]


def test_selection_against_sorted_hamming_distances(orc):
    rng = np.random.default_rng(2)
    n, words, R = 40, 2, 8
    codes = rng.integers(0, 2 ** 32, size=(n, words), dtype=np.uint64).astype(np.uint32)
    codes[17] = codes[5]                                   # a tie: the earlier index wins when only one fits
    q = rng.integers(0, 2 ** 32, size=words, dtype=np.uint64).astype(np.uint32)
    dist = [sum(bin(int(a) ^ int(b)).count("1") for a, b in zip(q, c)) for c in codes]
    want = sorted(sorted(range(n), key=lambda c: (dist[c], c))[:R])
    assert list(orc.l3_select(q, codes, R)) == want
    assert list(orc.l3_select(q, codes[:3], R)) == [0, 1, 2]           # fewer chunks than R: all of them
    assert list(orc.l3_select(codes[5], codes, 1)) == [5]              # exact match, tie with 17 -> lower index


def test_retrieve_finds_the_planted_chunk(orc):
    rng = np.random.default_rng(3)
    B, H, H_kv, d, pr, bits, R = 2, 4, 2, 32, 4, 128, 2
    P = rng.normal(size=(bits, d)).astype(np.float32)
    pool = rng.normal(size=(12, H_kv, pr, d)).astype(np.float32)
    q = rng.normal(size=(B, H, d)).astype(np.float32)
    bank = np.array([[7, 2, 9, 4, 0], [1, 3, 5, 6, 8]])
    bank_len = np.array([5, 3])
    # plant: page 9's keys of KV head 0 all point along the summed query of sequence 0's first group
    pool[9, 0] = (q[0, 0] + q[0, 1])[None, :]
    table, n_sel = orc.l3_retrieve(q, P, orc.l3_index(pool, P), bank, bank_len, R, H_kv)
    assert list(n_sel) == [2, 2] and table.shape == (B, H_kv, R)
    assert 9 in table[0, 0]                                             # distance 0 to the query's code
    assert set(table[1].ravel()) <= {1, 3, 5}                           # only pages of the bank's used part
    for b in range(B):
        for h in range(H_kv):                                           # bank (time) order
            order = [list(bank[b]).index(pg) for pg in table[b, h, :n_sel[b]]]
            assert order == sorted(order)
