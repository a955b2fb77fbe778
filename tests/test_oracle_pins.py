"""Pins for the CPU oracle: each test checks it against something other than itself --
a brute-force dense softmax, a library softmax-attention / autograd, closed forms,
finite differences, or an invariant the paper states (Theorem 1, Eq. 11-14, one-hot gate).
CPU only."""
import itertools
import math

import numpy as np
import pytest
import torch

W_SMALL = 3


def _problem(seed, B=2, H=2, T=9, d=5, N=(9, 9, 6), D=7, peaky=False):
    rng = np.random.default_rng(seed)
    Q = rng.standard_normal((B, H, T, d))
    K = [rng.standard_normal((B, H, n, d)) for n in N]
    V = [rng.standard_normal((B, H, n, d)) for n in N]
    X = rng.standard_normal((B, T, D))
    Wr = rng.standard_normal((D, 3)) * (1.0 if peaky else 0.1)
    br = rng.standard_normal(3) * 0.1
    return Q, K, V, X, Wr, br


def _mask(level, T, n, W, q_off, decode=False):
    """Visibility predicate written out independently of the oracle: L1 = last W keys ending at
    the query's own position, L2 = causal prefix, L3 = everything."""
    m = np.zeros((T, n), bool)
    for t in range(T):
        p = t + q_off
        for j in range(n):
            if decode or level == 2:
                m[t, j] = True
            elif level == 0:
                m[t, j] = (p - W < j <= p)
            else:
                m[t, j] = (j <= p)
    return m


def _dense_fast(Q, K, V, gate, W, q_off=0, tau=None, decode=False):
    """Brute force for Eq. 5: materialise every score, weight exp(score) by the gate of its
    level, normalise once."""
    B, H, T, d = Q.shape
    tau = 1 / math.sqrt(d) if tau is None else tau
    O = np.zeros((B, H, T, d))
    LSE = np.zeros((B, H, T))
    for b in range(B):
        for h in range(H):
            num = np.zeros((T, d))
            den = np.zeros(T)
            for l in range(3):
                n = K[l].shape[2]
                S = tau * Q[b, h] @ K[l][b, h].T
                E = np.exp(S) * _mask(l, T, n, W, q_off, decode) * gate[b][:, l:l + 1]
                num += E @ V[l][b, h]
                den += E.sum(1)
            with np.errstate(invalid="ignore", divide="ignore"):
                O[b, h] = np.where(den[:, None] > 0, num / den[:, None], 0.0)
                LSE[b, h] = np.log(den)
    return O, LSE


def _torch_bias_form(Q, K, V, gate, W, q_off=0, tau=None, decode=False):
    """Library pin: Eq. 5 equals ordinary softmax attention over the concatenated levels with
    the additive score bias ln(lambda) and -inf on masked pairs."""
    B, H, T, d = Q.shape[0], Q.shape[1], Q.shape[2], Q.shape[3]
    tau = 1 / math.sqrt(d) if tau is None else tau
    Kc = torch.cat(list(K), dim=2)
    Vc = torch.cat(list(V), dim=2)
    bias = []
    for l in range(3):
        n = K[l].shape[2]
        m = torch.from_numpy(_mask(l, T, n, W, q_off, decode))
        bl = torch.log(gate[:, :, l])[:, None, :, None].expand(B, 1, T, n)
        bias.append(torch.where(m[None, None], bl, torch.tensor(-math.inf, dtype=torch.float64)))
    bias = torch.cat(bias, dim=3)
    return torch.nn.functional.scaled_dot_product_attention(Q, Kc, Vc, attn_mask=bias, scale=tau)


@pytest.mark.parametrize("seed,W,q_off,N", [(0, 3, 0, (9, 9, 6)), (1, 20, 0, (9, 9, 0)), (2, 4, 5, (14, 14, 3)),
                                            (3, 1, 0, (9, 9, 1))])
def test_fast_equals_bruteforce_dense_softmax(orc, seed, W, q_off, N):
    Q, K, V, X, Wr, br = _problem(seed, N=N)
    gate, _ = orc.router(X, Wr, br)
    O, LSE = orc.fwd(Q, K, V, gate, W, q_off)
    Od, Ld = _dense_fast(Q, K, V, gate, W, q_off)
    np.testing.assert_allclose(O, Od, rtol=0, atol=1e-12)
    np.testing.assert_allclose(LSE, Ld, rtol=0, atol=1e-12)


@pytest.mark.parametrize("seed,W,peaky", [(0, 3, False), (5, 6, True)])
def test_fast_equals_library_attention_with_log_gate_bias(orc, seed, W, peaky):
    Q, K, V, X, Wr, br = _problem(seed, peaky=peaky)
    gate, _ = orc.router(X, Wr, br)
    O, _ = orc.fwd(Q, K, V, gate, W)
    tq = torch.from_numpy(Q)
    Ot = _torch_bias_form(tq, [torch.from_numpy(k) for k in K], [torch.from_numpy(v) for v in V],
                          torch.from_numpy(gate), W)
    np.testing.assert_allclose(O, Ot.numpy(), rtol=0, atol=1e-12)


def test_one_hot_gate_is_standard_attention_on_that_level(orc):
    Q, K, V, *_ = _problem(7)
    B, H, T, d = Q.shape
    for l in range(3):
        gate = np.zeros((B, T, 3))
        gate[..., l] = 1.0
        O, _ = orc.fwd(Q, K, V, gate, W_SMALL)
        m = torch.from_numpy(_mask(l, T, K[l].shape[2], W_SMALL, 0))
        Ot = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(Q), torch.from_numpy(K[l]), torch.from_numpy(V[l]), attn_mask=m[None, None])
        np.testing.assert_allclose(O, Ot.numpy(), atol=1e-12)
        Of, _ = orc.fwd(Q, K, V, gate, W_SMALL, mode="full")     # Alg. 1 agrees when the gate is one-hot
        np.testing.assert_allclose(Of, O, atol=1e-12)


def test_identical_levels_reduce_to_standard_attention(orc):
    # same K, V and same mask on every level (window >= T makes L1 causal like L2; decode makes all equal)
    rng = np.random.default_rng(11)
    B, H, T, d = 1, 2, 7, 4
    Q = rng.standard_normal((B, H, T, d))
    K1 = rng.standard_normal((B, H, T, d))
    V1 = rng.standard_normal((B, H, T, d))
    gate, _ = orc.router(rng.standard_normal((B, T, 5)), rng.standard_normal((5, 3)))
    O, _ = orc.fwd(Q, [K1, K1, K1], [V1, V1, V1], gate, 100, decode=True)
    Ot = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(Q), torch.from_numpy(K1), torch.from_numpy(V1))
    np.testing.assert_allclose(O, Ot.numpy(), atol=1e-12)
    # two causal levels only (Local-MKA): identical L1 (window >= T) and L2, L3 empty
    E = np.zeros((B, H, 0, d))
    O2, _ = orc.fwd(Q, [K1, K1, E], [V1, V1, E], gate, 100)
    Oc = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(Q), torch.from_numpy(K1), torch.from_numpy(V1), is_causal=True)
    np.testing.assert_allclose(O2, Oc.numpy(), atol=1e-12)


def test_uniform_gate_is_attention_over_concatenation(orc):
    Q, K, V, *_ = _problem(13)
    B, H, T, d = Q.shape
    gate = np.full((B, T, 3), 1 / 3)
    O, _ = orc.fwd(Q, K, V, gate, 100, decode=True)
    Kc, Vc = np.concatenate(K, 2), np.concatenate(V, 2)
    Ot = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(Q), torch.from_numpy(Kc), torch.from_numpy(Vc))
    np.testing.assert_allclose(O, Ot.numpy(), atol=1e-12)


@pytest.mark.parametrize("block", [1, 2, 3, 4, 7, 9, 64])
def test_theorem1_recursion_and_blockwise_equal_direct(orc, block):
    Q, K, V, X, Wr, br = _problem(17, N=(9, 9, 7))
    gate, _ = orc.router(X, Wr, br)
    O, LSE = orc.fwd(Q, K, V, gate, 4)
    Or, Lr = orc.fwd_recursive(Q, K, V, gate, 4, block=block)
    np.testing.assert_allclose(Or, O, atol=1e-12)
    np.testing.assert_allclose(Lr, LSE, atol=1e-12)


def test_max_shift_survives_huge_scores(orc):
    Q, K, V, X, Wr, br = _problem(19)
    gate, _ = orc.router(X, Wr, br)
    O, LSE = orc.fwd(Q, K, V, gate, 4, scale=400.0)      # |s| ~ 1e3: exp overflows without the shift
    Or, Lr = orc.fwd_recursive(Q, K, V, gate, 4, scale=400.0, block=3)
    assert np.isfinite(O).all() and np.isfinite(LSE).all()
    np.testing.assert_allclose(Or, O, atol=1e-10)
    np.testing.assert_allclose(Lr, LSE, rtol=1e-13)


def test_zero_query_closed_form_pins_masks_and_counts(orc):
    # Q = 0 => every score is 0: O_t = sum_l lam_l sum_vis v / sum_l lam_l n_l(t), LSE = ln sum_l lam_l n_l(t)
    rng = np.random.default_rng(23)
    B, H, T, d, W, q_off = 1, 1, 12, 3, 4, 2
    N = (14, 14, 5)
    Q = np.zeros((B, H, T, d))
    K = [rng.standard_normal((B, H, n, d)) for n in N]
    V = [rng.standard_normal((B, H, n, d)) for n in N]
    gate, _ = orc.router(rng.standard_normal((B, T, 4)), rng.standard_normal((4, 3)))
    O, LSE = orc.fwd(Q, K, V, gate, W, q_off)
    for t in range(T):
        p = t + q_off
        n1, n2, n3 = min(p + 1, W), p + 1, N[2]
        lam = gate[0, t]
        den = lam[0] * n1 + lam[1] * n2 + lam[2] * n3
        num = (lam[0] * V[0][0, 0, p - n1 + 1:p + 1].sum(0) + lam[1] * V[1][0, 0, :p + 1].sum(0)
               + lam[2] * V[2][0, 0].sum(0))
        np.testing.assert_allclose(O[0, 0, t], num / den, atol=1e-13)
        assert abs(LSE[0, 0, t] - math.log(den)) < 1e-13


def test_visible_ranges_match_mask_predicate(orc):
    for W, q_off, n in itertools.product([1, 2, 5, 40], [0, 3], [0, 1, 6, 11]):
        for level in range(3):
            m = _mask(level, 8, n, W, q_off)
            for t in range(8):
                lo, hi = orc.visible(level, t + q_off, W, n)
                expect = np.nonzero(m[t])[0]
                assert hi - lo == len(expect)
                if len(expect):
                    assert lo == expect[0] and hi == expect[-1] + 1
    assert orc.visible(0, 0, 4, 9, decode=True) == (0, 9)


def test_shift_invariance(orc):
    Q, K, V, X, Wr, br = _problem(29)
    g1, _ = orc.router(X, Wr, br)
    g2, _ = orc.router(X, Wr, br + 3.7)          # same constant on all three logits
    np.testing.assert_allclose(g1, g2, atol=1e-14)


def test_score_shift_leaves_output_and_moves_lse(orc):
    """A constant c added to EVERY score of a query row leaves O unchanged and moves LSE by c.  With one query row,
    adding c q / (tau |q|^2) to every key of every level adds exactly c to each of its scores."""
    rng = np.random.default_rng(30)
    B, H, d, N, c = 1, 2, 6, (5, 7, 4), 2.75
    Q = rng.standard_normal((B, H, 1, d))
    K = [rng.standard_normal((B, H, n, d)) for n in N]
    V = [rng.standard_normal((B, H, n, d)) for n in N]
    gate = np.array([[[0.2, 0.5, 0.3]]])
    tau = 1 / math.sqrt(d)
    q = Q[:, :, 0]
    delta = c * q / (tau * (q * q).sum(-1, keepdims=True))          # [B, H, d]
    Ks = [k + delta[:, :, None, :] for k in K]
    O1, L1 = orc.fwd(Q, K, V, gate, 1, decode=True)
    O2, L2 = orc.fwd(Q, Ks, V, gate, 1, decode=True)
    np.testing.assert_allclose(O2, O1, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(L2, L1 + c, rtol=1e-12, atol=1e-12)


def test_nothing_visible_gives_zero_output(orc):
    rng = np.random.default_rng(31)
    B, H, T, d = 1, 1, 3, 4
    E = np.zeros((B, H, 0, d))
    K3 = rng.standard_normal((B, H, 4, d))
    gate = np.zeros((B, T, 3))
    gate[..., 0] = 1.0                           # all weight on an empty level
    O, LSE = orc.fwd(rng.standard_normal((B, H, T, d)), [E, E, K3], [E, E, K3], gate, 2)
    assert (O == 0).all() and np.isneginf(LSE).all()


def test_full_mode_is_mixture_of_three_library_attentions(orc):
    Q, K, V, X, Wr, br = _problem(37, peaky=True)
    B, H, T, d = Q.shape
    gate, _ = orc.router(X, Wr, br)
    O, _ = orc.fwd(Q, K, V, gate, W_SMALL, mode="full")
    ref = np.zeros_like(Q)
    for l in range(3):
        m = torch.from_numpy(_mask(l, T, K[l].shape[2], W_SMALL, 0))
        a = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(Q), torch.from_numpy(K[l]), torch.from_numpy(V[l]), attn_mask=m[None, None]).numpy()
        ref += gate[:, None, :, l:l + 1] * a
    np.testing.assert_allclose(O, ref, atol=1e-12)
    Of, _ = orc.fwd(Q, K, V, gate, W_SMALL, mode="fast")
    assert np.abs(Of - O).max() > 1e-3           # Eq. 5 is NOT the mixture of per-level softmax outputs


# ---------------------------------------------------------------- router
def test_router_gates(orc):
    rng = np.random.default_rng(41)
    X = rng.standard_normal((3, 5, 8))
    Wr = rng.standard_normal((8, 3))
    br = rng.standard_normal(3)
    gate, idx = orc.router(X, Wr, br)
    np.testing.assert_allclose(gate.sum(-1), 1.0, atol=1e-15)
    ref = torch.softmax(torch.from_numpy(X) @ torch.from_numpy(Wr) + torch.from_numpy(br), -1).numpy()
    np.testing.assert_allclose(gate, ref, atol=1e-14)
    assert (idx == -1).all()
    g0, _ = orc.router(X, np.zeros((8, 3)), None)                      # W_r = 0 -> 1/3 each
    np.testing.assert_allclose(g0, 1 / 3, atol=1e-16)
    gb, _ = orc.router(X, np.zeros((8, 3)), np.array([0.0, math.log(2), math.log(3)]))
    np.testing.assert_allclose(gb, np.broadcast_to([1 / 6, 2 / 6, 3 / 6], gb.shape), atol=1e-15)
    gu, _ = orc.router(X, Wr, br, route=orc.ROUTE_UNIFORM)
    np.testing.assert_allclose(gu, 1 / 3, atol=1e-16)


def test_router_topk_all_orderings_and_ties(orc):
    vals = [0.0, 1.0, 2.0]
    cases = [list(p) for p in itertools.permutations(vals)] + [[1, 1, 0], [0, 1, 1], [1, 0, 1], [2, 2, 2], [0, 0, 1]]
    X = np.ones((len(cases), 1))
    for k, route in ((1, orc.ROUTE_TOP1), (2, orc.ROUTE_TOP2)):
        for i, g in enumerate(cases):
            gate, idx = orc.router(X[i:i + 1], np.zeros((1, 3)), np.array(g, float), route=route)
            order = sorted(range(3), key=lambda l: (-g[l], l))[:k]      # brute-force sort, ties -> lower level
            kept = sorted(order)
            assert list(idx[0][:k]) == kept and (k == 2 or idx[0][1] == -1)
            e = np.exp(np.array(g, float))
            ref = np.zeros(3)
            ref[kept] = e[kept] / e[kept].sum()
            np.testing.assert_allclose(gate[0], ref, atol=1e-15)
            assert all(gate[0][l] == 0.0 for l in range(3) if l not in kept)


# ---------------------------------------------------------------- decode
def test_decode_equals_last_prefill_row(orc):
    Q, K, V, X, Wr, br = _problem(43, T=9, N=(9, 9, 6))
    W = 4
    gate, _ = orc.router(X, Wr, br)
    O, LSE = orc.fwd(Q, K, V, gate, W)
    t = 8
    Kd = [K[0][:, :, t - W + 1:t + 1], K[1][:, :, :t + 1], K[2]]
    Vd = [V[0][:, :, t - W + 1:t + 1], V[1][:, :, :t + 1], V[2]]
    Od, Ld = orc.fwd(Q[:, :, t:t + 1], Kd, Vd, gate[:, t:t + 1], W, decode=True)
    np.testing.assert_allclose(Od[:, :, 0], O[:, :, t], atol=1e-13)
    np.testing.assert_allclose(Ld[:, :, 0], LSE[:, :, t], atol=1e-13)


def test_row_list_matches_full(orc):
    Q, K, V, X, Wr, br = _problem(47)
    gate, _ = orc.router(X, Wr, br)
    O, LSE = orc.fwd(Q, K, V, gate, 3)
    rows = [0, 4, 8]
    Or, Lr = orc.fwd(Q, K, V, gate, 3, rows=rows)
    np.testing.assert_array_equal(Or, O[:, :, rows])
    np.testing.assert_array_equal(Lr, LSE[:, :, rows])


# ---------------------------------------------------------------- backward
def _loss(orc, Q, K, V, X, Wr, br, dO, W, q_off=0):
    gate, _ = orc.router(X, Wr, br)
    O, _ = orc.fwd(Q, K, V, gate, W, q_off)
    return float((O * dO).sum())


def test_backward_finite_differences(orc):
    Q, K, V, X, Wr, br = _problem(53, B=1, H=2, T=6, d=4, N=(6, 6, 4), D=5, peaky=True)
    W = 3
    rng = np.random.default_rng(54)
    dO = rng.standard_normal(Q.shape)
    gate, _ = orc.router(X, Wr, br)
    g = orc.bwd(Q, K, V, gate, dO, W)
    dW, db = orc.router_bwd(X, g["dG"])
    eps = 1e-5

    def fd(arr, grad, picks):
        for idx in picks:
            old = arr[idx]
            arr[idx] = old + eps
            lp = _loss(orc, Q, K, V, X, Wr, br, dO, W)
            arr[idx] = old - eps
            lm = _loss(orc, Q, K, V, X, Wr, br, dO, W)
            arr[idx] = old
            num = (lp - lm) / (2 * eps)
            assert abs(num - grad[idx]) <= 1e-6 * max(1.0, abs(num)), (idx, num, grad[idx])

    def picks(shape, k=12):
        r = np.random.default_rng(99)
        return [tuple(int(r.integers(0, s)) for s in shape) for _ in range(k)]

    fd(Q, g["dQ"], picks(Q.shape))
    for l in range(3):
        fd(K[l], g["dK"][l], picks(K[l].shape))
        fd(V[l], g["dV"][l], picks(V[l].shape))
    fd(Wr, dW, picks(Wr.shape, 15))
    fd(br, db, [(0,), (1,), (2,)])


def test_backward_matches_torch_autograd(orc):
    Q, K, V, X, Wr, br = _problem(59, peaky=True)
    W = 4
    rng = np.random.default_rng(60)
    dO = rng.standard_normal(Q.shape)
    t = lambda a: torch.from_numpy(a.copy()).requires_grad_(True)
    tQ, tK, tV, tX, tW, tb = t(Q), [t(k) for k in K], [t(v) for v in V], torch.from_numpy(X), t(Wr), t(br)
    gate_t = torch.softmax(tX @ tW + tb, -1)
    Ot = _torch_bias_form(tQ, tK, tV, gate_t, W)
    (Ot * torch.from_numpy(dO)).sum().backward()
    gate, _ = orc.router(X, Wr, br)
    g = orc.bwd(Q, K, V, gate, dO, W)
    dW, db = orc.router_bwd(X, g["dG"])
    np.testing.assert_allclose(g["dQ"], tQ.grad.numpy(), atol=1e-12)
    for l in range(3):
        np.testing.assert_allclose(g["dK"][l], tK[l].grad.numpy(), atol=1e-12)
        np.testing.assert_allclose(g["dV"][l], tV[l].grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(dW, tW.grad.numpy(), atol=1e-11)
    np.testing.assert_allclose(db, tb.grad.numpy(), atol=1e-11)


def test_backward_invariants(orc):
    Q, K, V, X, Wr, br = _problem(61)
    rng = np.random.default_rng(62)
    dO = rng.standard_normal(Q.shape)
    gate, _ = orc.router(X, Wr, br)
    g = orc.bwd(Q, K, V, gate, dO, 3)
    np.testing.assert_allclose(g["G"].sum(-1), 0.0, atol=1e-13)      # sum_l G_l = 0 (sum_j dS = 0 per row)
    # one-hot gate: zero gradient to the other levels, standard attention backward on the kept one
    B, H, T, d = Q.shape
    oh = np.zeros((B, T, 3))
    oh[..., 1] = 1.0
    g1 = orc.bwd(Q, K, V, oh, dO, 3)
    for l in (0, 2):
        assert (g1["dK"][l] == 0).all() and (g1["dV"][l] == 0).all()
    tQ = torch.from_numpy(Q.copy()).requires_grad_(True)
    tK = torch.from_numpy(K[1].copy()).requires_grad_(True)
    tV = torch.from_numpy(V[1].copy()).requires_grad_(True)
    Ot = torch.nn.functional.scaled_dot_product_attention(tQ, tK, tV, is_causal=True)
    (Ot * torch.from_numpy(dO)).sum().backward()
    np.testing.assert_allclose(g1["dQ"], tQ.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(g1["dK"][1], tK.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(g1["dV"][1], tV.grad.numpy(), atol=1e-12)


def test_backward_row_list(orc):
    Q, K, V, X, Wr, br = _problem(67)
    rng = np.random.default_rng(68)
    dO = rng.standard_normal(Q.shape)
    gate, _ = orc.router(X, Wr, br)
    g = orc.bwd(Q, K, V, gate, dO, 3)
    rows = [1, 5, 8]
    gr = orc.bwd(Q, K, V, gate, dO, 3, rows=rows, want_kv=False)
    np.testing.assert_allclose(gr["dQ"], g["dQ"][:, :, rows], atol=1e-15)
    np.testing.assert_allclose(gr["dG"], g["dG"][:, rows], atol=1e-15)
