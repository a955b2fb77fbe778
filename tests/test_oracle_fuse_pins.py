"""Pins of the oracle's route-fusion (Alg. 2 step 6) against what the paper and linear algebra fix."""
import numpy as np
import pytest


def _levels(rng, B, n, D):
    return [rng.standard_normal((B, n, D)) for _ in range(3)]


def _gate(rng, B, n):
    g = rng.random((B, n, 3)) + 0.05
    return g / g.sum(-1, keepdims=True)


def test_one_hot_gate_selects_that_level_exactly(orc):
    rng = np.random.default_rng(0)
    L = _levels(rng, 2, 7, 5)
    for l in range(3):
        g = np.zeros((2, 7, 3)); g[:, :, l] = 1.0
        assert np.array_equal(orc.route_fuse(L, g), L[l])


def test_uniform_gate_is_the_mean_and_identical_levels_are_a_fixed_point(orc):
    rng = np.random.default_rng(1)
    L = _levels(rng, 1, 9, 4)
    g = np.full((1, 9, 3), 1.0 / 3.0)
    assert np.allclose(orc.route_fuse(L, g), (L[0] + L[1] + L[2]) / 3.0, rtol=0, atol=1e-15)
    same = [L[0], L[0].copy(), L[0].copy()]
    assert np.allclose(orc.route_fuse(same, _gate(rng, 1, 9)), L[0], rtol=0, atol=1e-15)    # gates sum to one


def test_brute_force_loops(orc):
    rng = np.random.default_rng(2)
    B, n, D = 2, 5, 3
    L, g = _levels(rng, B, n, D), _gate(rng, B, n)
    ref = np.zeros((B, n, D))
    for b in range(B):
        for j in range(n):
            for c in range(D):
                ref[b, j, c] = sum(g[b, j, l] * L[l][b, j, c] for l in range(3))
    assert np.allclose(orc.route_fuse(L, g), ref, rtol=0, atol=1e-15)
    # the gate is indexed by the ROW's own token: permuting the tokens of inputs and gate together permutes the output
    perm = rng.permutation(n)
    assert np.allclose(orc.route_fuse([x[:, perm] for x in L], g[:, perm]), ref[:, perm], rtol=0, atol=1e-15)


def test_fusing_projected_levels_equals_projecting_the_fused_representation(orc):
    """Alg. 2 steps 6-7: K = (sum_l lambda_l L_l) W_k.  By linearity that is sum_l lambda_l (L_l W_k), per head."""
    rng = np.random.default_rng(3)
    B, n, D, H, d = 2, 6, 8, 2, 4
    L, g = _levels(rng, B, n, D), _gate(rng, B, n)
    Wk = rng.standard_normal((D, H * d))
    K_of_fused = (orc.route_fuse(L, g) @ Wk).reshape(B, n, H, d).transpose(0, 2, 1, 3)
    proj = [(x @ Wk).reshape(B, n, H, d).transpose(0, 2, 1, 3) for x in L]
    assert np.allclose(orc.route_fuse(proj, g), K_of_fused, rtol=0, atol=1e-12)


def test_absent_level_contributes_nothing(orc):
    rng = np.random.default_rng(4)
    L, g = _levels(rng, 1, 4, 3), _gate(rng, 1, 4)
    two = orc.route_fuse([L[0], L[1], None], g)
    assert np.allclose(two, g[:, :, 0:1] * L[0] + g[:, :, 1:2] * L[1], rtol=0, atol=1e-15)
    with pytest.raises(ValueError):
        orc.route_fuse([None, None, None], g)
