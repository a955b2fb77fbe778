"""Pins of the oracle's causal L2 session summary (Alg. 1 loop over M_2 / Alg. 2 step 3)."""
import numpy as np


def test_prefix_mean_is_the_mean_of_each_prefix(orc):
    rng = np.random.default_rng(0)
    X = rng.standard_normal((2, 9, 4))
    M, S = orc.l2_summary(X, orc.SUMMARY_MEAN)
    for t in range(9):
        assert np.allclose(M[:, t], X[:, :t + 1].mean(axis=1), rtol=0, atol=1e-15)
    assert np.allclose(S, X.sum(axis=1), rtol=0, atol=1e-14)
    assert np.allclose(M, np.cumsum(X, axis=1) / np.arange(1, 10)[None, :, None], rtol=0, atol=1e-14)   # library scan


def test_constant_input_is_a_fixed_point_of_both_summaries(orc):
    X = np.broadcast_to(np.array([1.5, -2.0, 0.25]), (1, 12, 3)).copy()
    for kind in (orc.SUMMARY_MEAN, orc.SUMMARY_EMA):
        M, _ = orc.l2_summary(X, kind, beta=0.8)
        assert np.allclose(M, X, rtol=0, atol=1e-15)


def test_ema_closed_form_and_limits(orc):
    rng = np.random.default_rng(1)
    X = rng.standard_normal((1, 8, 2))
    beta = 0.7
    M, _ = orc.l2_summary(X, orc.SUMMARY_EMA, beta=beta)
    for t in range(8):      # m_t = beta^t x_0 + (1 - beta) sum_{i=1..t} beta^(t-i) x_i
        ref = beta ** t * X[:, 0] + (1 - beta) * sum(beta ** (t - i) * X[:, i] for i in range(1, t + 1))
        assert np.allclose(M[:, t], ref, rtol=0, atol=1e-14)
    assert np.array_equal(orc.l2_summary(X, orc.SUMMARY_EMA, beta=0.0)[0], X)                  # no memory
    assert np.allclose(orc.l2_summary(X, orc.SUMMARY_EMA, beta=1.0)[0], X[:, :1], atol=0)       # never updates


def test_summaries_are_causal(orc):
    rng = np.random.default_rng(2)
    X = rng.standard_normal((1, 10, 3))
    Y = X.copy()
    Y[:, 6:] += 5.0
    for kind in (orc.SUMMARY_MEAN, orc.SUMMARY_EMA):
        a, b = orc.l2_summary(X, kind)[0], orc.l2_summary(Y, kind)[0]
        assert np.array_equal(a[:, :6], b[:, :6]) and not np.allclose(a[:, 6:], b[:, 6:])


def test_a_session_can_be_summarised_in_chunks_with_the_carried_state(orc):
    rng = np.random.default_rng(3)
    X = rng.standard_normal((2, 11, 3))
    for kind in (orc.SUMMARY_MEAN, orc.SUMMARY_EMA):
        whole, s_whole = orc.l2_summary(X, kind, beta=0.85)
        first, s1 = orc.l2_summary(X[:, :4], kind, beta=0.85)
        second, s2 = orc.l2_summary(X[:, 4:], kind, beta=0.85, state=s1, n_prev=4)
        assert np.allclose(np.concatenate([first, second], axis=1), whole, rtol=0, atol=1e-14)
        assert np.allclose(s2, s_whole, rtol=0, atol=1e-14)
