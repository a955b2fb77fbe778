"""GPU parity of the causal L2 session summary (prefix mean / EMA scan) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from gpu_helpers import BF16_MAX, BF16_MEAN, F32_MAX, np64
from mka_inputs import approx_normal

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mka():
    import paper_2603_20586_b200 as m
    assert torch.cuda.is_available()
    return m


def _x(seed, B, T, D, dtype):
    return approx_normal(seed, 0, 0, B * T * D, 1.0, "cpu", dtype).view(B, T, D).cuda()


def _check(got, ref, dtype):
    e = np.abs(np64(got) - ref)
    if dtype == torch.bfloat16:
        assert e.max() <= BF16_MAX and e.mean() <= BF16_MEAN, (e.max(), e.mean())
    else:
        assert e.max() <= F32_MAX, e.max()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("kind", [0, 1])
@pytest.mark.parametrize("B,T,D", [(2, 300, 256), (1, 1, 64), (3, 129, 96), (1, 1000, 72), (150, 40, 64), (1, 2500, 4096)])
def test_l2_summary_matches_oracle(mka, orc, dtype, kind, B, T, D):
    X = _x(21, B, T, D, dtype)
    state = torch.full((B, D), 123.0, device="cuda")              # ignored on entry for a fresh session, written on exit
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    M2 = mka.mka_l2_summary(X, kind, beta=0.9, state=state, n_prev=0, ws=ws)
    assert mka.mka_device_status(ws) == 0
    ref, sref = orc.l2_summary(np64(X), kind, beta=0.9)
    _check(M2, ref, dtype)
    assert np.abs(np64(state) - sref).max() <= 1e-4 * max(1.0, np.abs(sref).max())


@pytest.mark.parametrize("kind", [0, 1])
def test_session_in_chunks_equals_one_call(mka, orc, kind):
    B, T, D, cut = 2, 777, 128, 301
    X = _x(22, B, T, D, torch.bfloat16)
    state = torch.zeros(B, D, device="cuda")
    first = mka.mka_l2_summary(X[:, :cut].contiguous(), kind, beta=0.95, state=state, n_prev=0)
    second = mka.mka_l2_summary(X[:, cut:].contiguous(), kind, beta=0.95, state=state, n_prev=cut)
    ref, sref = orc.l2_summary(np64(X), kind, beta=0.95)
    _check(torch.cat([first, second], 1), ref, torch.bfloat16)
    assert np.abs(np64(state) - sref).max() <= 1e-4 * max(1.0, np.abs(sref).max())


def test_l2_summary_is_causal_and_deterministic(mka):
    B, T, D = 1, 400, 64
    X = _x(23, B, T, D, torch.bfloat16)
    Y = X.clone()
    Y[:, 250:] += 3.0
    for kind in (0, 1):
        a, b, a2 = mka.mka_l2_summary(X, kind), mka.mka_l2_summary(Y, kind), mka.mka_l2_summary(X, kind)
        assert torch.equal(a[:, :250], b[:, :250]) and not torch.equal(a[:, 250:], b[:, 250:])
        assert torch.equal(a, a2)


def test_l2_summary_rejects_bad_arguments(mka):
    X = torch.zeros(1, 8, 20, dtype=torch.bfloat16, device="cuda")       # D not a multiple of 8
    with pytest.raises(mka.MkaError) as e:
        mka.mka_l2_summary(X)
    assert e.value.code == 2
    X = torch.zeros(1, 8, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mka.MkaError) as e:
        mka.mka_l2_summary(X, 1, beta=1.5)
    assert e.value.code == 1
    with pytest.raises(mka.MkaError) as e:
        mka.mka_l2_summary(X, 0, n_prev=5)                                 # a continued session needs its state
    assert e.value.code == 1
