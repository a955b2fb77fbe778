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


def _ws(mka, X, scratch):
    """256 bytes hold the status word only; the full scratch lets long, narrow inputs take the segmented form."""
    if scratch == "status":
        return torch.zeros(256, dtype=torch.uint8, device="cuda")
    return mka.mka_l2_summary_workspace(X)


SHAPES = [(2, 300, 256), (1, 1, 64), (3, 129, 96), (1, 1000, 72), (150, 40, 64), (1, 2500, 4096),
          (1, 512, 64), (1, 513, 64), (2, 1537, 192), (1, 8192, 128), (700, 520, 64)]


@pytest.mark.parametrize("scratch", ["status", "full"])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("kind", [0, 1])
@pytest.mark.parametrize("B,T,D", SHAPES)
def test_l2_summary_matches_oracle(mka, orc, dtype, kind, B, T, D, scratch):
    X = _x(21, B, T, D, dtype)
    state = torch.full((B, D), 123.0, device="cuda")              # ignored on entry for a fresh session, written on exit
    ws = _ws(mka, X, scratch)
    strips = B * -(-D * X.element_size() // 128)
    narrow = dtype == torch.bfloat16 or strips < 96
    assert mka.mka_l2_summary_kernel_kind(X, ws) == (1 if scratch == "full" and T >= 512 and narrow else 0)
    M2 = mka.mka_l2_summary(X, kind, beta=0.9, state=state, n_prev=0, ws=ws)
    assert mka.mka_device_status(ws) == 0
    ref, sref = orc.l2_summary(np64(X), kind, beta=0.9)
    _check(M2, ref, dtype)
    assert np.abs(np64(state) - sref).max() <= 1e-4 * max(1.0, np.abs(sref).max())


@pytest.mark.parametrize("scratch", ["status", "full"])
@pytest.mark.parametrize("kind", [0, 1])
@pytest.mark.parametrize("T,cut", [(777, 301), (3000, 1300)])
def test_session_in_chunks_equals_one_call(mka, orc, kind, scratch, T, cut):
    B, D = 2, 128
    X = _x(22, B, T, D, torch.bfloat16)
    state = torch.zeros(B, D, device="cuda")
    a, b = X[:, :cut].contiguous(), X[:, cut:].contiguous()
    wa, wb = _ws(mka, a, scratch), _ws(mka, b, scratch)
    first = mka.mka_l2_summary(a, kind, beta=0.95, state=state, n_prev=0, ws=wa)
    second = mka.mka_l2_summary(b, kind, beta=0.95, state=state, n_prev=cut, ws=wb)
    assert mka.mka_device_status(wa) == 0 and mka.mka_device_status(wb) == 0
    ref, sref = orc.l2_summary(np64(X), kind, beta=0.95)
    _check(torch.cat([first, second], 1), ref, torch.bfloat16)
    assert np.abs(np64(state) - sref).max() <= 1e-4 * max(1.0, np.abs(sref).max())


def test_segmented_form_is_causal_and_deterministic(mka):
    B, T, D = 1, 4000, 64
    X = _x(24, B, T, D, torch.bfloat16)
    Y = X.clone()
    Y[:, 2500:] += 3.0
    ws = mka.mka_l2_summary_workspace(X)
    assert mka.mka_l2_summary_kernel_kind(X, ws) == 1
    for kind in (0, 1):
        a, b, a2 = (mka.mka_l2_summary(Z, kind, ws=ws) for Z in (X, Y, X))
        assert torch.equal(a[:, :2500], b[:, :2500]) and not torch.equal(a[:, 2500:], b[:, 2500:])
        assert torch.equal(a, a2)


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
