"""The give-up path of the kernels' bounded waits, exercised without a fault or a hang.

Every wait inside the tensor-core forward and backward and the segmented summary has a wall-clock limit.  Here the
limit is set to a few milliseconds and a test hook withholds something a wait needs (the forward's last key tile; the
last query tile of the backward's dK/dV kernel, whose issuing warp polls two barriers in a loop of its own; one
segment's carried state): the wait runs out, every role of the CTA drains, tensor memory is freed, the kernel RETURNS, and the
status word of the workspace reads MKA_ERR_TIMEOUT.  The next ordinary call on the same stream must then match the
oracle, which shows that the context and the library are still healthy.
"""
import numpy as np
import pytest
import torch

from gpu_helpers import check, np64, problem

pytestmark = pytest.mark.gpu
MKA_ERR_TIMEOUT = 7


@pytest.fixture(scope="module")
def mka():
    import paper_2603_20586_b200 as m
    assert torch.cuda.is_available()
    return m


@pytest.fixture()
def short_limit(mka):
    old = mka.mka_set_wait_limit_us(3000)
    yield 3000
    mka.mka_set_wait_limit_us(old)


@pytest.mark.parametrize("d", [128, 64])
def test_forward_wait_runs_out_and_the_next_call_is_correct(mka, orc, short_limit, d):
    B, H, T, W, N = 1, 2, 300, 96, (300, 300, 160)
    P = problem(91, B, H, T, d, N, 32, torch.bfloat16, router_std=0.3)
    gate = mka.mka_router(P["X"], P["W_r"], None)
    ws = mka.alloc_workspace(mka.make_shape(B, H, T, d, 32, W), N, mka.MKA_WS_FWD, "cuda")
    stalled = mka.make_shape(B, H, T, d, 32, W, flags=mka.MKA_FLAG_TEST_STALL)
    assert mka.mka_fwd_kernel_kind(stalled, P["K"], P["V"]) == 1
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    mka.mka_fwd(stalled, P["Q"], P["K"], P["V"], gate, ws=ws)
    t1.record()
    assert mka.mka_device_status(ws) == MKA_ERR_TIMEOUT           # synchronises the stream: the kernel came back
    assert t0.elapsed_time(t1) < 1000.0                           # after about one limit, not after the one-second default
    # the same problem without the hook, same workspace, same stream
    shape = mka.make_shape(B, H, T, d, 32, W)
    O, LSE = mka.mka_fwd(shape, P["Q"], P["K"], P["V"], gate, ws=ws)
    assert mka.mka_device_status(ws) == 0
    rg, _ = orc.router(np64(P["X"]), np64(P["W_r"]))
    Or, Lr = orc.fwd(P["Q"], P["K"], P["V"], rg, W)
    check(O, Or, torch.bfloat16, "forward after a timed-out call")
    assert np.abs(np64(LSE) - Lr).max() <= 2e-3


@pytest.mark.parametrize("d", [128, 64])
def test_backward_wait_runs_out_and_the_next_call_is_correct(mka, orc, short_limit, d):
    B, H, T, W, N = 1, 2, 300, 96, (300, 300, 160)
    P = problem(93, B, H, T, d, N, 32, torch.bfloat16, router_std=0.3, with_dO=True)
    gate = mka.mka_router(P["X"], P["W_r"], None)
    shape = mka.make_shape(B, H, T, d, 32, W)
    O, LSE = mka.mka_fwd(shape, P["Q"], P["K"], P["V"], gate)
    assert mka.mka_bwd_kernel_kind(shape, P["K"], P["V"]) == 1
    ws = mka.alloc_workspace(shape, N, mka.MKA_WS_BWD, "cuda")
    stalled = mka.make_shape(B, H, T, d, 32, W, flags=mka.MKA_FLAG_TEST_STALL)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    mka.mka_bwd(stalled, P["Q"], P["K"], P["V"], gate, O, LSE, P["dO"], R=P["X"], ws=ws)
    t1.record()
    assert mka.mka_device_status(ws) == MKA_ERR_TIMEOUT
    assert t0.elapsed_time(t1) < 1000.0
    g = mka.mka_bwd(shape, P["Q"], P["K"], P["V"], gate, O, LSE, P["dO"], R=P["X"], ws=ws)
    assert mka.mka_device_status(ws) == 0
    rg, _ = orc.router(np64(P["X"]), np64(P["W_r"]))
    ref = orc.bwd(P["Q"], P["K"], P["V"], rg, P["dO"], W)
    check(g["dQ"], ref["dQ"], torch.bfloat16, "dQ after a timed-out call")
    for l in range(3):
        check(g["dK"][l], ref["dK"][l], torch.bfloat16, f"dK{l} after a timed-out call")
        check(g["dV"][l], ref["dV"][l], torch.bfloat16, f"dV{l} after a timed-out call")


def test_summary_look_back_runs_out_and_the_next_call_is_correct(mka, orc, short_limit):
    B, T, D = 1, 2048, 256                                        # eight 256-row segments (or four of 512) per strip
    from mka_inputs import approx_normal
    X = approx_normal(92, 0, 0, B * T * D, 1.0, "cpu", torch.bfloat16).view(B, T, D).cuda()
    ws = mka.mka_l2_summary_workspace(X).zero_()
    assert mka.mka_l2_summary_kernel_kind(X, ws) == 1
    mka.mka_l2_summary(X, mka.MKA_SUMMARY_MEAN | mka.MKA_SUMMARY_TEST_STALL, ws=ws)
    assert mka.mka_device_status(ws) == MKA_ERR_TIMEOUT
    M2 = mka.mka_l2_summary(X, mka.MKA_SUMMARY_MEAN, ws=ws)
    assert mka.mka_device_status(ws) == 0
    ref = orc.l2_summary(np64(X))[0]
    check(M2, ref, torch.bfloat16, "summary after a timed-out call")
