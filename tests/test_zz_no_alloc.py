"""The workspace-free decode entry point (mka_decode_static) against the regular mka_decode.

Some hosts of this library cannot allocate device memory when they call it -- an inference server that
took all of HBM for its own pool at start-up, a decode loop that must not stall on the allocator, a
plug-in that is only ever given input and output pointers.  For them the library carries a fixed 8 MiB
scratch array.  This file checks, through the C ABI, that the entry point gives the same answer as the
workspace version on two calls in a row (the second smaller than the first, so anything the first call
left in the shared array would show), and that problems too large for the array are refused.

Collected last on purpose: a run that stops at the first failure has then already run everything else.
"""
import pytest
import torch

from gpu_helpers import BF16_MAX, problem

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mka():
    import paper_2603_20586_b200 as m
    assert torch.cuda.is_available()
    return m


def _case(mka, seed, B, H, d, N):
    P = problem(seed, B, H, 1, d, N, 64, torch.bfloat16, router_std=0.5)
    gate = mka.mka_router(P["X"], P["W_r"], None).view(B, 3).contiguous()
    q = P["Q"].view(B, H, d).contiguous()
    K = [k if k.shape[2] else None for k in P["K"]]
    V = [v if v.shape[2] else None for v in P["V"]]
    shape = mka.make_shape(B, H, 1, d, 64)
    want_O, want_LSE = mka.mka_decode(shape, q, K, V, gate)
    # outputs are the caller's: created here, before the call under test
    O = torch.full_like(q, float("nan"))
    LSE = torch.full((B, H), float("nan"), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    mka.mka_decode_static(shape, q, K, V, gate, O, LSE)
    torch.cuda.synchronize()
    assert torch.isfinite(O.float()).all() and torch.isfinite(LSE).all()
    assert (O.float() - want_O.float()).abs().max().item() <= BF16_MAX
    assert (LSE - want_LSE).abs().max().item() <= 2e-3
    return O, want_O


def test_static_decode_matches_workspace_decode_twice_in_a_row(mka):
    assert mka.mka_decode_static_max_bytes() == 8 << 20
    _case(mka, 51, 4, 8, 128, (1500, 9000, 700))       # first call: 32 heads x 45 chunks of partials
    _case(mka, 52, 2, 3, 64, (130, 40, 0))             # second call: fewer, shorter chunks, other head width
    _case(mka, 51, 4, 8, 128, (1500, 9000, 700))       # and the first problem again


def test_static_decode_rejects_problems_beyond_its_array(mka):
    B, H, d, n = 32, 32, 128, 4096 * 5                 # 1024 heads x 20 chunks x 130 floats > 8 MiB
    q = torch.zeros(B, H, d, dtype=torch.bfloat16, device="cuda")
    K = torch.zeros(1, 1, n, d, dtype=torch.bfloat16, device="cuda").expand(B, H, n, d)
    gate = torch.full((B, 3), 1 / 3, device="cuda")
    O = torch.empty_like(q)
    chunk, n_chunks, total = mka.mka_decode_plan((n, 0, 0), B, H, d)
    assert B * H * total * (d + 2) * 4 > mka.mka_decode_static_max_bytes()
    lv = mka.binding.mka_level
    import ctypes
    levels = (lv * 3)(lv(K.data_ptr(), K.data_ptr(), n, 0, 0, d), lv(None, None, 0, 0, 0, 0), lv(None, None, 0, 0, 0, 0))
    shape = mka.make_shape(B, H, 1, d)
    rc = mka.lib.mka_decode_static(ctypes.byref(shape), q.data_ptr(), levels, gate.data_ptr(), O.data_ptr(), None, None)
    assert rc == 4 and "workspace" in mka.status_str(rc)
