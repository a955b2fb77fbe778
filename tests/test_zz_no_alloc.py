"""The workspace-free decode entry point (mka_decode_static) against the CPU oracle and the regular mka_decode.

Some hosts of this library cannot allocate device memory when they call it -- an inference server that
took all of HBM for its own pool at start-up, a decode loop that must not stall on the allocator, a
plug-in that is only ever given input and output pointers.  For them the library carries a fixed 8 MiB
scratch array.  This file checks, through the C ABI, that the entry point gives the oracle's answer (and the
workspace version's) on calls in a row (the second smaller than the first, so anything the first call
left in the shared array would show), with and without grouped heads, that a warm call leaves the device's free
memory where it was, and that problems too large for the array are refused.

Collected last on purpose: a run that stops at the first failure has then already run everything else.
"""
import numpy as np
import pytest
import torch

from gpu_helpers import BF16_MAX, BF16_MEAN, np64, problem
from mka_inputs import approx_normal

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mka():
    import paper_2603_20586_b200 as m
    assert torch.cuda.is_available()
    return m


def _case(mka, orc, seed, B, H, d, N, kv_heads=0):
    Hk = kv_heads or H
    P = problem(seed, B, Hk, 1, d, N, 64, torch.bfloat16, router_std=0.5)
    gate = mka.mka_router(P["X"], P["W_r"], None).view(B, 3).contiguous()
    q = approx_normal(seed, 70, 0, B * H * d, 1.0, "cpu", torch.bfloat16).view(B, H, d).cuda()
    K = [k if k.shape[2] else None for k in P["K"]]
    V = [v if v.shape[2] else None for v in P["V"]]
    shape = mka.make_shape(B, H, 1, d, 64, kv_heads=kv_heads)
    want_O, want_LSE = mka.mka_decode(shape, q, K, V, gate)
    # the oracle works on one KV head per query head: repeat every KV head over its group
    rep = lambda t: np64(t).repeat(H // Hk, axis=1)
    ref_O, ref_LSE = orc.fwd(np64(q)[:, :, None, :], [rep(k) for k in P["K"]], [rep(v) for v in P["V"]],
                             np64(gate)[:, None, :], 1, decode=True)
    ref_O, ref_LSE = ref_O[:, :, 0], ref_LSE[:, :, 0]
    # outputs are the caller's: created here, before the call under test
    O = torch.full_like(q, float("nan"))
    LSE = torch.full((B, H), float("nan"), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    mka.mka_decode_static(shape, q, K, V, gate, O, LSE)
    torch.cuda.synchronize()
    assert torch.isfinite(O.float()).all() and torch.isfinite(LSE).all()
    e = np.abs(np64(O) - ref_O)
    assert e.max() <= BF16_MAX and e.mean() <= BF16_MEAN
    assert np.abs(np64(LSE) - ref_LSE).max() <= 2e-3
    assert (O.float() - want_O.float()).abs().max().item() <= BF16_MAX
    assert (LSE - want_LSE).abs().max().item() <= 2e-3
    return shape, q, K, V, gate, O, LSE


def test_static_decode_matches_oracle_and_workspace_decode_on_calls_in_a_row(mka, orc):
    assert mka.mka_decode_static_max_bytes() == 8 << 20
    _case(mka, orc, 51, 4, 8, 128, (1500, 9000, 700))       # first call: 32 heads x 45 chunks of partials
    _case(mka, orc, 52, 2, 3, 64, (130, 40, 0))             # second call: fewer, shorter chunks, other head width
    _case(mka, orc, 51, 4, 8, 128, (1500, 9000, 700))       # and the first problem again


def test_static_decode_with_grouped_heads(mka, orc):
    """mka_decode hands grouped heads to the grouped-query kernel, the static entry keeps the plain kernel with a head
    map: two different kernels that must both give the oracle's answer."""
    _case(mka, orc, 53, 2, 8, 128, (700, 2600, 300), kv_heads=2)
    _case(mka, orc, 54, 3, 6, 64, (90, 1100, 0), kv_heads=3)


def test_static_decode_leaves_free_memory_unchanged(mka, orc):
    args = _case(mka, orc, 55, 2, 4, 128, (400, 3000, 200))    # warm: the array's address is known after this call
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        mka.mka_decode_static(*args)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0


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
