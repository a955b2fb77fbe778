"""GPU parity of the route-fusion / cache-write kernel (Alg. 2 steps 6-8) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from gpu_helpers import BF16_MAX, BF16_MEAN, F32_MAX, np64, problem
from mka_inputs import approx_normal

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mka():
    import paper_2603_20586_b200 as m
    assert torch.cuda.is_available()
    return m


def _aligned_levels(seed, B, H, n, d, dtype):
    mk = lambda tid: approx_normal(seed, tid, 0, B * H * n * d, 1.0, "cpu", dtype).view(B, H, n, d).cuda()
    return [mk(3 + 2 * l) for l in range(3)], [mk(4 + 2 * l) for l in range(3)]


def _gate(seed, B, n):
    g = approx_normal(seed, 20, 0, B * n * 3, 1.0, "cpu", torch.float32).view(B, n, 3).cuda()
    return torch.softmax(g, -1).contiguous()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("B,H,n,d", [(2, 3, 300, 128), (1, 2, 1, 64), (3, 1, 1031, 8), (1, 1, 77, 1024)])
def test_fuse_kv_matches_oracle(mka, orc, dtype, B, H, n, d):
    K, V = _aligned_levels(5, B, H, n, d, dtype)
    gate = _gate(5, B, n)
    ok_, ov_ = mka.mka_fuse_kv(K, V, gate)
    rk, rv = orc.route_fuse(K, np64(gate)), orc.route_fuse(V, np64(gate))
    for got, ref in ((ok_, rk), (ov_, rv)):
        e = np.abs(np64(got) - ref)
        if dtype == torch.bfloat16:
            assert e.max() <= BF16_MAX and e.mean() <= BF16_MEAN
            # one rounding of an fp32 sum: within half a bf16 ulp (plus the fp32 accumulation error) of the fp64 value
            assert np.all(e <= np.abs(ref) * 2.0 ** -8 + 1e-6)
        else:
            assert e.max() <= F32_MAX


def test_fuse_kv_appends_into_a_strided_cache_and_touches_nothing_else(mka, orc):
    B, H, n, d, off, cap = 2, 2, 100, 64, 37, 200
    K, V = _aligned_levels(6, B, H, n, d, torch.bfloat16)
    gate = _gate(6, B, n)
    ck = torch.full((B, H, cap, d + 32), 7.0, dtype=torch.bfloat16, device="cuda")
    cv = torch.full_like(ck, 7.0)
    mka.mka_fuse_kv(K, V, gate, out_k=ck[..., 8:8 + d], out_v=cv[..., 8:8 + d], dst_offset=off)
    rk = orc.route_fuse(K, np64(gate))
    assert np.abs(np64(ck[:, :, off:off + n, 8:8 + d]) - rk).max() <= BF16_MAX
    keep = torch.ones_like(ck, dtype=torch.bool)
    keep[:, :, off:off + n, 8:8 + d] = False
    assert bool((ck[keep] == 7.0).all()) and bool((cv[keep] == 7.0).all())


def test_fuse_kv_one_hot_zero_gate_and_absent_level(mka, orc):
    B, H, n, d = 1, 2, 130, 128
    K, V = _aligned_levels(7, B, H, n, d, torch.bfloat16)
    gate = torch.zeros(B, n, 3, device="cuda")
    gate[:, :, 1] = 1.0
    K[2].fill_(float("nan"))                        # a level whose gate is exactly 0 must not leak into the result
    ok_, ov_ = mka.mka_fuse_kv(K, V, gate)
    assert torch.equal(ok_, K[1]) and torch.equal(ov_, V[1])
    g2 = _gate(7, B, n)
    K2, V2 = [K[0], K[1], None], [V[0], V[1], None]
    ok2, _ = mka.mka_fuse_kv(K2, V2, g2)
    assert np.abs(np64(ok2) - orc.route_fuse(K2, np64(g2))).max() <= BF16_MAX


def test_decode_over_the_fused_cache_is_attention_on_the_fused_rows(mka, orc):
    """Alg. 2 steps 8-9 for one new token: one cache, one level, gate (1, 0, 0)."""
    B, H, n, d = 2, 4, 700, 128
    K, V = _aligned_levels(8, B, H, n, d, torch.bfloat16)
    gate = _gate(8, B, n)
    ck, cv = mka.mka_fuse_kv(K, V, gate)
    q = approx_normal(8, 2, 0, B * H * d, 1.0, "cpu", torch.bfloat16).view(B, H, d).cuda()
    one = torch.tensor([[1.0, 0.0, 0.0]], device="cuda").repeat(B, 1).contiguous()
    O, _ = mka.mka_decode(mka.make_shape(B, H, 1, d), q, [ck, None, None], [cv, None, None], one)
    none = torch.zeros(B, H, 0, d, dtype=torch.bfloat16)
    Or, _ = orc.fwd(q.view(B, H, 1, d), [ck, none, none], [cv, none, none], np64(one).reshape(B, 1, 3), 1, decode=True)
    e = np.abs(np64(O) - Or[:, :, 0])
    assert e.max() <= BF16_MAX and e.mean() <= BF16_MEAN


def test_fuse_kv_rejects_bad_arguments(mka):
    B, H, n, d = 1, 1, 16, 64
    K, V = _aligned_levels(9, B, H, n, d, torch.bfloat16)
    gate = _gate(9, B, n)
    small = torch.empty(B, H, 8, d, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mka.MkaError) as e:
        mka.mka_fuse_kv(K, V, gate, out_k=small, out_v=torch.empty_like(small))        # destination too short
    assert e.value.code == 2
    with pytest.raises(mka.MkaError) as e:
        mka.mka_fuse_kv([K[0], K[1][:, :, :8], K[2]], [V[0], V[1][:, :, :8], V[2]], gate)   # levels not token-aligned
    assert e.value.code == 2


def test_fuse_kv_into_a_paged_cache(mka, orc):
    """The fused rows land where the page table says, at a different offset per sequence; nothing else is touched."""
    B, H, n, d, pr = 3, 4, 50, 64, 16
    Ks = [approx_normal(71, 10 + l, 0, B * H * n * d, 1.0, "cpu", torch.bfloat16).view(B, H, n, d).cuda() for l in range(3)]
    Vs = [approx_normal(71, 20 + l, 0, B * H * n * d, 1.0, "cpu", torch.bfloat16).view(B, H, n, d).cuda() for l in range(3)]
    gate = torch.softmax(approx_normal(71, 30, 0, B * n * 3, 1.0, "cpu", torch.float32).view(B, n, 3), -1).cuda().contiguous()
    pages_per_seq = 8                                             # room for 128 rows per sequence
    gen = torch.Generator().manual_seed(71)
    table = torch.randperm(B * pages_per_seq + 2, generator=gen)[:B * pages_per_seq].int().view(B, pages_per_seq).cuda()
    pool_k = torch.full((B * pages_per_seq + 2, H, pr, d), 7.0, dtype=torch.bfloat16, device="cuda")
    pool_v = torch.full_like(pool_k, -7.0)
    offs = torch.tensor([0, 13, 40], dtype=torch.int32, device="cuda")
    base = 5
    mka.mka_fuse_kv_paged(Ks, Vs, gate, pool_k, pool_v, table, dst_offset=base, dst_offsets=offs)
    rk = orc.route_fuse(Ks, np64(gate))                           # [B, H, n, d]
    rv = orc.route_fuse(Vs, np64(gate))
    dense_k = pool_k[table.long()].permute(0, 2, 1, 3, 4).reshape(B, H, pages_per_seq * pr, d)
    dense_v = pool_v[table.long()].permute(0, 2, 1, 3, 4).reshape(B, H, pages_per_seq * pr, d)
    for b in range(B):
        o = base + int(offs[b])
        ek = np.abs(np64(dense_k[b, :, o:o + n]) - rk[b])
        ev = np.abs(np64(dense_v[b, :, o:o + n]) - rv[b])
        assert ek.max() <= BF16_MAX and ev.max() <= BF16_MAX and ek.mean() <= BF16_MEAN and ev.mean() <= BF16_MEAN
        untouched = torch.ones(pages_per_seq * pr, dtype=torch.bool, device="cuda")
        untouched[o:o + n] = False
        assert (dense_k[b][:, untouched] == 7.0).all() and (dense_v[b][:, untouched] == -7.0).all()
    used = torch.zeros(pool_k.shape[0], dtype=torch.bool, device="cuda")
    used[table.flatten().long()] = True
    assert (pool_k[~used] == 7.0).all()                           # pages that belong to nobody
