"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares,
validates arguments before touching CUDA, and its integer bookkeeping (decode split table, forward
tile ranges) matches a brute-force enumeration of the visibility predicate."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def mka():
    from paper_2603_20586_b200 import build
    build.build()
    import paper_2603_20586_b200 as m
    return m


def test_library_exports_every_declared_symbol(mka):
    hdr = open(os.path.join(ROOT, "include", "mka.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(mka_[a-z0-9_]+)\s*\(", hdr))
    assert {"mka_router", "mka_fwd", "mka_decode", "mka_bwd", "mka_workspace_bytes"} <= declared
    for name in declared:
        assert hasattr(mka.lib, name), name
    assert set(mka.binding.EXPORTS) <= declared | {"mka_status_str"}
    assert mka.status_str(0) == "ok" and "timed out" in mka.status_str(7)


def test_struct_sizes_match_header_layout(mka):
    b = mka.binding
    assert ctypes.sizeof(b.mka_level) == 48 and ctypes.sizeof(b.mka_level_grad) == 48
    assert ctypes.sizeof(b.mka_shape) == 48                       # twelve 4-byte fields, kv_heads last
    assert ctypes.sizeof(b.mka_paged_level) == 96                 # 4 pointers, 3 int64, int32 + padding, 4 int64
    assert ctypes.sizeof(b.mka_decode_plan_t) == 40 and ctypes.sizeof(b.mka_tile_range) == 32


def test_argument_validation_happens_before_any_launch(mka):
    b = mka.binding
    lv = (b.mka_level * 3)()
    bad_d = mka.make_shape(1, 1, 4, 48, window=4)
    assert mka.lib.mka_fwd(ctypes.byref(bad_d), None, lv, None, None, None, None, 0, None) == 2   # shape
    bad_w = mka.make_shape(1, 1, 4, 64, window=0)
    assert mka.lib.mka_fwd(ctypes.byref(bad_w), None, lv, None, None, None, None, 0, None) == 2
    ok = mka.make_shape(1, 1, 4, 64, window=4)
    assert mka.lib.mka_fwd(ctypes.byref(ok), None, lv, None, None, None, None, 0, None) == 1      # null Q
    lv[0] = b.mka_level(8, 16, -1, 0, 0, 64)
    assert mka.lib.mka_fwd(ctypes.byref(ok), None, lv, None, None, None, None, 0, None) == 2      # n < 0
    lv[0] = b.mka_level(8, 16, 4, 0, 0, 64)                                                     # misaligned k
    assert mka.lib.mka_fwd(ctypes.byref(ok), None, lv, None, None, None, None, 0, None) == 3
    dec = mka.make_shape(1, 1, 2, 64)
    assert mka.lib.mka_decode(ctypes.byref(dec), None, lv, None, None, None, None, 0, None) == 2  # T != 1
    assert mka.lib.mka_router(None, None, None, 4, 0, 0, 0, None, None, None, None) == 2
    assert mka.lib.mka_router(None, None, None, 4, 8, 0, 9, None, None, None, None) == 1
    assert mka.lib.mka_router(None, None, None, 0, 8, 0, 0, None, None, None, None) == 0          # empty is fine
    empty = mka.make_shape(0, 4, 16, 64, window=4)
    lv0 = (b.mka_level * 3)()
    assert mka.lib.mka_fwd(ctypes.byref(empty), None, lv0, None, None, None, None, 0, None) == 0
    full_bwd = mka.make_shape(1, 1, 4, 64, window=4, mode=b.MKA_MODE_FULL)
    gr = (b.mka_level_grad * 3)()
    assert mka.lib.mka_bwd(ctypes.byref(full_bwd), None, lv0, None, None, None, None, None, 0, None, gr, None, None,
                           None, None, 0, None) == 5


@pytest.mark.parametrize("n,B,H", [((4096, 32768, 8192), 32, 32), ((0, 100, 5), 1, 1), ((1, 1, 1), 2, 3),
                                   ((4096, 131072, 0), 1, 32), ((300, 300, 77), 1, 8), ((0, 0, 0), 1, 1)])
def test_decode_split_table_covers_each_row_exactly_once(mka, n, B, H):
    chunk, n_chunks, total = mka.mka_decode_plan(n, B, H, 128)
    assert chunk % 128 == 0 and 128 <= chunk <= 1024 and total == sum(n_chunks)
    for l in range(3):
        cover = np.zeros(n[l], int)
        for c in range(n_chunks[l]):
            lo, hi = c * chunk, min(n[l], (c + 1) * chunk)
            assert hi > lo                      # no empty chunk
            cover[lo:hi] += 1
        assert (cover == 1).all()
    ws = mka.mka_workspace_bytes(mka.make_shape(B, H, 1, 128), n, mka.binding.MKA_WS_DECODE)
    assert ws >= 256 + B * H * total * 130 * 4


def _vis(level, p, W, n):
    if level == 0:
        return [j for j in range(n) if p - W < j <= p]
    if level == 1:
        return [j for j in range(n) if j <= p]
    return list(range(n))


@pytest.mark.parametrize("T,W,q_off,N", [(300, 64, 0, (300, 300, 130)), (256, 512, 0, (256, 256, 0)),
                                         (130, 100, 700, (830, 830, 257)), (1, 1, 0, (1, 1, 1)),
                                         (640, 129, 3, (643, 500, 128))])
def test_forward_tile_ranges_match_mask_enumeration(mka, T, W, q_off, N):
    shape = mka.make_shape(1, 1, T, 128, window=W, q_offset=q_off)
    for q_tile in range((T + 127) // 128):
        rows = range(q_tile * 128, min(T, q_tile * 128 + 128))
        for level in range(3):
            first, end, ff, fe = mka.mka_fwd_tile_range(shape, N, level, q_tile)
            vis = [set(_vis(level, t + q_off, W, N[level])) for t in rows]
            union = set().union(*vis)
            n_tiles = (N[level] + 127) // 128
            touched = [kt for kt in range(n_tiles) if union & set(range(kt * 128, kt * 128 + 128))]
            if not touched:
                assert first == end
                continue
            assert (first, end) == (touched[0], touched[-1] + 1)
            assert touched == list(range(first, end))          # contiguous
            full = [kt for kt in range(first, end)
                    if all(set(range(kt * 128, kt * 128 + 128)) <= v for v in vis)]
            assert full == list(range(ff, fe)), (q_tile, level, full, ff, fe)


def test_widened_entry_points_validate_on_the_host(mka):
    """Paged, grouped-head, summary and recall entry points reject bad arguments before anything is launched."""
    b = mka.binding
    pl = (b.mka_paged_level * 3)()
    dec = mka.make_shape(1, 8, 1, 128)
    assert mka.lib.mka_decode_paged(ctypes.byref(dec), 3, None, pl, None, None, None, None, 0, None) == 2      # 8 heads on 3
    one = mka.make_shape(1, 32, 1, 128)
    assert mka.lib.mka_decode_paged(ctypes.byref(one), 1, None, pl, None, None, None, None, 0, None) == 2      # 32 heads per group
    pl[1] = b.mka_paged_level(16, 16, 16, None, 64, 4, 0, 12, 2048, 256, 128, 8)                                # 12 rows per page
    assert mka.lib.mka_decode_paged(ctypes.byref(dec), 2, None, pl, None, None, None, None, 0, None) == 2
    pl[1] = b.mka_paged_level(16, 16, 16, None, 6400, 4, 0, 16, 2048, 256, 128, 8)                              # table too narrow
    assert mka.lib.mka_decode_paged(ctypes.byref(dec), 2, None, pl, None, None, None, None, 0, None) == 2
    pl[1] = b.mka_paged_level(16, 16, 16, None, 64, 4, 0, 16, 2048, 256, 128, 8)
    assert mka.lib.mka_decode_paged(ctypes.byref(dec), 2, None, pl, None, None, None, None, 0, None) == 1      # null q
    fwd = mka.make_shape(1, 8, 64, 128, window=8)
    pl[1] = b.mka_paged_level(16, 16, 16, None, 64, 16, 0, 4, 2048, 256, 128, 8)                                # 4-row pages
    assert mka.lib.mka_fwd_paged(ctypes.byref(fwd), 2, None, pl, None, None, None, None, 0, None) == 2
    simt = mka.make_shape(1, 8, 64, 128, window=8, flags=1)
    assert mka.lib.mka_fwd_paged(ctypes.byref(simt), 2, None, pl, None, None, None, None, 0, None) == 5
    bad_group = mka.make_shape(1, 6, 4, 64, window=4, kv_heads=4)
    lv = (b.mka_level * 3)()
    assert mka.lib.mka_fwd(ctypes.byref(bad_group), None, lv, None, None, None, None, 0, None) == 2             # 6 heads on 4
    # summary
    assert mka.lib.mka_l2_summary(None, 1, 8, 20, 0, 0, 0.9, None, 0, None, None, 0, None) == 2                 # D % 8
    assert mka.lib.mka_l2_summary(None, 1, 8, 64, 0, 1, 1.5, None, 0, None, None, 0, None) == 1                 # beta
    assert mka.lib.mka_l2_summary(None, 0, 8, 64, 0, 0, 0.9, None, 0, None, None, 0, None) == 0                 # empty
    # recall
    assert mka.lib.mka_l3_index(None, 4, 2, 16, 96, 1, 1, 96, None, 64, None, None) == 2                        # d = 96
    assert mka.lib.mka_l3_index(None, 4, 2, 16, 128, 1, 1, 128, None, 48, None, None) == 2                      # 48 bits
    assert mka.lib.mka_l3_index(None, 0, 2, 16, 128, 1, 1, 128, None, 64, None, None) == 0                      # empty pool
    assert mka.lib.mka_l3_retrieve(None, 1, 8, 3, 128, None, 64, None, None, None, 8, 8, 4, 16, None, None, None, None) == 2
    assert mka.lib.mka_l3_retrieve(None, 1, 8, 2, 128, None, 64, None, None, None, 8, 8, 65, 16, None, None, None, None) == 2
    assert mka.lib.mka_l3_retrieve(None, 1, 8, 2, 128, None, 64, None, None, None, 8, 8, 4, 16, None, None, None, None) == 1


def test_summary_and_paged_workspace_queries(mka):
    b = mka.binding
    # 512 bytes + 8 bytes per (256-row segment, column)
    assert mka.lib.mka_l2_summary_workspace_bytes(1, 32768, 4096, 0) == 512 + 128 * 4096 * 8
    assert mka.lib.mka_l2_summary_workspace_bytes(2, 300, 64, 1) == 512 + 2 * 2 * 64 * 8
    full = mka.lib.mka_l2_summary_workspace_bytes(1, 32768, 4096, 0)
    assert mka.lib.mka_l2_summary_kernel_kind(1, 32768, 4096, 0, full) == 1
    assert mka.lib.mka_l2_summary_kernel_kind(1, 32768, 4096, 0, full - 1) == 0          # not enough scratch
    assert mka.lib.mka_l2_summary_kernel_kind(1, 400, 4096, 0, full) == 0                # short sequence
    assert mka.lib.mka_l2_summary_kernel_kind(1, 32768, 4096, 1, 1 << 30) == 0           # fp32 with 128 strips: strip form
    assert mka.lib.mka_l2_summary_kernel_kind(1, 32768, 1024, 1, 1 << 30) == 1           # fp32 with 32 strips
    # the paged decode's split: chunks of a multiple of 128 rows, every partial slot accounted for
    sh = mka.make_shape(4, 28, 1, 128)
    n = (4096, 131072, 8192)
    ws = mka.mka_decode_paged_workspace_bytes(sh, 4, n)
    slots = (ws - 256) // (4 * 28 * 130 * 4)
    assert (ws - 256) % (4 * 28 * 130 * 4) == 0 and 3 <= slots <= sum(-(-x // 128) for x in n)
    # grouped heads in the dense decode take the same split as the paged decode
    assert mka.mka_workspace_bytes(mka.make_shape(4, 28, 1, 128, kv_heads=4), n, b.MKA_WS_DECODE) == ws


def test_wait_limit_setter_clamps_and_returns_the_previous_value(mka):
    old = mka.mka_set_wait_limit_us(5)
    assert mka.mka_set_wait_limit_us(20_000_000) == 100          # 5 was raised to the floor
    assert mka.mka_set_wait_limit_us(0) == 10_000_000            # and 20 s lowered to the ceiling
    assert mka.mka_set_wait_limit_us(old) == 1_000_000           # 0 = the default
    assert old == 1_000_000
