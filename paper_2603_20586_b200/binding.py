"""Thin ctypes binding of the C-ABI library (``libmka_b200.so``): argument marshalling only.

Function names match ``include/mka.h``.  Tensors are ``torch`` CUDA tensors used purely as device
memory; every step of the path runs inside the library's kernels.  There is no fallback: if the
library has not been built the import fails, and every call raises ``MkaError`` on a non-zero status.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmka_b200.so")

MKA_BF16, MKA_F32 = 0, 1
MKA_MODE_FAST, MKA_MODE_FULL = 0, 1
MKA_ROUTE_SOFT, MKA_ROUTE_UNIFORM, MKA_ROUTE_TOP1, MKA_ROUTE_TOP2 = 0, 1, 2, 3
MKA_FLAG_FORCE_SIMT = 1
MKA_FLAG_TEST_STALL = 0x80000000
MKA_SUMMARY_MEAN, MKA_SUMMARY_EMA = 0, 1
MKA_SUMMARY_TEST_STALL = 0x40000000
MKA_WS_FWD, MKA_WS_DECODE, MKA_WS_BWD = 0, 1, 2
TILE = 128

EXPORTS = ["mka_status_str", "mka_router", "mka_workspace_bytes", "mka_fwd", "mka_decode", "mka_bwd",
           "mka_decode_plan", "mka_fwd_tile_range", "mka_device_status", "mka_fwd_kernel_kind",
           "mka_bwd_kernel_kind", "mka_fuse_kv", "mka_l2_summary", "mka_l2_summary_workspace_bytes", "mka_l2_summary_kernel_kind", "mka_decode_static", "mka_decode_static_max_bytes",
           "mka_decode_paged", "mka_decode_paged_workspace_bytes", "mka_l3_index", "mka_l3_retrieve", "mka_fwd_paged", "mka_fuse_kv_paged", "mka_set_wait_limit_us"]


class MkaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: status {code} ({status_str(code)})")


class mka_level(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("n", ctypes.c_int64),
                ("stride_b", ctypes.c_int64), ("stride_h", ctypes.c_int64), ("stride_n", ctypes.c_int64)]


class mka_level_grad(ctypes.Structure):
    _fields_ = [("dk", ctypes.c_void_p), ("dv", ctypes.c_void_p), ("n", ctypes.c_int64),
                ("stride_b", ctypes.c_int64), ("stride_h", ctypes.c_int64), ("stride_n", ctypes.c_int64)]


class mka_paged_level(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("page_table", ctypes.c_void_p),
                ("rows", ctypes.c_void_p), ("n", ctypes.c_int64), ("table_stride", ctypes.c_int64),
                ("table_head_stride", ctypes.c_int64), ("page_rows", ctypes.c_int32), ("stride_page", ctypes.c_int64), ("stride_h", ctypes.c_int64),
                ("stride_n", ctypes.c_int64), ("pool_pages", ctypes.c_int64)]


class mka_shape(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("T", ctypes.c_int32), ("d", ctypes.c_int32),
                ("D", ctypes.c_int32), ("window", ctypes.c_int32), ("q_offset", ctypes.c_int32),
                ("scale", ctypes.c_float), ("dtype", ctypes.c_int32), ("mode", ctypes.c_int32),
                ("flags", ctypes.c_uint32), ("kv_heads", ctypes.c_int32)]


class mka_decode_plan_t(ctypes.Structure):
    _fields_ = [("chunk_rows", ctypes.c_int64), ("n_chunks", ctypes.c_int64 * 3), ("total_chunks", ctypes.c_int64)]


class mka_tile_range(ctypes.Structure):
    _fields_ = [("first", ctypes.c_int64), ("end", ctypes.c_int64), ("full_first", ctypes.c_int64),
                ("full_end", ctypes.c_int64)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2603_20586_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    lib.mka_status_str.restype = ctypes.c_char_p
    lib.mka_status_str.argtypes = [ctypes.c_int]
    lib.mka_workspace_bytes.restype = ctypes.c_size_t
    lib.mka_workspace_bytes.argtypes = [ctypes.POINTER(mka_shape), ctypes.POINTER(ctypes.c_int64), ctypes.c_int32]
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    lib.mka_router.argtypes = [vp, vp, vp, i64, i32, i32, i32, vp, vp, vp, vp]
    lib.mka_fwd.argtypes = [ctypes.POINTER(mka_shape), vp, ctypes.POINTER(mka_level), vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.mka_decode.argtypes = lib.mka_fwd.argtypes
    lib.mka_bwd.argtypes = [ctypes.POINTER(mka_shape), vp, ctypes.POINTER(mka_level), vp, vp, vp, vp, vp, i32, vp,
                            ctypes.POINTER(mka_level_grad), vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.mka_decode_plan.argtypes = [ctypes.POINTER(ctypes.c_int64), i32, i32, i32, ctypes.POINTER(mka_decode_plan_t)]
    lib.mka_fwd_tile_range.argtypes = [ctypes.POINTER(mka_shape), ctypes.POINTER(ctypes.c_int64), i32, i64,
                                       ctypes.POINTER(mka_tile_range)]
    lib.mka_device_status.argtypes = [vp, vp]
    lib.mka_decode_static.argtypes = [ctypes.POINTER(mka_shape), vp, ctypes.POINTER(mka_level), vp, vp, vp, vp]
    lib.mka_decode_static_max_bytes.restype = ctypes.c_size_t
    lib.mka_decode_static_max_bytes.argtypes = []
    lib.mka_fwd_kernel_kind.argtypes = [ctypes.POINTER(mka_shape), ctypes.POINTER(mka_level)]
    lib.mka_fuse_kv.argtypes = [i32, i32, i64, i32, i32, ctypes.POINTER(mka_level), vp, ctypes.POINTER(mka_level_grad), i64, vp]
    lib.mka_l2_summary_workspace_bytes.restype = ctypes.c_size_t
    lib.mka_l2_summary_workspace_bytes.argtypes = [i32, i64, i32, i32]
    lib.mka_decode_paged_workspace_bytes.restype = ctypes.c_size_t
    lib.mka_decode_paged_workspace_bytes.argtypes = [ctypes.POINTER(mka_shape), i32, ctypes.POINTER(ctypes.c_int64)]
    lib.mka_decode_paged.argtypes = [ctypes.POINTER(mka_shape), i32, vp, ctypes.POINTER(mka_paged_level), vp, vp, vp, vp,
                                     ctypes.c_size_t, vp]
    lib.mka_fwd_paged.argtypes = lib.mka_decode_paged.argtypes
    lib.mka_fuse_kv_paged.argtypes = [i32, i32, i64, i32, i32, ctypes.POINTER(mka_level), vp, ctypes.POINTER(mka_paged_level), i64,
                                      vp, vp]
    lib.mka_l3_index.argtypes = [vp, i64, i32, i32, i32, i64, i64, i64, vp, i32, vp, vp]
    lib.mka_l3_retrieve.argtypes = [vp, i32, i32, i32, i32, vp, i32, vp, vp, vp, i64, i32, i32, i32, vp, vp, vp, vp]
    lib.mka_l2_summary_kernel_kind.argtypes = [i32, i64, i32, i32, ctypes.c_size_t]
    lib.mka_l2_summary.argtypes = [vp, i32, i64, i32, i32, i32, ctypes.c_float, vp, i64, vp, vp, ctypes.c_size_t, vp]
    lib.mka_bwd_kernel_kind.argtypes = [ctypes.POINTER(mka_shape), ctypes.POINTER(mka_level), vp]
    lib.mka_set_wait_limit_us.argtypes = [ctypes.c_uint32]
    for name in EXPORTS:
        if name not in ("mka_status_str", "mka_workspace_bytes", "mka_decode_static_max_bytes", "mka_l2_summary_workspace_bytes",
                        "mka_decode_paged_workspace_bytes", "mka_set_wait_limit_us"):
            getattr(lib, name).restype = ctypes.c_int
    lib.mka_set_wait_limit_us.restype = ctypes.c_uint32
    return lib


lib = _load()


def status_str(code: int) -> str:
    return lib.mka_status_str(code).decode()


def _check(code: int, where: str):
    if code != 0:
        raise MkaError(code, where)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return MKA_BF16
    if t.dtype == torch.float32:
        return MKA_F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _n_level(n) -> ctypes.Array:
    return (ctypes.c_int64 * 3)(*[int(x) for x in n])


def make_shape(B, H, T, d, D=0, window=1, q_offset=0, scale=0.0, dtype=MKA_BF16, mode=MKA_MODE_FAST, flags=0,
               kv_heads=0) -> mka_shape:
    return mka_shape(B, H, T, d, D, window, q_offset, scale, dtype, mode, flags, kv_heads)


def _levels(K: Sequence[Optional[torch.Tensor]], V: Sequence[Optional[torch.Tensor]]):
    arr = (mka_level * 3)()
    for l in range(3):
        k, v = K[l], V[l]
        if k is None or k.shape[2] == 0:
            arr[l] = mka_level(None, None, 0, 0, 0, 0)
            continue
        assert k.dim() == 4 and k.stride(3) == 1 and v.stride() == k.stride() and v.shape == k.shape
        arr[l] = mka_level(k.data_ptr(), v.data_ptr(), k.shape[2], k.stride(0), k.stride(1), k.stride(2))
    return arr


def mka_workspace_bytes(shape: mka_shape, n_level, which: int) -> int:
    return int(lib.mka_workspace_bytes(ctypes.byref(shape), _n_level(n_level), which))


def mka_decode_plan(n_level, B: int, H: int, d: int):
    plan = mka_decode_plan_t()
    _check(lib.mka_decode_plan(_n_level(n_level), B, H, d, ctypes.byref(plan)), "mka_decode_plan")
    return int(plan.chunk_rows), [int(x) for x in plan.n_chunks], int(plan.total_chunks)


def mka_fwd_tile_range(shape: mka_shape, n_level, level: int, q_tile: int):
    out = mka_tile_range()
    _check(lib.mka_fwd_tile_range(ctypes.byref(shape), _n_level(n_level), level, q_tile, ctypes.byref(out)),
           "mka_fwd_tile_range")
    return int(out.first), int(out.end), int(out.full_first), int(out.full_end)


def mka_router(R: torch.Tensor, W_r: torch.Tensor, b_r: Optional[torch.Tensor], route: int = MKA_ROUTE_SOFT,
               gate: Optional[torch.Tensor] = None, log2_gate: Optional[torch.Tensor] = None,
               route_idx: Optional[torch.Tensor] = None, stream=None):
    """R[..., D] -> gate[..., 3] (f32).  Outputs may be preallocated; missing ones are allocated here."""
    D = R.shape[-1]
    rows = R.numel() // D if D else 0
    assert R.is_contiguous() and W_r.is_contiguous() and W_r.dtype == torch.float32 and W_r.shape == (D, 3)
    lead = tuple(R.shape[:-1])
    if gate is None:
        gate = torch.empty(lead + (3,), dtype=torch.float32, device=R.device)
    _check(lib.mka_router(_ptr(R), _ptr(W_r), _ptr(b_r), rows, D, _dt(R), route, _ptr(gate), _ptr(log2_gate),
                          _ptr(route_idx), _stream(stream)), "mka_router")
    return gate


def alloc_workspace(shape: mka_shape, n_level, which: int, device) -> torch.Tensor:
    return torch.empty(mka_workspace_bytes(shape, n_level, which), dtype=torch.uint8, device=device)


def mka_fwd(shape: mka_shape, Q, K, V, gate, O=None, LSE=None, ws=None, stream=None, want_lse=True):
    assert Q.is_contiguous() and gate.is_contiguous() and gate.dtype == torch.float32
    if O is None:
        O = torch.empty_like(Q)
    if LSE is None and want_lse and shape.mode == MKA_MODE_FAST:
        LSE = torch.empty(Q.shape[:3], dtype=torch.float32, device=Q.device)
    n = [0 if k is None else k.shape[2] for k in K]
    if ws is None:
        ws = alloc_workspace(shape, n, MKA_WS_FWD, Q.device)
    _check(lib.mka_fwd(ctypes.byref(shape), _ptr(Q), _levels(K, V), _ptr(gate), _ptr(O), _ptr(LSE), _ptr(ws),
                       ws.numel(), _stream(stream)), "mka_fwd")
    return O, LSE


def mka_decode(shape: mka_shape, q, K, V, gate, O=None, LSE=None, ws=None, stream=None):
    assert q.is_contiguous() and gate.is_contiguous() and gate.dtype == torch.float32
    if O is None:
        O = torch.empty_like(q)
    if LSE is None:
        LSE = torch.empty(q.shape[:2], dtype=torch.float32, device=q.device)
    n = [0 if k is None else k.shape[2] for k in K]
    if ws is None:
        ws = alloc_workspace(shape, n, MKA_WS_DECODE, q.device)
    _check(lib.mka_decode(ctypes.byref(shape), _ptr(q), _levels(K, V), _ptr(gate), _ptr(O), _ptr(LSE), _ptr(ws),
                          ws.numel(), _stream(stream)), "mka_decode")
    return O, LSE


def _paged_levels(pools_k, pools_v, tables, rows, n):
    arr = (mka_paged_level * 3)()
    for l in range(3):
        k, v = pools_k[l], pools_v[l]
        if k is None or n[l] == 0:
            arr[l] = mka_paged_level(None, None, None, None, 0, 0, 0, 1, 0, 0, 0, 0)
            continue
        # pools [pages, H_kv, page_rows, d]; any strides with d contiguous
        assert k.dim() == 4 and k.stride(3) == 1 and v.stride() == k.stride() and v.shape == k.shape
        tab = tables[l]
        # [B, pages]: one table per sequence; [B, H_kv, pages]: one per (sequence, KV head)
        assert tab.dtype == torch.int32 and tab.dim() in (2, 3) and tab.stride(-1) == 1
        r = None if rows is None else rows[l]
        assert r is None or (r.dtype == torch.int32 and r.is_contiguous())
        arr[l] = mka_paged_level(k.data_ptr(), v.data_ptr(), tab.data_ptr(), _ptr(r), int(n[l]), tab.stride(0),
                                 tab.stride(1) if tab.dim() == 3 else 0, k.shape[2], k.stride(0), k.stride(1), k.stride(2),
                                 k.shape[0])
    return arr


def mka_fuse_kv_paged(K, V, gate, pool_k, pool_v, table, dst_offset=0, dst_offsets=None, stream=None):
    """Route-fusion of token-aligned levels K[l], V[l] ([B, H, n, d] or None) with gate [B, n, 3], appended to the paged
    cache pool_k / pool_v [pages, H, page_rows, d] through table int32 [B, pages] at logical rows dst_offset
    (+ dst_offsets[b]) + j."""
    ref = next(k for k in K if k is not None)
    B, H, n, d = ref.shape
    assert gate.is_contiguous() and gate.dtype == torch.float32 and tuple(gate.shape) == (B, n, 3)
    assert pool_k.dim() == 4 and pool_k.stride(3) == 1 and pool_v.stride() == pool_k.stride() and pool_k.dtype == ref.dtype
    assert table.dtype == torch.int32 and table.dim() == 2 and table.stride(1) == 1
    assert dst_offsets is None or (dst_offsets.dtype == torch.int32 and dst_offsets.is_contiguous())
    dst = mka_paged_level(pool_k.data_ptr(), pool_v.data_ptr(), table.data_ptr(), None, table.shape[1] * pool_k.shape[2],
                          table.stride(0), 0, pool_k.shape[2], pool_k.stride(0), pool_k.stride(1), pool_k.stride(2), pool_k.shape[0])
    _check(lib.mka_fuse_kv_paged(B, H, n, d, _dt(ref), _levels(K, V), _ptr(gate), ctypes.byref(dst), dst_offset, _ptr(dst_offsets),
                                 _stream(stream)), "mka_fuse_kv_paged")
    return pool_k, pool_v


def mka_fwd_paged(shape: mka_shape, H_kv: int, Q, pools_k, pools_v, tables, n, gate, rows=None, O=None, LSE=None, ws=None,
                  stream=None):
    """mka_fwd over paged levels with grouped-query head sharing (n[l]: upper bound of the rows on level l; rows[l]:
    int32 [B] rows of every sequence, or None)."""
    assert Q.is_contiguous() and gate.is_contiguous() and gate.dtype == torch.float32
    B, H, T, d = Q.shape
    if O is None:
        O = torch.empty_like(Q)
    if LSE is None:
        LSE = torch.empty(B, H, T, dtype=torch.float32, device=Q.device)
    if ws is None:
        ws = torch.zeros(256, dtype=torch.uint8, device=Q.device)
    _check(lib.mka_fwd_paged(ctypes.byref(shape), H_kv, _ptr(Q), _paged_levels(pools_k, pools_v, tables, rows, n), _ptr(gate),
                             _ptr(O), _ptr(LSE), _ptr(ws), ws.numel(), _stream(stream)), "mka_fwd_paged")
    return O, LSE


def mka_decode_paged_workspace_bytes(shape: mka_shape, H_kv: int, n) -> int:
    return int(lib.mka_decode_paged_workspace_bytes(ctypes.byref(shape), H_kv, _n_level(n)))


def mka_decode_paged(shape: mka_shape, H_kv: int, q, pools_k, pools_v, tables, n, gate, rows=None, O=None, LSE=None,
                     ws=None, stream=None):
    """Decode over paged levels with grouped-query head sharing.  pools_k[l], pools_v[l]: [pages, H_kv, page_rows, d]
    (or None); tables[l]: int32 [B, pages per sequence]; n[l]: upper bound of the rows; rows[l]: int32 [B] or None."""
    assert q.is_contiguous() and gate.is_contiguous() and gate.dtype == torch.float32
    if O is None:
        O = torch.empty_like(q)
    if LSE is None:
        LSE = torch.empty(q.shape[:2], dtype=torch.float32, device=q.device)
    if ws is None:
        ws = torch.empty(mka_decode_paged_workspace_bytes(shape, H_kv, n), dtype=torch.uint8, device=q.device)
    _check(lib.mka_decode_paged(ctypes.byref(shape), H_kv, _ptr(q), _paged_levels(pools_k, pools_v, tables, rows, n),
                                _ptr(gate), _ptr(O), _ptr(LSE), _ptr(ws), ws.numel(), _stream(stream)), "mka_decode_paged")
    return O, LSE


def mka_l3_index(pool_k, proj, codes=None, stream=None):
    """Sign-random-projection codes of every (page, KV head) of a key pool [pages, H_kv, page_rows, d] under
    proj [bits, d] f32; returns int32 [pages, H_kv, bits // 32] holding the code words' bit patterns."""
    assert pool_k.dim() == 4 and pool_k.stride(3) == 1 and proj.dtype == torch.float32 and proj.is_contiguous()
    P, H_kv, pr, d = pool_k.shape
    bits = proj.shape[0]
    if codes is None:
        codes = torch.empty(P, H_kv, bits // 32, dtype=torch.int32, device=pool_k.device)
    _check(lib.mka_l3_index(_ptr(pool_k), P, H_kv, pr, d, pool_k.stride(0), pool_k.stride(1), pool_k.stride(2), _ptr(proj),
                            bits, _ptr(codes), _stream(stream)), "mka_l3_index")
    return codes


def mka_l3_retrieve(q, H_kv: int, proj, codes, bank, bank_len, R: int, page_rows: int, table=None, n_sel=None, rows=None,
                    stream=None):
    """Recall lists of every (sequence, KV head): returns (table int32 [B, H_kv, R], n_sel int32 [B], rows int32 [B])."""
    assert q.is_contiguous() and bank.dtype == torch.int32 and bank.dim() == 2 and bank.stride(1) == 1
    assert bank_len.dtype == torch.int32 and bank_len.is_contiguous() and codes.is_contiguous()
    B, H, d = q.shape
    if table is None:
        table = torch.empty(B, H_kv, R, dtype=torch.int32, device=q.device)
    if n_sel is None:
        n_sel = torch.empty(B, dtype=torch.int32, device=q.device)
    if rows is None:
        rows = torch.empty(B, dtype=torch.int32, device=q.device)
    _check(lib.mka_l3_retrieve(_ptr(q), B, H, H_kv, d, _ptr(proj), proj.shape[0], _ptr(codes), _ptr(bank), _ptr(bank_len),
                               bank.stride(0), bank.shape[1], R, page_rows, _ptr(table), _ptr(n_sel), _ptr(rows),
                               _stream(stream)), "mka_l3_retrieve")
    return table, n_sel, rows


def mka_decode_static(shape: mka_shape, q, K, V, gate, O, LSE=None, stream=None):
    """Decode without a workspace, for callers that may not allocate: the partials go to the 8 MiB array
    built into the library.  This wrapper allocates nothing either -- `O` (and `LSE`, if wanted) must be
    passed in.  Raises MkaError(4) when the problem's split table does not fit the built-in array."""
    assert q.is_contiguous() and gate.is_contiguous() and gate.dtype == torch.float32 and O.is_contiguous()
    _check(lib.mka_decode_static(ctypes.byref(shape), _ptr(q), _levels(K, V), _ptr(gate), _ptr(O), _ptr(LSE),
                                 _stream(stream)), "mka_decode_static")
    return O, LSE


def mka_decode_static_max_bytes() -> int:
    return int(lib.mka_decode_static_max_bytes())


def mka_bwd(shape: mka_shape, Q, K, V, gate, O, LSE, dO, R=None, dQ=None, dK=None, dV=None, dG=None, dW_r=None,
            db_r=None, ws=None, stream=None, want_router_grad=True):
    for t in (Q, O, dO, gate, LSE):
        assert t.is_contiguous()
    dev = Q.device
    if dQ is None:
        dQ = torch.empty_like(Q)
    if dK is None:
        dK = [None if k is None else torch.empty_like(k) for k in K]
    if dV is None:
        dV = [None if v is None else torch.empty_like(v) for v in V]
    if dG is None:
        dG = torch.empty(gate.shape, dtype=torch.float32, device=dev)
    if R is not None and want_router_grad:
        assert R.is_contiguous()
        if dW_r is None:
            dW_r = torch.empty((R.shape[-1], 3), dtype=torch.float32, device=dev)
        if db_r is None:
            db_r = torch.empty((3,), dtype=torch.float32, device=dev)
    grads = (mka_level_grad * 3)()
    for l in range(3):
        if K[l] is None or K[l].shape[2] == 0:
            grads[l] = mka_level_grad(None, None, 0, 0, 0, 0)
        else:
            g = dK[l]
            assert g.stride(3) == 1 and dV[l].stride() == g.stride()
            grads[l] = mka_level_grad(g.data_ptr(), dV[l].data_ptr(), g.shape[2], g.stride(0), g.stride(1), g.stride(2))
    n = [0 if k is None else k.shape[2] for k in K]
    if ws is None:
        ws = alloc_workspace(shape, n, MKA_WS_BWD, dev)
    _check(lib.mka_bwd(ctypes.byref(shape), _ptr(Q), _levels(K, V), _ptr(gate), _ptr(O), _ptr(LSE), _ptr(dO),
                       _ptr(R), _dt(R) if R is not None else MKA_F32, _ptr(dQ), grads, _ptr(dG), _ptr(dW_r),
                       _ptr(db_r), _ptr(ws), ws.numel(), _stream(stream)), "mka_bwd")
    return {"dQ": dQ, "dK": dK, "dV": dV, "dG": dG, "dW_r": dW_r, "db_r": db_r}


def mka_fwd_kernel_kind(shape: mka_shape, K, V) -> int:
    return int(lib.mka_fwd_kernel_kind(ctypes.byref(shape), _levels(K, V)))


def mka_fuse_kv(K, V, gate, out_k=None, out_v=None, dst_offset=0, stream=None):
    """Route-fusion with cache write (Alg. 2 steps 6-8): rows [dst_offset, dst_offset+n) of out_k / out_v receive
    sum_l gate[b,j,l] * K[l][b,h,j,:] (and V likewise).  K, V: three [B,H,n,d] tensors or None; gate [B,n,3] f32."""
    ref = next(k for k in K if k is not None)
    B, H, n, d = ref.shape
    assert gate.is_contiguous() and gate.dtype == torch.float32 and tuple(gate.shape) == (B, n, 3)
    if out_k is None:
        out_k = torch.empty((B, H, dst_offset + n, d), dtype=ref.dtype, device=ref.device)
    if out_v is None:
        out_v = torch.empty_like(out_k)
    assert out_k.stride(3) == 1 and out_v.stride() == out_k.stride() and out_k.dtype == ref.dtype
    dst = mka_level_grad(out_k.data_ptr(), out_v.data_ptr(), out_k.shape[2], out_k.stride(0), out_k.stride(1), out_k.stride(2))
    _check(lib.mka_fuse_kv(B, H, n, d, _dt(ref), _levels(K, V), _ptr(gate), ctypes.byref(dst), dst_offset, _stream(stream)),
           "mka_fuse_kv")
    return out_k, out_v


def mka_l2_summary_workspace(X) -> torch.Tensor:
    """Scratch for mka_l2_summary's segmented form on input X (uint8 tensor on X's device)."""
    B, T, D = X.shape
    return torch.empty(int(lib.mka_l2_summary_workspace_bytes(B, T, D, _dt(X))), dtype=torch.uint8, device=X.device)


def mka_l2_summary_kernel_kind(X, ws=None) -> int:
    """1 when mka_l2_summary(X, ws=ws) would run the segmented form, 0 for the strip form."""
    B, T, D = X.shape
    return int(lib.mka_l2_summary_kernel_kind(B, T, D, _dt(X), 0 if ws is None else ws.numel()))


def mka_l2_summary(X, kind=MKA_SUMMARY_MEAN, beta=0.9, state=None, n_prev=0, M2=None, ws=None, stream=None):
    """Causal L2 session summary of X [B, T, D] (prefix mean or EMA); returns M2.  `state` [B, D] f32 carries a
    session across calls: read when n_prev > 0, written with the new state whenever it is given."""
    assert X.dim() == 3 and X.is_contiguous()
    B, T, D = X.shape
    if M2 is None:
        M2 = torch.empty_like(X)
    assert M2.is_contiguous() and M2.dtype == X.dtype
    if state is not None:
        assert state.is_contiguous() and state.dtype == torch.float32 and tuple(state.shape) == (B, D)
    _check(lib.mka_l2_summary(_ptr(X), B, T, D, _dt(X), kind, float(beta), _ptr(state), n_prev, _ptr(M2), _ptr(ws),
                              0 if ws is None else ws.numel(), _stream(stream)), "mka_l2_summary")
    return M2


def mka_bwd_kernel_kind(shape: mka_shape, K, V) -> int:
    """1 when mka_bwd would run the tensor-core kernels for this problem (gradients laid out like K, V)."""
    return int(lib.mka_bwd_kernel_kind(ctypes.byref(shape), _levels(K, V), None))


def mka_device_status(ws: torch.Tensor, stream=None) -> int:
    return int(lib.mka_device_status(_ptr(ws), _stream(stream)))


def mka_set_wait_limit_us(us: int) -> int:
    """Sets the limit of the kernels' internal waits (microseconds; 0 = the default of one second); returns the old one."""
    return int(lib.mka_set_wait_limit_us(int(us)))
