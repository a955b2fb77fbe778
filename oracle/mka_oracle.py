"""numpy front end of the CPU oracle (``mka_oracle.c``) -- TEST INFRASTRUCTURE ONLY.

Nothing in the product package may import this module; it exists so that the
tests, the smoke check and the benchmark's cpu-baseline leg can evaluate the
paper's definitions (Eq. 5, Alg. 1, the router, the derived backward) in fp64, and the steps around
them (route-fusion, session summary, paged grouped-query decode, L3 recall).

The wrappers only marshal arrays: they loop over (batch, head), hand one head
problem at a time to the C routines, and sum the per-head router-logit
gradients over heads (the gate is one per token, shared by all heads).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mka_oracle.c")
_LIB = os.path.join(_HERE, "libmka_oracle.so")
_lib = None

ROUTE_SOFT, ROUTE_UNIFORM, ROUTE_TOP1, ROUTE_TOP2 = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) if the library is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().orc_num_threads())


_DP = ctypes.POINTER(ctypes.c_double)
_LP = ctypes.POINTER(ctypes.c_int64)


def _p(a: Optional[np.ndarray]):
    if a is None:
        return ctypes.cast(None, _DP)
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_DP)


def _f64(a) -> np.ndarray:
    if hasattr(a, "detach"):  # torch tensor
        a = a.detach().to("cpu").double().numpy()
    return np.ascontiguousarray(a, dtype=np.float64)


def visible(level: int, p: int, W: int, n: int, decode: bool = False):
    lo, hi = ctypes.c_int64(), ctypes.c_int64()
    _load().orc_visible(ctypes.c_int(level), ctypes.c_int64(p), ctypes.c_int64(W), ctypes.c_int64(n),
                        ctypes.c_int(int(decode)), ctypes.byref(lo), ctypes.byref(hi))
    return lo.value, hi.value


def router(R, W_r, b_r=None, route: int = ROUTE_SOFT):
    """R[..., D], W_r[D, 3], b_r[3] -> gate[..., 3] (fp64), idx[..., 2] (int8)."""
    R = _f64(R)
    lead = R.shape[:-1]
    D = R.shape[-1]
    R2 = R.reshape(-1, D)
    W_r = _f64(W_r)
    assert W_r.shape == (D, 3)
    b = None if b_r is None else _f64(b_r)
    gate = np.empty((R2.shape[0], 3), np.float64)
    idx = np.empty((R2.shape[0], 2), np.int8)
    rc = _load().orc_router(_p(R2), _p(W_r), _p(b), ctypes.c_int64(R2.shape[0]), ctypes.c_int64(D),
                            ctypes.c_int(route), _p(gate), idx.ctypes.data_as(ctypes.POINTER(ctypes.c_int8)))
    assert rc == 0
    return gate.reshape(*lead, 3), idx.reshape(*lead, 2)


def _head_args(Qh, Ks, Vs, gate_b, W, q_off, tau, decode):
    T, d = Qh.shape
    args = [_p(Qh), ctypes.c_int64(T), ctypes.c_int64(d)]
    for l in range(3):
        n = Ks[l].shape[0]
        args += [_p(Ks[l]) if n else ctypes.cast(None, _DP), _p(Vs[l]) if n else ctypes.cast(None, _DP),
                 ctypes.c_int64(n)]
    args += [_p(gate_b), ctypes.c_int64(W), ctypes.c_int64(q_off), ctypes.c_double(tau), ctypes.c_int(int(decode))]
    return args


def _prep(Q, K, V, gate):
    Q = _f64(Q)
    K = [_f64(k) for k in K]
    V = [_f64(v) for v in V]
    gate = _f64(gate)
    B, H, T, d = Q.shape
    assert gate.shape == (B, T, 3)
    for l in range(3):
        assert K[l].shape == V[l].shape and K[l].shape[:2] == (B, H) and K[l].shape[3] == d
    return Q, K, V, gate, B, H, T, d


def _rows_arg(rows, T):
    if rows is None:
        return None, ctypes.cast(None, _LP), T
    r = np.ascontiguousarray(rows, dtype=np.int64)
    assert r.ndim == 1 and (r >= 0).all() and (r < T).all()
    return r, r.ctypes.data_as(_LP), r.shape[0]


def fwd(Q, K: Sequence, V: Sequence, gate, window: int, q_offset: int = 0, scale: Optional[float] = None,
        mode: str = "fast", decode: bool = False, rows=None, heads=None):
    """Forward of the operator.

    Q[B,H,T,d]; K[l], V[l] : [B,H,N_l,d]; gate[B,T,3].  mode "fast" = Eq. 5, "full" = Alg. 1.
    rows: optional 1-D list of query indices evaluated for every head (output then has
    len(rows) rows).  heads: optional list of (b, h) pairs; other heads are left as NaN.
    Returns O[B,H,R,d] and LSE[B,H,R] (LSE is None in "full" mode).
    """
    Q, K, V, gate, B, H, T, d = _prep(Q, K, V, gate)
    tau = (1.0 / np.sqrt(d)) if scale is None or scale <= 0 else float(scale)
    rkeep, rptr, R = _rows_arg(rows, T)
    O = np.full((B, H, R, d), np.nan)
    LSE = np.full((B, H, R), np.nan)
    lib = _load()
    pairs = heads if heads is not None else [(b, h) for b in range(B) for h in range(H)]
    for b, h in pairs:
        Ks = [np.ascontiguousarray(K[l][b, h]) for l in range(3)]
        Vs = [np.ascontiguousarray(V[l][b, h]) for l in range(3)]
        Qh = np.ascontiguousarray(Q[b, h])
        gb = np.ascontiguousarray(gate[b])
        o = np.empty((R, d))
        args = _head_args(Qh, Ks, Vs, gb, window, q_offset, tau, decode) + [rptr, ctypes.c_int64(R), _p(o)]
        if mode == "fast":
            ls = np.empty((R,))
            rc = lib.orc_fwd_fast_head(*args, _p(ls))
            LSE[b, h] = ls
        elif mode == "full":
            rc = lib.orc_fwd_full_head(*args)
        else:
            raise ValueError(mode)
        assert rc == 0
        O[b, h] = o
    return O, (LSE if mode == "fast" else None)


def fwd_recursive(Q, K, V, gate, window: int, q_offset: int = 0, scale: Optional[float] = None,
                  block: int = 128, decode: bool = False):
    """Eq. 6-8 / Eq. 11-14 evaluated level by level in key blocks (checks Theorem 1)."""
    Q, K, V, gate, B, H, T, d = _prep(Q, K, V, gate)
    tau = (1.0 / np.sqrt(d)) if scale is None or scale <= 0 else float(scale)
    O = np.empty((B, H, T, d))
    LSE = np.empty((B, H, T))
    lib = _load()
    for b in range(B):
        for h in range(H):
            Ks = [np.ascontiguousarray(K[l][b, h]) for l in range(3)]
            Vs = [np.ascontiguousarray(V[l][b, h]) for l in range(3)]
            o = np.empty((T, d))
            ls = np.empty((T,))
            rc = lib.orc_fwd_recursive_head(*_head_args(np.ascontiguousarray(Q[b, h]), Ks, Vs,
                                                        np.ascontiguousarray(gate[b]), window, q_offset, tau, decode),
                                            ctypes.c_int64(block), _p(o), _p(ls))
            assert rc == 0
            O[b, h], LSE[b, h] = o, ls
    return O, LSE


def bwd(Q, K, V, gate, dO, window: int, q_offset: int = 0, scale: Optional[float] = None,
        decode: bool = False, rows=None, heads=None, want_kv: bool = True):
    """Gradients of <dO, O> for the "fast" operator.

    Returns dict with dQ[B,H,R,d], dK[l], dV[l] ([B,H,N_l,d]; complete only when rows is
    None), G[B,H,R,3] (per-head router-logit gradient) and dG[B,R,3] = sum over heads.
    With `heads`, only those (b, h) pairs are evaluated (others NaN; dG then sums only them).
    """
    Q, K, V, gate, B, H, T, d = _prep(Q, K, V, gate)
    dO = _f64(dO)
    assert dO.shape == Q.shape
    tau = (1.0 / np.sqrt(d)) if scale is None or scale <= 0 else float(scale)
    rkeep, rptr, R = _rows_arg(rows, T)
    dQ = np.full((B, H, R, d), np.nan)
    G = np.full((B, H, R, 3), np.nan)
    dK = [np.full(K[l].shape, np.nan) for l in range(3)] if want_kv else None
    dV = [np.full(V[l].shape, np.nan) for l in range(3)] if want_kv else None
    lib = _load()
    pairs = heads if heads is not None else [(b, h) for b in range(B) for h in range(H)]
    null = ctypes.cast(None, _DP)
    for b, h in pairs:
        Ks = [np.ascontiguousarray(K[l][b, h]) for l in range(3)]
        Vs = [np.ascontiguousarray(V[l][b, h]) for l in range(3)]
        dq = np.empty((R, d))
        g = np.empty((R, 3))
        outs = []
        bufs = []
        for l in range(3):
            if want_kv:
                a, c = np.empty(Ks[l].shape), np.empty(Vs[l].shape)
                bufs.append((a, c))
                outs += [_p(a), _p(c)]
            else:
                outs += [null, null]
        rc = lib.orc_bwd_head(*_head_args(np.ascontiguousarray(Q[b, h]), Ks, Vs, np.ascontiguousarray(gate[b]),
                                          window, q_offset, tau, decode),
                              _p(np.ascontiguousarray(dO[b, h])), rptr, ctypes.c_int64(R), _p(dq), *outs, _p(g))
        assert rc == 0
        dQ[b, h], G[b, h] = dq, g
        if want_kv:
            for l in range(3):
                dK[l][b, h], dV[l][b, h] = bufs[l]
    dG = np.zeros((B, R, 3))
    for b, h in pairs:
        dG[b] += G[b, h]
    return {"dQ": dQ, "dK": dK, "dV": dV, "G": G, "dG": dG}


def router_bwd(R, dG):
    """dW_r[D,3] = sum over tokens of R^T dG, db_r[3] = sum dG (soft routing; the gate's
    softmax Jacobian is already folded into dG)."""
    R = _f64(R)
    dG = _f64(dG)
    D = R.shape[-1]
    dW = R.reshape(-1, D).T @ dG.reshape(-1, 3)
    return dW, dG.reshape(-1, 3).sum(0)


def route_fuse(levels: Sequence, gate) -> np.ndarray:
    """Route-fusion of Alg. 2 step 6: X_fused[b, j, :] = sum_l lambda[b, j, l] * L_l[b, j, :], in fp64.

    `levels` holds the three token-aligned level tensors; each is [B, n, D] (the paper's L_1, L_2, L_3) or
    [B, H, n, d] (their per-head key or value projections: because the projection of Alg. 2 step 7 is linear,
    fusing the projected levels equals projecting the fused representation), or None for an absent level,
    which contributes nothing.  `gate` is [B, n, 3]: the gate of the token the row belongs to.
    Plain definition, three explicit terms; no blocking.
    """
    g = _f64(gate)
    out = None
    for l in range(3):
        if levels[l] is None:
            continue
        x = _f64(levels[l])
        w = g[:, :, l]
        w = w[:, None, :, None] if x.ndim == 4 else w[:, :, None]
        term = w * x
        out = term if out is None else out + term
    if out is None:
        raise ValueError("no level present")
    return out


SUMMARY_MEAN, SUMMARY_EMA = 0, 1


def l2_summary(X, kind: int = SUMMARY_MEAN, beta: float = 0.9, state=None, n_prev: int = 0):
    """Causal session summary of Alg. 1 (the loop that fills M_2) / Alg. 2 step 3, in fp64: row t summarises X[:, :t+1].

    kind = SUMMARY_MEAN: prefix mean.  With a carried state (the running SUM of the n_prev earlier tokens of the
           session) M2[t] = (state + sum_{i<=t} x_i) / (n_prev + t + 1).
    kind = SUMMARY_EMA:  m_t = beta m_{t-1} + (1 - beta) x_t.  The paper does not say how the average starts; here the
           first token of a session initialises it (m_0 = x_0); with n_prev > 0 the carried state is m_{-1}.
    X is [B, T, D].  Returns (M2 [B, T, D], new state [B, D]): the state to carry into the session's next chunk.
    The recurrences are written out token by token.
    """
    X = _f64(X)
    B, T, D = X.shape
    M = np.empty_like(X)
    if kind == SUMMARY_MEAN:
        run = np.zeros((B, D)) if (state is None or n_prev == 0) else _f64(state).copy()
        for t in range(T):
            run = run + X[:, t]
            M[:, t] = run / float(n_prev + t + 1)
        return M, run
    if kind == SUMMARY_EMA:
        have = state is not None and n_prev > 0
        m = _f64(state).copy() if have else None
        for t in range(T):
            m = X[:, t].copy() if m is None else beta * m + (1.0 - beta) * X[:, t]
            M[:, t] = m
        return M, (m if m is not None else np.zeros((B, D)))
    raise ValueError("unknown summary kind")


def gather_pages(pool, table, rows: int, page_rows: int) -> np.ndarray:
    """Dense view of one sequence's rows of a paged level (the paged KV layout of the paper's inference setup for
    contexts beyond 32K).  pool is [P, H_kv, page_rows, d]; logical row r of the sequence lives in pool page
    table[r // page_rows] at offset r % page_rows.  Returns [H_kv, rows, d].  Written row by row."""
    pool = np.asarray(pool)
    out = np.empty((pool.shape[1], rows, pool.shape[3]), dtype=np.float64)
    for r in range(rows):
        out[:, r, :] = pool[int(table[r // page_rows]), :, r % page_rows, :]
    return out


def decode_paged(q, pools_k: Sequence, pools_v: Sequence, tables: Sequence, rows: Sequence, page_rows: int, gate,
                 scale: Optional[float] = None):
    """Single-token decode of Eq. 5 over paged levels with grouped-query sharing of the KV heads.

    q [B, H, d]; for level l: pools_k[l], pools_v[l] [P_l, H_kv, page_rows, d] (or None for an absent level),
    tables[l] [B, pages] page table (or [B, H_kv, pages]: one per KV head, as L3 recall produces), rows[l] [B] valid
    rows of every sequence; gate [B, 3].
    Query head h reads KV head h // (H / H_kv): consecutive query heads share one KV head.
    Every sequence is gathered into dense levels and handed to the dense decode (all gathered rows visible).
    Returns O [B, H, d], LSE [B, H]."""
    q = _f64(q)
    gate = _f64(gate)
    B, H, d = q.shape
    O = np.empty((B, H, d))
    LSE = np.empty((B, H))
    for b in range(B):
        Ks, Vs = [], []
        for l in range(3):
            if pools_k[l] is None or int(rows[l][b]) == 0:
                Ks.append(np.zeros((1, H, 0, d)))
                Vs.append(np.zeros((1, H, 0, d)))
                continue
            H_kv = np.asarray(pools_k[l]).shape[1]
            assert H % H_kv == 0
            tab = np.asarray(tables[l][b])
            if tab.ndim == 2:                                    # one recall list per KV head: gather head by head
                kd = np.concatenate([gather_pages(_f64(pools_k[l])[:, h:h + 1], tab[h], int(rows[l][b]), page_rows)
                                     for h in range(H_kv)], axis=0)
                vd = np.concatenate([gather_pages(_f64(pools_v[l])[:, h:h + 1], tab[h], int(rows[l][b]), page_rows)
                                     for h in range(H_kv)], axis=0)
            else:
                kd = gather_pages(_f64(pools_k[l]), tab, int(rows[l][b]), page_rows)
                vd = gather_pages(_f64(pools_v[l]), tab, int(rows[l][b]), page_rows)
            share = np.arange(H) // (H // H_kv)                  # KV head of every query head
            Ks.append(kd[share][None])
            Vs.append(vd[share][None])
        o, ls = fwd(q[b][None, :, None, :], Ks, Vs, gate[b].reshape(1, 1, 3), 1, scale=scale, decode=True)
        O[b] = o[0, :, 0, :]
        LSE[b] = ls[0, :, 0]
    return O, LSE


# ---- L3 recall: sign-random-projection codes and top-R selection (a reading; the paper names no hash) ----------------

def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def srp_code(x, proj) -> np.ndarray:
    """Code of one vector x[d] under proj[bits, d]: bit j = [proj[j] . x >= 0], the dot product taken as one fp32 fmaf
    chain over the columns.  Returns uint32[bits // 32], bit j in word j // 32 at position j % 32."""
    x, proj = _f32(x), _f32(proj)
    bits, d = proj.shape
    code = np.zeros(bits // 32, dtype=np.uint32)
    rc = _load().orc_srp_code(x.ctypes.data_as(ctypes.c_void_p), proj.ctypes.data_as(ctypes.c_void_p), ctypes.c_int64(d),
                              ctypes.c_int64(bits), code.ctypes.data_as(ctypes.c_void_p))
    assert rc == 0
    return code


def sum_rows_f32(x) -> np.ndarray:
    """Column sums of x[n, d] accumulated row by row in fp32."""
    x = _f32(x)
    s = np.zeros(x.shape[1], dtype=np.float32)
    _load().orc_sum_rows_f32(x.ctypes.data_as(ctypes.c_void_p), ctypes.c_int64(x.shape[0]), ctypes.c_int64(x.shape[1]),
                             s.ctypes.data_as(ctypes.c_void_p))
    return s


def l3_index(pool_k, proj) -> np.ndarray:
    """Codes of every (page, KV head) of a key pool [P, H_kv, page_rows, d]: the code of the sum of the page's keys.
    Returns uint32 [P, H_kv, bits // 32]."""
    pool_k = _f32(pool_k)
    P, H_kv = pool_k.shape[:2]
    out = np.zeros((P, H_kv, proj.shape[0] // 32), dtype=np.uint32)
    for pg in range(P):
        for h in range(H_kv):
            out[pg, h] = srp_code(sum_rows_f32(pool_k[pg, h]), proj)
    return out


def l3_select(qcode, codes, R: int):
    """Indices (ascending) of the min(R, n) rows of codes[n, words] nearest to qcode in Hamming distance, ties to the
    lower index."""
    codes = np.ascontiguousarray(codes, dtype=np.uint32)
    qcode = np.ascontiguousarray(qcode, dtype=np.uint32)
    n, words = codes.shape
    out = np.zeros(max(R, 1), dtype=np.int64)
    n_out = ctypes.c_int64(0)
    rc = _load().orc_l3_select(qcode.ctypes.data_as(ctypes.c_void_p), codes.ctypes.data_as(ctypes.c_void_p),
                               ctypes.c_int64(n), ctypes.c_int64(words), ctypes.c_int64(R),
                               out.ctypes.data_as(ctypes.c_void_p), ctypes.byref(n_out))
    assert rc == 0
    return out[:n_out.value].copy()


def l3_retrieve(q, proj, codes, bank, bank_len, R: int, H_kv: int):
    """Retrieve of Alg. 2 step 4 under the reading above.  q [B, H, d]; codes [P, H_kv, words] from l3_index;
    bank [B, n] pool pages of each sequence's long-term chunks in time order, bank_len [B] how many are in use.
    For every (sequence, KV head): the query is the fp32 sum of the query heads sharing the KV head (head order), its
    code is compared with the codes of the sequence's bank and the pool pages of the R nearest chunks are returned
    in bank order.  Returns (table int32 [B, H_kv, R], zero-padded; n_sel int32 [B])."""
    q = _f32(q)
    B, H, d = q.shape
    G = H // H_kv
    table = np.zeros((B, H_kv, R), dtype=np.int32)
    n_sel = np.zeros(B, dtype=np.int32)
    for b in range(B):
        n = int(bank_len[b])
        pages = np.asarray(bank[b][:n], dtype=np.int64)
        for h in range(H_kv):
            qc = srp_code(sum_rows_f32(q[b, h * G:(h + 1) * G]), proj)
            pos = l3_select(qc, codes[pages, h], R) if n else np.zeros(0, dtype=np.int64)
            table[b, h, :len(pos)] = pages[pos]
            n_sel[b] = len(pos)
    return table, n_sel


def fwd_paged(Q, pools_k: Sequence, pools_v: Sequence, tables: Sequence, n: Sequence[int], page_rows: int, gate,
              window: int, q_offset: int = 0, scale: Optional[float] = None):
    """Forward of the operator over paged levels with grouped-query sharing: every sequence's levels (n[l] rows each)
    are gathered through the page tables, the KV heads repeated over their groups, and the dense forward does the rest.
    Q [B, H, T, d]; pools [P_l, H_kv, page_rows, d] or None; tables[l] [B, pages] or [B, H_kv, pages]; gate [B, T, 3];
    n[l]: rows of level l, one number for all sequences or an array [B]."""
    Q = _f64(Q)
    gate = _f64(gate)
    B, H, T, d = Q.shape
    O = np.empty((B, H, T, d))
    LSE = np.empty((B, H, T))
    for b in range(B):
        Ks, Vs = [], []
        for l in range(3):
            n_b = int(np.asarray(n[l]).reshape(-1)[b if np.ndim(n[l]) else 0])
            if pools_k[l] is None or n_b == 0:
                Ks.append(np.zeros((1, H, 0, d)))
                Vs.append(np.zeros((1, H, 0, d)))
                continue
            pk, pv = _f64(pools_k[l]), _f64(pools_v[l])
            H_kv = pk.shape[1]
            tab = np.asarray(tables[l][b])
            if tab.ndim == 2:
                kd = np.concatenate([gather_pages(pk[:, h:h + 1], tab[h], n_b, page_rows) for h in range(H_kv)], axis=0)
                vd = np.concatenate([gather_pages(pv[:, h:h + 1], tab[h], n_b, page_rows) for h in range(H_kv)], axis=0)
            else:
                kd = gather_pages(pk, tab, n_b, page_rows)
                vd = gather_pages(pv, tab, n_b, page_rows)
            share = np.arange(H) // (H // H_kv)
            Ks.append(kd[share][None])
            Vs.append(vd[share][None])
        o, ls = fwd(Q[b:b + 1], Ks, Vs, gate[b:b + 1], window, q_offset=q_offset, scale=scale)
        O[b], LSE[b] = o[0], ls[0]
    return O, LSE
