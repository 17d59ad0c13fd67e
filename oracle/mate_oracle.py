"""ctypes front-end of the C oracle (test infrastructure only).

All floating-point arrays are converted to float64, which is exact for fp32 and bf16 inputs.
"""
import ctypes as C

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.oracle_fwd.restype = C.c_int
        _lib.oracle_bwd.restype = C.c_int
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _f64(x):
    return np.ascontiguousarray(np.asarray(x), dtype=np.float64)


def _i32(x):
    return np.ascontiguousarray(np.asarray(x), dtype=np.int32)


def _u8(x):
    return np.ascontiguousarray(np.asarray(x), dtype=np.uint8)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _g(P, global_len):
    return int(P if global_len is None else global_len)


def mask(row_ids, col_ids, P, view, radius=0, global_len=None):
    """Explicit attention pattern of Section 3 for one example: uint8 [N, N], M[k, j] = j in A_k.
    radius > 0: the bucketed pattern of Section 3.1 (buckets of `radius` positions of the view order
    behind a global section of global_len >= P positions; default: the prefix)."""
    r, c = _i32(row_ids).reshape(-1), _i32(col_ids).reshape(-1)
    N = r.shape[0]
    M = np.empty((N, N), dtype=np.uint8)
    _load().oracle_mask_bucketed(_p(r), _p(c), C.c_int(N), C.c_int(P), C.c_int(view), C.c_int(radius),
                                 C.c_int(_g(P, global_len)), _p(M))
    return M


def mask_sat(row_ids, col_ids, P):
    """Head-independent pattern of Section 2 (same row OR same column, plus the prefix): uint8 [N, N]."""
    r, c = _i32(row_ids).reshape(-1), _i32(col_ids).reshape(-1)
    N = r.shape[0]
    M = np.empty((N, N), dtype=np.uint8)
    _load().oracle_mask_sat(_p(r), _p(c), C.c_int(N), C.c_int(P), _p(M))
    return M


def cell_mean(logits, row_ids, col_ids, P, max_row_id, max_col_id):
    """Mean of the token logits per table cell (Section 4.1).  Returns mean f64 and count int32,
    both [B, max_row_id+1, max_col_id+1]."""
    x, r, c = _f64(logits), _i32(row_ids), _i32(col_ids)
    B, N = r.shape
    assert x.shape == (B, N)
    mean = np.empty((B, max_row_id + 1, max_col_id + 1), dtype=np.float64)
    cnt = np.empty((B, max_row_id + 1, max_col_id + 1), dtype=np.int32)
    _load().oracle_cell_mean(_p(x), _p(r), _p(c), C.c_int(B), C.c_int(N), C.c_int(P), C.c_int(max_row_id),
                             C.c_int(max_col_id), _p(mean), _p(cnt))
    return mean, cnt


def useful_pairs(row_ids, col_ids, P, head_view, radius=0, global_len=None):
    r, c, hv = _i32(row_ids), _i32(col_ids), _u8(head_view)
    B, N = r.shape
    out = np.zeros((B, hv.shape[0]), dtype=np.int64)
    _load().oracle_useful_pairs(_p(r), _p(c), C.c_int(B), C.c_int(hv.shape[0]), C.c_int(N),
                                C.c_int(P), _p(hv), C.c_int(radius), C.c_int(_g(P, global_len)), _p(out))
    return out


def fwd(Q, K, V, row_ids, col_ids, P, head_view, scale, radius=0, global_len=None):
    """Masked softmax attention (Section 3 head formula).  Returns O [B,H,N,d], LSE [B,H,N] (f64)."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    r, c, hv = _i32(row_ids), _i32(col_ids), _u8(head_view)
    B, H, N, d = Q.shape
    assert K.shape == Q.shape and V.shape == Q.shape and r.shape == (B, N) and c.shape == (B, N)
    assert hv.shape == (H,)
    O = np.empty_like(Q)
    LSE = np.empty((B, H, N), dtype=np.float64)
    rc = _load().oracle_fwd(_p(Q), _p(K), _p(V), _p(r), _p(c), C.c_int(B), C.c_int(H), C.c_int(N),
                            C.c_int(d), C.c_int(P), _p(hv), C.c_double(scale), C.c_int(radius),
                            C.c_int(_g(P, global_len)), _p(O), _p(LSE))
    assert rc == 0
    return O, LSE


def bwd(Q, K, V, dO, row_ids, col_ids, P, head_view, scale, radius=0, global_len=None):
    """Analytic backward of `fwd`.  Returns dQ, dK, dV (f64)."""
    Q, K, V, dO = _f64(Q), _f64(K), _f64(V), _f64(dO)
    r, c, hv = _i32(row_ids), _i32(col_ids), _u8(head_view)
    B, H, N, d = Q.shape
    assert K.shape == Q.shape and V.shape == Q.shape and dO.shape == Q.shape
    assert r.shape == (B, N) and c.shape == (B, N) and hv.shape == (H,)
    dQ, dK, dV = np.empty_like(Q), np.empty_like(Q), np.empty_like(Q)
    rc = _load().oracle_bwd(_p(Q), _p(K), _p(V), _p(dO), _p(r), _p(c), C.c_int(B), C.c_int(H),
                            C.c_int(N), C.c_int(d), C.c_int(P), _p(hv), C.c_double(scale), C.c_int(radius),
                            C.c_int(_g(P, global_len)), _p(dQ), _p(dK), _p(dV))
    assert rc == 0
    return dQ, dK, dV


def plan(row_ids, col_ids, P, view, max_id):
    """Per-view stable order.  Returns perm, inv_perm int32 [B,N] and seg_off int32 [B,max_id+2]."""
    r, c = _i32(row_ids), _i32(col_ids)
    B, N = r.shape
    perm = np.empty((B, N), dtype=np.int32)
    inv = np.empty((B, N), dtype=np.int32)
    seg = np.empty((B, max_id + 2), dtype=np.int32)
    _load().oracle_plan(_p(r), _p(c), C.c_int(B), C.c_int(N), C.c_int(P), C.c_int(view),
                        C.c_int(max_id), _p(perm), _p(inv), _p(seg))
    return perm, inv, seg
