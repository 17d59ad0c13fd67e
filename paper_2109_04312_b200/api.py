"""ctypes binding of libmate.so (same names as the C entry points; marshalling only)."""
import ctypes as C
import os

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libmate.so")

IMPL_AUTO, IMPL_SIMT, IMPL_TCGEN05 = 0, 1, 2
FLAG_VIEW_ORDER, FLAG_BULK_TILES, FLAG_GATHER_TILES = 4, 8, 16   # or-ed to the implementation choice (see mate.h)
VIEW_ROW, VIEW_COL = 0, 1
_BF16, _F32 = 0, 1

_lib = None


class MateError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__("%s failed: %s (%d)" % (where, _status_string(status), status))


def library_path() -> str:
    """MATE_LIB (read when the library is first loaded) selects another build of the same library:
    the profiling build, libmate_trace.so."""
    return os.environ.get("MATE_LIB") or _LIB_PATH


def _load():
    """Loads the CUDA library; there is no fallback: a missing library is an error."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(
            "libmate.so is not built: run `python -m paper_2109_04312_b200.build` "
            "(needs nvcc); there is no CPU or PyTorch fallback")
    lib = C.CDLL(path)
    vp, i32, u32, f32, sz = C.c_void_p, C.c_int, C.c_uint, C.c_float, C.c_size_t
    lib.mate_status_string.restype = C.c_char_p
    lib.mate_status_string.argtypes = [i32]
    lib.mate_plan.restype = i32
    lib.mate_plan.argtypes = [vp, vp, i32, i32, i32, vp, i32, i32, i32, vp, C.POINTER(vp)]
    lib.mate_plan_bucketed.restype = i32
    lib.mate_plan_bucketed.argtypes = [vp, vp, i32, i32, i32, vp, i32, i32, i32, i32, vp, C.POINTER(vp)]
    lib.mate_plan_varlen.restype = i32
    lib.mate_plan_varlen.argtypes = [vp, vp, i32, i32, vp, vp, i32, i32, i32, i32, vp, C.POINTER(vp)]
    lib.mate_plan_packed.restype = i32
    lib.mate_plan_packed.argtypes = [vp, vp, i32, vp, vp, vp, i32, i32, i32, vp, C.POINTER(vp)]
    lib.mate_plan_bucketed_global.restype = i32
    lib.mate_plan_bucketed_global.argtypes = [vp, vp, i32, i32, vp, vp, vp, i32, i32, i32, i32, vp, C.POINTER(vp)]
    lib.mate_plan_sat.restype = i32
    lib.mate_plan_sat.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32, vp, C.POINTER(vp)]
    lib.mate_plan_get.restype = i32
    lib.mate_plan_get.argtypes = [vp, i32, vp, vp, vp]
    lib.mate_plan_useful_pairs.restype = i32
    lib.mate_plan_useful_pairs.argtypes = [vp, vp]
    lib.mate_plan_status.restype = i32
    lib.mate_plan_status.argtypes = [vp, vp]
    lib.mate_debug_expire_wait.restype = i32
    lib.mate_debug_expire_wait.argtypes = [vp, vp]
    lib.mate_plan_destroy.restype = i32
    lib.mate_plan_destroy.argtypes = [vp]
    lib.mate_attn_workspace_bytes.restype = i32
    lib.mate_attn_workspace_bytes.argtypes = [vp, i32, i32, u32, C.POINTER(sz), C.POINTER(sz)]
    lib.mate_attn_fwd.restype = i32
    lib.mate_attn_fwd.argtypes = [vp, vp, vp, vp, i32, i32, f32, vp, vp, vp, sz, u32, vp]
    lib.mate_attn_bwd.restype = i32
    lib.mate_attn_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, vp, vp, vp, vp, sz, u32, vp]
    lib.mate_cell_mean.restype = i32
    lib.mate_cell_mean.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.mate_attn_bwd_noalloc.restype = i32
    lib.mate_attn_bwd_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, vp, vp, vp, vp]
    _lib = lib
    return lib


def _status_string(status):
    try:
        return _load().mate_status_string(status).decode()
    except Exception:
        return "?"


def _check(status, where):
    if status != 0:
        raise MateError(status, where)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype_code(t):
    if t.dtype == torch.bfloat16:
        return _BF16
    if t.dtype == torch.float32:
        return _F32
    raise TypeError("libmate takes bfloat16 or float32 tensors, got %s" % t.dtype)


def _dev(t, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
        raise ValueError("%s must be a contiguous CUDA tensor" % name)
    return C.c_void_p(t.data_ptr())


class Plan:
    """Owner of a mate_plan_t*: the pre-computed per-view order (see mate_plan)."""

    def __init__(self, handle, B, N, P, H, max_row_id, max_col_id, device):
        self._h = handle
        self.B, self.N, self.P, self.H = B, N, P, H
        self.max_id = (max_row_id, max_col_id)
        self.device = device
        self.T = None          # packed plans: total number of tokens (tensors are [H, T, d])
        self._ws = {}

    def _split(self, Q):
        """Checks a tensor's shape against the plan; returns (d, shape of the row statistic)."""
        if self.T is not None:
            if Q.dim() != 3 or tuple(Q.shape[:2]) != (self.H, self.T):
                raise ValueError("a packed plan takes [H, T, d] tensors")
            return Q.shape[2], (self.H, self.T)
        if Q.dim() != 4 or tuple(Q.shape[:3]) != (self.B, self.H, self.N):
            raise ValueError("tensor shapes do not match the plan")
        return Q.shape[3], (self.B, self.H, self.N)

    def get(self, view):
        """(perm, inv_perm, seg_off) of one view as numpy int32 arrays."""
        perm = np.empty((self.B, self.N), np.int32)
        inv = np.empty((self.B, self.N), np.int32)
        seg = np.empty((self.B, self.max_id[view] + 2), np.int32)
        _check(_load().mate_plan_get(self._h, view, perm.ctypes.data, inv.ctypes.data, seg.ctypes.data),
               "mate_plan_get")
        return perm, inv, seg

    def useful_pairs(self):
        out = np.empty((self.B, self.H), np.int64)
        _check(_load().mate_plan_useful_pairs(self._h, out.ctypes.data), "mate_plan_useful_pairs")
        return out

    def status(self):
        _check(_load().mate_plan_status(self._h, _stream()), "mate_plan_status")

    def debug_expire_wait(self):
        """Test hook: makes a bounded device wait give up (see mate_debug_expire_wait in mate.h)."""
        _check(_load().mate_debug_expire_wait(self._h, _stream()), "mate_debug_expire_wait")

    def destroy(self):
        if self._h is not None:
            _load().mate_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def mate_plan_bucketed(row_ids, col_ids, prefix_len, head_view, radius, max_row_id=None, max_col_id=None) -> Plan:
    """Plan of the bucketed variant (see mate_plan_bucketed in mate.h); radius = 0 is the exact pattern."""
    return mate_plan(row_ids, col_ids, prefix_len, head_view, max_row_id, max_col_id, radius=radius)


def mate_plan_packed(row_ids, col_ids, cu_seqlens, prefix_lens, head_view, max_row_id=None, max_col_id=None) -> Plan:
    """Plan of a packed batch (see mate_plan_packed in mate.h): row_ids, col_ids are int32 CUDA tensors [T],
    example b owning the tokens cu_seqlens[b] .. cu_seqlens[b + 1] - 1; Q, K, V, O and the gradients are then
    [H, T, d] and LSE is [H, T]."""
    if row_ids.dtype != torch.int32 or col_ids.dtype != torch.int32 or row_ids.shape != col_ids.shape \
            or row_ids.dim() != 1:
        raise ValueError("row_ids / col_ids must be int32 tensors of the same [T] shape")
    cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
    pf = np.ascontiguousarray(np.asarray(prefix_lens, dtype=np.int32))
    B = int(pf.shape[0])
    if cu.shape != (B + 1,) or int(cu[-1]) != int(row_ids.shape[0]):
        raise ValueError("cu_seqlens must have B + 1 entries and end at T")
    hv = np.ascontiguousarray(np.asarray(head_view, dtype=np.uint8))
    if max_row_id is None:
        max_row_id = max(int(row_ids.max().item()), 0) if row_ids.numel() else 0
    if max_col_id is None:
        max_col_id = max(int(col_ids.max().item()), 0) if col_ids.numel() else 0
    handle = C.c_void_p()
    with torch.cuda.device(row_ids.device):
        _check(_load().mate_plan_packed(_dev(row_ids, "row_ids"), _dev(col_ids, "col_ids"), B, cu.ctypes.data,
                                        pf.ctypes.data, hv.ctypes.data, int(hv.shape[0]), int(max_row_id),
                                        int(max_col_id), _stream(), C.byref(handle)), "mate_plan_packed")
    n_max = max(int(np.diff(cu).max()), 1)
    plan = Plan(handle, B, n_max, pf.tolist(), int(hv.shape[0]), int(max_row_id), int(max_col_id), row_ids.device)
    plan.T = int(cu[-1])
    return plan


def mate_plan_varlen(row_ids, col_ids, prefix_lens, head_view, radius=0, max_row_id=None, max_col_id=None) -> Plan:
    """Plan with one prefix length per example (see mate_plan_varlen in mate.h): prefix_lens has B entries."""
    return mate_plan(row_ids, col_ids, [int(x) for x in prefix_lens], head_view, max_row_id, max_col_id,
                     radius=radius)


def mate_plan(row_ids, col_ids, prefix_len, head_view, max_row_id=None, max_col_id=None, radius=0) -> Plan:
    """row_ids, col_ids: int32 CUDA tensors [B, N]; head_view: sequence of 0 (row) / 1 (column);
    prefix_len: one int, or a list of B ints (one per example)."""
    if row_ids.dtype != torch.int32 or col_ids.dtype != torch.int32 or row_ids.shape != col_ids.shape \
            or row_ids.dim() != 2:
        raise ValueError("row_ids / col_ids must be int32 tensors of the same [B, N] shape")
    B, N = row_ids.shape
    hv = np.ascontiguousarray(np.asarray(head_view, dtype=np.uint8))
    if max_row_id is None:
        max_row_id = max(int(row_ids.max().item()), 0)
    if max_col_id is None:
        max_col_id = max(int(col_ids.max().item()), 0)
    handle = C.c_void_p()
    with torch.cuda.device(row_ids.device):
        lib = _load()
        common = (_dev(row_ids, "row_ids"), _dev(col_ids, "col_ids"), B, N)
        tail = (hv.ctypes.data, int(hv.shape[0]), int(max_row_id), int(max_col_id))
        if isinstance(prefix_len, (list, tuple, np.ndarray)):
            pf = np.ascontiguousarray(np.asarray(prefix_len, dtype=np.int32))
            if pf.shape != (B,):
                raise ValueError("prefix_len must have one entry per example")
            _check(lib.mate_plan_varlen(*common, pf.ctypes.data, *tail, int(radius), _stream(), C.byref(handle)),
                   "mate_plan_varlen")
            prefix_len = pf.tolist()
        elif radius:
            _check(lib.mate_plan_bucketed(*common, int(prefix_len), *tail, int(radius), _stream(),
                                          C.byref(handle)), "mate_plan_bucketed")
        else:
            _check(lib.mate_plan(*common, int(prefix_len), *tail, _stream(), C.byref(handle)), "mate_plan")
    return Plan(handle, B, N, prefix_len, int(hv.shape[0]), int(max_row_id), int(max_col_id), row_ids.device)


def mate_plan_bucketed_global(row_ids, col_ids, prefix_lens, global_lens, head_view, radius, max_row_id=None,
                              max_col_id=None) -> Plan:
    """Bucketed plan whose global section (global_lens[b] >= prefix_lens[b] positions of every head's own order)
    may reach beyond the prefix (see mate_plan_bucketed_global in mate.h).  Scalars are taken for every example."""
    B, N = row_ids.shape
    pf = np.ascontiguousarray(np.broadcast_to(np.asarray(prefix_lens, dtype=np.int32), (B,)))
    gl = np.ascontiguousarray(np.broadcast_to(np.asarray(global_lens, dtype=np.int32), (B,)))
    hv = np.ascontiguousarray(np.asarray(head_view, dtype=np.uint8))
    if max_row_id is None:
        max_row_id = max(int(row_ids.max().item()), 0)
    if max_col_id is None:
        max_col_id = max(int(col_ids.max().item()), 0)
    handle = C.c_void_p()
    with torch.cuda.device(row_ids.device):
        _check(_load().mate_plan_bucketed_global(_dev(row_ids, "row_ids"), _dev(col_ids, "col_ids"), B, N, pf.ctypes.data,
                                                 gl.ctypes.data, hv.ctypes.data, int(hv.shape[0]), int(max_row_id),
                                                 int(max_col_id), int(radius), _stream(), C.byref(handle)),
               "mate_plan_bucketed_global")
    return Plan(handle, B, N, pf.tolist(), int(hv.shape[0]), int(max_row_id), int(max_col_id), row_ids.device)


def mate_plan_sat(row_ids, col_ids, prefix_len, n_heads, max_row_id=None, max_col_id=None) -> Plan:
    """Plan of the head-independent row-or-column pattern (see mate_plan_sat in mate.h)."""
    if row_ids.dtype != torch.int32 or col_ids.dtype != torch.int32 or row_ids.shape != col_ids.shape \
            or row_ids.dim() != 2:
        raise ValueError("row_ids / col_ids must be int32 tensors of the same [B, N] shape")
    B, N = row_ids.shape
    if max_row_id is None:
        max_row_id = max(int(row_ids.max().item()), 0)
    if max_col_id is None:
        max_col_id = max(int(col_ids.max().item()), 0)
    handle = C.c_void_p()
    with torch.cuda.device(row_ids.device):
        _check(_load().mate_plan_sat(_dev(row_ids, "row_ids"), _dev(col_ids, "col_ids"), B, N, int(prefix_len),
                                     int(n_heads), int(max_row_id), int(max_col_id), _stream(), C.byref(handle)),
               "mate_plan_sat")
    return Plan(handle, B, N, prefix_len, int(n_heads), int(max_row_id), int(max_col_id), row_ids.device)


def mate_attn_workspace_bytes(plan, d, dtype, impl=IMPL_AUTO):
    f, b = C.c_size_t(0), C.c_size_t(0)
    _check(_load().mate_attn_workspace_bytes(plan._h, int(d), dtype, impl, C.byref(f), C.byref(b)),
           "mate_attn_workspace_bytes")
    return f.value, b.value


def _workspace(plan, nbytes, key):
    if nbytes == 0:
        return None
    ws = plan._ws.get(key)
    if ws is None or ws.numel() < nbytes:
        ws = torch.empty(nbytes, dtype=torch.uint8, device=plan.device)
        plan._ws[key] = ws
    return ws


def mate_attn_fwd(plan, Q, K, V, scale=None, impl=IMPL_AUTO, out=None, lse=None, workspace=None):
    """Q, K, V: [B, H, N, d] CUDA tensors (bf16 or f32), or [H, T, d] for a packed plan.  Returns (O, LSE)
    in original token order."""
    d, stat_shape = plan._split(Q)
    if K.shape != Q.shape or V.shape != Q.shape:
        raise ValueError("tensor shapes do not match the plan")
    dt = _dtype_code(Q)
    if scale is None:
        scale = 1.0 / float(d) ** 0.5
    O = torch.empty_like(Q) if out is None else out
    LSE = torch.empty(stat_shape, dtype=torch.float32, device=Q.device) if lse is None else lse
    need, _ = mate_attn_workspace_bytes(plan, d, dt, impl)
    ws = workspace if workspace is not None else _workspace(plan, need, "fwd")
    with torch.cuda.device(Q.device):
        _check(_load().mate_attn_fwd(plan._h, _dev(Q, "Q"), _dev(K, "K"), _dev(V, "V"), d, dt,
                                     float(scale), _dev(O, "O"), _dev(LSE, "LSE"),
                                     C.c_void_p(ws.data_ptr()) if ws is not None else None,
                                     ws.numel() if ws is not None else 0, impl, _stream()),
               "mate_attn_fwd")
    return O, LSE


def mate_attn_bwd(plan, Q, K, V, O, LSE, dO, scale=None, impl=IMPL_AUTO, workspace=None):
    """Returns (dQ, dK, dV)."""
    d, _ = plan._split(Q)
    for t in (K, V, O, dO):
        if t.shape != Q.shape or t.dtype != Q.dtype:
            raise ValueError("K, V, O, dO must match Q in shape and dtype")
    dt = _dtype_code(Q)
    if scale is None:
        scale = 1.0 / float(d) ** 0.5
    dQ, dK, dV = torch.empty_like(Q), torch.empty_like(Q), torch.empty_like(Q)
    _, need = mate_attn_workspace_bytes(plan, d, dt, impl)
    ws = workspace if workspace is not None else _workspace(plan, need, "bwd")
    with torch.cuda.device(Q.device):
        _check(_load().mate_attn_bwd(plan._h, _dev(Q, "Q"), _dev(K, "K"), _dev(V, "V"), _dev(O, "O"),
                                     _dev(LSE, "LSE"), _dev(dO, "dO"), d, dt, float(scale),
                                     _dev(dQ, "dQ"), _dev(dK, "dK"), _dev(dV, "dV"),
                                     C.c_void_p(ws.data_ptr()) if ws is not None else None,
                                     ws.numel() if ws is not None else 0, impl, _stream()),
               "mate_attn_bwd")
    return dQ, dK, dV


def mate_cell_mean(plan, logits, col_ids, want_count=True, out=None):
    """Mean of the token logits per table cell (see mate_cell_mean in mate.h).  logits: float32 [B, N];
    col_ids: the int32 [B, N] tensor the plan was made from.  Returns (mean, count) of shape
    [B, max_row_id + 1, max_col_id + 1] (count is None when not wanted)."""
    if logits.dtype != torch.float32 or tuple(logits.shape) != (plan.B, plan.N):
        raise ValueError("logits must be a float32 [B, N] tensor")
    if col_ids.dtype != torch.int32 or tuple(col_ids.shape) != (plan.B, plan.N):
        raise ValueError("col_ids must be the int32 [B, N] tensor given to mate_plan")
    shape = (plan.B, plan.max_id[0] + 1, plan.max_id[1] + 1)
    if out is not None:  # (mean, count) tensors of an earlier call, written in place
        mean, count = out
        want_count = count is not None
    else:
        mean = torch.empty(shape, dtype=torch.float32, device=logits.device)
        count = torch.empty(shape, dtype=torch.int32, device=logits.device) if want_count else None
    with torch.cuda.device(logits.device):
        _check(_load().mate_cell_mean(plan._h, _dev(logits, "logits"), _dev(col_ids, "col_ids"), _dev(mean, "mean"),
                                      _dev(count, "count") if want_count else None, _stream()), "mate_cell_mean")
    return mean, count


def mate_attn_bwd_noalloc(plan, Q, K, V, O, LSE, dO, dQ, dK, dV, scale=None):
    """Backward for callers that may not allocate device memory (for example inside a loop whose
    framework owns every byte of the device): the caller passes the three output tensors and the
    library uses its built-in scratch array, so neither this function nor the C entry point
    allocates anything.  B*H*N is limited to 1,048,576.  Calls must not overlap on the GPU."""
    d, _ = plan._split(Q)
    for t in (K, V, O, dO, dQ, dK, dV):
        if t.shape != Q.shape or t.dtype != Q.dtype:
            raise ValueError("K, V, O, dO, dQ, dK, dV must match Q in shape and dtype")
    if scale is None:
        scale = 1.0 / float(d) ** 0.5
    with torch.cuda.device(Q.device):
        _check(_load().mate_attn_bwd_noalloc(plan._h, _dev(Q, "Q"), _dev(K, "K"), _dev(V, "V"),
                                             _dev(O, "O"), _dev(LSE, "LSE"), _dev(dO, "dO"), d,
                                             _dtype_code(Q), float(scale), _dev(dQ, "dQ"),
                                             _dev(dK, "dK"), _dev(dV, "dV"), _stream()),
               "mate_attn_bwd_noalloc")
    return dQ, dK, dV
