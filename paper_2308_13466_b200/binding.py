"""ctypes binding of libsat_b200.so: one Python function per C entry point, same names.

Argument marshalling only — every step of the path runs in the library's CUDA kernels.
Device tensors are torch CUDA tensors (fp32, last dimension contiguous); their row
stride is passed as the leading dimension.  Host arrays are numpy arrays.
There is no CPU fallback: importing this module fails loudly when the library is
missing or cannot be loaded.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from .build import lib_path

SAT_OK, SAT_EINVAL, SAT_ESTATE, SAT_ENOMEM, SAT_ECUDA, SAT_EDATA = 0, -1, -2, -3, -4, -5
SAT_HOST, SAT_DEVICE = 0, 1
SAT_ALL_PARTS = -1
SAT_PART_GIVEN, SAT_PART_CONTIG_BLOCKS, SAT_PART_BFS_BLOCKS = 0, 1, 2
SAT_ACT_NONE, SAT_ACT_RELU = 0, 1
SAT_LOSS_SOFTMAX_CE, SAT_LOSS_SIGMOID_BCE = 0, 1
SAT_BWD_ACCUMULATE, SAT_BWD_MASK_G_IN, SAT_BWD_G_OUT_MASKED, SAT_BWD_GRAD_HISTORY = 1, 2, 4, 8
SAT_FWD_PUSH = 0x100
SAT_FWD_HALO_GLOBAL = 0x200
SAT_FWD_INPUT_GLOBAL = 0x400
SAT_ROWS_INNER, SAT_ROWS_HALO = 0, 1
SAT_CACHE_ZERO, SAT_CACHE_COPY = 0, 1

_STATUS_NAMES = {0: "SAT_OK", -1: "SAT_EINVAL", -2: "SAT_ESTATE", -3: "SAT_ENOMEM", -4: "SAT_ECUDA", -5: "SAT_EDATA"}


class SatError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{_STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class sat_pred_params(C.Structure):
    _fields_ = [("Wx", C.c_void_p), ("Uh", C.c_void_p), ("b", C.c_void_p), ("Wg", C.c_void_p), ("bg", C.c_void_p),
                ("h", C.c_int32), ("cell", C.c_int32), ("version", C.c_uint64)]


SAT_CELL_LSTM, SAT_CELL_GRU = 0, 1


def _load():
    # SAT_B200_DEBUG=1 selects the bounds-checking build of the same sources (libsat_b200_dbg.so)
    path = lib_path(debug=os.environ.get("SAT_B200_DEBUG", "0") == "1")
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2308_13466_b200.build` "
                          "(there is no fallback implementation)")
    lib = C.CDLL(path)
    lib.sat_last_error.restype = C.c_char_p
    lib.sat_last_error.argtypes = [C.c_void_p]
    return lib


_lib = _load()

# every symbol the header declares
EXPORTS = [
    "sat_create", "sat_destroy", "sat_last_error", "sat_sync_status", "sat_graph_load", "sat_graph_dinv", "sat_partition",
    "sat_part_sizes", "sat_part_lists", "sat_slot_map", "sat_gather_rows", "sat_cache_init", "sat_predict",
    "sat_predict_state", "sat_layer_fwd", "sat_layer_bwd", "sat_cache_update", "sat_cache_commit", "sat_cache_state",
    "sat_cache_read", "sat_cache_export", "sat_cache_import", "sat_cache_set_state", "sat_loss_grad", "sat_sgd_step", "sat_sgd_steps",
    "sat_dense_nn", "sat_dense_nt", "sat_dense_tn", "sat_dense_tn_static", "sat_launch_count", "sat_profile_families", "sat_profile_enable", "sat_profile_select", "sat_profile_read",
    "sat_codec_plan", "sat_codec_encode", "sat_codec_decode", "sat_cache_requantise", "sat_staleness", "sat_pred_grad", "sat_grad_history_read", "sat_grad_history_write", "sat_gat_fwd", "sat_gat_bwd", "sat_gat_scores", "sat_profile_l2_rates", "sat_debug_poke_index", "sat_spmm_plan",
]


def _check(ctx, status):
    if status != SAT_OK:
        msg = _lib.sat_last_error(ctx).decode() if ctx else "no context"
        raise SatError(status, msg)


def _dev(t):
    """Device pointer of a torch CUDA tensor (or None)."""
    if t is None:
        return None
    assert t.is_cuda, "expected a CUDA tensor"
    return C.c_void_p(t.data_ptr())


def _ld(t):
    """Leading dimension (row stride in elements) of a 2-D tensor whose rows are contiguous."""
    assert t.dim() == 2 and (t.shape[1] <= 1 or t.stride(1) == 1)
    return int(t.stride(0)) if t.shape[0] > 1 else max(int(t.stride(0)), int(t.shape[1]))


def _host(a, dtype):
    if a is None:
        return None, None
    a = np.ascontiguousarray(a, dtype=dtype)
    return a, a.ctypes.data_as(C.c_void_p)


# --------------------------------------------------------------------------------------
def sat_create(device: int = 0, stream: int = 0):
    ctx = C.c_void_p()
    st = _lib.sat_create(C.byref(ctx), C.c_int(device), C.c_void_p(stream))
    if st != SAT_OK:
        raise SatError(st, "sat_create failed")
    return ctx


def sat_destroy(ctx):
    _check(None, _lib.sat_destroy(ctx))


def sat_last_error(ctx) -> str:
    return _lib.sat_last_error(ctx).decode()


def sat_sync_status(ctx):
    _check(ctx, _lib.sat_sync_status(ctx))


def sat_graph_load(ctx, rowptr, col, n=None, ptr_space=None):
    """rowptr / col: numpy arrays (host) or torch CUDA tensors (device)."""
    if isinstance(rowptr, np.ndarray):
        rp, rpp = _host(rowptr, np.int64)
        cl, clp = _host(col, np.int32)
        n = rp.shape[0] - 1 if n is None else n
        nnz = cl.shape[0]
        space = SAT_HOST
    else:
        rpp, clp = _dev(rowptr), _dev(col)
        n = rowptr.shape[0] - 1 if n is None else n
        nnz = col.shape[0]
        space = SAT_DEVICE
    if ptr_space is not None:
        space = ptr_space
    _check(ctx, _lib.sat_graph_load(ctx, C.c_int32(n), C.c_int64(nnz), rpp, clp, C.c_int(space)))


def sat_graph_dinv(ctx, n: int) -> np.ndarray:
    out = np.empty(n, dtype=np.float32)
    _check(ctx, _lib.sat_graph_dinv(ctx, out.ctypes.data_as(C.c_void_p)))
    return out


def sat_partition(ctx, M: int, method: int, part_of_node=None):
    if part_of_node is None:
        ptr, space = None, SAT_HOST
    elif isinstance(part_of_node, np.ndarray):
        keep, ptr = _host(part_of_node, np.int32)
        space = SAT_HOST
    else:
        ptr, space = _dev(part_of_node), SAT_DEVICE
    _check(ctx, _lib.sat_partition(ctx, C.c_int32(M), C.c_int(method), ptr, C.c_int(space)))


def sat_part_sizes(ctx, m: int):
    """(n_inner, n_halo, nnz_local, n_push, nnz_hrow)"""
    ni, nh, npush = C.c_int32(), C.c_int32(), C.c_int32()
    nl, nhr = C.c_int64(), C.c_int64()
    _check(ctx, _lib.sat_part_sizes(ctx, C.c_int32(m), C.byref(ni), C.byref(nh), C.byref(nl), C.byref(npush), C.byref(nhr)))
    return ni.value, nh.value, nl.value, npush.value, nhr.value


def sat_part_lists(ctx, m: int) -> dict:
    ni, nh, nl, npush, nhr = sat_part_sizes(ctx, m)
    out = dict(
        inner_gid=np.empty(ni, np.int32), halo_gid=np.empty(nh, np.int32), halo_slot=np.empty(nh, np.int32),
        push_local=np.empty(npush, np.int32), push_slot=np.empty(npush, np.int32),
        loc_rowptr=np.empty(ni + 1, np.int64), loc_col=np.empty(nl, np.int32),
        hrow_ptr=np.empty(nh + 1, np.int64), hrow_col=np.empty(nhr, np.int32))
    p = lambda k: out[k].ctypes.data_as(C.c_void_p)
    _check(ctx, _lib.sat_part_lists(ctx, C.c_int32(m), p("inner_gid"), p("halo_gid"), p("halo_slot"), p("push_local"),
                                    p("push_slot"), p("loc_rowptr"), p("loc_col"), p("hrow_ptr"), p("hrow_col")))
    return out


def sat_slot_map(ctx, n: int):
    """(part[n], slot[n], n_slots)"""
    part = np.empty(n, np.int32)
    slot = np.empty(n, np.int32)
    ns = C.c_int32()
    _check(ctx, _lib.sat_slot_map(ctx, part.ctypes.data_as(C.c_void_p), slot.ctypes.data_as(C.c_void_p), C.byref(ns)))
    return part, slot, ns.value


def sat_gather_rows(ctx, part: int, which: int, x, out):
    _check(ctx, _lib.sat_gather_rows(ctx, C.c_int32(part), C.c_int(which), _dev(x), C.c_int32(_ld(x)), C.c_int32(x.shape[1]),
                                     _dev(out), C.c_int32(_ld(out))))


def sat_cache_init(ctx, widths, tau: int, mode: int = SAT_CACHE_ZERO, init=None):
    n = len(widths)
    w = (C.c_int32 * max(n, 1))(*widths)
    arr = None
    if init is not None:
        arr = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in init])
    _check(ctx, _lib.sat_cache_init(ctx, C.c_int32(n), w, C.c_int32(tau), C.c_int(mode), arr))


def make_pred_params(Wx, Uh, b, Wg, bg, h: int, version: int = 0, cell: int = 0) -> sat_pred_params:
    """version != 0 promises that the values of all five arrays stay the same for as long as the same version is passed.
    cell: SAT_CELL_LSTM (Wx [d, 4h], Uh [h, 4h], b [4h]) or SAT_CELL_GRU (Wx [d, 3h], Uh [h, 3h], b [4h])."""
    for t in (Wx, Uh, b, Wg, bg):
        assert t.is_cuda and t.is_contiguous()
    gates = 3 if cell == SAT_CELL_GRU else 4
    assert Wx.shape[1] == gates * h and tuple(Uh.shape) == (h, gates * h) and b.numel() == 4 * h
    p = sat_pred_params(Wx.data_ptr(), Uh.data_ptr(), b.data_ptr(), Wg.data_ptr(), bg.data_ptr(), h, cell, version)
    p._keep = (Wx, Uh, b, Wg, bg)
    return p


def sat_predict(ctx, layer: int, part: int, params, reuse_state: int, halo_out):
    pp = None if params is None else C.byref(params)
    _check(ctx, _lib.sat_predict(ctx, C.c_int32(layer), C.c_int32(part), pp, C.c_int(reuse_state), _dev(halo_out),
                                 C.c_int32(_ld(halo_out))))


def sat_predict_state(ctx, layer: int, n_slots: int, h: int) -> np.ndarray:
    out = np.empty((n_slots, h), np.float32)
    _check(ctx, _lib.sat_predict_state(ctx, C.c_int32(layer), out.ctypes.data_as(C.c_void_p), C.c_int32(h)))
    return out


def sat_layer_fwd(ctx, part: int, layer: int, h_in, h_halo, W, bias, act: int, h_out):
    d_in, d_out = int(W.shape[0]), int(W.shape[1])
    assert W.is_contiguous() and (bias is None or bias.is_contiguous())
    _check(ctx, _lib.sat_layer_fwd(ctx, C.c_int32(part), C.c_int32(layer), C.c_int32(d_in), C.c_int32(d_out),
                                   _dev(h_in), C.c_int32(_ld(h_in)),
                                   _dev(h_halo), C.c_int32(_ld(h_halo) if h_halo is not None else 0),
                                   _dev(W), _dev(bias), C.c_int(act), _dev(h_out), C.c_int32(_ld(h_out))))


def sat_layer_bwd(ctx, part: int, layer: int, g_out, W, g_W, g_b, accumulate: int, g_in=None, g_halo=None):
    assert W.is_contiguous() and g_W.is_contiguous()
    _check(ctx, _lib.sat_layer_bwd(ctx, C.c_int32(part), C.c_int32(layer), _dev(g_out), C.c_int32(_ld(g_out)), _dev(W),
                                   _dev(g_W), _dev(g_b), C.c_int(accumulate),
                                   _dev(g_in), C.c_int32(_ld(g_in) if g_in is not None else 0),
                                   _dev(g_halo), C.c_int32(_ld(g_halo) if g_halo is not None else 0)))


def sat_cache_update(ctx, part: int, layer: int, h_out):
    _check(ctx, _lib.sat_cache_update(ctx, C.c_int32(part), C.c_int32(layer), _dev(h_out), C.c_int32(_ld(h_out))))


def sat_cache_commit(ctx):
    _check(ctx, _lib.sat_cache_commit(ctx))


def sat_cache_state(ctx):
    """(write_idx, n_valid)"""
    w, v = C.c_int32(), C.c_int32()
    _check(ctx, _lib.sat_cache_state(ctx, C.byref(w), C.byref(v)))
    return w.value, v.value


def sat_cache_set_state(ctx, write_idx: int, n_valid: int):
    _check(ctx, _lib.sat_cache_set_state(ctx, C.c_int32(write_idx), C.c_int32(n_valid)))


def sat_cache_read(ctx, layer: int, age: int, n_slots: int, width: int) -> np.ndarray:
    out = np.empty((n_slots, width), np.float32)
    _check(ctx, _lib.sat_cache_read(ctx, C.c_int32(layer), C.c_int32(age), out.ctypes.data_as(C.c_void_p)))
    return out


def sat_cache_export(ctx, layer: int, tau: int, n_slots: int, width: int) -> np.ndarray:
    out = np.empty((tau + 1, n_slots, width), np.float32)
    _check(ctx, _lib.sat_cache_export(ctx, C.c_int32(layer), out.ctypes.data_as(C.c_void_p)))
    return out


def sat_cache_import(ctx, layer: int, ring: np.ndarray):
    ring = np.ascontiguousarray(ring, dtype=np.float32)
    _check(ctx, _lib.sat_cache_import(ctx, C.c_int32(layer), ring.ctypes.data_as(C.c_void_p)))


def sat_loss_grad(ctx, part: int, kind: int, z, labels, loss_sum, g):
    """labels: int32 [n] (CE) or uint8 [n, C] (BCE) CUDA tensor; loss_sum: float64 CUDA scalar tensor or None."""
    _check(ctx, _lib.sat_loss_grad(ctx, C.c_int32(part), C.c_int(kind), C.c_int32(z.shape[1]), _dev(z), C.c_int32(_ld(z)),
                                   _dev(labels), _dev(loss_sum), _dev(g), C.c_int32(_ld(g))))


def sat_sgd_steps(ctx, ws, gs, lr: float):
    """w <- w - lr g for a list of (contiguous CUDA fp32) parameter tensors and their gradients, in one launch per 16."""
    n = len(ws)
    assert n == len(gs) and all(w.is_contiguous() and g.is_contiguous() and w.numel() == g.numel() for w, g in zip(ws, gs))
    counts = (C.c_int64 * n)(*[int(w.numel()) for w in ws])
    wp = (C.c_void_p * n)(*[w.data_ptr() for w in ws])
    gp = (C.c_void_p * n)(*[g.data_ptr() for g in gs])
    _check(ctx, _lib.sat_sgd_steps(ctx, C.c_int32(n), counts, wp, gp, C.c_float(lr)))


def sat_sgd_step(ctx, w, g, lr: float):
    assert w.is_contiguous() and g.is_contiguous() and w.numel() == g.numel()
    _check(ctx, _lib.sat_sgd_step(ctx, C.c_int64(w.numel()), _dev(w), _dev(g), C.c_float(lr)))


def sat_dense_nn(ctx, A, W, bias, out):
    """out[m, n] = A[m, k] W[k, n] + bias"""
    assert W.is_contiguous()
    _check(ctx, _lib.sat_dense_nn(ctx, C.c_int64(A.shape[0]), C.c_int32(W.shape[1]), C.c_int32(W.shape[0]), _dev(A), C.c_int32(_ld(A)),
                                  _dev(W), _dev(bias), _dev(out), C.c_int32(_ld(out))))


def sat_dense_nt(ctx, A, W, out):
    """out[m, n] = A[m, k] W[n, k]^T"""
    assert W.is_contiguous()
    _check(ctx, _lib.sat_dense_nt(ctx, C.c_int64(A.shape[0]), C.c_int32(W.shape[0]), C.c_int32(W.shape[1]), _dev(A), C.c_int32(_ld(A)),
                                  _dev(W), _dev(out), C.c_int32(_ld(out))))


def sat_dense_tn(ctx, A, Bm, out):
    """out[m, n] = A[rows, m]^T Bm[rows, n]  (out dense)"""
    assert out.is_contiguous()
    _check(ctx, _lib.sat_dense_tn(ctx, C.c_int64(A.shape[0]), C.c_int32(A.shape[1]), C.c_int32(Bm.shape[1]), _dev(A), C.c_int32(_ld(A)),
                                  _dev(Bm), C.c_int32(_ld(Bm)), _dev(out)))


def sat_pred_grad(ctx, layer: int, params, row_weight, g_Wx, g_Uh, g_b, g_Wg, g_bg, want_loss: bool = False):
    """Gradient of the predictor objective of cached layer `layer` into the CUDA fp32 arrays g_* (dense, shapes of the
    parameters); row_weight: CUDA fp32 [sum_m b_m] or None.  Returns the loss when want_loss (synchronises), else None."""
    loss = C.c_double(0.0)
    _check(ctx, _lib.sat_pred_grad(ctx, C.c_int32(layer), C.byref(params), _dev(row_weight), _dev(g_Wx), _dev(g_Uh), _dev(g_b),
                                   _dev(g_Wg), _dev(g_bg), C.byref(loss) if want_loss else None))
    return float(loss.value) if want_loss else None


def sat_grad_history_read(ctx, layer: int, which: int, n_slots: int, width: int) -> np.ndarray:
    """Committed (which = 0) or running (which = 1) gradient-side history of layer `layer` as a host array [n_slots, width]."""
    out = np.empty((n_slots, width), np.float32)
    _check(ctx, _lib.sat_grad_history_read(ctx, C.c_int32(layer), C.c_int(which), out.ctypes.data_as(C.c_void_p)))
    return out


def sat_grad_history_write(ctx, layer: int, width: int, hist):
    """hist: host array [n_slots, width] that becomes the committed history, or None to clear it."""
    if hist is None:
        _check(ctx, _lib.sat_grad_history_write(ctx, C.c_int32(layer), C.c_int32(width), None))
        return
    hist = np.ascontiguousarray(hist, dtype=np.float32)
    _check(ctx, _lib.sat_grad_history_write(ctx, C.c_int32(layer), C.c_int32(width), hist.ctypes.data_as(C.c_void_p)))


def sat_gat_fwd(ctx, part: int, layer: int, h_in, h_halo, W, a_src, a_dst, bias, act: int, h_out):
    """Graph-attention layer forward; all arguments CUDA fp32 tensors (2-D ones with row strides that are multiples of 4)."""
    d_in, d_out = int(W.shape[0]), int(W.shape[1])
    assert W.is_contiguous() and a_src.is_contiguous() and a_dst.is_contiguous() and (bias is None or bias.is_contiguous())
    _check(ctx, _lib.sat_gat_fwd(ctx, C.c_int32(part), C.c_int32(layer), C.c_int32(d_in), C.c_int32(d_out), _dev(h_in), C.c_int32(_ld(h_in)),
                                 _dev(h_halo), C.c_int32(_ld(h_halo) if h_halo is not None and h_halo.shape[0] else d_in + (-d_in) % 4),
                                 _dev(W), _dev(a_src), _dev(a_dst), _dev(bias), C.c_int(act), _dev(h_out), C.c_int32(_ld(h_out))))


def sat_gat_bwd(ctx, part: int, layer: int, g_out, h_out, h_in, h_halo, W, a_src, a_dst, g_W, g_a_src, g_a_dst, g_b, accumulate: int, g_in):
    d_in = int(W.shape[0])
    _check(ctx, _lib.sat_gat_bwd(ctx, C.c_int32(part), C.c_int32(layer), _dev(g_out), C.c_int32(_ld(g_out)), _dev(h_out),
                                 C.c_int32(_ld(h_out) if h_out is not None else 0), _dev(h_in), C.c_int32(_ld(h_in)), _dev(h_halo),
                                 C.c_int32(_ld(h_halo) if h_halo is not None and h_halo.shape[0] else d_in + (-d_in) % 4), C.c_int32(d_in),
                                 _dev(W), _dev(a_src), _dev(a_dst), _dev(g_W), _dev(g_a_src), _dev(g_a_dst), _dev(g_b), C.c_int(accumulate),
                                 _dev(g_in), C.c_int32(_ld(g_in) if g_in is not None else 0)))


def sat_gat_scores(ctx, layer: int, n: int, nb: int):
    """(s_src of the inner rows [n], s_dst [n], s_src of the halo positions [nb]) kept by sat_gat_fwd for `layer`."""
    s_in = np.empty(n, dtype=np.float32)
    s_dst = np.empty(n, dtype=np.float32)
    s_halo = np.empty(max(nb, 1), dtype=np.float32)
    _check(ctx, _lib.sat_gat_scores(ctx, C.c_int32(layer), s_in.ctypes.data_as(C.c_void_p), s_dst.ctypes.data_as(C.c_void_p),
                                    s_halo.ctypes.data_as(C.c_void_p)))
    return s_in, s_dst, s_halo[:nb]


def sat_staleness(ctx, part: int, h_fresh, h_used_halo, sq_sum):
    """sq_sum (CUDA float64 [1]) = squared Frobenius norm of (fresh embeddings of the halo nodes - embeddings used for them)."""
    d = int(h_used_halo.shape[1])
    _check(ctx, _lib.sat_staleness(ctx, C.c_int32(part), C.c_int32(d), _dev(h_fresh), C.c_int32(_ld(h_fresh)), _dev(h_used_halo),
                                   C.c_int32(_ld(h_used_halo)), _dev(sq_sum)))


def sat_codec_plan(ctx, x, precision: int, row_offsets):
    """Sizes of the encoded rows of x (CUDA fp32 [rows, d]): fills row_offsets (CUDA int64 [rows + 1]), returns the total."""
    total = C.c_int64(0)
    _check(ctx, _lib.sat_codec_plan(ctx, _dev(x), C.c_int32(_ld(x)), C.c_int64(x.shape[0]), C.c_int32(x.shape[1]), C.c_int32(precision),
                                    _dev(row_offsets), C.byref(total)))
    return int(total.value)


def sat_codec_encode(ctx, x, precision: int, row_offsets, out):
    """Writes the encoded rows of x into out (CUDA uint8, at least the planned total)."""
    _check(ctx, _lib.sat_codec_encode(ctx, _dev(x), C.c_int32(_ld(x)), C.c_int64(x.shape[0]), C.c_int32(x.shape[1]), C.c_int32(precision),
                                      _dev(row_offsets), _dev(out), C.c_int64(out.numel())))


def sat_codec_decode(ctx, data, row_offsets, precision: int, x):
    """Decodes rows into x (CUDA fp32 [rows, d]); malformed rows surface as SAT_EDATA from sat_sync_status."""
    _check(ctx, _lib.sat_codec_decode(ctx, _dev(data), C.c_int64(data.numel()), _dev(row_offsets), C.c_int64(x.shape[0]), C.c_int32(x.shape[1]), C.c_int32(precision),
                                      _dev(x), C.c_int32(_ld(x))))


def sat_cache_requantise(ctx, layer: int, age: int, precision: int) -> int:
    """Replaces committed snapshot `age` of cached layer `layer` by its encode + decode image; returns the encoded size."""
    total = C.c_int64(0)
    _check(ctx, _lib.sat_cache_requantise(ctx, C.c_int32(layer), C.c_int32(age), C.c_int32(precision), C.byref(total)))
    return int(total.value)


def sat_dense_tn_static(stream: int, A, Bm, out):
    """out[m, n] = A[rows, m]^T Bm[rows, n] without any allocation: the split partial sums live in an array built into the
    library (for callers that must not call cudaMalloc).  Needs no context; `stream` is a raw cudaStream_t (0 = default).
    Raises SatError with the library's message, e.g. when m * n exceeds the built-in scratch."""
    assert out.is_contiguous()
    err = C.create_string_buffer(256)
    st = _lib.sat_dense_tn_static(C.c_void_p(stream), C.c_int64(A.shape[0]), C.c_int32(A.shape[1]), C.c_int32(Bm.shape[1]), _dev(A),
                                  C.c_int32(_ld(A)), _dev(Bm), C.c_int32(_ld(Bm)), _dev(out), err, C.c_int32(256))
    if st != SAT_OK:
        raise SatError(st, err.value.decode())


def sat_launch_count(ctx) -> int:
    c = C.c_int64()
    _check(ctx, _lib.sat_launch_count(ctx, C.byref(c)))
    return c.value


def sat_debug_poke_index(ctx, which: int, pos: int, value: int) -> int:
    """Debug build only: overwrite one entry of an internal index array; returns the old value."""
    old = C.c_int32(0)
    _check(ctx, _lib.sat_debug_poke_index(ctx, C.c_int(which), C.c_int64(pos), C.c_int32(value), C.byref(old)))
    return int(old.value)


def sat_profile_l2_rates(ctx, row_floats: int):
    """(stream GB/s, random-row gather GB/s) out of an L2-resident 64 MiB buffer, measured now."""
    a, b = C.c_double(), C.c_double()
    _check(ctx, _lib.sat_profile_l2_rates(ctx, C.c_int32(row_floats), C.byref(a), C.byref(b)))
    return float(a.value), float(b.value)


def sat_spmm_plan(ctx, part: int, d: int):
    """(source blocks, work items, partial-sum rows) of the forward aggregation at width d for `part`."""
    nb, ni, ns = C.c_int32(), C.c_int64(), C.c_int64()
    _check(ctx, _lib.sat_spmm_plan(ctx, C.c_int32(part), C.c_int32(d), C.byref(nb), C.byref(ni), C.byref(ns)))
    return int(nb.value), int(ni.value), int(ns.value)


def sat_profile_families() -> int:
    return int(_lib.sat_profile_families())


def sat_profile_enable(ctx, enable: bool):
    _check(ctx, _lib.sat_profile_enable(ctx, C.c_int(1 if enable else 0)))


def sat_profile_select(ctx, names=None):
    """Restrict the per-family event bracketing to the named families (None = all of them)."""
    mask = (1 << 64) - 1
    if names is not None:
        order = []
        for f in range(sat_profile_families()):
            name = C.c_char_p()
            calls = C.c_int64()
            ms, by, fl = C.c_double(), C.c_double(), C.c_double()
            _check(ctx, _lib.sat_profile_read(ctx, C.c_int32(f), C.byref(name), C.byref(calls), C.byref(ms), C.byref(by), C.byref(fl)))
            order.append(name.value.decode())
        mask = 0
        for n in names:
            mask |= 1 << order.index(n)
    _check(ctx, _lib.sat_profile_select(ctx, C.c_uint64(mask)))


def sat_profile_read(ctx) -> dict:
    """{family name: dict(calls, ms, bytes, flops)} of the calls bracketed since sat_profile_enable(True)."""
    out = {}
    for f in range(sat_profile_families()):
        name = C.c_char_p()
        calls = C.c_int64()
        ms, by, fl = C.c_double(), C.c_double(), C.c_double()
        _check(ctx, _lib.sat_profile_read(ctx, C.c_int32(f), C.byref(name), C.byref(calls), C.byref(ms), C.byref(by), C.byref(fl)))
        out[name.value.decode()] = dict(calls=calls.value, ms=ms.value, bytes=by.value, flops=fl.value)
    return out
