"""ctypes binding of libslicegcn.so -- argument marshalling only.

Every function has the name of the C entry point it calls (see include/slicegcn.h for the
semantics) and raises SliceGCNError when the call returns a non-zero status.  Pointers may be
given as torch tensors (their data_ptr() is taken), numpy arrays (host memory), ints or None.
There is no Python or CPU fallback: importing this module fails loudly when the CUDA library
has not been built.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char, c_char_p, c_double, c_float, c_int32, c_int64, c_uint32, c_void_p
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libslicegcn.so")

OK, ERR_INVALID_ARG, ERR_OUT_OF_RANGE, ERR_OVERFLOW, ERR_ALLOC, ERR_CUDA, ERR_UNSUPPORTED = range(7)
F32, BF16 = 0, 1
ORDER_AUTO, AGG_FIRST, XFORM_FIRST = 0, 1, 2
RULE_CEIL, RULE_FLOOR_PLUS_1 = 0, 1
SYMMETRIZE, ADD_SELF_LOOPS, INPUT_ON_DEVICE, NORM_MEAN, NORM_SUM = 1, 2, 4, 8, 16
MAX_SLICES = 64
DEVSTATUS_BAD_LABEL = 32

EXPORTS = [
    "slicegcn_last_error", "slicegcn_slice_strategy", "slicegcn_graph_create", "slicegcn_graph_create_from_csr",
    "slicegcn_graph_info", "slicegcn_graph_export", "slicegcn_graph_device_status", "slicegcn_graph_destroy", "slicegcn_spmm_workspace_bytes",
    "slicegcn_spmm", "slicegcn_spmm_static_scratch", "slicegcn_layer_saved_bytes", "slicegcn_layer_saved_layout", "slicegcn_layer_workspace_bytes", "slicegcn_layer_forward",
    "slicegcn_layer_backward", "slicegcn_model_create", "slicegcn_model_destroy", "slicegcn_model_invalidate_caches", "slicegcn_model_param_count",
    "slicegcn_model_param_elems", "slicegcn_model_num_tensors", "slicegcn_model_tensor_info", "slicegcn_model_slices",
    "slicegcn_model_layer_order", "slicegcn_train_workspace_bytes", "slicegcn_train_epoch", "slicegcn_train_epoch_dropout", "slicegcn_train_epoch_sliced", "slicegcn_forward_logits", "slicegcn_train_epoch_host", "slicegcn_train_epochs_host", "slicegcn_profile_begin", "slicegcn_profile_begin_sampled",
    "slicegcn_profile_end",
]


class SliceGCNError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"slicegcn status {status}: {message}")
        self.status = status


class LayerDesc(ctypes.Structure):
    _fields_ = [("num_slices", c_int32), ("in_starts", POINTER(c_int32)), ("in_width", c_int32), ("in_cols", c_int32),
                ("in_ld", c_int64), ("h_s", c_int32), ("out_ld", c_int64), ("dtype", c_int32), ("order", c_int32),
                ("W_agg", c_void_p), ("W_self", c_void_p), ("b", c_void_p), ("b_self", c_void_p), ("E", c_void_p)]


class ModelDesc(ctypes.Structure):
    _fields_ = [("in_d", c_int32), ("hidden", c_int32), ("num_layers", c_int32), ("num_classes", c_int32),
                ("num_slices", c_int32), ("slice_size_scale", c_double), ("slice_rule", c_int32), ("use_ff", c_int32),
                ("use_se", c_int32), ("use_self", c_int32), ("use_b_self", c_int32), ("dtype", c_int32),
                ("order", c_int32), ("cache_input_aggregate", c_int32)]


class OptDesc(ctypes.Structure):
    _fields_ = [("lr0", c_double), ("beta1", c_double), ("beta2", c_double), ("eps", c_double),
                ("weight_decay", c_double), ("epoch", c_int32), ("total_epochs", c_int32)]


class DropoutDesc(ctypes.Structure):
    _fields_ = [("rate", c_double), ("masks", POINTER(c_void_p)), ("mask_ld", c_int64)]


def make_dropout_desc(rate: float, masks: Sequence, mask_ld: int) -> DropoutDesc:
    """masks: one device tensor (bytes, n x mask_ld) per layer but the last."""
    d = DropoutDesc()
    arr = (c_void_p * max(len(masks), 1))(*[_ptr(t) for t in masks])
    d._keep = (arr, list(masks))       # keep the pointer array and the tensors alive with the struct
    d.rate, d.masks, d.mask_ld = rate, ctypes.cast(arr, POINTER(c_void_p)), mask_ld
    return d


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it first (python -m paper_2408_11500_b200.build); "
                          "this package has no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    lib.slicegcn_last_error.restype = c_char_p
    for name in EXPORTS:
        if name != "slicegcn_last_error":
            getattr(lib, name).restype = c_int32
    return lib


_lib = _load()


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if isinstance(x, c_void_p):
        return x.value
    raise TypeError(f"cannot take a pointer from {type(x)}")


def _vp(x) -> c_void_p:
    return c_void_p(_ptr(x))


def _check(status: int):
    if status != OK:
        raise SliceGCNError(status, _lib.slicegcn_last_error().decode())


def slicegcn_last_error() -> str:
    return _lib.slicegcn_last_error().decode()


def slicegcn_slice_strategy(in_d: int, p: int, scale: float = 1.0, rule: int = RULE_CEIL) -> Tuple[List[Tuple[int, int]], int]:
    n = max(int(p), 1)
    starts = (c_int32 * n)()
    ends = (c_int32 * n)()
    size = c_int32()
    _check(_lib.slicegcn_slice_strategy(c_int32(in_d), c_int32(p), c_double(scale), c_int32(rule), starts, ends,
                                        byref(size)))
    return [(starts[i], ends[i]) for i in range(p)], size.value


# ------------------------------------------------------------------------------------------ graph

def slicegcn_graph_create(n: int, src, dst, flags: int, stream=None, n_edges: Optional[int] = None) -> c_void_p:
    if n_edges is None:
        n_edges = int(src.shape[0]) if src is not None else 0
    if isinstance(src, np.ndarray):
        assert src.dtype == np.int32 and dst.dtype == np.int32 and src.flags.c_contiguous and dst.flags.c_contiguous
    h = c_void_p()
    _check(_lib.slicegcn_graph_create(c_int64(n), c_int64(n_edges), _vp(src), _vp(dst), c_uint32(flags), _vp(stream),
                                      byref(h)))
    return h


def slicegcn_graph_create_from_csr(n: int, rowptr, colidx, flags: int, stream=None) -> c_void_p:
    h = c_void_p()
    _check(_lib.slicegcn_graph_create_from_csr(c_int64(n), _vp(rowptr), _vp(colidx), c_uint32(flags), _vp(stream),
                                               byref(h)))
    return h


def slicegcn_graph_info(g) -> Dict[str, int]:
    n, nnz, seg = c_int64(), c_int64(), c_int64()
    sym = c_int32()
    _check(_lib.slicegcn_graph_info(g, byref(n), byref(nnz), byref(sym), byref(seg)))
    return {"n": n.value, "nnz": nnz.value, "symmetric": bool(sym.value), "n_segments": seg.value}


def slicegcn_graph_export(g) -> Dict[str, np.ndarray]:
    info = slicegcn_graph_info(g)
    rowptr = np.empty(info["n"] + 1, np.int32)
    colidx = np.empty(max(info["nnz"], 1), np.int32)
    deg = np.empty(info["n"], np.int32)
    dinv = np.empty(info["n"], np.float32)
    _check(_lib.slicegcn_graph_export(g, _vp(rowptr), _vp(colidx), _vp(deg), _vp(dinv)))
    return {"rowptr": rowptr, "colidx": colidx[:info["nnz"]], "deg": deg, "dinv": dinv}


def slicegcn_graph_device_status(g) -> int:
    v = c_int32()
    _check(_lib.slicegcn_graph_device_status(g, byref(v)))
    return v.value


def slicegcn_graph_destroy(g) -> None:
    _check(_lib.slicegcn_graph_destroy(g))


# ------------------------------------------------------------------------------------------ spmm

def slicegcn_spmm_workspace_bytes(g, width: int) -> int:
    b = c_int64()
    _check(_lib.slicegcn_spmm_workspace_bytes(g, c_int32(width), byref(b)))
    return b.value


def slicegcn_spmm(g, transpose: int, in_dtype: int, out_dtype: int, X, ldx: int, Y, ldy: int, width: int,
                  workspace=None, workspace_bytes: int = 0, stream=None) -> None:
    _check(_lib.slicegcn_spmm(g, c_int32(transpose), c_int32(in_dtype), c_int32(out_dtype), _vp(X), c_int64(ldx), _vp(Y),
                              c_int64(ldy), c_int32(width), _vp(workspace), c_int64(workspace_bytes), _vp(stream)))


def slicegcn_spmm_static_scratch(g, transpose: int, in_dtype: int, out_dtype: int, X, ldx: int, Y, ldy: int, width: int,
                                 stream=None) -> None:
    """slicegcn_spmm for callers that cannot allocate: the hub-row scratch is an 8 MiB buffer built into the
    library (shared by all calls; overlapping calls race).  Raises SliceGCNError(ERR_UNSUPPORTED) when the graph
    and width need more."""
    _check(_lib.slicegcn_spmm_static_scratch(g, c_int32(transpose), c_int32(in_dtype), c_int32(out_dtype), _vp(X),
                                             c_int64(ldx), _vp(Y), c_int64(ldy), c_int32(width), _vp(stream)))


# ------------------------------------------------------------------------------------------ layer

def make_layer_desc(num_slices: int, in_starts: Sequence[int], in_width: int, in_cols: int, in_ld: int, h_s: int,
                    out_ld: int, dtype: int, order: int, W_agg, W_self=None, b=None, b_self=None, E=None) -> LayerDesc:
    d = LayerDesc()
    arr = (c_int32 * max(len(in_starts), 1))(*in_starts)
    d._keep = arr                      # keep the host array alive with the struct
    d.num_slices = num_slices
    d.in_starts = ctypes.cast(arr, POINTER(c_int32))
    d.in_width, d.in_cols, d.in_ld, d.h_s, d.out_ld = in_width, in_cols, in_ld, h_s, out_ld
    d.dtype, d.order = dtype, order
    d.W_agg, d.W_self, d.b, d.b_self, d.E = _ptr(W_agg), _ptr(W_self), _ptr(b), _ptr(b_self), _ptr(E)
    return d


def slicegcn_layer_saved_bytes(g, d: LayerDesc) -> int:
    b = c_int64()
    _check(_lib.slicegcn_layer_saved_bytes(g, byref(d), byref(b)))
    return b.value


def slicegcn_layer_saved_layout(g, d: LayerDesc) -> Dict[str, int]:
    zo, zl, mo, ml, zc = c_int64(), c_int64(), c_int64(), c_int64(), c_int32()
    _check(_lib.slicegcn_layer_saved_layout(g, byref(d), byref(zo), byref(zl), byref(zc), byref(mo), byref(ml)))
    return {"zt_offset": zo.value, "zt_ld": zl.value, "zt_cols": zc.value, "mask_offset": mo.value, "mask_ld": ml.value}


def slicegcn_layer_workspace_bytes(g, d: LayerDesc) -> int:
    b = c_int64()
    _check(_lib.slicegcn_layer_workspace_bytes(g, byref(d), byref(b)))
    return b.value


def slicegcn_layer_forward(g, d: LayerDesc, H_in, H_out, saved, saved_bytes: int, workspace, workspace_bytes: int,
                           stream=None) -> None:
    _check(_lib.slicegcn_layer_forward(g, byref(d), _vp(H_in), _vp(H_out), _vp(saved), c_int64(saved_bytes),
                                       _vp(workspace), c_int64(workspace_bytes), _vp(stream)))


def slicegcn_layer_backward(g, d: LayerDesc, H_in, saved, dH_out, dout_ld: int, dH_in, din_ld: int, dW_agg, dW_self,
                            db, db_self, dE, workspace, workspace_bytes: int, stream=None) -> None:
    _check(_lib.slicegcn_layer_backward(g, byref(d), _vp(H_in), _vp(saved), _vp(dH_out), c_int64(dout_ld), _vp(dH_in),
                                        c_int64(din_ld), _vp(dW_agg), _vp(dW_self), _vp(db), _vp(db_self), _vp(dE),
                                        _vp(workspace), c_int64(workspace_bytes), _vp(stream)))


# ------------------------------------------------------------------------------------------ model

def slicegcn_model_create(in_d: int, hidden: int, num_layers: int, num_classes: int, num_slices: int = 1,
                          slice_size_scale: float = 1.0, slice_rule: int = RULE_CEIL, use_ff: bool = False,
                          use_se: bool = False, use_self: bool = True, use_b_self: bool = False, dtype: int = F32,
                          order: int = ORDER_AUTO, cache_input_aggregate: bool = False) -> c_void_p:
    d = ModelDesc(in_d, hidden, num_layers, num_classes, num_slices, slice_size_scale, slice_rule, int(use_ff),
                  int(use_se), int(use_self), int(use_b_self), dtype, order, int(cache_input_aggregate))
    h = c_void_p()
    _check(_lib.slicegcn_model_create(byref(d), byref(h)))
    return h


def slicegcn_model_destroy(m) -> None:
    _check(_lib.slicegcn_model_destroy(m))


def slicegcn_model_invalidate_caches(m) -> None:
    _check(_lib.slicegcn_model_invalidate_caches(m))


def slicegcn_model_param_count(m) -> int:
    c = c_int64()
    _check(_lib.slicegcn_model_param_count(m, byref(c)))
    return c.value


def slicegcn_model_param_elems(m) -> int:
    c = c_int64()
    _check(_lib.slicegcn_model_param_elems(m, byref(c)))
    return c.value


def slicegcn_model_num_tensors(m) -> int:
    c = c_int32()
    _check(_lib.slicegcn_model_num_tensors(m, byref(c)))
    return c.value


def slicegcn_model_tensor_info(m, t: int) -> Tuple[str, int, Tuple[int, int, int]]:
    name = (c_char * 32)()
    off = c_int64()
    dims = (c_int32 * 3)()
    _check(_lib.slicegcn_model_tensor_info(m, c_int32(t), name, byref(off), dims))
    return name.value.decode(), off.value, (dims[0], dims[1], dims[2])


def slicegcn_model_slices(m, p: int) -> Tuple[List[Tuple[int, int]], int, int]:
    starts = (c_int32 * p)()
    ends = (c_int32 * p)()
    size, hs = c_int32(), c_int32()
    _check(_lib.slicegcn_model_slices(m, starts, ends, byref(size), byref(hs)))
    return [(starts[i], ends[i]) for i in range(p)], size.value, hs.value


def slicegcn_model_layer_order(m, layer: int) -> int:
    o = c_int32()
    _check(_lib.slicegcn_model_layer_order(m, c_int32(layer), byref(o)))
    return o.value


def slicegcn_train_workspace_bytes(m, g) -> int:
    b = c_int64()
    _check(_lib.slicegcn_train_workspace_bytes(m, g, byref(b)))
    return b.value


def make_opt_desc(lr0: float = 1e-3, epoch: int = 0, total_epochs: int = 500, beta1: float = 0.9, beta2: float = 0.999,
                  eps: float = 1e-8, weight_decay: float = 0.0) -> OptDesc:
    return OptDesc(lr0, beta1, beta2, eps, weight_decay, epoch, total_epochs)


def slicegcn_train_epoch(m, g, X, x_ld: int, labels, train_idx, n_train: int, params, grads, adam_m, adam_v,
                         opt: Optional[OptDesc], logits_out, loss_out, workspace, workspace_bytes: int,
                         stream=None) -> None:
    _check(_lib.slicegcn_train_epoch(m, g, _vp(X), c_int64(x_ld), _vp(labels), _vp(train_idx), c_int64(n_train),
                                     _vp(params), _vp(grads), _vp(adam_m), _vp(adam_v),
                                     byref(opt) if opt is not None else None, _vp(logits_out), _vp(loss_out),
                                     _vp(workspace), c_int64(workspace_bytes), _vp(stream)))


def slicegcn_train_epoch_dropout(m, g, X, x_ld: int, labels, train_idx, n_train: int, params, grads, adam_m, adam_v,
                                 opt: Optional[OptDesc], drop: Optional[DropoutDesc], logits_out, loss_out, workspace,
                                 workspace_bytes: int, stream=None) -> None:
    _check(_lib.slicegcn_train_epoch_dropout(m, g, _vp(X), c_int64(x_ld), _vp(labels), _vp(train_idx), c_int64(n_train),
                                             _vp(params), _vp(grads), _vp(adam_m), _vp(adam_v),
                                             byref(opt) if opt is not None else None,
                                             byref(drop) if drop is not None else None, _vp(logits_out), _vp(loss_out),
                                             _vp(workspace), c_int64(workspace_bytes), _vp(stream)))


EXCHANGE_GATHER_H, EXCHANGE_SUM_DXFF, EXCHANGE_SUM_GRADS = 1, 2, 3
ExchangeFn = ctypes.CFUNCTYPE(c_int32, c_void_p, c_int32, c_void_p, c_int64, c_int64, c_int32, c_int32, c_int32, c_void_p)


def slicegcn_train_epoch_sliced(m, g, X, x_ld: int, labels, train_idx, n_train: int, params, grads, adam_m, adam_v,
                                opt: Optional[OptDesc], slice_begin: int, slice_end: int, exchange, logits_out, loss_out,
                                workspace, workspace_bytes: int, stream=None) -> None:
    """exchange(what, buf_address, rows, ld, col0, cols, dtype, stream_address) -> status (0 = OK), or None."""
    def trampoline(_ctx, what, buf, rows, ld, col0, cols, dtype, st):
        try:
            return int(exchange(what, buf, rows, ld, col0, cols, dtype, st) or 0)
        except Exception:          # an exception must not cross the C frames
            return ERR_INVALID_ARG
    fn = ExchangeFn(trampoline) if exchange is not None else ctypes.cast(None, ExchangeFn)
    _check(_lib.slicegcn_train_epoch_sliced(m, g, _vp(X), c_int64(x_ld), _vp(labels), _vp(train_idx), c_int64(n_train),
                                            _vp(params), _vp(grads), _vp(adam_m), _vp(adam_v),
                                            byref(opt) if opt is not None else None, c_int32(slice_begin), c_int32(slice_end),
                                            fn, None, _vp(logits_out), _vp(loss_out), _vp(workspace), c_int64(workspace_bytes),
                                            _vp(stream)))


def slicegcn_forward_logits(m, g, X, x_ld: int, params, logits_out, workspace, workspace_bytes: int, stream=None) -> None:
    _check(_lib.slicegcn_forward_logits(m, g, _vp(X), c_int64(x_ld), _vp(params), _vp(logits_out), _vp(workspace),
                                        c_int64(workspace_bytes), _vp(stream)))


def slicegcn_train_epoch_host(m, g, X_host, x_ld: int, labels_host, X_stage, labels_stage, train_idx, n_train: int, params,
                              grads, adam_m, adam_v, opt: Optional[OptDesc], loss_dev, loss_host, workspace,
                              workspace_bytes: int, stream=None) -> None:
    _check(_lib.slicegcn_train_epoch_host(m, g, _vp(X_host), c_int64(x_ld), _vp(labels_host), _vp(X_stage), _vp(labels_stage),
                                          _vp(train_idx), c_int64(n_train), _vp(params), _vp(grads), _vp(adam_m),
                                          _vp(adam_v), byref(opt) if opt is not None else None, _vp(loss_dev),
                                          _vp(loss_host), _vp(workspace), c_int64(workspace_bytes), _vp(stream)))


def slicegcn_train_epochs_host(m, g, X_host, x_ld: int, labels_host, X_stage0, X_stage1, labels_stage0, labels_stage1, train_idx,
                               n_train: int, params, grads, adam_m, adam_v, opt: OptDesc, num_epochs: int, losses_dev,
                               losses_host, workspace, workspace_bytes: int, stream=None) -> None:
    _check(_lib.slicegcn_train_epochs_host(m, g, _vp(X_host), c_int64(x_ld), _vp(labels_host), _vp(X_stage0), _vp(X_stage1),
                                           _vp(labels_stage0), _vp(labels_stage1), _vp(train_idx), c_int64(n_train),
                                           _vp(params), _vp(grads), _vp(adam_m), _vp(adam_v), byref(opt), c_int32(num_epochs),
                                           _vp(losses_dev), _vp(losses_host), _vp(workspace), c_int64(workspace_bytes),
                                           _vp(stream)))


def slicegcn_profile_begin() -> None:
    _check(_lib.slicegcn_profile_begin())


def slicegcn_profile_begin_sampled(stride: int) -> None:
    _check(_lib.slicegcn_profile_begin_sampled(c_int32(stride)))


def slicegcn_profile_end() -> Dict[str, float]:
    ms, by = c_double(), c_double()
    calls, launches = c_int64(), c_int64()
    _check(_lib.slicegcn_profile_end(byref(ms), byref(calls), byref(by), byref(launches)))
    return {"spmm_ms": ms.value, "spmm_calls": calls.value, "spmm_bytes": by.value, "kernel_launches": launches.value}


# ------------------------------------------------------------------------------------------ parameter marshalling

def tensor_table(m) -> List[Tuple[str, int, Tuple[int, int, int]]]:
    return [slicegcn_model_tensor_info(m, t) for t in range(slicegcn_model_num_tensors(m))]


def named_param_shapes(m) -> Dict[str, Tuple[int, ...]]:
    """Shapes under the per-slice names pack_params() accepts."""
    shapes: Dict[str, Tuple[int, ...]] = {}
    for name, _, dims in tensor_table(m):
        if name.startswith(("W_agg.", "W_self.")):
            for i in range(dims[0]):
                shapes[f"{name}.{i}"] = (dims[1], dims[2])
        elif name.startswith(("b.", "b_self.")):
            for i in range(dims[0]):
                shapes[f"{name}.{i}"] = (dims[1],)
        elif name == "E":
            shapes[name] = (dims[0], dims[1])
        elif dims[1] == 1:
            shapes[name] = (dims[0],)
        else:
            shapes[name] = (dims[0], dims[1])
    return shapes


def pack_params(m, named: Dict[str, np.ndarray]) -> np.ndarray:
    """Per-slice named arrays ("W_agg.<l>.<i>", "b.<l>.<i>", "E", "Wc1", ...) -> the flat fp32 buffer."""
    flat = np.zeros(slicegcn_model_param_elems(m), np.float32)
    for name, off, dims in tensor_table(m):
        cnt = dims[0] * dims[1] * dims[2]
        if name in named:
            flat[off:off + cnt] = np.asarray(named[name], np.float32).reshape(-1)
        else:                               # per-layer tensors are stored slice-major
            per = cnt // dims[0]
            for i in range(dims[0]):
                flat[off + i * per: off + (i + 1) * per] = np.asarray(named[f"{name}.{i}"], np.float32).reshape(-1)
    return flat


def unpack_params(m, flat: np.ndarray) -> Dict[str, np.ndarray]:
    """Inverse of pack_params (per-slice names for the per-layer tensors)."""
    out: Dict[str, np.ndarray] = {}
    for name, off, dims in tensor_table(m):
        cnt = dims[0] * dims[1] * dims[2]
        data = np.asarray(flat[off:off + cnt])
        if name.startswith(("W_agg.", "W_self.")):
            for i in range(dims[0]):
                out[f"{name}.{i}"] = data.reshape(dims)[i].copy()
        elif name.startswith(("b.", "b_self.")):
            for i in range(dims[0]):
                out[f"{name}.{i}"] = data.reshape(dims[0], dims[1])[i].copy()
        elif name == "E":
            out[name] = data.reshape(dims[0], dims[1]).copy()
        elif dims[1] == 1:
            out[name] = data.copy()
        else:
            out[name] = data.reshape(dims[0], dims[1]).copy()
    return out


def slicegcn_graph_degrees(g) -> np.ndarray:
    """deg [n] alone (the CSR arrays of a large graph stay on the device)."""
    info = slicegcn_graph_info(g)
    deg = np.empty(info["n"], np.int32)
    _check(_lib.slicegcn_graph_export(g, None, None, _vp(deg), None))
    return deg
