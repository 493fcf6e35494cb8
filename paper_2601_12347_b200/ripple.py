"""Thin Python binding over the C ABI of libripple.so (include/ripple.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  PyTorch is
used for device memory (inputs may be CUDA tensors, results come back as CUDA tensor views) and
for the stream.  There is no fallback: if the library has not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# RIPPLE_LIB_PATH: load another build of the library (kernel experiments); default: the in-tree build
LIB_PATH = os.environ.get("RIPPLE_LIB_PATH") or os.path.join(_HERE, "libripple.so")

MAX_LAYERS = 8
OK, ERR_INVALID_ARG, ERR_VERTEX_RANGE, ERR_CAPACITY, ERR_OOM, ERR_CUDA, ERR_TIMEOUT = range(7)
MEM_HOST, MEM_DEVICE = 0, 1
AGG_SUM, AGG_MEAN, AGG_WSUM_GCN, AGG_MAX, AGG_MIN, AGG_WSUM_EDGE = 0, 1, 2, 3, 4, 5
LAYER_SAGE, LAYER_GRAPHCONV, LAYER_GIN, LAYER_GAT = 0, 1, 2, 3
ACT_IDENTITY, ACT_RELU = 0, 1
OP_ADD_EDGE, OP_DEL_EDGE, OP_SET_FEATURE, OP_DEL_VERTEX = 0, 1, 2, 3
SCATTER_AUTO, SCATTER_PUSH, SCATTER_PULL, SCATTER_REGATHER, SCATTER_PUSH_BULK = 0, 1, 2, 3, 4
GEMM_AUTO, GEMM_FP32, GEMM_TF32 = 0, 1, 2

UPDATE_DTYPE = np.dtype([("op", "<i4"), ("u", "<i4"), ("v", "<i4")])

EXPORTED = [
    "ripple_create", "ripple_apply_batch", "ripple_apply_batch_weighted", "ripple_get_embeddings",
    "ripple_get_aggregate", "ripple_get_affected", "ripple_export_graph", "ripple_export_graph_weighted",
    "ripple_get_degrees", "ripple_recompute_full", "ripple_reserve_vertices",
    "ripple_export_graph_static", "ripple_set_timing", "ripple_probe_reduction_rate", "ripple_probe_gather_rate",
    "ripple_get_stats", "ripple_last_error", "ripple_destroy", "ripple_version",
]
# partitioned execution (include/ripple_part.h); the first 18 return a status
EXPORTED_PART = [
    "ripple_part_exports_get", "ripple_part_set_peer", "ripple_part_ipc_export", "ripple_part_ipc_open",
    "ripple_part_set_halos", "ripple_part_bootstrap_layer", "ripple_part_begin", "ripple_part_hop_send",
    "ripple_part_hop_compute", "ripple_part_end", "ripple_part_rows_sent",
    "ripple_router_create", "ripple_router_partition_shape", "ripple_router_partition_fill",
    "ripple_router_route", "ripple_router_batch_shape", "ripple_router_batch_fill", "ripple_router_global_ids",
    "ripple_router_destroy", "ripple_router_owner", "ripple_router_local_id", "ripple_router_global_id",
    "ripple_router_is_high_degree", "ripple_router_load",
]
MAX_PEERS = 16


class RippleError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"ripple status {status}: {message}")
        self.status = status


class _Graph(ctypes.Structure):
    _fields_ = [("num_vertices", ctypes.c_int64), ("num_edges", ctypes.c_int64),
                ("src", ctypes.c_void_p), ("dst", ctypes.c_void_p), ("mem", ctypes.c_int32),
                ("weight", ctypes.c_void_p)]


class _Layer(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("d_in", ctypes.c_int32), ("d_hidden", ctypes.c_int32),
                ("d_out", ctypes.c_int32), ("act", ctypes.c_int32), ("eps", ctypes.c_float),
                ("Wa", ctypes.c_void_p), ("Wb", ctypes.c_void_p), ("ba", ctypes.c_void_p),
                ("bb", ctypes.c_void_p)]


class _Options(ctypes.Structure):
    _fields_ = [("slack", ctypes.c_double), ("pool_edges", ctypes.c_int64),
                ("max_batch", ctypes.c_int64), ("scatter_mode", ctypes.c_int32),
                ("gemm_mode", ctypes.c_int32), ("timing", ctypes.c_int32),
                ("pre_transform", ctypes.c_int32), ("no_graphs", ctypes.c_int32), ("device", ctypes.c_int32), ("stream", ctypes.c_void_p),
                ("regather_threshold", ctypes.c_float), ("rebuild_budget", ctypes.c_float),
                ("n_local", ctypes.c_int32)]


class _Stats(ctypes.Structure):
    _A = ctypes.c_int64 * (MAX_LAYERS + 1)
    _I = ctypes.c_int32 * (MAX_LAYERS + 1)
    _F = ctypes.c_float * (MAX_LAYERS + 1)
    _fields_ = [("num_layers", ctypes.c_int32), ("num_edges", ctypes.c_int64),
                ("n_ops", ctypes.c_int64), ("n_added", ctypes.c_int64), ("n_deleted", ctypes.c_int64),
                ("n_noop_add", ctypes.c_int64), ("n_noop_del", ctypes.c_int64),
                ("n_superseded", ctypes.c_int64), ("n_feature", ctypes.c_int64),
                ("affected", _A), ("senders", _A), ("active_edges", _A), ("scatter_pull", _I),
                ("in_edges", _A), ("message_width", _I),
                ("pool_used", ctypes.c_int64), ("pool_size", ctypes.c_int64),
                ("ms_total", ctypes.c_float), ("ms_graph", ctypes.c_float),
                ("ms_frontier", _F), ("ms_scatter", _F), ("ms_update", _F),
                ("ms_scatter_kernel", _F), ("ms_regather", _F), ("ms_bootstrap", ctypes.c_float), ("gpu_launches", ctypes.c_int64), ("n_expanded", ctypes.c_int64),
                ("rows_rebuilt", _A), ("pool_free", ctypes.c_int64), ("pool_lost", ctypes.c_int64)]


class _PartExports(ctypes.Structure):
    _fields_ = [("accumulator", ctypes.c_void_p * (MAX_LAYERS + 1)), ("accumulator_ld", ctypes.c_int64 * (MAX_LAYERS + 1)),
                ("embeddings", ctypes.c_void_p * (MAX_LAYERS + 1)), ("embeddings_ld", ctypes.c_int64 * (MAX_LAYERS + 1)),
                ("frontier_bitmap", ctypes.c_void_p), ("out_degrees", ctypes.c_void_p),
                ("num_vertices", ctypes.c_int64)]


class _PartIpc(ctypes.Structure):
    _fields_ = [("accumulator", (ctypes.c_ubyte * 64) * (MAX_LAYERS + 1)),
                ("embeddings", (ctypes.c_ubyte * 64) * (MAX_LAYERS + 1)),
                ("frontier_bitmap", ctypes.c_ubyte * 64), ("out_degrees", ctypes.c_ubyte * 64),
                ("accumulator_ld", ctypes.c_int64 * (MAX_LAYERS + 1)),
                ("embeddings_ld", ctypes.c_int64 * (MAX_LAYERS + 1)), ("num_vertices", ctypes.c_int64),
                ("num_layers", ctypes.c_int32)]


_lib = None


def load_library(path: Optional[str] = None):
    """dlopen libripple.so and declare the prototypes.  Raises if the library is not there."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} not found: build it with `python -m paper_2601_12347_b200.build` "
            "(there is no CPU fallback)")
    lib = ctypes.CDLL(path)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    P = ctypes.POINTER
    lib.ripple_create.argtypes = [P(_Graph), vp, i32, P(_Layer), i32, i32, P(_Options), P(vp)]
    lib.ripple_apply_batch.argtypes = [vp, vp, i64, vp, i64, i32]
    lib.ripple_apply_batch_weighted.argtypes = [vp, vp, i64, vp, i64, vp, i32]
    lib.ripple_export_graph_weighted.argtypes = [vp, vp, vp, vp, i64]
    lib.ripple_get_embeddings.argtypes = [vp, i32, P(vp), P(i64)]
    lib.ripple_get_aggregate.argtypes = [vp, i32, P(vp), P(i64), P(i32), P(i32)]
    lib.ripple_get_affected.argtypes = [vp, i32, P(vp), P(i64)]
    lib.ripple_export_graph.argtypes = [vp, vp, vp, i64]
    lib.ripple_get_degrees.argtypes = [vp, P(vp), P(vp)]
    lib.ripple_recompute_full.argtypes = [vp]
    lib.ripple_get_stats.argtypes = [vp, P(_Stats)]
    lib.ripple_last_error.argtypes = [vp]
    lib.ripple_last_error.restype = ctypes.c_char_p
    lib.ripple_destroy.argtypes = [vp]
    lib.ripple_destroy.restype = None
    lib.ripple_version.argtypes = []
    lib.ripple_version.restype = ctypes.c_char_p
    lib.ripple_export_graph_static.argtypes = [vp, vp, vp, i64]
    lib.ripple_set_timing.argtypes = [vp, i32]
    lib.ripple_probe_reduction_rate.argtypes = [i32, i64, i32, i64, i32, P(ctypes.c_float)]
    lib.ripple_probe_gather_rate.argtypes = [i32, i64, i32, i64, P(ctypes.c_float)]
    lib.ripple_reserve_vertices.argtypes = [vp, i64]
    for name in EXPORTED[:16]:
        getattr(lib, name).restype = i32
    # partitioned execution
    lib.ripple_part_exports_get.argtypes = [vp, P(_PartExports)]
    lib.ripple_part_set_peer.argtypes = [vp, i32, P(_PartExports)]
    lib.ripple_part_ipc_export.argtypes = [vp, P(_PartIpc)]
    lib.ripple_part_ipc_open.argtypes = [vp, i32, P(_PartIpc)]
    lib.ripple_part_set_halos.argtypes = [vp, i32, i32, vp, vp]
    lib.ripple_part_bootstrap_layer.argtypes = [vp, i32]
    lib.ripple_part_begin.argtypes = [vp, vp, i64, vp, i64, vp, vp, i32]
    lib.ripple_part_hop_send.argtypes = [vp, i32]
    lib.ripple_part_hop_compute.argtypes = [vp, i32]
    lib.ripple_part_end.argtypes = [vp]
    lib.ripple_part_rows_sent.argtypes = [vp, vp]
    lib.ripple_router_create.argtypes = [i32, i64, vp, i64, vp, vp, i32, i64, i64, i64, P(vp)]
    lib.ripple_router_partition_shape.argtypes = [vp, i32, P(i64), P(i64), P(i64), P(i64)]
    lib.ripple_router_partition_fill.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp]
    lib.ripple_router_route.argtypes = [vp, vp, i64]
    lib.ripple_router_batch_shape.argtypes = [vp, i32, P(i64), P(i64), P(i64)]
    lib.ripple_router_batch_fill.argtypes = [vp, i32, vp, vp, vp, vp, P(i32), vp, vp]
    lib.ripple_router_global_ids.argtypes = [vp, i32, vp, i64]
    for name in EXPORTED_PART[:18]:
        getattr(lib, name).restype = i32
    lib.ripple_router_destroy.argtypes = [vp]
    lib.ripple_router_destroy.restype = None
    for name in ("ripple_router_owner", "ripple_router_local_id", "ripple_router_is_high_degree"):
        getattr(lib, name).argtypes = [vp, i32]
        getattr(lib, name).restype = i32
    lib.ripple_router_global_id.argtypes = [vp, i32, i32]
    lib.ripple_router_global_id.restype = i32
    lib.ripple_router_load.argtypes = [vp, i32]
    lib.ripple_router_load.restype = i64
    _lib = lib
    return lib


class _DevArray:
    """Exposes borrowed device memory through __cuda_array_interface__ (no copy)."""

    def __init__(self, ptr: int, shape: Tuple[int, ...], typestr: str, strides=None, owner=None):
        self.__cuda_array_interface__ = {"shape": shape, "typestr": typestr, "data": (ptr, False),
                                         "version": 2, "strides": strides}
        self._owner = owner


def _is_torch_cuda(x) -> bool:
    return hasattr(x, "is_cuda") and bool(x.is_cuda)


class Ripple:
    """One resident graph + model + cached embeddings on the current CUDA device.

    model: object with `.agg` and `.layers` (kind, d_in, d_out, act, d_hidden, eps per layer);
    weights: per layer a dict of fp32 numpy arrays (Wa, ba and, by kind, Wb, bb), input-major.
    src / dst / features: numpy arrays (host) or CUDA torch tensors (device).
    """

    def __init__(self, n: int, src, dst, features, model, weights: Sequence[Dict[str, np.ndarray]],
                 slack: float = 0.0, pool_edges: int = 0, max_batch: int = 0,
                 scatter_mode: int = SCATTER_AUTO, gemm_mode: int = GEMM_AUTO, timing: bool = False,
                 pre_transform: bool = True, graphs: bool = True, stream=None,
                 regather_threshold: float = 0.0, rebuild_budget: float = 0.0, edge_weights=None,
                 n_local: int = 0):
        import torch
        self._torch = torch
        self.lib = load_library()
        self.n = int(n)
        self.n_local = int(n_local)
        self.model, self.weights = model, weights
        self.L = len(model.layers)
        self.dims = [model.layers[0].d_in] + [l.d_out for l in model.layers]
        self.h = ctypes.c_void_p(None)
        keep = []
        g = _Graph()
        g.num_vertices = self.n
        if _is_torch_cuda(src):
            assert src.dtype == torch.int32 and dst.dtype == torch.int32
            src, dst = src.contiguous(), dst.contiguous()
            g.num_edges, g.src, g.dst, g.mem = src.numel(), src.data_ptr(), dst.data_ptr(), MEM_DEVICE
        else:
            src = np.ascontiguousarray(src, dtype=np.int32)
            dst = np.ascontiguousarray(dst, dtype=np.int32)
            g.num_edges, g.src, g.dst, g.mem = src.size, src.ctypes.data, dst.ctypes.data, MEM_HOST
        keep += [src, dst]
        if edge_weights is not None:       # one stored weight per edge (AGG_WSUM_EDGE), same memory space as src / dst
            if _is_torch_cuda(edge_weights):
                assert g.mem == MEM_DEVICE and edge_weights.dtype == torch.float32
                edge_weights = edge_weights.contiguous()
                g.weight = edge_weights.data_ptr()
            else:
                assert g.mem == MEM_HOST
                edge_weights = np.ascontiguousarray(edge_weights, dtype=np.float32)
                g.weight = edge_weights.ctypes.data
            assert edge_weights.shape[0] == g.num_edges
            keep.append(edge_weights)
        if _is_torch_cuda(features):
            assert features.dtype == torch.float32
            features = features.contiguous()
            fptr, fmem = features.data_ptr(), MEM_DEVICE
        else:
            features = np.ascontiguousarray(features, dtype=np.float32)
            fptr, fmem = features.ctypes.data, MEM_HOST
        assert tuple(features.shape) == (self.n, self.dims[0])
        layers = (_Layer * self.L)()
        for i, (ly, w) in enumerate(zip(model.layers, weights)):
            layers[i].kind, layers[i].d_in, layers[i].d_hidden = int(ly.kind), int(ly.d_in), int(ly.d_hidden)
            layers[i].d_out, layers[i].act, layers[i].eps = int(ly.d_out), int(ly.act), float(ly.eps)
            for name in ("Wa", "Wb", "ba", "bb"):
                a = w.get(name)
                if a is not None:
                    a = np.ascontiguousarray(a, dtype=np.float32)
                    keep.append(a)
                    setattr(layers[i], name, a.ctypes.data)
        opt = _Options()
        opt.slack, opt.pool_edges, opt.max_batch = float(slack), int(pool_edges), int(max_batch)
        opt.scatter_mode, opt.gemm_mode, opt.timing = int(scatter_mode), int(gemm_mode), int(bool(timing))
        opt.pre_transform = 0 if pre_transform else 1
        opt.no_graphs = 0 if graphs else 1
        opt.regather_threshold = float(regather_threshold)
        opt.rebuild_budget = float(rebuild_budget)
        opt.n_local = int(n_local)     # > 0: one worker of a partitioned execution (see partitioned.py)
        opt.device = torch.cuda.current_device()
        self._stream = stream if stream is not None else torch.cuda.Stream()
        opt.stream = self._stream.cuda_stream
        torch.cuda.current_stream().synchronize()
        st = self.lib.ripple_create(ctypes.byref(g), fptr, fmem, layers, self.L, int(model.agg),
                                    ctypes.byref(opt), ctypes.byref(self.h))
        if st != OK:
            msg = self.lib.ripple_last_error(None).decode()
            self.h = ctypes.c_void_p(None)
            raise RippleError(st, msg)

    # ---- lifetime ------------------------------------------------------------------------
    def close(self):
        if getattr(self, "h", None) and self.h.value:
            self.lib.ripple_destroy(self.h)
            self.h = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st != OK:
            raise RippleError(st, self.lib.ripple_last_error(self.h).decode())

    @property
    def stream(self):
        return self._stream

    # ---- the hot path ----------------------------------------------------------------------
    def apply_batch(self, ups, feat_rows=None, op_weights=None) -> None:
        """ups: numpy array of UPDATE_DTYPE (host) or CUDA int32 tensor [n, 3] (device);
        feat_rows: [n_rows, d0] fp32 in the same memory space; op_weights: [n] fp32 in the same
        memory space, the weight of every ADD_EDGE (graphs with stored edge weights only)."""
        if _is_torch_cuda(ups):
            ups = ups.contiguous()
            n, uptr, mem = ups.shape[0], ups.data_ptr(), MEM_DEVICE
            if feat_rows is None:
                nr, fptr = 0, None
            else:
                feat_rows = feat_rows.contiguous()
                nr, fptr = feat_rows.shape[0], feat_rows.data_ptr()
        else:
            if hasattr(ups, "numpy"):      # pinned host tensor [n, 3] int32
                n, uptr = ups.shape[0], ups.data_ptr()
            else:
                ups = np.ascontiguousarray(ups, dtype=UPDATE_DTYPE)
                n, uptr = ups.size, ups.ctypes.data
            mem = MEM_HOST
            if feat_rows is None:
                nr, fptr = 0, None
            elif hasattr(feat_rows, "numpy"):
                nr, fptr = feat_rows.shape[0], feat_rows.data_ptr()
            else:
                feat_rows = np.ascontiguousarray(feat_rows, dtype=np.float32)
                nr, fptr = feat_rows.shape[0], feat_rows.ctypes.data
        if op_weights is None:
            self._check(self.lib.ripple_apply_batch(self.h, uptr, n, fptr, nr, mem))
            return
        if mem == MEM_DEVICE:
            op_weights = op_weights.contiguous()
            wptr = op_weights.data_ptr()
        elif hasattr(op_weights, "numpy"):
            wptr = op_weights.data_ptr()
        else:
            op_weights = np.ascontiguousarray(op_weights, dtype=np.float32)
            wptr = op_weights.ctypes.data
        assert op_weights.shape[0] == n
        self._check(self.lib.ripple_apply_batch_weighted(self.h, uptr, n, fptr, nr, wptr, mem))

    def set_timing(self, on: bool) -> None:
        self._check(self.lib.ripple_set_timing(self.h, int(bool(on))))

    def reserve_vertices(self, n: int) -> None:
        """Raises the id capacity to n: the new ids are isolated vertices with zero features.  Views
        obtained earlier (embeddings, aggregate, affected, degrees) are invalid afterwards."""
        self._check(self.lib.ripple_reserve_vertices(self.h, int(n)))
        self.n = int(n)

    def recompute_full(self) -> None:
        self._check(self.lib.ripple_recompute_full(self.h))

    # ---- read-out (borrowed device memory, valid until the next apply / recompute / close) ----
    def _matrix(self, fn, layer: int, width: int):
        ptr, ld = ctypes.c_void_p(), ctypes.c_int64()
        self._check(fn(self.h, layer, ctypes.byref(ptr), ctypes.byref(ld)))
        arr = _DevArray(ptr.value, (self.n, width), "<f4", strides=(4 * ld.value, 4), owner=self)
        return self._torch.as_tensor(arr, device="cuda")

    def embeddings(self, layer: int):
        return self._matrix(self.lib.ripple_get_embeddings, layer, self.dims[layer])

    def aggregate(self, layer: int):
        """(tensor view N x width, transformed): the cached aggregate of `layer`; if transformed,
        its rows are sums of W_n^T h_u instead of h_u."""
        ptr, ld = ctypes.c_void_p(), ctypes.c_int64()
        width, tr = ctypes.c_int32(), ctypes.c_int32()
        self._check(self.lib.ripple_get_aggregate(self.h, layer, ctypes.byref(ptr), ctypes.byref(ld),
                                                  ctypes.byref(width), ctypes.byref(tr)))
        arr = _DevArray(ptr.value, (self.n, width.value), "<f4", strides=(4 * ld.value, 4), owner=self)
        return self._torch.as_tensor(arr, device="cuda"), bool(tr.value)

    def affected(self, layer: int):
        ptr, cnt = ctypes.c_void_p(), ctypes.c_int64()
        self._check(self.lib.ripple_get_affected(self.h, layer, ctypes.byref(ptr), ctypes.byref(cnt)))
        if cnt.value == 0:
            return self._torch.zeros(0, dtype=self._torch.int32, device="cuda")
        return self._torch.as_tensor(_DevArray(ptr.value, (cnt.value,), "<i4", owner=self), device="cuda")

    def degrees(self):
        po, pi = ctypes.c_void_p(), ctypes.c_void_p()
        self._check(self.lib.ripple_get_degrees(self.h, ctypes.byref(po), ctypes.byref(pi)))
        mk = lambda p: self._torch.as_tensor(_DevArray(p.value, (self.n,), "<i4", owner=self), device="cuda")
        return mk(po), mk(pi)

    def export_graph(self) -> Tuple[np.ndarray, np.ndarray]:
        """Canonical CSR over out-edges (host arrays): rowptr[N+1], col ascending per row."""
        e = self.stats()["num_edges"]
        rowptr = np.zeros(self.n + 1, dtype=np.int64)
        col = np.zeros(max(e, 1), dtype=np.int32)
        self._check(self.lib.ripple_export_graph(self.h, rowptr.ctypes.data, col.ctypes.data, col.size))
        return rowptr, col[: rowptr[-1]]

    def export_graph_weighted(self) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """export_graph() plus the stored weight of every edge, in the order of col."""
        e = self.stats()["num_edges"]
        rowptr = np.zeros(self.n + 1, dtype=np.int64)
        col = np.zeros(max(e, 1), dtype=np.int32)
        w = np.zeros(max(e, 1), dtype=np.float32)
        self._check(self.lib.ripple_export_graph_weighted(self.h, rowptr.ctypes.data, col.ctypes.data,
                                                          w.ctypes.data, col.size))
        return rowptr, col[: rowptr[-1]], w[: rowptr[-1]]

    def export_graph_static(self) -> Tuple[np.ndarray, np.ndarray]:
        """Same result as export_graph() through the entry point that allocates no device memory.

        For processes in which every byte of device memory already belongs to a framework's
        caching allocator, or callers that cannot afford the synchronisation an allocation may
        imply.  Works for graphs of up to 262 144 vertices and 2 097 152 edges; larger graphs
        raise RippleError (status ERR_CAPACITY).  The first call on a device performs a one-time
        address look-up and should come before any stream capture; concurrent calls on one device
        share the library's fixed staging arrays and must be serialised by the caller."""
        e = self.stats()["num_edges"]
        rowptr = np.zeros(self.n + 1, dtype=np.int64)
        col = np.zeros(max(e, 1), dtype=np.int32)
        self._check(self.lib.ripple_export_graph_static(self.h, rowptr.ctypes.data, col.ctypes.data, col.size))
        return rowptr, col[: rowptr[-1]]

    def stats(self) -> dict:
        s = _Stats()
        self._check(self.lib.ripple_get_stats(self.h, ctypes.byref(s)))
        L = self.L
        out = {k: getattr(s, k) for k in ("num_layers", "num_edges", "n_ops", "n_added", "n_deleted",
                                          "n_noop_add", "n_noop_del", "n_superseded", "n_feature",
                                          "pool_used", "pool_size", "pool_free", "pool_lost", "ms_total", "ms_graph",
                                          "ms_bootstrap", "gpu_launches", "n_expanded")}
        for k in ("affected", "senders", "active_edges", "scatter_pull", "in_edges", "message_width", "rows_rebuilt", "ms_frontier", "ms_scatter",
                  "ms_update", "ms_scatter_kernel", "ms_regather"):
            out[k] = list(getattr(s, k))[: L + 1]
        return out


def probe_reduction_rate(n_rows: int, row_floats: int, n_messages: int, pattern: int = 0, device: int = -1) -> float:
    """Milliseconds for n_messages rows of row_floats floats issued as 16-byte vector reductions
    into rows of a window of n_rows rows (best of three passes).  pattern 0: uniformly random
    rows, 1: consecutive rows, 2: random rows with a popular head."""
    lib = load_library()
    ms = ctypes.c_float()
    st = lib.ripple_probe_reduction_rate(int(device), int(n_rows), int(row_floats), int(n_messages), int(pattern),
                                         ctypes.byref(ms))
    if st:
        raise RippleError(st, "reduction probe failed")
    return float(ms.value)


def probe_gather_rate(n_rows: int, row_floats: int, n_gathers: int, device: int = -1) -> float:
    """Milliseconds for n_gathers whole rows of row_floats floats read from pseudo-random rows of a
    window of n_rows rows (best of three passes)."""
    lib = load_library()
    ms = ctypes.c_float()
    st = lib.ripple_probe_gather_rate(int(device), int(n_rows), int(row_floats), int(n_gathers), ctypes.byref(ms))
    if st:
        raise RippleError(st, "gather probe failed")
    return float(ms.value)


def version() -> str:
    return load_library().ripple_version().decode()
