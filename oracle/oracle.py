"""ctypes front end of the CPU oracle (ripple_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the benchmark's CPU-baseline
leg.  It never imports the CUDA binding and the CUDA binding never imports it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, List, Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_lib = None

UPDATE_DTYPE = np.dtype([("op", "<i4"), ("u", "<i4"), ("v", "<i4")])


def build(force: bool = False) -> str:
    """Compile the oracle with gcc; returns the shared object's path."""
    src = os.path.join(_HERE, "ripple_oracle.c")
    out = os.path.join(_HERE, "_ripple_oracle.so")
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O3", "-fopenmp", "-shared", "-fPIC", "-o", out, src, "-lm"])
    return out


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    vp, i32, i64, dbl = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_double
    lib.orc_create.argtypes = [i32, i64, vp, vp, vp, i32, vp, i32]
    lib.orc_create.restype = vp
    lib.orc_create_weighted.argtypes = [i32, i64, vp, vp, vp, vp, i32, vp, i32]
    lib.orc_create_weighted.restype = vp
    lib.orc_set_batch_weights.argtypes = [vp, vp]
    lib.orc_set_batch_weights.restype = None
    lib.orc_export_weights.argtypes = [vp, vp]
    lib.orc_export_weights.restype = None
    lib.orc_set_layer.argtypes = [vp, i32, i32, i32, i32, dbl, vp, vp, vp, vp]
    lib.orc_set_layer.restype = None
    lib.orc_destroy.argtypes = [vp]
    lib.orc_destroy.restype = None
    for name in ("orc_full", "orc_bootstrap"):
        getattr(lib, name).argtypes = [vp]
        getattr(lib, name).restype = None
    for name in ("orc_apply_incremental", "orc_apply_incremental_pull", "orc_apply_scoped"):
        getattr(lib, name).argtypes = [vp, vp, i64, vp, i64]
        getattr(lib, name).restype = i32
    for name in ("orc_H", "orc_S", "orc_Den", "orc_full_H", "orc_full_S"):
        getattr(lib, name).argtypes = [vp, i32]
        getattr(lib, name).restype = ctypes.POINTER(ctypes.c_double)
    lib.orc_affected.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_int)]
    lib.orc_affected.restype = ctypes.POINTER(ctypes.c_int)
    lib.orc_active_edges.argtypes = [vp, i32]
    lib.orc_active_edges.restype = ctypes.c_long
    lib.orc_counts.argtypes = [vp, vp]
    lib.orc_counts.restype = None
    lib.orc_num_edges.argtypes = [vp]
    lib.orc_num_edges.restype = i64
    lib.orc_degrees.argtypes = [vp, vp, vp]
    lib.orc_degrees.restype = None
    lib.orc_export_csr.argtypes = [vp, vp, vp]
    lib.orc_export_csr.restype = None
    lib.orc_row_from_prev.argtypes = [vp, i32, i32, vp, i64, vp, vp]
    lib.orc_row_from_prev.restype = None
    lib.orc_rows_from_prev.argtypes = [vp, i32, vp, i64, vp, i64, vp, vp]
    lib.orc_rows_from_prev.restype = None
    lib.orc_apply_structure.argtypes = [vp, vp, i64, i64]
    lib.orc_apply_structure.restype = i32
    lib.orc_num_threads.argtypes = []
    lib.orc_num_threads.restype = i32
    _lib = lib
    return lib


def num_threads() -> int:
    return int(_load().orc_num_threads())


class Oracle:
    """One oracle state: graph, features, weights and the cached H^l / S^l.

    model: an object with `.agg` and `.layers` (each with kind, d_in, d_out, act, d_hidden, eps);
    weights: one dict per layer with fp32 arrays Wa, ba and (SAGE, GIN) Wb, (GIN) bb.
    """

    def __init__(self, n: int, src: np.ndarray, dst: np.ndarray, feat: np.ndarray, model, weights,
                 bootstrap: bool = True, edge_weights: Optional[np.ndarray] = None):
        lib = _load()
        self.lib = lib
        self.n = int(n)
        self.dims = [model.layers[0].d_in] + [l.d_out for l in model.layers]
        self.L = len(model.layers)
        src = np.ascontiguousarray(src, dtype=np.int32)
        dst = np.ascontiguousarray(dst, dtype=np.int32)
        feat = np.ascontiguousarray(feat, dtype=np.float32)
        assert feat.shape == (self.n, self.dims[0])
        dims = np.asarray(self.dims, dtype=np.int32)
        if edge_weights is not None:
            edge_weights = np.ascontiguousarray(edge_weights, dtype=np.float32)
            assert edge_weights.shape == src.shape
        self.h = lib.orc_create_weighted(self.n, src.size, src.ctypes.data, dst.ctypes.data,
                                         edge_weights.ctypes.data if edge_weights is not None else None,
                                         feat.ctypes.data, self.L, dims.ctypes.data, int(model.agg))
        for i, (ly, w) in enumerate(zip(model.layers, weights)):
            def p(name):
                a = w.get(name)
                if a is None:
                    return None
                a = np.ascontiguousarray(a, dtype=np.float32)
                w[name] = a
                return a.ctypes.data
            lib.orc_set_layer(self.h, i + 1, int(ly.kind), int(ly.d_hidden), int(ly.act),
                              float(ly.eps), p("Wa"), p("Wb"), p("ba"), p("bb"))
        if bootstrap:
            lib.orc_bootstrap(self.h)

    def close(self):
        if self.h:
            self.lib.orc_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- updates -----------------------------------------------------------------------
    def _apply(self, fn, ups: np.ndarray, feat_rows: Optional[np.ndarray], op_weights=None) -> int:
        ups = np.ascontiguousarray(ups, dtype=UPDATE_DTYPE)
        if feat_rows is None:
            feat_rows = np.zeros((0, self.dims[0]), dtype=np.float32)
        feat_rows = np.ascontiguousarray(feat_rows, dtype=np.float32)
        if op_weights is not None:     # one weight per operation; read for edge additions only
            op_weights = np.ascontiguousarray(op_weights, dtype=np.float32)
            assert op_weights.shape == (ups.size,)
            self.lib.orc_set_batch_weights(self.h, op_weights.ctypes.data)
        try:
            return int(fn(self.h, ups.ctypes.data, ups.size, feat_rows.ctypes.data, feat_rows.shape[0]))
        finally:
            self.lib.orc_set_batch_weights(self.h, None)

    def apply_incremental(self, ups, feat_rows=None, pull: bool = False, op_weights=None) -> int:
        """The incremental algorithm.  pull: messages are gathered per affected sink on all host
        cores instead of being pushed along the senders' out-lists by one thread; only the order
        of the additions differs.  op_weights: the weight of every ADD_EDGE of the batch (an array
        with one entry per operation) for the weighted sum with per-edge weights."""
        fn = self.lib.orc_apply_incremental_pull if pull else self.lib.orc_apply_incremental
        return self._apply(fn, ups, feat_rows, op_weights)

    def apply_scoped(self, ups, feat_rows=None, op_weights=None) -> int:
        return self._apply(self.lib.orc_apply_scoped, ups, feat_rows, op_weights)

    def apply_structure(self, ups, n_rows: int, op_weights=None) -> int:
        """Graph state and affected sets only (no embedding arithmetic; H and S go stale)."""
        ups = np.ascontiguousarray(ups, dtype=UPDATE_DTYPE)
        if op_weights is not None:
            op_weights = np.ascontiguousarray(op_weights, dtype=np.float32)
            self.lib.orc_set_batch_weights(self.h, op_weights.ctypes.data)
        try:
            return int(self.lib.orc_apply_structure(self.h, ups.ctypes.data, ups.size, int(n_rows)))
        finally:
            self.lib.orc_set_batch_weights(self.h, None)

    def bootstrap(self):
        self.lib.orc_bootstrap(self.h)

    # ---- read-out (views into the oracle's memory; copy if they must outlive a call) -----
    def _mat(self, ptr, rows, cols) -> np.ndarray:
        return np.ctypeslib.as_array(ptr, shape=(rows, cols))

    def H(self, l: int) -> np.ndarray:
        return self._mat(self.lib.orc_H(self.h, l), self.n, self.dims[l])

    def S(self, l: int) -> np.ndarray:
        return self._mat(self.lib.orc_S(self.h, l), self.n, self.dims[l - 1])

    def Den(self, l: int) -> np.ndarray:
        """Attention layers: the cached denominator sum of every vertex (S holds the numerator)."""
        return np.ctypeslib.as_array(self.lib.orc_Den(self.h, l), shape=(self.n,))

    def full(self) -> List[np.ndarray]:
        """O-full on the current graph and features: [H^0, H^1, .., H^L] (fresh copies)."""
        self.lib.orc_full(self.h)
        return [self._mat(self.lib.orc_full_H(self.h, l), self.n, self.dims[l]).copy()
                for l in range(self.L + 1)]

    def full_S(self, l: int) -> np.ndarray:
        return self._mat(self.lib.orc_full_S(self.h, l), self.n, self.dims[l - 1]).copy()

    def affected(self, l: int) -> np.ndarray:
        cnt = ctypes.c_int(0)
        p = self.lib.orc_affected(self.h, l, ctypes.byref(cnt))
        if cnt.value == 0:
            return np.zeros(0, dtype=np.int32)
        return np.ctypeslib.as_array(p, shape=(cnt.value,)).astype(np.int32)

    def active_edges(self, l: int) -> int:
        return int(self.lib.orc_active_edges(self.h, l))

    def counts(self) -> Dict[str, int]:
        out = np.zeros(5, dtype=np.int64)
        self.lib.orc_counts(self.h, out.ctypes.data)
        return dict(zip(("added", "deleted", "noop_add", "noop_del", "superseded"), out.tolist()))

    def num_edges(self) -> int:
        return int(self.lib.orc_num_edges(self.h))

    def degrees(self) -> Tuple[np.ndarray, np.ndarray]:
        do = np.zeros(self.n, dtype=np.int32)
        di = np.zeros(self.n, dtype=np.int32)
        self.lib.orc_degrees(self.h, do.ctypes.data, di.ctypes.data)
        return do, di

    def export_csr(self) -> Tuple[np.ndarray, np.ndarray]:
        rowptr = np.zeros(self.n + 1, dtype=np.int64)
        col = np.zeros(max(1, self.num_edges()), dtype=np.int32)
        self.lib.orc_export_csr(self.h, rowptr.ctypes.data, col.ctypes.data)
        return rowptr, col[: rowptr[-1]]

    def export_weights(self) -> np.ndarray:
        """The stored weight of every edge, in the order of export_csr()'s column array."""
        w = np.zeros(max(1, self.num_edges()), dtype=np.float32)
        self.lib.orc_export_weights(self.h, w.ctypes.data)
        return w[: self.num_edges()]

    def row_from_prev(self, l: int, v: int, Hprev: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
        """(S^l_v, h^l_v) by the layer definition from a caller-supplied fp32 H^{l-1}."""
        assert Hprev.dtype == np.float32 and Hprev.flags.c_contiguous
        ld = Hprev.shape[1]
        S = np.zeros(self.dims[l - 1], dtype=np.float64)
        h = np.zeros(self.dims[l], dtype=np.float64)
        self.lib.orc_row_from_prev(self.h, l, int(v), Hprev.ctypes.data, ld, S.ctypes.data,
                                   h.ctypes.data)
        return S, h

    def rows_from_prev(self, l: int, ids: np.ndarray, Hprev: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
        """row_from_prev for every vertex of ids: (S rows, h rows), fp64, in the order of ids."""
        assert Hprev.dtype == np.float32 and Hprev.flags.c_contiguous
        ids = np.ascontiguousarray(ids, dtype=np.int32)
        S = np.zeros((ids.size, self.dims[l - 1]), dtype=np.float64)
        h = np.zeros((ids.size, self.dims[l]), dtype=np.float64)
        self.lib.orc_rows_from_prev(self.h, l, ids.ctypes.data, ids.size, Hprev.ctypes.data,
                                    Hprev.shape[1], S.ctypes.data, h.ctypes.data)
        return S, h
