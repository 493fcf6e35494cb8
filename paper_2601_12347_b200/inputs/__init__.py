"""Seeded synthetic inputs: graphs, features, weights and update streams.

This module serves both the CUDA path and the CPU oracle and therefore holds none of the
method's arithmetic: it only draws graphs, feature rows, weight matrices and batches of updates.
Everything is a pure function of the seeds given, so both sides see identical inputs.

The graphs stand in for the public datasets the paper measures on (Table 2): "sparse" has the
vertex / edge / feature / class counts of the citation graph, "dense" those of the product graph.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

OP_ADD_EDGE = 0
OP_DEL_EDGE = 1
OP_SET_FEATURE = 2
OP_DEL_VERTEX = 3

# one update record: for edge ops (u, v) = (source, sink); for a feature update u is the vertex
# and v the index of its row in the batch's feature payload
UPDATE_DTYPE = np.dtype([("op", "<i4"), ("u", "<i4"), ("v", "<i4")])

KIND_SAGE = 0      # h = act(W_self h_v + W_neigh agg_v + b)
KIND_GRAPHCONV = 1  # h = act(W agg_v + b)            (no self term)
KIND_GIN = 2       # h = act(W2 relu(W1 ((1+eps) h_v + agg_v) + b1) + b2)
KIND_GAT = 3       # h = act(sum_u softmax_u(z_uv) h_u), z_uv = rect(a_src . W h_u + a_dst . W h_v)   (Eq. 3)

AGG_SUM = 0
AGG_MEAN = 1
AGG_WSUM_GCN = 2   # coefficient 1/sqrt(deg_out(u) * deg_in(v))
AGG_MAX = 3        # element-wise maximum over the in-neighbours (monotonic; zeros if there are none)
AGG_MIN = 4        # element-wise minimum, likewise
AGG_WSUM_EDGE = 5  # weighted sum with a stored weight per edge (the paper's GC-W workload)

ACT_IDENTITY = 0
ACT_RELU = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SUBSTREAM = {"graph": 1, "features": 2, "weights": 3, "updates": 4, "warmup": 5, "perm": 6,
              "drop": 7, "order": 8, "edge_weights": 9, "update_weights": 10}


def _rng(seed: int, stream: str) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([int(seed), _SUBSTREAM[stream]]))


# --------------------------------------------------------------------------------------------
# native helper (R-MAT pair draws)
# --------------------------------------------------------------------------------------------
_lib = None


def build_native(force: bool = False) -> str:
    """Compile the R-MAT pair generator with gcc; returns the path of the shared object."""
    src = os.path.join(_HERE, "rmat_gen.c")
    out = os.path.join(_HERE, "_rmat_gen.so")
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", out, src])
    return out


def _native():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build_native())
        lib.rmat_pairs.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int64, ctypes.c_int,
                                   ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                   ctypes.c_void_p, ctypes.c_void_p]
        lib.rmat_pairs.restype = None
        _lib = lib
    return _lib


# --------------------------------------------------------------------------------------------
# graphs
# --------------------------------------------------------------------------------------------
def _sorted_unique(k: np.ndarray) -> np.ndarray:
    """Sorted distinct values (in-place sort + neighbour compare)."""
    k.sort()
    if k.size == 0:
        return k
    keep = np.empty(k.size, dtype=bool)
    keep[0] = True
    np.not_equal(k[1:], k[:-1], out=keep[1:])
    return k[keep]


def er_graph(n: int, m: int, seed: int) -> Tuple[np.ndarray, np.ndarray]:
    """Directed G(n, M): exactly m distinct ordered pairs, no self-loops."""
    rng = _rng(seed, "graph")
    keys = np.empty(0, dtype=np.int64)
    while keys.size < m:
        need = m - keys.size
        u = rng.integers(0, n, size=need + need // 8 + 16, dtype=np.int64)
        v = rng.integers(0, n, size=u.size, dtype=np.int64)
        k = (u * n + v)[u != v]
        k = k[~np.isin(k, keys)]
        _, first = np.unique(k, return_index=True)
        k = k[np.sort(first)][:need]
        keys = np.concatenate([keys, k])
    return (keys // n).astype(np.int32), (keys % n).astype(np.int32)


def rmat_graph(n: int, m: int, seed: int, a: float = 0.57, b: float = 0.19, c: float = 0.19
               ) -> Tuple[np.ndarray, np.ndarray]:
    """R-MAT graph with exactly m distinct directed edges on n vertices, no self-loops.

    scale = ceil(log2 n); pairs with an endpoint >= n, self-loops and duplicates are rejected.
    Candidates are drawn in rounds; if a round overshoots, a seeded uniformly random subset of
    the distinct pairs is dropped.  Vertex ids are then relabelled by one seeded permutation and
    the edge order is shuffled.
    """
    lib = _native()
    scale = max(1, int(np.ceil(np.log2(n))))
    keys = np.empty(0, dtype=np.int64)
    drawn = 0
    yield_ = 1.0 / 1.35        # distinct new pairs per candidate, re-estimated after every round
    while keys.size < m:
        need = m - keys.size
        cnt = int(need * 1.35) + 1024 if drawn == 0 else int(need / max(yield_, 0.02) * 1.05) + 1024
        u = np.empty(cnt, dtype=np.int32)
        v = np.empty(cnt, dtype=np.int32)
        lib.rmat_pairs(ctypes.c_uint64(seed), ctypes.c_uint64(drawn), cnt, scale, a, b, c,
                       u.ctypes.data, v.ctypes.data)
        drawn += cnt
        ok = (u < n) & (v < n) & (u != v)
        k = u[ok].astype(np.int64) * n + v[ok]
        del u, v, ok
        before = keys.size
        keys = _sorted_unique(np.concatenate([keys, k])) if before else _sorted_unique(k)
        yield_ = max(keys.size - before, 1) / cnt
    if keys.size > m:
        drop = _rng(seed, "drop").choice(keys.size, size=keys.size - m, replace=False)
        mask = np.ones(keys.size, dtype=bool)
        mask[drop] = False
        keys = keys[mask]
    perm = _rng(seed, "perm").permutation(n).astype(np.int32)
    order = _rng(seed, "order").permutation(m)
    src = perm[keys // n][order]
    dst = perm[keys % n][order]
    return np.ascontiguousarray(src, dtype=np.int32), np.ascontiguousarray(dst, dtype=np.int32)


def edge_weights(m: int, seed: int, stream: str = "edge_weights") -> np.ndarray:
    """m fp32 edge weights ~ U(0.1, 1), in the order of the graph's edge arrays."""
    return _rng(seed, stream).uniform(0.1, 1.0, size=m).astype(np.float32)


def features(n: int, d: int, seed: int, stream: str = "features") -> np.ndarray:
    """n x d fp32 rows ~ N(0, 1)."""
    return _rng(seed, stream).standard_normal((n, d), dtype=np.float32)


# --------------------------------------------------------------------------------------------
# models
# --------------------------------------------------------------------------------------------
@dataclass
class LayerSpec:
    kind: int
    d_in: int
    d_out: int
    act: int
    d_hidden: int = 0          # GIN: width of the MLP's hidden layer; attention: width of W h
    eps: float = 0.0           # GIN: eps; attention: slope of the logit for negative arguments (1 = linear)


@dataclass
class ModelSpec:
    agg: int
    layers: List[LayerSpec]

    @property
    def dims(self) -> List[int]:
        return [self.layers[0].d_in] + [l.d_out for l in self.layers]

    @property
    def self_term(self) -> bool:
        return self.layers[0].kind != KIND_GRAPHCONV

    @property
    def src_norm(self) -> bool:
        return self.agg == AGG_WSUM_GCN


def sage_model(dims: List[int], agg: int = AGG_MEAN, last_act: int = ACT_IDENTITY) -> ModelSpec:
    L = len(dims) - 1
    return ModelSpec(agg, [LayerSpec(KIND_SAGE, dims[i], dims[i + 1],
                                     ACT_RELU if i < L - 1 else last_act) for i in range(L)])


def graphconv_model(dims: List[int], agg: int, last_act: int = ACT_IDENTITY) -> ModelSpec:
    L = len(dims) - 1
    return ModelSpec(agg, [LayerSpec(KIND_GRAPHCONV, dims[i], dims[i + 1],
                                     ACT_RELU if i < L - 1 else last_act) for i in range(L)])


def gin_model(d0: int, hidden: int, n_layers: int, eps: float = 0.0,
              last_act: int = ACT_IDENTITY) -> ModelSpec:
    dims = [d0] + [hidden] * n_layers
    return ModelSpec(AGG_SUM, [LayerSpec(KIND_GIN, dims[i], dims[i + 1],
                                         ACT_RELU if i < n_layers - 1 else last_act,
                                         d_hidden=hidden, eps=eps) for i in range(n_layers)])


def gat_model(d: int, n_layers: int, d_att: int = 8, slope: float = 1.0,
              act: int = ACT_IDENTITY) -> ModelSpec:
    """Attention layers: every layer keeps the width d (the output is a convex combination of
    in-neighbour rows); d_att is the width of W h that the attention vector a reads."""
    return ModelSpec(AGG_SUM, [LayerSpec(KIND_GAT, d, d, act, d_hidden=d_att, eps=slope)
                               for _ in range(n_layers)])


def _glorot(rng: np.random.Generator, fan_in: int, fan_out: int) -> np.ndarray:
    a = np.sqrt(6.0 / (fan_in + fan_out))
    return rng.uniform(-a, a, size=(fan_in, fan_out)).astype(np.float32)


def make_weights(model: ModelSpec, seed: int, zero_bias: bool = True) -> List[Dict[str, np.ndarray]]:
    """Glorot-uniform matrices (input-major: fan_in x fan_out, row-major), one dict per layer.

    SAGE: Wa = W_self, Wb = W_neigh, ba.   GraphConv: Wa, ba.   GIN: Wa (d_in x hid), ba,
    Wb (hid x d_out), bb.   Attention: Wa = W (d_in x d_att), ba / bb = halves of a (never zeroed).  Biases are zero unless zero_bias is False (then small uniform).
    """
    rng = _rng(seed, "weights")
    out = []
    for l in model.layers:
        def bias(n):
            if zero_bias:
                return np.zeros(n, dtype=np.float32)
            return rng.uniform(-0.1, 0.1, size=n).astype(np.float32)
        if l.kind == KIND_SAGE:
            w = {"Wa": _glorot(rng, l.d_in, l.d_out), "Wb": _glorot(rng, l.d_in, l.d_out),
                 "ba": bias(l.d_out)}
        elif l.kind == KIND_GRAPHCONV:
            w = {"Wa": _glorot(rng, l.d_in, l.d_out), "ba": bias(l.d_out)}
        elif l.kind == KIND_GAT:   # Wa = W (d_in x d_att); ba, bb = the source and sink halves of a
            a = _glorot(rng, 2 * l.d_hidden, 1).reshape(-1)
            w = {"Wa": _glorot(rng, l.d_in, l.d_hidden), "ba": a[:l.d_hidden].copy(),
                 "bb": a[l.d_hidden:].copy()}
        else:
            w = {"Wa": _glorot(rng, l.d_in, l.d_hidden), "ba": bias(l.d_hidden),
                 "Wb": _glorot(rng, l.d_hidden, l.d_out), "bb": bias(l.d_out)}
        out.append(w)
    return out


# --------------------------------------------------------------------------------------------
# update streams
# --------------------------------------------------------------------------------------------
class UpdateStream:
    """Batches of edge additions, edge deletions and feature replacements.

    Each update's type is drawn i.i.d. from (p_add, p_del, p_feat).  An addition is a uniform
    ordered pair u != v that is not an edge of the current graph; a deletion is uniform over the
    current edges; a feature update names a uniform vertex and carries a fresh N(0,1) row.  No
    pair and no feature vertex appears twice within one batch.  The stream keeps its own record
    of which edges exist, so it needs no feedback from whoever applies the batches.

    With `hubs` given (an array of vertex ids), endpoints are restricted to hubs: additions join
    two hubs, a deletion removes a uniform current out-edge of a uniformly drawn hub, feature
    updates name hubs.

    A fourth entry in `mix` is the share of vertex deletions (a uniform vertex; every edge at it
    goes, its feature row becomes zeros; the id may be named again by later updates).
    """

    def __init__(self, n: int, src: np.ndarray, dst: np.ndarray, d0: int, seed: int,
                 stream: str = "updates", mix: Tuple[float, float, float] = (0.4, 0.4, 0.2),
                 hubs: Optional[np.ndarray] = None):
        self.n = int(n)
        self.d0 = int(d0)
        self.rng = _rng(seed, stream)
        self.mix = np.asarray(mix, dtype=np.float64)
        self.init_keys = np.sort(src.astype(np.int64) * self.n + dst.astype(np.int64))
        self.e0 = self.init_keys.size
        self.touched: Dict[int, bool] = {}       # pair key -> currently an edge?
        self.added: List[int] = []               # live edges that are not initial edges
        self.added_pos: Dict[int, int] = {}
        self.hubs = None if hubs is None else np.asarray(hubs, dtype=np.int64)
        self.n_edges = self.e0
        self.wrng = _rng(seed, "update_weights")   # weights of added edges: a stream of its own
        self.init_in_keys = None
        if self.mix.size > 3 and self.mix[3] > 0:   # in-edge index, only needed to delete vertices
            self.init_in_keys = np.sort(dst.astype(np.int64) * self.n + src.astype(np.int64))

    # -- membership ---------------------------------------------------------------------
    def _in_init(self, key: int) -> bool:
        i = int(np.searchsorted(self.init_keys, key))
        return i < self.e0 and int(self.init_keys[i]) == key

    def _present(self, key: int) -> bool:
        t = self.touched.get(key)
        return self._in_init(key) if t is None else t

    def _set(self, key: int, present: bool) -> None:
        was_init = self._in_init(key)
        self.touched[key] = present
        if not was_init:
            if present:
                self.added_pos[key] = len(self.added)
                self.added.append(key)
            else:
                i = self.added_pos.pop(key)
                last = self.added.pop()
                if last != key:
                    self.added[i] = last
                    self.added_pos[last] = i
        self.n_edges += 1 if present else -1

    def _remove_vertex(self, w: int) -> None:
        n = self.n
        lo, hi = np.searchsorted(self.init_keys, [w * n, (w + 1) * n])
        keys = [int(k) for k in self.init_keys[lo:hi]]
        lo, hi = np.searchsorted(self.init_in_keys, [w * n, (w + 1) * n])
        keys += [int(k % n) * n + w for k in self.init_in_keys[lo:hi]]
        keys += [k for k in self.added if k // n == w or k % n == w]
        for key in set(keys):
            if self._present(key):
                self._set(key, False)

    # -- draws --------------------------------------------------------------------------
    def _draw_vertex(self) -> int:
        if self.hubs is not None:
            return int(self.hubs[self.rng.integers(0, self.hubs.size)])
        return int(self.rng.integers(0, self.n))

    def _draw_add(self, in_batch) -> int:
        while True:
            u, v = self._draw_vertex(), self._draw_vertex()
            key = u * self.n + v
            if u != v and key not in in_batch and not self._present(key):
                return key

    def _draw_del(self, in_batch) -> Optional[int]:
        if self.n_edges - len(in_batch) <= 0:
            return None
        for _ in range(100000):
            if self.hubs is not None:
                u = self._draw_vertex()
                lo = int(np.searchsorted(self.init_keys, u * self.n))
                hi = int(np.searchsorted(self.init_keys, (u + 1) * self.n))
                if hi == lo:
                    continue
                key = int(self.init_keys[self.rng.integers(lo, hi)])
            else:
                r = int(self.rng.integers(0, self.e0 + len(self.added)))
                key = int(self.init_keys[r]) if r < self.e0 else self.added[r - self.e0]
            if key not in in_batch and self._present(key):
                return key
        return None

    def next_batch(self, b: int) -> Tuple[np.ndarray, np.ndarray]:
        """Returns (updates[b] of UPDATE_DTYPE, feature_rows[n_feat, d0] fp32)."""
        kinds = self.rng.choice(self.mix.size, size=b, p=self.mix)
        ups = np.zeros(b, dtype=UPDATE_DTYPE)
        rows: List[np.ndarray] = []
        in_batch = set()
        feat_seen = set()
        for i, k in enumerate(kinds):
            if k == OP_DEL_EDGE:
                key = self._draw_del(in_batch)
                if key is None:
                    k = OP_ADD_EDGE
            if k == OP_ADD_EDGE:
                key = self._draw_add(in_batch)
            if k == OP_DEL_VERTEX:
                ups[i] = (OP_DEL_VERTEX, self._draw_vertex(), 0)
            elif k == OP_SET_FEATURE:
                while True:
                    v = self._draw_vertex()
                    if v not in feat_seen:
                        break
                feat_seen.add(v)
                ups[i] = (OP_SET_FEATURE, v, len(rows))
                rows.append(self.rng.standard_normal(self.d0, dtype=np.float32))
            else:
                in_batch.add(key)
                ups[i] = (k, key // self.n, key % self.n)
        # the stream's own record of the graph, operation by operation
        for rec in ups:
            if rec["op"] == OP_DEL_VERTEX:
                self._remove_vertex(int(rec["u"]))
            elif rec["op"] != OP_SET_FEATURE:
                key, want = int(rec["u"]) * self.n + int(rec["v"]), rec["op"] == OP_ADD_EDGE
                if self._present(key) != want:
                    self._set(key, bool(want))
        feat = np.stack(rows) if rows else np.zeros((0, self.d0), dtype=np.float32)
        return ups, np.ascontiguousarray(feat, dtype=np.float32)


    def next_batch_weighted(self, b: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """next_batch plus one fp32 weight ~ U(0.1, 1) per update (it matters for edge additions only)."""
        ups, feat = self.next_batch(b)
        return ups, feat, self.wrng.uniform(0.1, 1.0, size=b).astype(np.float32)


def top_out_degree(n: int, src: np.ndarray, frac: float = 0.01) -> np.ndarray:
    """Ids of the ceil(frac * n) vertices of largest out-degree (ties broken by lower id)."""
    deg = np.bincount(src, minlength=n)
    k = int(np.ceil(frac * n))
    order = np.lexsort((np.arange(n), -deg))
    return np.sort(order[:k]).astype(np.int32)


# --------------------------------------------------------------------------------------------
# named workloads
# --------------------------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    n: int
    e: int
    graph: str                 # "er" | "rmat"
    model: ModelSpec
    seed: int = 0
    batch_sizes: Tuple[int, ...] = (100,)
    n_batches: int = 100
    extra: dict = field(default_factory=dict)


def workloads() -> Dict[str, Workload]:
    n_s, e_s = 169_343, 1_166_243
    n_d, e_d = 2_449_029, 123_718_280
    return {
        "tiny": Workload("tiny", 2000, 20000, "er", sage_model([32, 32, 16]), 0, (100,), 10),
        "sparse": Workload("sparse", n_s, e_s, "rmat", sage_model([128, 256, 40]), 0,
                           (1, 10, 100, 1000), 100),
        "sparse-deep-gin": Workload("sparse-deep-gin", n_s, e_s, "rmat", gin_model(128, 256, 3), 0,
                                    (100, 1000), 100),
        "sparse-deep-gcn": Workload("sparse-deep-gcn", n_s, e_s, "rmat",
                                    graphconv_model([128, 256, 256, 40], AGG_WSUM_GCN), 0,
                                    (100, 1000), 100),
        "dense-2l": Workload("dense-2l", n_d, e_d, "rmat", sage_model([100, 256, 47]), 0,
                             (10, 100, 1000, 10000), 100),
        # a smaller graph of the same kind and the same model as dense-2l: larger than L2, small
        # enough to profile (a few GB on the device)
        "mid-2l": Workload("mid-2l", 1_000_000, 30_000_000, "rmat", sage_model([100, 256, 47]), 0,
                           (1000,), 20),
        "mid-3l": Workload("mid-3l", 1_000_000, 30_000_000, "rmat", sage_model([100, 256, 256, 47]), 0,
                           (1000,), 20),
        "dense-3l": Workload("dense-3l", n_d, e_d, "rmat", sage_model([100, 256, 256, 47]), 0,
                             (10, 100, 1000, 10000), 100),
        "dense-4l": Workload("dense-4l", n_d, e_d, "rmat", sage_model([100, 256, 256, 256, 47]), 0,
                             (100, 1000), 20),
        # ultra-dense second graph shaped like the paper's social-network dataset (Table 2: 233 K
        # vertices, 114.9 M edges, average in-degree 492, 602 features, 41 classes)
        "reddit-2l": Workload("reddit-2l", 232_965, 114_900_000, "rmat", sage_model([602, 256, 41]), 0,
                              (10, 100, 1000), 20),
        "reddit-4l": Workload("reddit-4l", 232_965, 114_900_000, "rmat",
                              sage_model([602, 256, 256, 256, 41]), 0, (100, 1000), 20),
        # GraphConv with max (the paper's GC-X workload, Sec. 6.1): hybrid-incremental propagation
        "sparse-gcx": Workload("sparse-gcx", n_s, e_s, "rmat", graphconv_model([128, 256, 40], AGG_MAX), 0,
                               (1, 10, 100, 1000), 100),
        "mid-gcx-2l": Workload("mid-gcx-2l", 1_000_000, 30_000_000, "rmat", graphconv_model([100, 256, 47], AGG_MAX), 0,
                               (1000,), 20),
        "dense-gcx-2l": Workload("dense-gcx-2l", n_d, e_d, "rmat", graphconv_model([100, 256, 47], AGG_MAX), 0,
                                 (10, 100, 1000), 20),
        # GraphConv with a stored weight per edge (the paper's GC-W workload, Sec. 6.1.1)
        "sparse-gcw": Workload("sparse-gcw", n_s, e_s, "rmat", graphconv_model([128, 256, 40], AGG_WSUM_EDGE), 0,
                               (1, 10, 100, 1000), 100, {"edge_weights": True}),
        "dense-gcw-2l": Workload("dense-gcw-2l", n_d, e_d, "rmat", graphconv_model([100, 256, 47], AGG_WSUM_EDGE), 0,
                                 (100, 1000), 20, {"edge_weights": True}),
        # attention layers (the paper's GA-A workload, Sec. 6.1.1): hybrid-incremental propagation; the
        # layer of Eq. 3 keeps its input's width, logits go through the leaky rectifier of the cited architecture
        "sparse-gat": Workload("sparse-gat", n_s, e_s, "rmat", gat_model(128, 2, d_att=8, slope=0.2), 0,
                               (1, 10, 100, 1000), 100),
        "mid-gat-2l": Workload("mid-gat-2l", 1_000_000, 30_000_000, "rmat", gat_model(100, 2, d_att=8, slope=0.2), 0,
                               (1000,), 20),
        "dense-gat-2l": Workload("dense-gat-2l", n_d, e_d, "rmat", gat_model(100, 2, d_att=8, slope=0.2), 0,
                                 (10, 100, 1000), 20),
        "dense-gat-3l": Workload("dense-gat-3l", n_d, e_d, "rmat", gat_model(100, 3, d_att=8, slope=0.2), 0,
                                 (100, 1000), 20),
        # all five update types of Sec. 3.1: 2 % of the updates delete a vertex
        "sparse-vdel": Workload("sparse-vdel", n_s, e_s, "rmat", sage_model([128, 256, 40]), 0, (100, 1000), 100,
                                {"mix": (0.39, 0.39, 0.2, 0.02), "max_batch": 65536}),
        # hub stress: every endpoint is one of the top-1 % out-degree vertices of the initial graph
        "dense-3l-hub-feature": Workload("dense-3l-hub-feature", n_d, e_d, "rmat",
                                         sage_model([100, 256, 256, 47]), 0, (1, 10, 100, 1000), 20,
                                         {"hubs": True, "mix": (0.0, 0.0, 1.0)}),
        "dense-3l-hub-delete": Workload("dense-3l-hub-delete", n_d, e_d, "rmat",
                                        sage_model([100, 256, 256, 47]), 0, (1, 10, 100, 1000), 20,
                                        {"hubs": True, "mix": (0.1, 0.8, 0.1)}),
    }


def make_stream(w: Workload, src: np.ndarray, dst: np.ndarray, seed: Optional[int] = None,
                stream: str = "updates") -> "UpdateStream":
    """The update stream of a named workload (hub-restricted for the hub-stress workloads)."""
    hubs = top_out_degree(w.n, src) if w.extra.get("hubs") else None
    return UpdateStream(w.n, src, dst, w.model.dims[0], w.seed if seed is None else seed, stream=stream,
                        mix=w.extra.get("mix", (0.4, 0.4, 0.2)), hubs=hubs)


def make_graph(w: Workload) -> Tuple[np.ndarray, np.ndarray]:
    if w.graph == "er":
        return er_graph(w.n, w.e, w.seed)
    return rmat_graph(w.n, w.e, w.seed)
