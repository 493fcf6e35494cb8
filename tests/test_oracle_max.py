"""Pins for the oracle's monotonic (max) aggregation, Sec. 3.4.2: full inference against a dense
brute force, the paper's three worked cases, and the hybrid-incremental route against full
recomputation, including which vertices it may call affected.  No GPU needed."""
import os
import sys

import numpy as np
import pytest

sys.path.insert(0, os.path.dirname(__file__))
import test_oracle_pins as P  # noqa: E402
from test_oracle_vertex_ops import random_batch, replay  # noqa: E402

from paper_2601_12347_b200 import inputs as I  # noqa: E402
from oracle.oracle import Oracle  # noqa: E402


def dense_full_max(n, src, dst, X, model, weights):
    """GraphConv with an element-wise maximum (minimum) over the in-neighbours, written with an
    explicit n x n adjacency matrix: x_v = max_{u : A[u, v]} h_u (zeros if v has no in-neighbour)."""
    red = np.min if model.agg == I.AGG_MIN else np.max
    A = np.zeros((n, n), dtype=bool)
    A[src, dst] = True
    H = [X.astype(np.float64)]
    for ly, w in zip(model.layers, weights):
        agg = np.zeros((n, H[-1].shape[1]))
        for v in range(n):
            nb = np.nonzero(A[:, v])[0]
            if nb.size:
                agg[v] = red(H[-1][nb], axis=0)
        Z = agg @ w["Wa"].astype(np.float64) + w["ba"]
        H.append(np.maximum(Z, 0.0) if ly.act == I.ACT_RELU else Z)
    return H


def max_model(dims, agg=I.AGG_MAX):
    return I.graphconv_model(dims, agg)


AGGS = [I.AGG_MAX, I.AGG_MIN]


@pytest.mark.parametrize("agg", AGGS, ids=["max", "min"])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_full_matches_dense_definition(seed, agg):
    m = max_model([5, 6, 4, 3], agg)
    n = 14
    src, dst = P.random_graph(n, 30, seed)
    X = I.features(n, 5, seed)
    W = I.make_weights(m, seed, zero_bias=False)
    o = Oracle(n, src, dst, X, m, W)
    ref = dense_full_max(n, src, dst, X, m, W)
    full = o.full()
    for l in range(4):
        assert P.rel_err(full[l], ref[l]) < 1e-12
        assert P.rel_err(o.H(l), ref[l]) < 1e-12          # the bootstrap state
    deg_in = np.bincount(dst, minlength=n)
    assert np.all(o.full_S(1)[deg_in == 0] == 0.0)
    v = int(np.argmax(deg_in))
    nb = src[dst == v]
    red = np.min if agg == I.AGG_MIN else np.max
    assert np.array_equal(o.full_S(1)[v], red(X[nb].astype(np.float64), axis=0))


def _three_cases():
    """Sec. 3.4.2, Fig. "max cases": A aggregates B (5) and C; the cached maximum at A and the
    change at C decide between no-op, incremental update and recomputation."""
    spec = {}
    for line in open(os.path.join(P.GOLD, "max_cases.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split(":")
            spec[k] = [float(x) for x in v.split()]
    return spec


@pytest.mark.parametrize("case", ["noop", "incremental", "recompute"])
def test_worked_cases_of_the_paper(case):
    spec = _three_cases()
    b, c_old, c_new, a_before, a_after = spec[case]
    A_, B_, C_ = 0, 1, 2
    src = np.array([B_, C_], dtype=np.int32)
    dst = np.array([A_, A_], dtype=np.int32)
    m = max_model([1, 1])
    X = np.array([[0.0], [b], [c_old]], dtype=np.float32)
    W = [{"Wa": np.ones((1, 1), dtype=np.float32), "ba": np.zeros(1, dtype=np.float32)}]
    o = Oracle(3, src, dst, X, m, W)
    assert o.S(1)[A_, 0] == a_before
    assert o.apply_incremental(P.ups_array([(I.OP_SET_FEATURE, C_, 0)]), np.array([[c_new]], dtype=np.float32)) == 0
    assert o.S(1)[A_, 0] == a_after and o.H(1)[A_, 0] == a_after
    assert np.array_equal(o.affected(0), np.array([C_], dtype=np.int32))
    want = np.array([A_], dtype=np.int32) if a_after != a_before else np.zeros(0, dtype=np.int32)
    assert np.array_equal(o.affected(1), want)             # an unchanged maximum is not propagated


@pytest.mark.parametrize("agg", AGGS, ids=["max", "min"])
@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_hybrid_incremental_equals_full_recompute(seed, agg):
    m = max_model([6, 8, 5, 4], agg)
    L = 3
    n = 40
    src, dst = P.random_graph(n, 150, 60 + seed)
    X = I.features(n, 6, seed)
    W = I.make_weights(m, seed, zero_bias=False)
    o = Oracle(n, src, dst, X, m, W)
    edges = set(zip(src.tolist(), dst.tolist()))
    Xcur = X.copy()
    rng = np.random.default_rng(seed)
    pruned = 0
    o.full()   # fills the full-recompute buffers that full_S views
    for b in range(12):
        rows = I.features(5, 6, 900 + 20 * seed + b)
        recs = random_batch(rng, n, edges, int(rng.integers(1, 12)), 5, p_vertex=0.08)
        S_old = [None] + [o.full_S(l).copy() for l in range(1, L + 1)]
        H_old = [o.H(l).copy() for l in range(L + 1)]
        edges, feat = replay(edges, recs)
        for v, r in feat.items():
            Xcur[v] = rows[r] if r >= 0 else 0.0
        assert o.apply_incremental(P.ups_array(recs), rows) == 0
        e = sorted(edges)
        ref = dense_full_max(n, np.array([a for a, _ in e], dtype=np.int32),
                             np.array([c for _, c in e], dtype=np.int32), Xcur, m, W)
        full = o.full()
        for l in range(L + 1):
            assert P.rel_err(o.H(l), ref[l]) < 1e-12, (seed, b, l)
            assert P.rel_err(full[l], ref[l]) < 1e-12
        for l in range(1, L + 1):
            S_new = o.full_S(l)
            assert np.array_equal(o.S(l), S_new), (seed, b, l)            # the cached maxima are exact copies
            changed = np.nonzero(np.any(S_new != S_old[l], axis=1))[0].astype(np.int32)
            assert np.array_equal(o.affected(l), changed), (seed, b, l)   # affected = cached row changed
            moved = np.nonzero(np.any(o.H(l) != H_old[l], axis=1))[0]
            assert set(moved.tolist()) <= set(changed.tolist())
        # the structural frontier of the same batch would be larger: pruning happened somewhere
        reach = set(v for (u, v) in edges if u in feat)
        pruned += len(reach - set(o.affected(1).tolist()))
    assert pruned > 0


def test_empty_in_list_transitions_and_negative_maxima():
    """A sink without in-neighbours caches zeros, which is not a maximum: gaining its first
    in-neighbour with negative features must lower the row below zero, losing the last one must
    return it to zero."""
    m = max_model([2, 2])
    for ly in m.layers:
        ly.act = I.ACT_IDENTITY
    X = np.array([[0.5, 0.5], [-3.0, -1.0], [-2.0, -4.0], [9.0, 9.0]], dtype=np.float32)
    W = [{"Wa": np.eye(2, dtype=np.float32), "ba": np.zeros(2, dtype=np.float32)}]
    src = np.array([3], dtype=np.int32)
    dst = np.array([3], dtype=np.int32)          # vertex 0 starts isolated
    o = Oracle(4, src, dst, X, m, W)
    assert np.all(o.S(1)[0] == 0.0)
    assert o.apply_incremental(P.ups_array([(I.OP_ADD_EDGE, 1, 0)])) == 0
    assert np.array_equal(o.S(1)[0], [-3.0, -1.0])
    assert o.apply_incremental(P.ups_array([(I.OP_ADD_EDGE, 2, 0)])) == 0
    assert np.array_equal(o.S(1)[0], [-2.0, -1.0])
    assert o.apply_incremental(P.ups_array([(I.OP_DEL_EDGE, 1, 0)])) == 0
    assert np.array_equal(o.S(1)[0], [-2.0, -4.0])
    assert o.apply_incremental(P.ups_array([(I.OP_DEL_EDGE, 2, 0)])) == 0
    assert np.all(o.S(1)[0] == 0.0) and np.array_equal(o.affected(1), np.array([0], dtype=np.int32))
    full = o.full()
    assert np.array_equal(o.H(1), full[1])


def test_gin_layers_are_refused():
    m = I.gin_model(4, 4, 2)
    m.agg = I.AGG_MAX
    src, dst = P.random_graph(10, 20, 1)
    o = Oracle(10, src, dst, I.features(10, 4, 1), m, I.make_weights(m, 1))
    assert o.apply_incremental(P.ups_array([(I.OP_ADD_EDGE, 0, 1)])) != 0


def dense_full_sage_max(n, src, dst, X, model, weights):
    A = np.zeros((n, n), dtype=bool)
    A[src, dst] = True
    red = np.min if model.agg == I.AGG_MIN else np.max
    H = [X.astype(np.float64)]
    for ly, w in zip(model.layers, weights):
        agg = np.zeros((n, H[-1].shape[1]))
        for v in range(n):
            nb = np.nonzero(A[:, v])[0]
            if nb.size:
                agg[v] = red(H[-1][nb], axis=0)
        Z = H[-1] @ w["Wa"].astype(np.float64) + agg @ w["Wb"].astype(np.float64) + w["ba"]
        H.append(np.maximum(Z, 0.0) if ly.act == I.ACT_RELU else Z)
    return H


@pytest.mark.parametrize("agg", AGGS, ids=["max", "min"])
@pytest.mark.parametrize("seed", [0, 1])
def test_self_term_with_a_monotonic_aggregator(seed, agg):
    """SAGE layers: h = act(W_self h_v + W_neigh max_u h_u + b).  A vertex is affected when its
    cached maximum or its own previous-layer row changed."""
    m = I.sage_model([6, 8, 5, 4], agg)
    L, n = 3, 40
    src, dst = P.random_graph(n, 150, 70 + seed)
    X = I.features(n, 6, seed)
    W = I.make_weights(m, seed, zero_bias=False)
    o = Oracle(n, src, dst, X, m, W)
    edges = set(zip(src.tolist(), dst.tolist()))
    Xcur = X.copy()
    rng = np.random.default_rng(seed)
    o.full()
    for b in range(10):
        rows = I.features(5, 6, 400 + 20 * seed + b)
        recs = random_batch(rng, n, edges, int(rng.integers(1, 12)), 5, p_vertex=0.08)
        S_old = [None] + [o.full_S(l).copy() for l in range(1, L + 1)]
        H_old = [o.H(l).copy() for l in range(L + 1)]
        edges, feat = replay(edges, recs)
        for v, r in feat.items():
            Xcur[v] = rows[r] if r >= 0 else 0.0
        assert o.apply_incremental(P.ups_array(recs), rows) == 0
        e = sorted(edges)
        ref = dense_full_sage_max(n, np.array([a for a, _ in e], dtype=np.int32),
                                  np.array([c for _, c in e], dtype=np.int32), Xcur, m, W)
        o.full()
        for l in range(L + 1):
            assert P.rel_err(o.H(l), ref[l]) < 1e-12, (seed, b, l)
        for l in range(1, L + 1):
            S_new = o.full_S(l)
            assert np.array_equal(o.S(l), S_new)
            changed = set(np.nonzero(np.any(S_new != S_old[l], axis=1))[0].tolist())
            own = set(np.nonzero(np.any(o.H(l - 1).astype(np.float32) != H_old[l - 1].astype(np.float32), axis=1))[0].tolist())
            assert set(o.affected(l).tolist()) == changed | own, (seed, b, l)


def test_min_is_the_mirror_image_of_max():
    """With the identity activation, negating features and the first layer's weights turns a
    min model into the max model of the negated inputs: the two oracles must agree row by row."""
    n = 30
    src, dst = P.random_graph(n, 100, 5)
    X = I.features(n, 4, 5)
    mmax, mmin = max_model([4, 3], I.AGG_MAX), max_model([4, 3], I.AGG_MIN)
    for ly in mmax.layers + mmin.layers:
        ly.act = I.ACT_IDENTITY
    W = I.make_weights(mmax, 5, zero_bias=False)
    Wneg = [{"Wa": -W[0]["Wa"], "ba": W[0]["ba"]}]
    omax = Oracle(n, src, dst, -X, mmax, Wneg)
    omin = Oracle(n, src, dst, X, mmin, W)
    assert np.array_equal(omax.H(1), omin.H(1)) and np.array_equal(omax.S(1), -omin.S(1))
    rows = I.features(3, 4, 6)
    recs = [(I.OP_SET_FEATURE, 2, 0), (I.OP_DEL_EDGE, int(src[0]), int(dst[0])), (I.OP_ADD_EDGE, 1, 7),
            (I.OP_SET_FEATURE, 9, 1), (I.OP_DEL_VERTEX, 11, 0)]
    assert omax.apply_incremental(P.ups_array(recs), -rows) == 0
    assert omin.apply_incremental(P.ups_array(recs), rows) == 0
    assert np.array_equal(omax.H(1), omin.H(1)) and np.array_equal(omax.S(1), -omin.S(1))
    assert np.array_equal(omax.affected(1), omin.affected(1))


@pytest.mark.parametrize("agg", AGGS, ids=["max", "min"])
def test_scoped_recompute_route_agrees_for_monotonic_aggregators(agg):
    """The scoped route (Sec. 3.2) recomputes every structurally reachable vertex; its embeddings must
    equal full recomputation, and its affected sets must contain the pruned ones of the hybrid route."""
    m = max_model([6, 8, 4], agg)
    n = 40
    src, dst = P.random_graph(n, 150, 8)
    X = I.features(n, 6, 8)
    W = I.make_weights(m, 8, zero_bias=False)
    a, b = Oracle(n, src, dst, X, m, W), Oracle(n, src, dst, X, m, W)
    stream = I.UpdateStream(n, src, dst, 6, 8)
    for _ in range(6):
        ups, rows = stream.next_batch(5)
        assert a.apply_incremental(ups, rows) == 0
        assert b.apply_scoped(ups, rows) == 0
        full = a.full()
        for l in range(3):
            assert P.rel_err(a.H(l), full[l]) < 1e-12 and P.rel_err(b.H(l), full[l]) < 1e-12
        for l in range(1, 3):
            assert set(a.affected(l).tolist()) <= set(b.affected(l).tolist())
