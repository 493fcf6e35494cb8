"""Pins of the oracle's route for the weighted sum with a stored weight per edge (Table 1; the
GC-W workload of Sec. 6.1.1): S_v = sum over in-neighbours u of alpha_uv h_u, messages
alpha_uv (h_u - h_u^-) along surviving edges, alpha_uv h_u along an added edge, -alpha_uv h_u^- along
a deleted one (Sec. 3.3.3, "other linear aggregators").

Reading where the paper is silent: weights are static.  An edge keeps the weight it was created
with for as long as it exists at batch boundaries: adding an edge that exists is a counted no-op
whatever weight comes with it, also when an earlier operation of the same batch deleted it.
"""
import numpy as np
import pytest

from paper_2601_12347_b200 import inputs as I
from oracle.oracle import Oracle

import test_oracle_pins as P


def dense_weighted(n, edges_w, X, model, W):
    """H^l = act(A_w^T H^{l-1} W + b) with the explicit n x n weight matrix (fp64)."""
    A = np.zeros((n, n))
    for (u, v), w in edges_w.items():
        A[u, v] = float(np.float32(w))
    H = [X.astype(np.float64)]
    for ly, wl in zip(model.layers, W):
        z = (A.T @ H[-1]) @ wl["Wa"].astype(np.float64) + wl["ba"].astype(np.float64)
        H.append(np.maximum(z, 0) if ly.act == I.ACT_RELU else z)
    return H


def setup(n=40, m=220, seed=3, dims=(5, 6, 3)):
    model = I.graphconv_model(list(dims), I.AGG_WSUM_EDGE)
    src, dst = P.random_graph(n, m, seed)
    w = I.edge_weights(m, seed)
    X = I.features(n, dims[0], seed)
    W = I.make_weights(model, seed, zero_bias=False)
    edges = {(int(a), int(b)): float(c) for a, b, c in zip(src, dst, w)}
    return n, src, dst, w, X, model, W, edges


def stored_weights(o):
    rowptr, col = o.export_csr()
    w = o.export_weights()
    return {(u, int(col[j])): float(w[j]) for u in range(len(rowptr) - 1) for j in range(rowptr[u], rowptr[u + 1])}


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_full_matches_the_weighted_dense_matrix_definition(seed):
    n, src, dst, w, X, model, W, edges = setup(seed=seed, dims=(5, 7, 4, 3))
    o = Oracle(n, src, dst, X, model, W, edge_weights=w)
    ref = dense_weighted(n, edges, X, model, W)
    full = o.full()
    for l in range(len(ref)):
        assert P.rel_err(full[l], ref[l]) < 1e-12
        assert P.rel_err(o.H(l), ref[l]) < 1e-12
    assert stored_weights(o) == {k: float(np.float32(v)) for k, v in edges.items()}


def test_hand_case_star_with_weights():
    # 1 -> 0 (0.5), 2 -> 0 (2.0), 0 -> 3 (4.0); one layer, identity matrix
    model = I.ModelSpec(I.AGG_WSUM_EDGE, [I.LayerSpec(I.KIND_GRAPHCONV, 2, 2, I.ACT_IDENTITY)])
    W = [{"Wa": np.eye(2, dtype=np.float32), "ba": np.zeros(2, dtype=np.float32)}]
    X = np.array([[1, 2], [10, 20], [100, 200], [7, 7]], dtype=np.float32)
    src = np.array([1, 2, 0], dtype=np.int32)
    dst = np.array([0, 0, 3], dtype=np.int32)
    o = Oracle(4, src, dst, X, model, W, edge_weights=np.array([0.5, 2.0, 4.0], dtype=np.float32))
    assert np.array_equal(o.H(1), np.array([[205, 410], [0, 0], [0, 0], [4, 8]], dtype=np.float64))
    # add 3 -> 0 with weight 0.25, delete 1 -> 0, change the row of vertex 2
    ups = P.ups_array([(I.OP_ADD_EDGE, 3, 0), (I.OP_DEL_EDGE, 1, 0), (I.OP_SET_FEATURE, 2, 0)])
    rows = np.array([[1, 1]], dtype=np.float32)
    assert o.apply_incremental(ups, rows, op_weights=np.array([0.25, 9.0, 9.0], dtype=np.float32)) == 0
    assert np.array_equal(o.H(1)[0], np.array([2.0 * 1 + 0.25 * 7, 2.0 * 1 + 0.25 * 7]))
    assert np.array_equal(o.affected(1), np.array([0], dtype=np.int32))


def test_unit_weights_reduce_to_the_plain_sum():
    n, src, dst, w, X, model, W, edges = setup(seed=5)
    plain = I.graphconv_model([5, 6, 3], I.AGG_SUM)
    a = Oracle(n, src, dst, X, model, W, edge_weights=np.ones_like(w))
    b = Oracle(n, src, dst, X, plain, W)
    stream = I.UpdateStream(n, src, dst, 5, 5)
    for _ in range(6):
        ups, rows = stream.next_batch(12)
        assert a.apply_incremental(ups, rows) == 0        # no weights given: additions carry weight 1
        assert b.apply_incremental(ups, rows) == 0
        for l in range(3):
            assert np.array_equal(a.H(l), b.H(l))
            assert np.array_equal(a.affected(l), b.affected(l))


@pytest.mark.parametrize("route", ["push", "pull", "scoped"])
def test_incremental_equals_full_recompute_every_batch(route):
    n, src, dst, w, X, model, W, edges = setup(n=60, m=400, seed=11, dims=(5, 6, 6, 3))
    o = Oracle(n, src, dst, X, model, W, edge_weights=w)
    stream = I.UpdateStream(n, src, dst, 5, 11, mix=(0.38, 0.38, 0.2, 0.04))
    Xcur = X.copy()
    for b in range(12):
        ups, rows, ow = stream.next_batch_weighted(2 + 3 * b)
        before = dict(edges)
        # literal replay, one operation after the other
        for i, r in enumerate(ups):
            op, u, v = int(r["op"]), int(r["u"]), int(r["v"])
            if op == I.OP_ADD_EDGE:
                edges.setdefault((u, v), float(ow[i]))
            elif op == I.OP_DEL_EDGE:
                edges.pop((u, v), None)
            elif op == I.OP_DEL_VERTEX:
                for k in [k for k in edges if u in k]:
                    del edges[k]
                Xcur[u] = 0.0
            else:
                Xcur[u] = rows[v]
        for k in edges:      # an edge that exists before and after the batch keeps its weight
            if k in before:
                edges[k] = before[k]
        if route == "scoped":
            assert o.apply_scoped(ups, rows, op_weights=ow) == 0
        else:
            assert o.apply_incremental(ups, rows, pull=route == "pull", op_weights=ow) == 0
        assert stored_weights(o) == {k: float(np.float32(v)) for k, v in edges.items()}, b
        ref = dense_weighted(n, edges, Xcur, model, W)
        full = o.full()
        for l in range(4):
            assert P.rel_err(full[l], ref[l]) < 1e-12
            assert P.rel_err(o.H(l), ref[l]) < 1e-9, (route, b, l)
        for l in range(1, 4):
            assert P.rel_err(o.S(l), o.full_S(l)) < 1e-9


@pytest.mark.parametrize("pull", [False, True], ids=["push", "pull"])
@pytest.mark.parametrize("op", ["add", "del", "feat", "feat+add+del"])
def test_single_update_rules(op, pull):
    n, src, dst, w, X, model, W, edges = setup(n=30, m=120, seed=5)
    o = Oracle(n, src, dst, X, model, W, edge_weights=w)
    X2 = X.copy()
    rows, ow = None, None
    if op == "add":
        u, v = next((a, b) for a in range(n) for b in range(n) if a != b and (a, b) not in edges)
        ups, ow = P.ups_array([(I.OP_ADD_EDGE, u, v)]), np.array([0.375], dtype=np.float32)
        edges[(u, v)] = 0.375
    elif op == "del":
        u, v = int(src[17]), int(dst[17])
        ups = P.ups_array([(I.OP_DEL_EDGE, u, v)])
        del edges[(u, v)]
    elif op == "feat":
        rows = I.features(1, 5, 99)
        ups = P.ups_array([(I.OP_SET_FEATURE, 9, 0)])
        X2[9] = rows[0]
    else:
        u, wv = int(src[17]), int(dst[17])
        v = next(b for b in range(n) if b != u and (u, b) not in edges)
        rows = I.features(1, 5, 98)
        ups = P.ups_array([(I.OP_SET_FEATURE, u, 0), (I.OP_ADD_EDGE, u, v), (I.OP_DEL_EDGE, u, wv)])
        ow = np.array([9.0, 0.625, 9.0], dtype=np.float32)
        X2[u] = rows[0]
        edges[(u, v)] = 0.625
        del edges[(u, wv)]
    assert o.apply_incremental(ups, rows, pull=pull, op_weights=ow) == 0
    ref = dense_weighted(n, edges, X2, model, W)
    for l in range(3):
        assert P.rel_err(o.H(l), ref[l]) < 1e-10, (op, l)


def test_existing_edges_keep_their_weight_and_add_then_delete_restores_everything():
    n, src, dst, w, X, model, W, edges = setup(n=30, m=120, seed=7)
    o = Oracle(n, src, dst, X, model, W, edge_weights=w)
    base = [o.H(l).copy() for l in range(3)]
    eu, ev = int(src[3]), int(dst[3])
    # adding an edge that exists: counted no-op, whatever weight comes with it -- also after a deletion in the same batch
    for recs in ([(I.OP_ADD_EDGE, eu, ev)], [(I.OP_DEL_EDGE, eu, ev), (I.OP_ADD_EDGE, eu, ev)]):
        assert o.apply_incremental(P.ups_array(recs), op_weights=np.full(len(recs), 77.0, dtype=np.float32)) == 0
        assert o.counts()["noop_add"] == 1 and o.counts()["added"] == 0 and o.counts()["deleted"] == 0
        assert stored_weights(o)[(eu, ev)] == float(w[3])
        for l in range(3):
            assert np.array_equal(o.H(l), base[l])
    u, v = next((a, b) for a in range(n) for b in range(n) if a != b and (a, b) not in edges)
    assert o.apply_incremental(P.ups_array([(I.OP_ADD_EDGE, u, v)]), op_weights=np.array([0.7], dtype=np.float32)) == 0
    assert stored_weights(o)[(u, v)] == float(np.float32(0.7))
    assert o.apply_incremental(P.ups_array([(I.OP_DEL_EDGE, u, v)])) == 0
    assert stored_weights(o) == {k: float(np.float32(x)) for k, x in edges.items()}
    for l in range(3):
        assert P.rel_err(o.H(l), base[l]) < 1e-12


def test_mutation_check_weight_of_the_right_edge():
    """A plausible mistake -- scaling a message by the wrong edge's weight -- cannot hide: with all
    weights distinct powers of two the sums identify every (edge, weight) pairing."""
    n = 6
    src = np.array([0, 0, 1, 2, 3], dtype=np.int32)
    dst = np.array([1, 2, 2, 3, 1], dtype=np.int32)
    w = np.array([1, 2, 4, 8, 16], dtype=np.float32)
    model = I.ModelSpec(I.AGG_WSUM_EDGE, [I.LayerSpec(I.KIND_GRAPHCONV, 1, 1, I.ACT_IDENTITY)])
    W = [{"Wa": np.ones((1, 1), dtype=np.float32), "ba": np.zeros(1, dtype=np.float32)}]
    X = np.array([[1], [10], [100], [1000], [0], [0]], dtype=np.float32)
    o = Oracle(n, src, dst, X, model, W, edge_weights=w)
    assert o.H(1)[:, 0].tolist() == [0, 1 * 1 + 16 * 1000, 2 * 1 + 4 * 10, 8 * 100, 0, 0]
    rows = np.array([[3]], dtype=np.float32)
    for pull in (False, True):
        assert o.apply_incremental(P.ups_array([(I.OP_SET_FEATURE, 0, 0)]), rows, pull=pull) == 0
        assert o.H(1)[:, 0].tolist() == [0, 1 * 3 + 16 * 1000, 2 * 3 + 4 * 10, 8 * 100, 0, 0]
        rows = rows * 2 - 3     # 3 again
