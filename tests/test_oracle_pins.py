"""Pins for the CPU oracle: it is checked against things other than itself.

  * the layer definition written as dense adjacency-matrix algebra (tiny graphs),
  * closed forms and hand-computed cases that fix edge direction, normalisation and widths,
  * the paper's worked example (tests/golden/fig4_edge_addition.txt),
  * the defining invariant of the method (Sec. 3.3.2, Sec. 5): after every batch the incremental
    result equals full recomputation on the updated graph, at every layer,
  * a structural brute force for the affected sets (computation-tree signatures),
  * the numeric footprint of a batch under identity activations.
"""
import os

import numpy as np
import pytest

from oracle.oracle import Oracle
from paper_2601_12347_b200 import inputs as I

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------------------------
# helpers
# ---------------------------------------------------------------------------------------------
def dense_full(n, src, dst, X, model, weights):
    """Eq. 1-2 with an explicit n x n adjacency matrix (A[u, v] = 1 for edge u -> v)."""
    A = np.zeros((n, n))
    A[src, dst] = 1.0
    deg_out, deg_in = A.sum(1), A.sum(0)
    H = [X.astype(np.float64)]
    for ly, w in zip(model.layers, weights):
        c = np.ones(n)
        norm = np.ones(n)
        if model.agg == I.AGG_WSUM_GCN:
            c = np.where(deg_out > 0, 1.0 / np.sqrt(np.maximum(deg_out, 1)), 0.0)
            norm = np.where(deg_in > 0, 1.0 / np.sqrt(np.maximum(deg_in, 1)), 0.0)
        elif model.agg == I.AGG_MEAN:
            norm = np.where(deg_in > 0, 1.0 / np.maximum(deg_in, 1), 0.0)
        agg = norm[:, None] * (A.T @ (c[:, None] * H[-1]))
        Wa = w["Wa"].astype(np.float64)
        if ly.kind == I.KIND_SAGE:
            Z = H[-1] @ Wa + agg @ w["Wb"].astype(np.float64) + w["ba"]
        elif ly.kind == I.KIND_GRAPHCONV:
            Z = agg @ Wa + w["ba"]
        else:
            T = np.maximum(((1.0 + ly.eps) * H[-1] + agg) @ Wa + w["ba"], 0.0)
            Z = T @ w["Wb"].astype(np.float64) + w["bb"]
        H.append(np.maximum(Z, 0.0) if ly.act == I.ACT_RELU else Z)
    return H


def all_models(d0=5, hid=6, out=3, acts_identity=False):
    la = I.ACT_IDENTITY
    ms = {
        "sage_mean": I.sage_model([d0, hid, out], I.AGG_MEAN),
        "sage_sum": I.sage_model([d0, hid, out], I.AGG_SUM),
        "sage_mean_3l": I.sage_model([d0, hid, hid, out], I.AGG_MEAN),
        "gc_sum": I.graphconv_model([d0, hid, out], I.AGG_SUM),
        "gc_mean": I.graphconv_model([d0, hid, hid, out], I.AGG_MEAN),
        "gcn_wsum": I.graphconv_model([d0, hid, hid, out], I.AGG_WSUM_GCN),
        "gin": I.gin_model(d0, hid, 3),
    }
    if acts_identity:
        for m in ms.values():
            for ly in m.layers:
                ly.act = la
    return ms


def random_graph(n, m, seed):
    return I.er_graph(n, m, seed)


def rel_err(a, b):
    return float(np.max(np.abs(a - b) / (1.0 + np.abs(b)))) if a.size else 0.0


def ups_array(recs):
    a = np.zeros(len(recs), dtype=I.UPDATE_DTYPE)
    for i, r in enumerate(recs):
        a[i] = r
    return a


# ---------------------------------------------------------------------------------------------
# O-full against the definition
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", list(all_models().keys()))
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_full_matches_dense_matrix_definition(name, seed):
    model = all_models()[name]
    n, m = 12, 40
    src, dst = random_graph(n, m, seed)
    # self-loops are ordinary edges: add one
    src = np.append(src, 3).astype(np.int32)
    dst = np.append(dst, 3).astype(np.int32)
    X = I.features(n, model.dims[0], seed)
    W = I.make_weights(model, seed, zero_bias=False)
    o = Oracle(n, src, dst, X, model, W)
    ref = dense_full(n, src, dst, X, model, W)
    got = o.full()
    for l in range(len(ref)):
        assert rel_err(got[l], ref[l]) < 1e-12, (name, l)
        assert rel_err(o.H(l), ref[l]) < 1e-12  # bootstrap state is the same thing


def test_closed_form_sum_identity():
    """Sum aggregation, no self term, identity activation, zero bias: H^L = (A^T)^L X W1..WL
    (the algebra behind the cancellation example of Sec. 3.3.3)."""
    n, m = 10, 30
    src, dst = random_graph(n, m, 7)
    model = I.graphconv_model([4, 5, 6, 3], I.AGG_SUM)
    for ly in model.layers:
        ly.act = I.ACT_IDENTITY
    X = I.features(n, 4, 7)
    W = I.make_weights(model, 7)
    A = np.zeros((n, n))
    A[src, dst] = 1
    ref = X.astype(np.float64)
    P = np.eye(n)
    for w in W:
        ref = ref @ w["Wa"].astype(np.float64)
        P = A.T @ P
    ref = P @ ref
    o = Oracle(n, src, dst, X, model, W)
    assert rel_err(o.H(3), ref) < 1e-12


def test_hand_cases_direction_and_normalisation():
    """Directed path 0 -> 1 -> 2 and a star, numbers small enough to check by hand.
    Edge (u, v): v aggregates u (Sec. 3.2: an addition (u, v) alters the sink v)."""
    eye = np.eye(2, dtype=np.float32)
    X = np.array([[1, 2], [10, 20], [100, 200]], dtype=np.float32)
    src = np.array([0, 1], dtype=np.int32)
    dst = np.array([1, 2], dtype=np.int32)
    # GraphConv, sum, W = I: h1 = [0, x0, x1], h2 = [0, 0, x0]
    m = I.graphconv_model([2, 2, 2], I.AGG_SUM)
    W = [{"Wa": eye.copy(), "ba": np.zeros(2, np.float32)} for _ in range(2)]
    o = Oracle(3, src, dst, X, m, W)
    assert np.array_equal(o.H(1), np.array([[0, 0], [1, 2], [10, 20]], dtype=np.float64))
    assert np.array_equal(o.H(2), np.array([[0, 0], [0, 0], [1, 2]], dtype=np.float64))
    # SAGE mean with W_self = I, W_neigh = 2I; star 1 -> 0, 2 -> 0; vertex 0 has in-degree 2,
    # vertices 1 and 2 are isolated on the in-side (aggregate 0).
    src = np.array([1, 2], dtype=np.int32)
    dst = np.array([0, 0], dtype=np.int32)
    m = I.sage_model([2, 2], I.AGG_MEAN)
    W = [{"Wa": eye.copy(), "Wb": 2 * eye, "ba": np.array([0.5, -0.5], np.float32)}]
    o = Oracle(3, src, dst, X, m, W)
    # h_0 = x0 + 2 * mean(x1, x2) + b = [1,2] + [110, 220] + [.5,-.5]
    assert np.array_equal(o.H(1)[0], np.array([111.5, 221.5]))
    assert np.array_equal(o.H(1)[1], np.array([10.5, 19.5]))
    assert np.array_equal(o.S(1)[0], np.array([110.0, 220.0]))  # un-normalised aggregate
    # weighted sum: edges 0->2, 1->2, 0->1: c_0 = 1/sqrt(2), c_1 = 1; deg_in(2) = 2
    src = np.array([0, 1, 0], dtype=np.int32)
    dst = np.array([2, 2, 1], dtype=np.int32)
    m = I.graphconv_model([2, 2], I.AGG_WSUM_GCN)
    W = [{"Wa": eye.copy(), "ba": np.zeros(2, np.float32)}]
    o = Oracle(3, src, dst, X, m, W)
    want2 = (X[0].astype(np.float64) / np.sqrt(2) + X[1]) / np.sqrt(2)
    want1 = X[0].astype(np.float64) / np.sqrt(2) / 1.0
    assert np.allclose(o.H(1)[2], want2, rtol=1e-15)
    assert np.allclose(o.H(1)[1], want1, rtol=1e-15)
    assert np.array_equal(o.H(1)[0], np.zeros(2))
    # GIN with eps = 0.5: h = W2 relu(W1 (1.5 h_v + sum) + b1) + b2, single edge 0 -> 1
    src = np.array([0], dtype=np.int32)
    dst = np.array([1], dtype=np.int32)
    m = I.gin_model(2, 2, 1, eps=0.5)
    W = [{"Wa": eye.copy(), "ba": np.array([-20, 0], np.float32), "Wb": 3 * eye,
          "bb": np.array([1, 1], np.float32)}]
    o = Oracle(3, src, dst, X, m, W)
    # vertex 1: t = 1.5*[10,20] + [1,2] = [16,32]; relu(t + [-20,0]) = [0,32]; *3 + 1 = [1,97]
    assert np.array_equal(o.H(1)[1], np.array([1.0, 97.0]))


def test_cancellation_example_of_the_paper():
    """Sec. 3.3.3: with sum and a linear layer, h2_D after the update equals w2 (h1_C + h1_A),
    i.e. the delta message replaces A's old contribution exactly."""
    # D's in-neighbours are A and C
    A_, B_, C_, D_, E_ = range(5)
    src, dst, add = _fig4()
    m = I.graphconv_model([3, 3, 3], I.AGG_SUM)
    for ly in m.layers:
        ly.act = I.ACT_IDENTITY
    X = I.features(5, 3, 3)
    W = I.make_weights(m, 3)
    o = Oracle(5, src, dst, X, m, W)
    assert o.apply_incremental(ups_array([(I.OP_ADD_EDGE, add[0], add[1])])) == 0
    h1 = o.H(1)
    want = (h1[C_] + h1[A_]) @ W[1]["Wa"].astype(np.float64)
    assert np.allclose(o.H(2)[D_], want, rtol=1e-12, atol=1e-14)


# ---------------------------------------------------------------------------------------------
# the paper's worked example
# ---------------------------------------------------------------------------------------------
def _fig4():
    spec = {}
    for line in open(os.path.join(GOLD, "fig4_edge_addition.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split(":")
        spec[k] = v.split()
    e = [tuple(int(x) for x in t.split(">")) for t in spec["edges"]]
    src = np.array([a for a, _ in e], dtype=np.int32)
    dst = np.array([b for _, b in e], dtype=np.int32)
    add = tuple(int(x) for x in spec["add"][0].split(">"))
    _fig4.hops = {k: np.array([int(x) for x in spec[k]], dtype=np.int32) for k in ("hop1", "hop2", "hop3")}
    return src, dst, add


@pytest.mark.parametrize("route", ["incremental", "scoped"])
def test_worked_example_affected_sets(route):
    src, dst, add = _fig4()
    hops = _fig4.hops
    m = I.graphconv_model([4, 4, 4, 4], I.AGG_SUM)
    X = I.features(5, 4, 1)
    W = I.make_weights(m, 1)
    o = Oracle(5, src, dst, X, m, W)
    before = [o.H(l).copy() for l in range(4)]
    fn = o.apply_incremental if route == "incremental" else o.apply_scoped
    assert fn(ups_array([(I.OP_ADD_EDGE, add[0], add[1])])) == 0
    assert o.affected(0).size == 0
    assert np.array_equal(o.affected(1), hops["hop1"])
    assert np.array_equal(o.affected(2), hops["hop2"])
    assert np.array_equal(o.affected(3), hops["hop3"])
    # C and E are untouched by a 2-layer model (Sec. 2.2)
    for v in (2, 4):
        assert np.array_equal(o.H(1)[v], before[1][v]) and np.array_equal(o.H(2)[v], before[2][v])
    full = o.full()
    for l in range(4):
        assert rel_err(o.H(l), full[l]) < 1e-12
    # deleting the edge again touches the same vertices (Sec. 3.2, edge deletion)
    assert fn(ups_array([(I.OP_DEL_EDGE, add[0], add[1])])) == 0
    assert np.array_equal(o.affected(2), hops["hop2"])
    for l in range(4):
        assert rel_err(o.H(l), before[l]) < 1e-12


# ---------------------------------------------------------------------------------------------
# the defining invariant, every model, many batches
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("pull", [False, True], ids=["push", "pull"])
@pytest.mark.parametrize("name", list(all_models().keys()))
def test_incremental_equals_full_recompute_every_batch(name, pull):
    model = all_models()[name]
    n, m = 60, 400
    src, dst = random_graph(n, m, 11)
    X = I.features(n, model.dims[0], 11)
    W = I.make_weights(model, 11, zero_bias=False)
    inc = Oracle(n, src, dst, X, model, W)
    rc = Oracle(n, src, dst, X, model, W)
    stream = I.UpdateStream(n, src, dst, model.dims[0], 11)
    e = m
    for b in range(12):
        ups, rows = stream.next_batch(1 + 3 * b)
        assert inc.apply_incremental(ups, rows, pull=pull) == 0
        assert rc.apply_scoped(ups, rows) == 0
        c = inc.counts()
        e += c["added"] - c["deleted"]
        assert inc.num_edges() == e == stream.n_edges
        full = inc.full()
        for l in range(model_layers(model) + 1):
            assert rel_err(inc.H(l), full[l]) < 1e-9, (name, b, l)
            assert rel_err(rc.H(l), full[l]) < 1e-12, (name, b, l)
            assert np.array_equal(inc.affected(l), rc.affected(l))
        for l in range(1, model_layers(model) + 1):
            assert rel_err(inc.S(l), inc.full_S(l)) < 1e-9
        # graph state: canonical CSR agrees between the two routes and with a fresh rebuild
        rp, col = inc.export_csr()
        rp2, col2 = rc.export_csr()
        assert np.array_equal(rp, rp2) and np.array_equal(col, col2)
        do, di = inc.degrees()
        assert np.array_equal(do, np.diff(rp))
        assert np.array_equal(di, np.bincount(col, minlength=n))


def model_layers(model):
    return len(model.layers)


@pytest.mark.parametrize("pull", [False, True], ids=["push", "pull"])
@pytest.mark.parametrize("name", ["sage_mean", "gc_sum", "gcn_wsum", "gin"])
@pytest.mark.parametrize("op", ["add", "del", "feat", "feat+add+del"])
def test_single_update_rules(name, op, pull):
    """One update per batch: added edge (old contribution 0), deleted edge (new contribution 0),
    changed vertex (new minus old) -- Sec. 3.3.3."""
    model = all_models()[name]
    n, m = 30, 120
    src, dst = random_graph(n, m, 5)
    X = I.features(n, model.dims[0], 5)
    W = I.make_weights(model, 5, zero_bias=False)
    o = Oracle(n, src, dst, X, model, W)
    present = set(zip(src.tolist(), dst.tolist()))
    if op == "add":
        u, v = next((a, b) for a in range(n) for b in range(n) if a != b and (a, b) not in present)
        ups, rows = ups_array([(I.OP_ADD_EDGE, u, v)]), None
        src2, dst2, X2 = np.append(src, u), np.append(dst, v), X
    elif op == "del":
        u, v = int(src[17]), int(dst[17])
        ups, rows = ups_array([(I.OP_DEL_EDGE, u, v)]), None
        src2, dst2, X2 = np.delete(src, 17), np.delete(dst, 17), X
    elif op == "feat":
        rows = I.features(1, model.dims[0], 99)
        ups = ups_array([(I.OP_SET_FEATURE, 9, 0)])
        X2 = X.copy()
        X2[9] = rows[0]
        src2, dst2 = src, dst
    else:
        # the three rules meet at one source: its row changes, it gains an edge (the whole new term
        # arrives, and no delta message travels along that edge) and loses one (the whole old term leaves)
        u = int(src[17])
        w = int(dst[17])
        v = next(b for b in range(n) if b != u and (u, b) not in present)
        rows = I.features(1, model.dims[0], 98)
        ups = ups_array([(I.OP_SET_FEATURE, u, 0), (I.OP_ADD_EDGE, u, v), (I.OP_DEL_EDGE, u, w)])
        X2 = X.copy()
        X2[u] = rows[0]
        src2, dst2 = np.append(np.delete(src, 17), u), np.append(np.delete(dst, 17), v)
    assert o.apply_incremental(ups, rows, pull=pull) == 0
    ref = dense_full(n, src2.astype(np.int32), dst2.astype(np.int32), X2, model, W)
    for l in range(len(ref)):
        assert rel_err(o.H(l), ref[l]) < 1e-10, (name, op, l)


# ---------------------------------------------------------------------------------------------
# affected sets
# ---------------------------------------------------------------------------------------------
def _signatures(n, edges, fver, model, L):
    """Structural signature of every vertex's l-hop computation tree, l = 0..L."""
    ins = {v: [] for v in range(n)}
    outdeg = [0] * n
    for (u, v) in edges:
        ins[v].append(u)
        outdeg[u] += 1
    sig = [[("x", v, fver[v]) for v in range(n)]]
    for _ in range(L):
        prev = sig[-1]
        cur = []
        for v in range(n):
            nb = frozenset((u, prev[u], outdeg[u] if model.src_norm else 0) for u in ins[v])
            cur.append((prev[v] if model.self_term else None, nb))
        sig.append([hash(c) for c in cur])
    return sig


@pytest.mark.parametrize("name", ["sage_mean", "gc_sum", "gcn_wsum", "gin"])
def test_affected_sets_match_structural_brute_force(name):
    model = all_models()[name]
    L = len(model.layers)
    n, m = 40, 100
    src, dst = random_graph(n, m, 21)
    X = I.features(n, model.dims[0], 21)
    W = I.make_weights(model, 21)
    o = Oracle(n, src, dst, X, model, W)
    stream = I.UpdateStream(n, src, dst, model.dims[0], 21)
    edges = set(zip(src.tolist(), dst.tolist()))
    fver = [0] * n
    for b in range(10):
        ups, rows = stream.next_batch(1 + b % 4)
        old = _signatures(n, edges, fver, model, L)
        for r in ups:
            if r["op"] == I.OP_ADD_EDGE:
                edges.add((int(r["u"]), int(r["v"])))
            elif r["op"] == I.OP_DEL_EDGE:
                edges.discard((int(r["u"]), int(r["v"])))
            else:
                fver[int(r["u"])] += 1
        new = _signatures(n, edges, fver, model, L)
        assert o.apply_incremental(ups, rows) == 0
        for l in range(L + 1):
            want = np.array([v for v in range(n) if old[l][v] != new[l][v]], dtype=np.int32)
            assert np.array_equal(o.affected(l), want), (name, b, l)


@pytest.mark.parametrize("name", ["sage_mean", "gc_mean", "gcn_wsum", "gin"])
def test_numeric_footprint_equals_affected_sets(name):
    """With identity activations and generic data the rows that full recomputation changes are
    exactly A_l; with ReLU they are a subset."""
    for ident in (True, False):
        model = all_models(acts_identity=ident)[name]
        L = len(model.layers)
        n, m = 50, 160
        src, dst = random_graph(n, m, 31)
        X = I.features(n, model.dims[0], 31)
        W = I.make_weights(model, 31, zero_bias=False)
        o = Oracle(n, src, dst, X, model, W)
        stream = I.UpdateStream(n, src, dst, model.dims[0], 31)
        for b in range(6):
            before = o.full()
            ups, rows = stream.next_batch(2)
            assert o.apply_incremental(ups, rows) == 0
            after = o.full()
            for l in range(L + 1):
                changed = np.nonzero(np.any(before[l] != after[l], axis=1))[0].astype(np.int32)
                if ident and name != "gin":   # GIN keeps an inner ReLU
                    assert np.array_equal(changed, o.affected(l)), (name, b, l)
                else:
                    assert np.all(np.isin(changed, o.affected(l)))
            # frontier never shrinks for models with a self term (Sec. 3.5: a_l >= a_{l-1})
            if model.self_term:
                for l in range(1, L + 1):
                    assert o.affected(l).size >= o.affected(l - 1).size


# ---------------------------------------------------------------------------------------------
# batch semantics and degenerate cases
# ---------------------------------------------------------------------------------------------
def _small(name="sage_mean", seed=41):
    model = all_models()[name]
    n, m = 25, 90
    src, dst = random_graph(n, m, seed)
    X = I.features(n, model.dims[0], seed)
    W = I.make_weights(model, seed, zero_bias=False)
    return n, src, dst, X, model, W


def test_empty_batch_and_identical_feature_change_nothing():
    n, src, dst, X, model, W = _small()
    o = Oracle(n, src, dst, X, model, W)
    before = [o.H(l).copy() for l in range(3)]
    assert o.apply_incremental(ups_array([])) == 0
    assert all(o.affected(l).size == 0 for l in range(3))
    # a feature update that repeats the stored values is still structurally affected, but its
    # delta message is exactly zero
    rows = X[[7]].copy()
    assert o.apply_incremental(ups_array([(I.OP_SET_FEATURE, 7, 0)]), rows) == 0
    assert np.array_equal(o.affected(0), np.array([7], dtype=np.int32))
    assert o.affected(1).size >= 1
    for l in range(3):
        assert np.array_equal(o.H(l), before[l])


def test_add_then_delete_restores_graph_and_embeddings():
    n, src, dst, X, model, W = _small("gcn_wsum")
    o = Oracle(n, src, dst, X, model, W)
    rp0, col0 = o.export_csr()
    before = [o.H(l).copy() for l in range(4)]
    present = set(zip(src.tolist(), dst.tolist()))
    u, v = next((a, b) for a in range(n) for b in range(n) if a != b and (a, b) not in present)
    assert o.apply_incremental(ups_array([(I.OP_ADD_EDGE, u, v)])) == 0
    assert o.num_edges() == src.size + 1
    assert o.apply_incremental(ups_array([(I.OP_DEL_EDGE, u, v)])) == 0
    rp1, col1 = o.export_csr()
    assert np.array_equal(rp0, rp1) and np.array_equal(col0, col1)
    for l in range(4):
        assert rel_err(o.H(l), before[l]) < 1e-12


def test_repeated_items_in_one_batch_have_sequential_net_effect():
    n, src, dst, X, model, W = _small()
    present = set(zip(src.tolist(), dst.tolist()))
    missing = [(a, b) for a in range(n) for b in range(n) if a != b and (a, b) not in present]
    (u, v), (mu, mv) = missing[0], missing[5]
    eu, ev = int(src[0]), int(dst[0])
    rows = I.features(3, model.dims[0], 77)
    recs = [
        (I.OP_ADD_EDGE, u, v), (I.OP_DEL_EDGE, u, v),          # net: nothing
        (I.OP_DEL_EDGE, eu, ev), (I.OP_ADD_EDGE, eu, ev),      # net: nothing
        (I.OP_ADD_EDGE, eu, ev),                               # again: still an edge
        (I.OP_SET_FEATURE, 4, 0), (I.OP_SET_FEATURE, 4, 2),    # last payload wins
        (I.OP_DEL_EDGE, int(src[1]), int(dst[1])),             # a real deletion
        (I.OP_ADD_EDGE, int(src[2]), int(dst[2])),             # adding an existing edge: no-op
        (I.OP_DEL_EDGE, mu, mv),                               # deleting a missing edge: no-op
        (I.OP_ADD_EDGE, 6, 6),                                 # a self-loop is an ordinary edge
    ]
    o = Oracle(n, src, dst, X, model, W)
    assert o.apply_incremental(ups_array(recs), rows) == 0
    c = o.counts()
    assert c["deleted"] == 1 and c["added"] == 1
    assert c["noop_add"] == 2 and c["noop_del"] == 2 and c["superseded"] == 3
    src2 = np.append(np.delete(src, 1), 6).astype(np.int32)
    dst2 = np.append(np.delete(dst, 1), 6).astype(np.int32)
    X2 = X.copy()
    X2[4] = rows[2]
    ref = dense_full(n, src2, dst2, X2, model, W)
    for l in range(3):
        assert rel_err(o.H(l), ref[l]) < 1e-10
    assert np.array_equal(o.affected(0), np.array([4], dtype=np.int32))


def test_message_order_does_not_matter():
    """Sec. 3.3.3, aggregation at the inbox: any arrival order gives the same sum."""
    n, src, dst, X, model, W = _small("gin")
    stream = I.UpdateStream(n, src, dst, model.dims[0], 5)
    ups, rows = stream.next_batch(12)
    a = Oracle(n, src, dst, X, model, W)
    b = Oracle(n, src, dst, X, model, W)
    assert a.apply_incremental(ups, rows) == 0
    perm = np.random.default_rng(0).permutation(ups.size)
    assert b.apply_incremental(ups[perm], rows) == 0
    for l in range(4):
        assert np.array_equal(a.affected(l), b.affected(l))
        assert rel_err(a.H(l), b.H(l)) < 1e-12


def test_invalid_batches_are_rejected_without_side_effects():
    n, src, dst, X, model, W = _small()
    o = Oracle(n, src, dst, X, model, W)
    before = [o.H(l).copy() for l in range(3)]
    rp0, col0 = o.export_csr()
    good = (I.OP_DEL_EDGE, int(src[0]), int(dst[0]))
    assert o.apply_incremental(ups_array([good, (I.OP_ADD_EDGE, 0, n)])) < 0
    assert o.apply_incremental(ups_array([good, (I.OP_ADD_EDGE, -1, 2)])) < 0
    assert o.apply_incremental(ups_array([good, (7, 1, 2)])) < 0
    assert o.apply_incremental(ups_array([good, (I.OP_SET_FEATURE, 1, 0)]), None) < 0  # no payload row
    rp1, col1 = o.export_csr()
    assert np.array_equal(rp0, rp1) and np.array_equal(col0, col1)
    for l in range(3):
        assert np.array_equal(o.H(l), before[l])


def test_row_from_prev_matches_full():
    n, src, dst, X, model, W = _small("gcn_wsum")
    o = Oracle(n, src, dst, X, model, W)
    full = o.full()
    for l in range(1, 4):
        prev = np.ascontiguousarray(full[l - 1].astype(np.float32))
        ref = dense_full(n, src, dst, X, model, W)
        for v in (0, 5, 24):
            S, h = o.row_from_prev(l, v, prev)
            assert np.allclose(h, ref[l][v], rtol=1e-5, atol=1e-6)
        ids = np.array([24, 0, 5, 5], dtype=np.int32)     # the many-rows form returns the same rows, in order
        Sm, hm = o.rows_from_prev(l, ids, prev)
        for i, v in enumerate(ids):
            S, h = o.row_from_prev(l, int(v), prev)
            assert np.array_equal(Sm[i], S) and np.array_equal(hm[i], h)


# ---------------------------------------------------------------------------------------------
# the tiny configuration end to end (the smallest of the build's named workloads)
# ---------------------------------------------------------------------------------------------
def test_tiny_config_invariant_10_batches():
    w = I.workloads()["tiny"]
    src, dst = I.make_graph(w)
    X = I.features(w.n, w.model.dims[0], w.seed)
    W = I.make_weights(w.model, w.seed)
    o = Oracle(w.n, src, dst, X, w.model, W)
    stream = I.UpdateStream(w.n, src, dst, w.model.dims[0], w.seed)
    for b in range(w.n_batches):
        ups, rows = stream.next_batch(100)
        assert o.apply_incremental(ups, rows) == 0
        full = o.full()
        for l in range(3):
            assert rel_err(o.H(l), full[l]) < 1e-9
        sizes = [o.affected(l).size for l in range(3)]
        assert sizes[0] <= sizes[1] <= sizes[2] <= w.n


def test_structure_only_route_matches_incremental_route():
    """orc_apply_structure follows graph and affected sets exactly like the incremental route."""
    for name in ("sage_mean", "gcn_wsum"):
        model = all_models()[name]
        n, m = 80, 500
        src, dst = random_graph(n, m, 3)
        X = I.features(n, model.dims[0], 3)
        W = I.make_weights(model, 3)
        a = Oracle(n, src, dst, X, model, W)
        b = Oracle(n, src, dst, X, model, W, bootstrap=False)
        stream = I.UpdateStream(n, src, dst, model.dims[0], 3)
        for _ in range(8):
            ups, rows = stream.next_batch(15)
            assert a.apply_incremental(ups, rows) == 0
            assert b.apply_structure(ups, rows.shape[0]) == 0
            for l in range(len(model.layers) + 1):
                assert np.array_equal(a.affected(l), b.affected(l))
            for l in range(1, len(model.layers) + 1):
                assert a.active_edges(l) == b.active_edges(l)
            assert a.counts() == b.counts()
            ra, ca = a.export_csr()
            rb, cb = b.export_csr()
            assert np.array_equal(ra, rb) and np.array_equal(ca, cb)
