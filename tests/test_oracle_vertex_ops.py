"""Pins for the oracle's vertex operations (Sec. 3.2: a vertex deletion deletes every incident
edge and then propagates from the vertex as root; Sec. 4.1: a vertex addition arrives as the edge
addition that creates the endpoint).  Nothing here needs a GPU.

The oracle derives a batch's net effect from sorted tables; these tests replay the same
operations literally, one after the other, on Python sets and compare."""
import os
import sys

import numpy as np
import pytest

sys.path.insert(0, os.path.dirname(__file__))
import test_oracle_pins as P  # noqa: E402  (dense-matrix definition, structural signatures, fixtures)

from paper_2601_12347_b200 import inputs as I  # noqa: E402
from oracle.oracle import Oracle  # noqa: E402


def replay(edges, ups):
    """Literal sequential application.  Returns (edge set, {vertex: payload row or -1 for zeros})."""
    E = set(edges)
    feat = {}
    for op, u, v in ups:
        if op == I.OP_ADD_EDGE:
            E.add((u, v))
        elif op == I.OP_DEL_EDGE:
            E.discard((u, v))
        elif op == I.OP_SET_FEATURE:
            feat[u] = v
        else:
            E = {p for p in E if u not in p}
            feat[u] = -1
    return E, feat


def random_batch(rng, n, edges, size, n_rows, p_vertex=0.15):
    """Ops that deliberately collide: pairs are drawn around a few vertices, some of which are
    deleted in the middle of the batch."""
    hot = rng.choice(n, size=min(n, 6), replace=False)
    present = sorted(edges)
    recs = []
    for _ in range(size):
        r = rng.random()
        if r < p_vertex:
            recs.append((I.OP_DEL_VERTEX, int(rng.choice(hot)), 0))
        elif r < 0.45:
            u = int(rng.choice(hot)) if rng.random() < 0.7 else int(rng.integers(n))
            v = int(rng.choice(hot)) if rng.random() < 0.5 else int(rng.integers(n))
            recs.append((I.OP_ADD_EDGE, u, v))
        elif r < 0.75:
            if present and rng.random() < 0.7:
                u, v = present[int(rng.integers(len(present)))]
            else:
                u, v = int(rng.choice(hot)), int(rng.integers(n))
            recs.append((I.OP_DEL_EDGE, int(u), int(v)))
        else:
            recs.append((I.OP_SET_FEATURE, int(rng.choice(hot)) if rng.random() < 0.5 else int(rng.integers(n)),
                         int(rng.integers(n_rows))))
    return recs


def edges_of(o):
    rowptr, col = o.export_csr()
    return {(u, int(col[j])) for u in range(len(rowptr) - 1) for j in range(rowptr[u], rowptr[u + 1])}


@pytest.mark.parametrize("name", ["sage_mean", "gc_sum", "gcn_wsum", "gin"])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_net_effect_equals_literal_replay(name, seed):
    model = P.all_models()[name]
    L = len(model.layers)
    n, m = 30, 120
    src, dst = P.random_graph(n, m, 50 + seed)
    X = I.features(n, model.dims[0], seed)
    W = I.make_weights(model, seed)
    o = Oracle(n, src, dst, X, model, W)
    edges = set(zip(src.tolist(), dst.tolist()))
    Xcur = X.copy()
    rng = np.random.default_rng(seed)
    for b in range(8):
        rows = I.features(4, model.dims[0], 1000 + 10 * seed + b)
        recs = random_batch(rng, n, edges, int(rng.integers(1, 25)), 4)
        new_edges, feat = replay(edges, recs)
        assert o.apply_incremental(P.ups_array(recs), rows, pull=(seed + b) % 2 == 1) == 0   # both delivery orders
        assert edges_of(o) == new_edges, (name, seed, b)
        c = o.counts()
        assert c["added"] == len(new_edges - edges) and c["deleted"] == len(edges - new_edges)
        assert np.array_equal(o.affected(0), np.array(sorted(feat), dtype=np.int32))
        for v, r in feat.items():
            Xcur[v] = rows[r] if r >= 0 else 0.0
        edges = new_edges
        e = sorted(edges)
        ref = P.dense_full(n, np.array([a for a, _ in e], dtype=np.int32), np.array([b_ for _, b_ in e], dtype=np.int32),
                           Xcur, model, W)
        for l in range(L + 1):
            assert P.rel_err(o.H(l), ref[l]) < 1e-9, (name, seed, b, l)
        do, di = o.degrees()
        assert do.sum() == len(edges) and di.sum() == len(edges)


def signatures(n, edges, fver, over, model, L):
    """Structural signature of every vertex's l-hop computation tree.  fver[v] counts the feature
    events of v; over[u] counts the batches that changed u's out-list: the recurrence treats the
    source coefficient of such a vertex as changed (C_l includes the sources of edge changes), even
    when an addition and a deletion leave its out-degree where it was."""
    ins = {v: [] for v in range(n)}
    for (u, v) in edges:
        ins[v].append(u)
    sig = [[("x", v, fver[v]) for v in range(n)]]
    for _ in range(L):
        prev = sig[-1]
        cur = []
        for v in range(n):
            nb = frozenset((u, prev[u], over[u] if model.src_norm else 0) for u in ins[v])
            cur.append((prev[v] if model.self_term else None, nb))
        sig.append([hash(c) for c in cur])
    return sig


@pytest.mark.parametrize("name", ["sage_mean", "gc_sum", "gcn_wsum", "gin"])
def test_affected_sets_with_vertex_deletions_match_structural_brute_force(name):
    model = P.all_models()[name]
    L = len(model.layers)
    n, m = 40, 110
    src, dst = P.random_graph(n, m, 23)
    X = I.features(n, model.dims[0], 23)
    W = I.make_weights(model, 23)
    edges = set(zip(src.tolist(), dst.tolist()))
    fver = [0] * n
    over = [0] * n
    rng = np.random.default_rng(23)
    for route in ("incremental", "scoped", "structure"):
        o = Oracle(n, src, dst, X, model, W)
        edges = set(zip(src.tolist(), dst.tolist()))
        for b in range(8):
            rows = I.features(3, model.dims[0], 500 + b)
            recs = random_batch(rng, n, edges, 1 + b % 5, 3, p_vertex=0.3)
            old = signatures(n, edges, fver, over, model, L)
            before = edges
            edges, feat = replay(edges, recs)
            for v in feat:
                fver[v] += 1
            for u in {p[0] for p in before ^ edges}:
                over[u] += 1
            new = signatures(n, edges, fver, over, model, L)
            ups = P.ups_array(recs)
            rc = {"incremental": lambda: o.apply_incremental(ups, rows), "scoped": lambda: o.apply_scoped(ups, rows),
                  "structure": lambda: o.apply_structure(ups, 3)}[route]()
            assert rc == 0
            for l in range(L + 1):
                want = np.array([v for v in range(n) if old[l][v] != new[l][v]], dtype=np.int32)
                assert np.array_equal(o.affected(l), want), (name, route, b, l)


def test_worked_example_vertex_deletion():
    """Sec. 3.2: deleting C removes C->A, C->D, E->C and B->C; A and D, downstream of C, update."""
    src, dst, add = P._fig4()
    spec = {}
    for line in open(os.path.join(P.GOLD, "fig4_edge_addition.txt")):
        if ":" in line and not line.startswith("#"):
            k, v = line.strip().split(":")
            spec[k] = v.split()
    victim = int(spec["delete_vertex"][0])
    gone = {tuple(int(x) for x in t.split(">")) for t in spec["deleted_edges"]}
    downstream = [int(x) for x in spec["deleted_downstream"]]
    m = I.graphconv_model([4, 4, 4], I.AGG_SUM)
    X = I.features(5, 4, 1)
    W = I.make_weights(m, 1)
    o = Oracle(5, src, dst, X, m, W)
    assert o.apply_incremental(P.ups_array([(I.OP_ADD_EDGE, add[0], add[1])])) == 0
    before = edges_of(o)
    assert o.apply_incremental(P.ups_array([(I.OP_DEL_VERTEX, victim, 0)])) == 0
    assert before - edges_of(o) == gone and edges_of(o) <= before
    assert o.counts()["deleted"] == 4
    a1 = set(o.affected(1).tolist())
    assert set(downstream) <= a1
    assert a1 == set(downstream) | {victim}       # C itself is the sink of E->C and B->C
    do, di = o.degrees()
    assert do[victim] == 0 and di[victim] == 0
    assert np.all(o.H(0)[victim] == 0.0)
    full = o.full()
    for l in range(3):
        assert P.rel_err(o.H(l), full[l]) < 1e-12


def test_counters_and_ordering_around_a_deletion():
    n, src, dst, X, model, W = P._small()
    present = sorted(set(zip(src.tolist(), dst.tolist())))
    w = int(src[0])
    out_w = [p for p in present if p[0] == w]
    in_w = [p for p in present if p[1] == w and p[0] != w]
    missing = [(w, b) for b in range(n) if (w, b) not in set(present) and b != w]
    other = next(p for p in present if w not in p)
    rows = I.features(2, model.dims[0], 5)
    recs = [
        (I.OP_ADD_EDGE, missing[0][0], missing[0][1]),   # superseded: the vertex is deleted later
        (I.OP_DEL_EDGE, out_w[0][0], out_w[0][1]),       # superseded likewise (the deletion removes it)
        (I.OP_DEL_EDGE, missing[1][0], missing[1][1]),   # superseded likewise (would have been a no-op)
        (I.OP_SET_FEATURE, w, 0),                        # overridden by the deletion: zeros win
        (I.OP_DEL_VERTEX, w, 0),
        (I.OP_ADD_EDGE, missing[2][0], missing[2][1]),   # after the deletion: a real addition
        (I.OP_ADD_EDGE, out_w[-1][0], out_w[-1][1]),     # re-adds an edge the deletion removed: net nothing
        (I.OP_DEL_EDGE, other[0], other[1]),             # unrelated real deletion
        (I.OP_SET_FEATURE, other[0], 1),
    ]
    o = Oracle(n, src, dst, X, model, W)
    assert o.apply_incremental(P.ups_array(recs), rows) == 0
    c = o.counts()
    n_incident = len(out_w) + len(in_w)
    assert c["superseded"] == 3
    assert c["added"] == 1
    assert c["noop_add"] == 1 and c["noop_del"] == 0
    assert c["deleted"] == n_incident - 1 + 1            # all incident edges but the re-added one, plus `other`
    assert np.all(o.H(0)[w] == 0.0)
    assert np.array_equal(o.H(0)[other[0]], rows[1].astype(np.float64))
    want, _ = replay(set(present), recs)
    assert edges_of(o) == want
    # a second batch re-creates the vertex: features and edges attach to the same id
    recs2 = [(I.OP_SET_FEATURE, w, 1), (I.OP_ADD_EDGE, w, other[1]), (I.OP_ADD_EDGE, other[0], w)]
    assert o.apply_incremental(P.ups_array(recs2), rows) == 0
    want2, _ = replay(want, recs2)
    assert edges_of(o) == want2
    full = o.full()
    for l in range(len(model.layers) + 1):
        assert P.rel_err(o.H(l), full[l]) < 1e-9


def test_vertex_deletion_rejects_bad_ids_and_accepts_isolated_vertices():
    n, src, dst, X, model, W = P._small()
    o = Oracle(n, src, dst, X, model, W)
    H = [o.H(l).copy() for l in range(3)]
    assert o.apply_incremental(P.ups_array([(I.OP_DEL_VERTEX, n, 0)])) != 0
    assert o.apply_incremental(P.ups_array([(I.OP_DEL_VERTEX, -1, 0)])) != 0
    for l in range(3):
        assert np.array_equal(o.H(l), H[l])
    # twice in one batch, and again in the next: the second time nothing is left to remove
    assert o.apply_incremental(P.ups_array([(I.OP_DEL_VERTEX, 3, 0), (I.OP_DEL_VERTEX, 3, 0)])) == 0
    assert o.apply_incremental(P.ups_array([(I.OP_DEL_VERTEX, 3, 0)])) == 0
    assert o.counts()["deleted"] == 0
    assert np.array_equal(o.affected(0), np.array([3], dtype=np.int32))   # structural: still a feature event
    full = o.full()
    for l in range(3):
        assert P.rel_err(o.H(l), full[l]) < 1e-9
