"""Vertex deletion and re-creation on the GPU against the oracle (Sec. 3.2: a vertex deletion
deletes every incident edge and propagates from the vertex as root; Sec. 4.1: a vertex addition
arrives as the edge addition that names the new endpoint)."""
import os
import sys

import numpy as np
import pytest

sys.path.insert(0, os.path.dirname(__file__))
import test_gpu_parity as G  # noqa: E402  (env fixture, graph / frontier / value checks)
from test_gpu_parity import env  # noqa: E402,F401
from test_oracle_vertex_ops import random_batch  # noqa: E402

from paper_2601_12347_b200 import inputs as I  # noqa: E402

pytestmark = pytest.mark.gpu


def edge_set(src, dst):
    return set(zip(src.tolist(), dst.tolist()))


@pytest.mark.parametrize("name", list(G.small_models().keys()))
def test_colliding_batches_with_vertex_deletions(env, name):
    """Edge operations before and after the deletion of their endpoints, repeated deletions,
    feature rows overridden by a deletion and the other way round."""
    ripple, Oracle = env
    model = G.small_models()[name]
    L = len(model.layers)
    n, m = 300, 2500
    src, dst = I.er_graph(n, m, 5)
    X = I.features(n, model.dims[0], 5)
    W = I.make_weights(model, 5, zero_bias=False)
    rp = ripple.Ripple(n, src, dst, X, model, W)
    orc = Oracle(n, src, dst, X, model, W)
    rng = np.random.default_rng(5)
    edges = edge_set(src, dst)
    seen_expanded = 0
    for b in range(24):
        rows = I.features(6, model.dims[0], 700 + b)
        recs = random_batch(rng, n, edges, int(rng.integers(1, 60)), 6, p_vertex=0.1)
        ups = G.ups_array(recs)
        rp.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        G.check_graph(rp, orc)
        G.check_frontiers(rp, orc, L)
        seen_expanded += rp.stats()["n_expanded"]
        rowptr, col = orc.export_csr()
        edges = {(u, int(col[j])) for u in range(n) for j in range(rowptr[u], rowptr[u + 1])}
        if b % 4 == 3:
            G.check_values(rp, orc.full(), L, [None] + [orc.full_S(l) for l in range(1, L + 1)])
    assert seen_expanded > 0
    rp.close()


@pytest.mark.parametrize("mem", ["host", "device"])
def test_hub_deletion_and_recreation(env, mem):
    """A vertex with thousands of in- and out-edges is deleted (host batch: full-batch launch
    geometry; device batch: geometry of the few given operations, replayed as a captured graph),
    then re-created under the same id."""
    import torch
    ripple, Oracle = env
    model = I.sage_model([12, 64, 24, 8], I.AGG_MEAN)
    L = 3
    n = 5000
    src, dst = I.er_graph(n, 20000, 9)
    have = edge_set(src, dst)
    hub = 17
    extra = [(hub, v) for v in range(100, 2600) if (hub, v) not in have]
    extra += [(u, hub) for u in range(1000, 4200) if (u, hub) not in have and u != hub]
    extra += [(hub, hub)]
    src = np.concatenate([src, np.array([a for a, _ in extra], dtype=np.int32)])
    dst = np.concatenate([dst, np.array([b for _, b in extra], dtype=np.int32)])
    X = I.features(n, 12, 9)
    W = I.make_weights(model, 9, zero_bias=False)
    rp = ripple.Ripple(n, src, dst, X, model, W, max_batch=8192)
    orc = Oracle(n, src, dst, X, model, W)
    rows = I.features(2, 12, 99)

    def apply(recs):
        ups = G.ups_array(recs)
        if mem == "device":
            u = torch.from_numpy(np.stack([ups["op"], ups["u"], ups["v"]], axis=1).astype(np.int32)).cuda()
            rp.apply_batch(u, torch.from_numpy(rows).cuda())
        else:
            rp.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        G.check_graph(rp, orc)
        G.check_frontiers(rp, orc, L)
        G.check_values(rp, orc.full(), L, [None] + [orc.full_S(l) for l in range(1, L + 1)])

    do, di = rp.degrees()
    deg = int(do[hub]) + int(di[hub])
    assert deg > 5000
    apply([(I.OP_ADD_EDGE, 3, 4), (I.OP_DEL_VERTEX, hub, 0), (I.OP_SET_FEATURE, 8, 1)])
    st = rp.stats()
    assert st["n_expanded"] == deg and st["n_deleted"] == deg - 1     # the self-loop is stored in both lists
    do, di = rp.degrees()
    assert int(do[hub]) == 0 and int(di[hub]) == 0
    assert float(rp.embeddings(0)[hub].abs().max()) == 0.0
    # the same id comes back: features first, then edges in both directions
    apply([(I.OP_SET_FEATURE, hub, 0), (I.OP_ADD_EDGE, hub, 5), (I.OP_ADD_EDGE, 6, hub), (I.OP_ADD_EDGE, hub, hub)])
    assert rp.stats()["n_added"] == 3
    # deleted again together with a neighbour, with edge operations on both sides of the deletions
    apply([(I.OP_ADD_EDGE, hub, 7), (I.OP_DEL_VERTEX, hub, 0), (I.OP_DEL_VERTEX, 5, 0), (I.OP_ADD_EDGE, hub, 9),
           (I.OP_DEL_VERTEX, hub, 0), (I.OP_ADD_EDGE, 5, hub)])
    # three more batches of three operations: a chain is captured at its second appearance and
    # replayed from the third on, here with a vertex deletion inside the replayed batch
    apply([(I.OP_ADD_EDGE, 20, 21), (I.OP_DEL_VERTEX, 30, 0), (I.OP_SET_FEATURE, 31, 0)])
    apply([(I.OP_ADD_EDGE, 22, 23), (I.OP_DEL_VERTEX, 32, 0), (I.OP_SET_FEATURE, 33, 1)])
    rp.close()


def test_expansion_beyond_the_batch_capacity_is_rejected(env):
    ripple, Oracle = env
    model = I.sage_model([8, 16, 4], I.AGG_SUM)
    n = 2000
    src, dst = I.er_graph(n, 6000, 13)
    have = edge_set(src, dst)
    extra = [(1, v) for v in range(2, 1500) if (1, v) not in have]
    src = np.concatenate([src, np.array([a for a, _ in extra], dtype=np.int32)])
    dst = np.concatenate([dst, np.array([b for _, b in extra], dtype=np.int32)])
    X = I.features(n, 8, 13)
    W = I.make_weights(model, 13)
    rp = ripple.Ripple(n, src, dst, X, model, W, max_batch=1024)
    orc = Oracle(n, src, dst, X, model, W)
    before = [rp.embeddings(l).clone() for l in range(3)]
    ups = G.ups_array([(I.OP_ADD_EDGE, 5, 6), (I.OP_DEL_VERTEX, 1, 0), (I.OP_SET_FEATURE, 9, 0)])
    with pytest.raises(ripple.RippleError) as ei:
        rp.apply_batch(ups, I.features(1, 8, 1))
    assert ei.value.status == ripple.ERR_CAPACITY and "max_batch" in str(ei.value)
    G.check_graph(rp, orc)
    for l in range(3):
        assert bool((rp.embeddings(l) == before[l]).all())
    # the context is still usable, and a deletion that fits goes through
    small = int(np.argmin(np.bincount(src, minlength=n) + np.bincount(dst, minlength=n) + (np.arange(n) == 1) * 10**6))
    ups = G.ups_array([(I.OP_DEL_VERTEX, small, 0), (I.OP_ADD_EDGE, 5, 6)])
    rp.apply_batch(ups, None)
    assert orc.apply_incremental(ups, None) == 0
    G.check_graph(rp, orc)
    G.check_frontiers(rp, orc, 2)
    G.check_values(rp, orc.full(), 2)
    # out-of-range vertex: rejected like any other bad id
    with pytest.raises(ripple.RippleError) as ei:
        rp.apply_batch(G.ups_array([(I.OP_DEL_VERTEX, n, 0)]), None)
    assert ei.value.status == ripple.ERR_VERTEX_RANGE
    G.check_graph(rp, orc)
    rp.close()


@pytest.mark.parametrize("batch", [100, 1000])
def test_all_five_update_types_100_consecutive_batches(env, batch):
    """The sparse workload with 2 % vertex deletions in the stream (Sec. 3.1: five update types)."""
    ripple, Oracle = env
    w = I.workloads()["sparse-vdel"]
    src, dst = I.make_graph(w)
    X = I.features(w.n, w.model.dims[0], w.seed)
    W = I.make_weights(w.model, w.seed)
    L = len(w.model.layers)
    rp = ripple.Ripple(w.n, src, dst, X, w.model, W, max_batch=w.extra["max_batch"])
    orc = Oracle(w.n, src, dst, X, w.model, W)
    stream = I.make_stream(w, src, dst)
    expanded = 0
    for b in range(100):
        ups, rows = stream.next_batch(batch)
        rp.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        G.check_frontiers(rp, orc, L)
        expanded += rp.stats()["n_expanded"]
        if b % 25 == 24:
            G.check_graph(rp, orc)
            G.check_values(rp, [orc.H(l) for l in range(L + 1)], L)
    assert expanded > 0
    G.check_graph(rp, orc)
    G.check_values(rp, orc.full(), L, [None] + [orc.full_S(l) for l in range(1, L + 1)])
    assert rp.stats()["num_edges"] == stream.n_edges
    rp.close()


# ---------------------------------------------------------------------------------------------
# growing the vertex set (ripple_reserve_vertices)
# ---------------------------------------------------------------------------------------------
def _reserve_models():
    return {
        "sage_mean": I.sage_model([18, 36, 10], I.AGG_MEAN),
        "gc_sum_3l": I.graphconv_model([18, 36, 20, 10], I.AGG_SUM),     # no self term: an isolated vertex still has act(bias) rows
        "gcn_wsum": I.graphconv_model([18, 36, 10], I.AGG_WSUM_GCN),
        "gin": I.gin_model(18, 24, 2, eps=0.25),
        "gc_max": I.graphconv_model([18, 36, 10], I.AGG_MAX),
        "gat": I.gat_model(20, 2, d_att=4, slope=0.2),
        "sage_wide": I.sage_model([40, 160, 24], I.AGG_MEAN),
    }


@pytest.mark.parametrize("name", list(_reserve_models().keys()))
def test_reserved_vertices_are_isolated_vertices_and_can_be_attached(env, name):
    ripple, Oracle = env
    model = _reserve_models()[name]
    L = len(model.layers)
    n, spare = 500, 70
    src, dst = I.er_graph(n, 3500, 17)
    X = I.features(n + spare, model.dims[0], 17)
    X[n:] = 0
    W = I.make_weights(model, 17, zero_bias=False)
    rp = ripple.Ripple(n, src, dst, X[:n], model, W)
    orc = Oracle(n + spare, src, dst, X, model, W)          # the oracle has had the ids all along, as isolated vertices
    stream = I.UpdateStream(n, src, dst, model.dims[0], 17)
    for _ in range(3):                                       # same size three times: a captured chain exists before the growth
        ups, rows = stream.next_batch(20)
        rp.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
    before = [rp.embeddings(l).clone() for l in range(L + 1)]
    with pytest.raises(ripple.RippleError):
        rp.reserve_vertices(n)
    rp.reserve_vertices(n + spare)
    full = orc.full()
    for l in range(L + 1):
        got = rp.embeddings(l)
        assert got.shape[0] == n + spare
        assert bool((got[:n] == before[l]).all()), "rows of the old vertices changed"
    G.check_values(rp, full, L)
    rng = np.random.default_rng(3)
    nxt = n
    for b in range(6):
        ups, rows = stream.next_batch(20)
        extra = G.ups_array([(I.OP_ADD_EDGE, nxt, int(rng.integers(0, n))), (I.OP_ADD_EDGE, int(rng.integers(0, n)), nxt + 1),
                             (I.OP_ADD_EDGE, nxt + 2, nxt + 3), (I.OP_SET_FEATURE, nxt, rows.shape[0]),
                             (I.OP_ADD_EDGE, nxt + 1, nxt)])
        nxt += 4
        ups = np.concatenate([ups, extra])
        rows = np.concatenate([rows, I.features(1, model.dims[0], 200 + b)])
        rp.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        G.check_frontiers(rp, orc, L)
    rowptr, col = rp.export_graph()
    orp, ocol = orc.export_csr()
    assert np.array_equal(rowptr, orp) and np.array_equal(col, ocol)
    G.check_values(rp, orc.full(), L)
    rp.reserve_vertices(n + spare + 33)                      # once more, to a capacity that is no multiple of 32
    assert rp.embeddings(L).shape[0] == n + spare + 33
    rp.apply_batch(G.ups_array([(I.OP_ADD_EDGE, n + spare + 32, 0)]))
    assert rp.stats()["n_added"] == 1
    rp.close()
