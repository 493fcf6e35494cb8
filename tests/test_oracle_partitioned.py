"""Pins for the oracle of the distributed execution model (Sec. 4): routing and vertex placement
(Sec. 4.3, 4.4, Alg. 1) by hand-made cases for every branch, and the workers' result against the
single-machine oracle's full recomputation on the same global graph (the paper's claim that the
distributed execution flow computes what a single machine computes), with the hop sets against the
single-machine incremental route and the combiner's effect on the number of rows sent."""
import numpy as np
import pytest

from oracle.oracle import Oracle
from oracle.partitioned import Cluster, Server
from paper_2601_12347_b200 import inputs as I


def ups_array(recs):
    a = np.zeros(len(recs), dtype=I.UPDATE_DTYPE)
    for i, r in enumerate(recs):
        a[i] = r
    return a


# ---------------------------------------------------------------------------------------------
# routing and placement
# ---------------------------------------------------------------------------------------------
def _server(routing="locality"):
    # 8 placed vertices on 2 partitions, vertex 3 has in-degree 5 (average degree 6 / 8: high), ids 8.. are new
    owner = np.array([0, 0, 0, 0, 1, 1, 1, 1, -1, -1, -1, -1], dtype=np.int64)
    src = np.array([0, 1, 2, 4, 5, 6], dtype=np.int32)
    dst = np.array([3, 3, 3, 3, 3, 7], dtype=np.int32)
    return Server(2, owner, src, dst, routing=routing)


def test_high_in_degree_set_is_twice_the_average_degree():
    s = _server()
    assert s.hd == {3}          # in-degree 5 > 2 * 6 / 8; vertex 7 has 1, not above 1.5


def test_local_edge_goes_to_its_partition_only():
    s = _server()
    r = s.route(ups_array([(I.OP_ADD_EDGE, 0, 1), (I.OP_DEL_EDGE, 6, 7)]))
    assert r[0] == [(0, I.OP_ADD_EDGE, 0, 1, True)]
    assert r[1] == [(1, I.OP_DEL_EDGE, 6, 7, True)]


def test_cut_edge_goes_to_the_source_and_a_no_compute_copy_to_the_sink():
    s = _server()
    r = s.route(ups_array([(I.OP_ADD_EDGE, 1, 5), (I.OP_DEL_EDGE, 4, 3)]))
    assert r[0] == [(0, I.OP_ADD_EDGE, 1, 5, True), (1, I.OP_DEL_EDGE, 4, 3, False)]
    assert r[1] == [(0, I.OP_ADD_EDGE, 1, 5, False), (1, I.OP_DEL_EDGE, 4, 3, True)]


def test_feature_update_goes_to_the_owner():
    s = _server()
    r = s.route(ups_array([(I.OP_SET_FEATURE, 6, 0), (I.OP_SET_FEATURE, 2, 1)]))
    assert r[0] == [(1, I.OP_SET_FEATURE, 2, 1, True)] and r[1] == [(0, I.OP_SET_FEATURE, 6, 0, True)]


def test_new_source_joins_a_high_in_degree_sink():
    s = _server()
    s.load[:] = [10, 4]                                   # partition 1 is the lighter one
    s.route(ups_array([(I.OP_ADD_EDGE, 8, 3)]))          # sink 3 is high in-degree, lives on 0
    assert s.owner[8] == 0 and s.load[0] == 11


def test_new_source_of_an_ordinary_sink_goes_to_the_least_loaded_partition():
    s = _server()
    s.load[:] = [10, 4]
    r = s.route(ups_array([(I.OP_ADD_EDGE, 8, 2)]))      # sink 2 is not high in-degree
    assert s.owner[8] == 1 and s.load[1] == 5
    assert r[1] == [(0, I.OP_ADD_EDGE, 8, 2, True)] and r[0] == [(0, I.OP_ADD_EDGE, 8, 2, False)]


def test_edge_without_existing_endpoints_goes_to_the_least_loaded_partition():
    s = _server()
    s.load[:] = [3, 9]
    r = s.route(ups_array([(I.OP_ADD_EDGE, 8, 9)]))
    assert s.owner[8] == 0 and s.owner[9] == 0 and s.load[0] == 5
    assert r[0] == [(0, I.OP_ADD_EDGE, 8, 9, True)] and r[1] == []


def test_new_sink_of_an_existing_source_takes_the_final_else():
    s = _server()
    s.load[:] = [9, 3]
    s.route(ups_array([(I.OP_ADD_EDGE, 0, 10)]))
    assert s.owner[10] == 1 and s.owner[0] == 0


def test_ties_go_to_the_lowest_partition_and_load_counts_placements():
    s = _server()
    assert list(s.load) == [4, 4]
    s.route(ups_array([(I.OP_ADD_EDGE, 8, 9), (I.OP_ADD_EDGE, 10, 11)]))
    assert list(s.owner[8:12]) == [0, 0, 1, 1] and list(s.load) == [6, 6]


def test_hash_routing_places_by_id_modulo_partitions():
    s = _server("hash")
    s.route(ups_array([(I.OP_ADD_EDGE, 8, 3), (I.OP_ADD_EDGE, 9, 11)]))
    assert s.owner[8] == 0 and s.owner[9] == 1 and s.owner[11] == 1


def test_high_in_degree_set_is_refreshed_after_the_stated_number_of_updates():
    owner = np.zeros(6, dtype=np.int64)
    s = Server(2, owner, np.array([0], dtype=np.int32), np.array([1], dtype=np.int32), hd_refresh=4)
    assert s.hd == {1}                                     # in-degree 1 > 2 * 1 / 6
    s = Server(2, owner, np.array([0, 1, 2], dtype=np.int32), np.array([1, 2, 0], dtype=np.int32), hd_refresh=4)
    assert s.hd == set()                                   # every in-degree is 1 = 2 * 3 / 6
    s.route(ups_array([(I.OP_ADD_EDGE, 3, 5), (I.OP_ADD_EDGE, 4, 5), (I.OP_ADD_EDGE, 0, 5)]))
    assert s.hd == set()                                   # three updates seen: not refreshed yet
    s.route(ups_array([(I.OP_ADD_EDGE, 1, 5)]))
    assert s.hd == {5}                                     # in-degree 4 > 2 * 7 / 6


def test_no_op_updates_leave_the_in_degrees_alone():
    s = _server()
    s.route(ups_array([(I.OP_ADD_EDGE, 0, 3), (I.OP_DEL_EDGE, 1, 2)]))     # existing edge, missing edge
    assert s.in_degree[3] == 5 and s.in_degree[2] == 0 and s.n_edges == 6


# ---------------------------------------------------------------------------------------------
# workers, combiner, remote send: the cluster computes what one machine computes
# ---------------------------------------------------------------------------------------------
def rel_err(a, b):
    return float(np.max(np.abs(a - b) / (1.0 + np.abs(b)))) if a.size else 0.0


MODELS = {
    "sage_mean": lambda: I.sage_model([5, 6, 3], I.AGG_MEAN),
    "sage_sum_3l": lambda: I.sage_model([5, 6, 6, 3], I.AGG_SUM),
    "gc_sum": lambda: I.graphconv_model([5, 6, 3], I.AGG_SUM),
    "gcn_wsum_3l": lambda: I.graphconv_model([5, 6, 6, 3], I.AGG_WSUM_GCN),
    "gin": lambda: I.gin_model(5, 6, 3),
}


def _cluster(name, P, n=60, m=240, seed=7, spare=0, routing="locality"):
    model = MODELS[name]()
    src, dst = I.er_graph(n, m, seed)
    X = I.features(n + spare, model.dims[0], seed)
    X[n:] = 0
    W = I.make_weights(model, seed, zero_bias=False)
    orc = Oracle(n + spare, src, dst, X, model, W)
    L = len(model.layers)
    owner = np.full(n + spare, -1, dtype=np.int64)
    owner[:n] = np.random.default_rng(seed).integers(0, P, size=n)
    full = orc.full()
    cl = Cluster(P, owner, n + spare, src, dst, X, model, W, full, [None] + [orc.full_S(l) for l in range(1, L + 1)],
                 routing=routing)
    return model, src, dst, orc, cl, L


@pytest.mark.parametrize("P", [2, 3])
@pytest.mark.parametrize("name", list(MODELS.keys()))
def test_cluster_equals_single_machine_every_batch(name, P):
    n = 60
    model, src, dst, orc, cl, L = _cluster(name, P, n=n)
    stream = I.UpdateStream(n, src, dst, model.dims[0], 7)
    for b in range(10):
        ups, rows = stream.next_batch(1 + 4 * (b % 3))
        cl.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        full = orc.full()
        for l in range(L + 1):
            assert rel_err(cl.gather(l, n), full[l]) < 1e-10, (name, P, b, l)
            assert cl.affected[l] == orc.affected(l).tolist(), (name, P, b, l)


def test_repeated_pairs_and_no_ops_in_one_batch():
    n = 60
    model, src, dst, orc, cl, L = _cluster("sage_mean", 2, n=n)
    e0 = (int(src[0]), int(dst[0]))
    have = set(zip(src.tolist(), dst.tolist()))
    miss = next((a, b) for a in range(n) for b in range(n) if a != b and (a, b) not in have and cl.server.owner[a] != cl.server.owner[b])
    ups = ups_array([(I.OP_DEL_EDGE, *e0), (I.OP_ADD_EDGE, *e0), (I.OP_ADD_EDGE, *miss), (I.OP_DEL_EDGE, *miss),
                     (I.OP_ADD_EDGE, *miss), (I.OP_ADD_EDGE, int(src[3]), int(dst[3])), (I.OP_SET_FEATURE, 5, 0),
                     (I.OP_SET_FEATURE, 5, 1)])
    rows = I.features(2, 5, 99)
    cl.apply_batch(ups, rows)
    assert orc.apply_incremental(ups, rows) == 0
    full = orc.full()
    for l in range(L + 1):
        assert rel_err(cl.gather(l, n), full[l]) < 1e-10
        assert cl.affected[l] == orc.affected(l).tolist()


@pytest.mark.parametrize("routing", ["locality", "hash"])
def test_vertices_created_by_edge_additions_are_placed_and_computed(routing):
    n, spare = 50, 10
    model, src, dst, orc, cl, L = _cluster("sage_mean", 3, n=n, m=200, spare=spare, routing=routing)
    rng = np.random.default_rng(1)
    new_ids = list(range(n, n + spare))
    for b in range(5):
        a, c = new_ids[2 * b], new_ids[2 * b + 1]
        ups = ups_array([(I.OP_ADD_EDGE, a, int(rng.integers(0, n))), (I.OP_SET_FEATURE, a, 0),
                         (I.OP_ADD_EDGE, int(rng.integers(0, n)), c), (I.OP_ADD_EDGE, a, c)])
        rows = I.features(1, 5, 100 + b)
        cl.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        full = orc.full()
        assert cl.server.owner[a] >= 0 and cl.server.owner[c] >= 0
        placed = cl.server.owner >= 0     # ids no edge has named yet live on no worker
        for l in range(L + 1):
            assert rel_err(cl.gather(l, n + spare)[placed], full[l][placed]) < 1e-10, (b, l)
            assert cl.affected[l] == orc.affected(l).tolist()


def test_combiner_sends_one_row_per_worker_and_remote_sink():
    # a star: hub 0 on partition 0 points at 30 sinks on partition 1, which also receive from 1 and 2 (partition 0)
    n = 40
    srcs = [0] * 30 + [1] * 30 + [2] * 30
    dsts = list(range(5, 35)) * 3
    src, dst = np.array(srcs, dtype=np.int32), np.array(dsts, dtype=np.int32)
    model = I.graphconv_model([4, 4, 2], I.AGG_SUM)
    X = I.features(n, 4, 2)
    W = I.make_weights(model, 2)
    orc = Oracle(n, src, dst, X, model, W)
    owner = np.array([0] * 5 + [1] * 35, dtype=np.int64)
    cl = Cluster(2, owner, n, src, dst, X, model, W, orc.full(), [None, orc.full_S(1), orc.full_S(2)])
    ups = ups_array([(I.OP_SET_FEATURE, 0, 0), (I.OP_SET_FEATURE, 1, 1), (I.OP_SET_FEATURE, 2, 2)])
    rows = I.features(3, 4, 3)
    cl.apply_batch(ups, rows)
    assert orc.apply_incremental(ups, rows) == 0
    assert cl.halo_rows_sent[1] == 30          # 90 messages cross the cut, 30 combined rows are sent
    assert orc.active_edges(1) == 90
    assert rel_err(cl.gather(2, n), orc.full()[2]) < 1e-12


# ---------------------------------------------------------------------------------------------
# vertex deletion: expanded by the server
# ---------------------------------------------------------------------------------------------
def test_vertex_deletion_is_replaced_by_its_edge_deletions_and_a_zero_row():
    s = _server()
    r = s.route(ups_array([(I.OP_DEL_VERTEX, 3, 0)]))          # in-edges from 0, 1, 2 (partition 0) and 4, 5 (partition 1)
    assert r[0] == [(0, I.OP_DEL_EDGE, 0, 3, True), (0, I.OP_DEL_EDGE, 1, 3, True), (0, I.OP_DEL_EDGE, 2, 3, True),
                    (0, I.OP_DEL_EDGE, 4, 3, False), (0, I.OP_DEL_EDGE, 5, 3, False), (0, I.OP_SET_FEATURE, 3, -1, True)]
    assert r[1] == [(0, I.OP_DEL_EDGE, 4, 3, True), (0, I.OP_DEL_EDGE, 5, 3, True)]
    assert s.in_degree[3] == 0 and s.n_edges == 1
    r = s.route(ups_array([(I.OP_ADD_EDGE, 6, 3), (I.OP_DEL_VERTEX, 6, 0)]))   # an edge added earlier in the batch goes too
    assert (1, I.OP_DEL_EDGE, 6, 3, True) in r[1] and (1, I.OP_DEL_EDGE, 6, 7, True) in r[1]
    assert s.n_edges == 0


@pytest.mark.parametrize("P", [2, 3])
@pytest.mark.parametrize("name", ["sage_mean", "gcn_wsum_3l", "gin"])
def test_cluster_with_vertex_deletions_equals_single_machine(name, P):
    n = 60
    model, src, dst, orc, cl, L = _cluster(name, P, n=n)
    stream = I.UpdateStream(n, src, dst, model.dims[0], 7, mix=(0.35, 0.35, 0.2, 0.1))
    for b in range(10):
        ups, rows = stream.next_batch(1 + 4 * (b % 3))
        cl.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        full = orc.full()
        for l in range(L + 1):
            assert rel_err(cl.gather(l, n), full[l]) < 1e-9, (name, P, b, l)
            assert cl.affected[l] == orc.affected(l).tolist(), (name, P, b, l)


# ---------------------------------------------------------------------------------------------
# stored edge weights (the paper's GC-W runs distributed too, Sec. 6.3.1)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("P", [2, 3])
def test_cluster_with_stored_edge_weights_equals_single_machine(P):
    n = 60
    model = I.graphconv_model([5, 6, 6, 3], I.AGG_WSUM_EDGE)
    src, dst = I.er_graph(n, 240, 9)
    ew = I.edge_weights(src.size, 9)
    X = I.features(n, 5, 9)
    W = I.make_weights(model, 9, zero_bias=False)
    orc = Oracle(n, src, dst, X, model, W, edge_weights=ew)
    owner = np.random.default_rng(9).integers(0, P, size=n)
    cl = Cluster(P, owner, n, src, dst, X, model, W, orc.full(), [None] + [orc.full_S(l) for l in (1, 2, 3)],
                 edge_weights=ew)
    stream = I.UpdateStream(n, src, dst, 5, 9)
    for b in range(10):
        ups, rows, ow = stream.next_batch_weighted(1 + 4 * (b % 3))
        cl.apply_batch(ups, rows, ow)
        assert orc.apply_incremental(ups, rows, op_weights=ow) == 0
        full = orc.full()
        for l in range(4):
            assert rel_err(cl.gather(l, n), full[l]) < 1e-10, (P, b, l)
            assert cl.affected[l] == orc.affected(l).tolist()
