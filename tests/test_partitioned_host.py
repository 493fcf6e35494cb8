"""Host side of the partitioned execution (no GPU): the library's router against the oracle's server on
random streams (routing, placement by Alg. 1 and by hashing, the high in-degree set and its refresh,
global-to-local ids, halo slots), its error paths, and the phase sequence of a multi-process run as
two gloo ranks that drive the oracle's workers and exchange the combined halo rows for real."""
import os
import socket
import sys

import numpy as np
import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle.oracle import Oracle
from oracle.partitioned import Cluster as OracleCluster, Server
from paper_2601_12347_b200 import build as B
from paper_2601_12347_b200 import inputs as I


@pytest.fixture(scope="module")
def PT():
    B.build_library()
    from paper_2601_12347_b200 import partitioned
    return partitioned


def ups_array(recs):
    a = np.zeros(len(recs), dtype=I.UPDATE_DTYPE)
    for i, r in enumerate(recs):
        a[i] = r
    return a


def _graph(n=300, m=1500, spare=60, P=3, seed=3):
    src, dst = I.er_graph(n, m, seed)
    owner = np.full(n + spare, -1, dtype=np.int32)
    owner[:n] = np.random.default_rng(seed).integers(0, P, size=n)
    return n, spare, src, dst, owner


@pytest.mark.parametrize("routing", ["locality", "hash"])
def test_router_routes_like_the_oracle_server(PT, routing):
    n, spare, src, dst, owner = _graph()
    r = PT.Router(3, owner, src, dst, routing=PT.ROUTE_LOCALITY if routing == "locality" else PT.ROUTE_HASH,
                  hd_refresh=50, spare_local=spare, halo_capacity=n + spare)
    s = Server(3, owner, src, dst, routing=routing, hd_refresh=50)
    stream = I.UpdateStream(n, src, dst, 4, 3, mix=(0.38, 0.38, 0.2, 0.04))    # vertex deletions too: the router expands them
    rng = np.random.default_rng(5)
    nxt = n
    for b in range(30):
        ups, _ = stream.next_batch(20)
        if nxt < n + spare - 3:     # vertices that the stream creates: new source, new sink, both new
            ups = np.concatenate([ups, ups_array([(I.OP_ADD_EDGE, nxt, int(rng.integers(0, n))),
                                                  (I.OP_ADD_EDGE, int(rng.integers(0, n)), nxt + 1),
                                                  (I.OP_ADD_EDGE, nxt + 2, nxt + 3)])])
            nxt += 4
        r.route(ups)
        want = s.route(ups)
        for p in range(3):
            lu, nc, row_of, _, _, _, op_of = r.batch(p)
            got = [(int(x["op"]), r.global_id(p, int(x["u"])),
                    r.global_id(p, int(x["v"])) if x["op"] != I.OP_SET_FEATURE else int(row_of[x["v"]]), bool(c == 0))
                   for x, c in zip(lu, nc)]
            assert got == [(op, u, v, comp) for (_, op, u, v, comp) in want[p]], (b, p)
            assert op_of.tolist() == [i for (i, _, _, _, _) in want[p]], (b, p)     # where in the batch each one comes from
    assert all(r.owner(v) == s.owner[v] for v in range(n + spare))
    assert all(r.is_high_degree(v) == (v in s.hd) for v in range(n + spare))
    assert [r.load(p) for p in range(3)] == s.load.tolist()


def test_partition_holds_every_edge_with_a_local_endpoint_and_halo_tables_point_home(PT):
    n, spare, src, dst, owner = _graph(spare=0)
    r = PT.Router(3, owner, src, dst)
    seen = set()
    for p in range(3):
        n_local, nv, ls, ld, gof, ho, hr, edge_of = r.partition(p)
        assert n_local % 32 == 0 and nv == n_local + n
        own = gof[:n_local]
        assert sorted(own[own >= 0].tolist()) == np.nonzero(owner == p)[0].tolist()
        assert (np.diff(own[own >= 0]) > 0).all()                      # local ids in ascending global id
        edges = set(zip(gof[ls].tolist(), gof[ld].tolist()))
        assert np.array_equal(src[edge_of], gof[ls]) and np.array_equal(dst[edge_of], gof[ld])   # the global edge behind each
        want = {(u, v) for u, v in zip(src.tolist(), dst.tolist()) if owner[u] == p or owner[v] == p}
        assert edges == want
        seen |= edges
        for h in range(ho.size):                                        # a halo slot names its owner's local id
            g = gof[n_local + h]
            assert owner[g] == ho[h] != p and r.local_id(g) == hr[h] and r.global_id(int(ho[h]), int(hr[h])) == g
        halos = set(gof[n_local:n_local + ho.size].tolist())
        cut = {v for u, v in want if owner[v] != p} | {u for u, v in want if owner[u] != p}
        assert halos == cut
    assert seen == set(zip(src.tolist(), dst.tolist()))


def test_new_halo_slots_are_reported_with_the_batch_that_creates_them(PT):
    owner = np.array([0, 0, 1, 1], dtype=np.int32)
    src, dst = np.array([0], dtype=np.int32), np.array([1], dtype=np.int32)
    r = PT.Router(2, owner, src, dst, halo_capacity=4)
    r.route(ups_array([(I.OP_ADD_EDGE, 0, 2), (I.OP_ADD_EDGE, 1, 2), (I.OP_ADD_EDGE, 3, 0)]))
    lu, nc, _, first, ho, hr, op_of = r.batch(0)
    assert first == 0 and ho.tolist() == [1, 1] and hr.tolist() == [r.local_id(2), r.local_id(3)]
    assert op_of.tolist() == [0, 1, 2]
    assert nc.tolist() == [0, 0, 1] and lu["v"].tolist()[:2] == [32, 32] and lu["u"].tolist()[2] == 33
    lu, nc, _, first, ho, hr, _ = r.batch(1)
    assert ho.tolist() == [0, 0] and hr.tolist() == [0, 1] and nc.tolist() == [1, 1, 0]
    r.route(ups_array([(I.OP_DEL_EDGE, 0, 2)]))
    assert r.batch(0)[4].size == 0 and r.batch(0)[3] == 2                # nothing new, next free slot is 2


def test_router_refuses_bad_ids_unknown_ops_and_overflow(PT):
    from paper_2601_12347_b200 import ripple
    owner = np.array([0, 0, 1, 1, -1, -1], dtype=np.int32)
    src, dst = np.array([0], dtype=np.int32), np.array([1], dtype=np.int32)
    r = PT.Router(2, owner, src, dst, halo_capacity=1, spare_local=0)
    for bad in ([(I.OP_DEL_VERTEX, 9, 0)], [(I.OP_ADD_EDGE, 0, 9)], [(7, 0, 1)]):
        with pytest.raises(ripple.RippleError):
            r.route(ups_array(bad))
    r.route(ups_array([(I.OP_ADD_EDGE, 0, 2)]))
    with pytest.raises(ripple.RippleError) as e:
        r.route(ups_array([(I.OP_ADD_EDGE, 0, 3)]))                      # worker 0 has one halo slot
    assert e.value.status == ripple.ERR_CAPACITY
    with pytest.raises(ripple.RippleError):
        PT.Router(2, np.array([0, 5], dtype=np.int32), src, dst)


# ---------------------------------------------------------------------------------------------
# two processes: the phase sequence with real message exchange (oracle workers stand in for the GPUs)
# ---------------------------------------------------------------------------------------------
def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2601_12347_b200 import partitioned as PT
    n = 80
    model = I.sage_model([5, 6, 3], I.AGG_MEAN)
    L = 2
    src, dst = I.er_graph(n, 400, 11)
    X = I.features(n, 5, 11)
    W = I.make_weights(model, 11, zero_bias=False)
    owner = np.random.default_rng(11).integers(0, world, size=n).astype(np.int32)
    orc = Oracle(n, src, dst, X, model, W)
    cl = OracleCluster(world, owner, n, src, dst, X, model, W, orc.full(), [None] + [orc.full_S(l) for l in (1, 2)])
    me = cl.workers[rank]                       # this process drives one worker only
    router = PT.Router(world, owner, src, dst)  # every process runs a replica of the router
    stream = I.UpdateStream(n, src, dst, 5, 11)
    for b in range(6):
        ups, rows = stream.next_batch(9)
        router.route(ups)
        lu, nc, row_of, _, _, _, _ = router.batch(rank)
        ops = [(i, int(x["op"]), router.global_id(rank, int(x["u"])),
                router.global_id(rank, int(x["v"])) if x["op"] != I.OP_SET_FEATURE else int(x["v"]), bool(c == 0))
               for i, (x, c) in enumerate(zip(lu, nc))]
        A, old = me.apply(ops, PT.payload_rows(rows, row_of, 5) if row_of.size else rows[:0])
        dist.barrier()
        for l in range(1, L + 1):
            halo = me.send(l, A, old)
            boxes = [None] * world
            dist.all_gather_object(boxes, {int(v): (int(router.owner(v)), m) for v, m in halo.items()})   # remote send
            for r, box in enumerate(boxes):
                if r != rank:
                    me.receive({v: m for v, (p, m) in box.items() if p == rank})
            dist.barrier()
            A, old = me.compute(l, A)
            dist.barrier()
        assert orc.apply_incremental(ups, rows) == 0
    full = orc.full()
    worst = 0.0
    for l in range(L + 1):
        for v, row in me.H[l].items():
            worst = max(worst, float(np.max(np.abs(row - full[l][v]) / (1 + np.abs(full[l][v])))))
    out[rank] = (worst, len(me.H[0]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_processes_run_the_phases_with_real_exchange(PT):
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert sum(res[r][1] for r in range(world)) == 80
    for r in range(world):
        assert res[r][0] < 1e-10


def test_payload_rows_of_a_worker_have_zeros_for_deleted_vertices(PT):
    rows = np.arange(12, dtype=np.float32).reshape(3, 4)
    out = PT.payload_rows(rows, np.array([2, -1, 0], dtype=np.int32), 4)
    assert np.array_equal(out, np.stack([rows[2], np.zeros(4, dtype=np.float32), rows[0]]))
    assert PT.payload_rows(None, np.array([-1], dtype=np.int32), 4).tolist() == [[0.0] * 4]
    assert PT.payload_rows(rows, np.zeros(0, dtype=np.int32), 4) is None


def test_vertex_deletion_reaches_both_workers_of_every_cut_edge(PT):
    owner = np.array([0, 0, 1, 1], dtype=np.int32)
    src = np.array([0, 2, 1, 0], dtype=np.int32)      # 0->1 (local to 0), 2->0 and 0->3 (cut), 1->2 (cut)
    dst = np.array([1, 0, 2, 3], dtype=np.int32)
    r = PT.Router(2, owner, src, dst, halo_capacity=4)
    r.route(ups_array([(I.OP_DEL_VERTEX, 0, 0)]))
    lu, nc, row_of, _, _, _, op_of = r.batch(0)
    g = lambda p, x: r.global_id(p, int(x))
    ops0 = [(int(x["op"]), g(0, x["u"]), g(0, x["v"]) if x["op"] != I.OP_SET_FEATURE else int(row_of[x["v"]]), int(c)) for x, c in zip(lu, nc)]
    assert ops0 == [(I.OP_DEL_EDGE, 0, 1, 0), (I.OP_DEL_EDGE, 0, 3, 0), (I.OP_DEL_EDGE, 2, 0, 1), (I.OP_SET_FEATURE, 0, -1, 0)]
    assert op_of.tolist() == [0, 0, 0, 0]
    lu, nc, _, _, _, _, _ = r.batch(1)
    ops1 = [(int(x["op"]), g(1, x["u"]), g(1, x["v"]), int(c)) for x, c in zip(lu, nc)]
    assert ops1 == [(I.OP_DEL_EDGE, 0, 3, 1), (I.OP_DEL_EDGE, 2, 0, 0)]
