"""Partitioned execution (Sec. 4) on the device: P workers, each a context of its own holding one vertex
partition, run in one process on one GPU (the phases of a hop run worker after worker; nothing waits
on the device).  After every batch the rows gathered from the owners must equal the single-machine
oracle's full recomputation on the global graph, the union of the workers' hop sets the oracle's hop
sets, and the number of halo rows sent the oracle cluster's (one combined row per worker and remote
sink)."""
import numpy as np
import pytest

from paper_2601_12347_b200 import inputs as I
from tolerances import TOL

import test_gpu_parity as G

pytestmark = pytest.mark.gpu

env = G.env

MODELS = {
    "sage_mean": lambda: I.sage_model([18, 36, 10], I.AGG_MEAN),
    "sage_sum_3l": lambda: I.sage_model([18, 36, 20, 10], I.AGG_SUM),
    "gc_sum": lambda: I.graphconv_model([18, 36, 10], I.AGG_SUM),
    "gcn_wsum_3l": lambda: I.graphconv_model([18, 36, 20, 10], I.AGG_WSUM_GCN),
    "gin_3l": lambda: I.gin_model(18, 24, 3, eps=0.25),
    "sage_wide": lambda: I.sage_model([40, 160, 24], I.AGG_MEAN),
}


def max_err(got, ref):
    return float(np.max(np.abs(got.astype(np.float64) - ref) / (1.0 + np.abs(ref)))) if ref.size else 0.0


def setup(name, P, n, m, seed, spare=0):
    from oracle.partitioned import Cluster as OracleCluster
    from paper_2601_12347_b200.partitioned import Cluster
    model = MODELS[name]()
    L = len(model.layers)
    src, dst = I.er_graph(n, m, seed)
    have = set(zip(src.tolist(), dst.tolist()))
    extra = [(0, int(v)) for v in range(1, min(n, 300)) if (0, int(v)) not in have]      # a hub that cuts every partition
    src = np.concatenate([src, np.array([a for a, _ in extra], dtype=np.int32)])
    dst = np.concatenate([dst, np.array([b for _, b in extra], dtype=np.int32)])
    X = I.features(n + spare, model.dims[0], seed)
    X[n:] = 0
    W = I.make_weights(model, seed, zero_bias=False)
    owner = np.full(n + spare, -1, dtype=np.int32)
    owner[:n] = np.random.default_rng(seed).integers(0, P, size=n)
    return model, L, src, dst, X, W, owner, Cluster, OracleCluster


@pytest.mark.parametrize("P", [2, 3])
@pytest.mark.parametrize("name", list(MODELS.keys()))
def test_workers_compute_what_one_machine_computes(env, name, P):
    ripple, Oracle = env
    n = 700
    model, L, src, dst, X, W, owner, Cluster, OracleCluster = setup(name, P, n, 5000, 3)
    orc = Oracle(n, src, dst, X, model, W)
    full = orc.full()
    ocl = OracleCluster(P, owner, n, src, dst, X, model, W, full, [None] + [orc.full_S(l) for l in range(1, L + 1)])
    cl = Cluster(P, owner, src, dst, X, model, W)
    for l in range(L + 1):
        assert max_err(cl.embeddings(l, n), full[l]) <= TOL, f"bootstrap, layer {l}"
    stream = I.UpdateStream(n, src, dst, model.dims[0], 3)
    for b, bs in enumerate([1, 1, 2, 7, 33, 100, 1, 250, 64, 5]):
        ups, rows = stream.next_batch(bs)
        cl.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        ocl.apply_batch(ups, rows)
        for l in range(L + 1):
            assert np.array_equal(cl.affected(l), orc.affected(l)), (name, P, b, l)
        assert cl.rows_sent()[1:] == ocl.halo_rows_sent[1:], (name, P, b)
        if b % 3 == 2 or b == 9:
            full = orc.full()
            for l in range(L + 1):
                assert max_err(cl.embeddings(l, n), full[l]) <= TOL, (name, P, b, l)
    cl.close()


@pytest.mark.parametrize("routing", ["locality", "hash"])
def test_vertices_created_by_the_stream_are_placed_and_computed(env, routing):
    ripple, Oracle = env
    from paper_2601_12347_b200 import partitioned as PT
    n, spare, P = 400, 40, 3
    model, L, src, dst, X, W, owner, Cluster, _ = setup("sage_mean", P, n, 3000, 5, spare=spare)
    orc = Oracle(n + spare, src, dst, X, model, W)
    cl = Cluster(P, owner, src, dst, X, model, W, routing=PT.ROUTE_LOCALITY if routing == "locality" else PT.ROUTE_HASH,
                 spare_local=spare)
    rng = np.random.default_rng(1)
    stream = I.UpdateStream(n, src, dst, model.dims[0], 5)
    nxt = n
    for b in range(8):
        ups, rows = stream.next_batch(20)
        extra = G.ups_array([(I.OP_ADD_EDGE, nxt, int(rng.integers(0, n))), (I.OP_ADD_EDGE, int(rng.integers(0, n)), nxt + 1),
                             (I.OP_ADD_EDGE, nxt + 2, nxt + 3), (I.OP_SET_FEATURE, nxt, rows.shape[0])])
        nxt += 4
        ups = np.concatenate([ups, extra])
        rows = np.concatenate([rows, I.features(1, model.dims[0], 100 + b)])
        cl.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        for l in range(L + 1):
            assert np.array_equal(cl.affected(l), orc.affected(l)), (b, l)
    full = orc.full()
    placed = np.array([cl.router.owner(v) >= 0 for v in range(n + spare)])
    assert placed[:nxt].all() and not placed[nxt:].any()
    for l in range(L + 1):
        assert max_err(cl.embeddings(l, n + spare)[placed], full[l][placed]) <= TOL, l
    cl.close()


def test_one_partition_is_the_single_machine_case(env):
    ripple, Oracle = env
    n = 300
    model, L, src, dst, X, W, owner, Cluster, _ = setup("gc_sum", 1, n, 2000, 9)
    owner[:] = 0
    orc = Oracle(n, src, dst, X, model, W)
    cl = Cluster(1, owner, src, dst, X, model, W)
    stream = I.UpdateStream(n, src, dst, model.dims[0], 9)
    for _ in range(5):
        ups, rows = stream.next_batch(30)
        cl.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
    assert cl.rows_sent()[1:] == [0] * L
    full = orc.full()
    for l in range(L + 1):
        assert max_err(cl.embeddings(l, n), full[l]) <= TOL
    cl.close()


def test_partitioned_context_refuses_what_it_cannot_do(env):
    ripple, Oracle = env
    from paper_2601_12347_b200.partitioned import Cluster
    n = 200
    model, L, src, dst, X, W, owner, _, _ = setup("sage_mean", 2, n, 1000, 4)
    cl = Cluster(2, owner, src, dst, X, model, W)
    w = cl.workers[0]
    with pytest.raises(ripple.RippleError):
        w.apply_batch(G.ups_array([(I.OP_ADD_EDGE, 0, 1)]))
    with pytest.raises(ripple.RippleError):
        w.recompute_full()
    with pytest.raises(ripple.RippleError):
        w.begin(G.ups_array([(I.OP_DEL_VERTEX, 0, 0)]), None, np.zeros(1, dtype=np.uint8))
    # a worker whose halo slots name a peer that was never registered refuses to exchange
    from paper_2601_12347_b200 import partitioned as PT
    lone, _ = PT._make_worker(cl.router, 1, X, model, W)
    with pytest.raises(ripple.RippleError):
        lone.bootstrap_layer(1)
    with pytest.raises(ripple.RippleError):
        lone.set_halos(0, np.array([99], dtype=np.int32), np.array([0], dtype=np.int32))
    # ... and one whose halo slot names a vertex its owner does not have
    for r, wk in enumerate(cl.workers):
        lone.set_peer(r, wk.exports())
    lone.set_halos(0, np.array([0], dtype=np.int32), np.array([cl.workers[0].n + 5], dtype=np.int32))
    with pytest.raises(ripple.RippleError) as e:
        lone.bootstrap_layer(1)
    assert e.value.status == ripple.ERR_VERTEX_RANGE
    lone.close()
    cl.close()
    model = I.graphconv_model([18, 36, 10], I.AGG_MAX)
    with pytest.raises(ripple.RippleError):
        Cluster(2, owner, src, dst, X, model, I.make_weights(model, 1))


# ---------------------------------------------------------------------------------------------
# one worker per process: CUDA IPC mappings of the peers' buffers, barriers between the phases.  Both
# processes use the one GPU of the test box; their kernels never wait for each other (every phase call
# returns when its device work is done, the barrier is on the host).
# ---------------------------------------------------------------------------------------------
def _ipc_rank(rank, world, port, out):
    import datetime
    import os
    import torch
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world, timeout=datetime.timedelta(seconds=120))
    torch.cuda.set_device(0)
    from oracle.oracle import Oracle
    from paper_2601_12347_b200.partitioned import DistributedWorker
    n = 600
    model = I.sage_model([18, 36, 10], I.AGG_MEAN)
    src, dst = I.er_graph(n, 4000, 13)
    X = I.features(n, 18, 13)
    W = I.make_weights(model, 13, zero_bias=False)
    owner = np.random.default_rng(13).integers(0, world, size=n).astype(np.int32)
    dw = DistributedWorker(owner, src, dst, X, model, W)
    orc = Oracle(n, src, dst, X, model, W)
    stream = I.UpdateStream(n, src, dst, 18, 13)
    sent = 0
    for _ in range(6):
        ups, rows = stream.next_batch(40)
        dw.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        sent += sum(dw.worker.rows_sent())
    full = orc.full()
    nl = dw.worker.n_local
    gof = np.array([dw.router.global_id(rank, i) for i in range(nl)])
    worst = 0.0
    for l in range(3):
        h = dw.worker.embeddings(l).cpu().numpy()[:nl][gof >= 0].astype(np.float64)
        ref = full[l][gof[gof >= 0]]
        worst = max(worst, float(np.max(np.abs(h - ref) / (1.0 + np.abs(ref)))))
    mine = sorted(gof[dw.worker.affected(2).cpu().numpy()].tolist())
    out[rank] = (worst, int((gof >= 0).sum()), sent, mine, orc.affected(2).tolist())
    dist.barrier()
    dw.close()
    dist.destroy_process_group()


def test_one_worker_per_process_with_ipc_mappings(env):
    import socket
    import torch.multiprocessing as mp
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_ipc_rank, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert sum(res[r][1] for r in range(world)) == 600
    assert all(res[r][0] <= TOL for r in range(world)), [res[r][0] for r in range(world)]
    assert all(res[r][2] > 0 for r in range(world))                      # rows did cross between the processes
    assert sorted(res[0][3] + res[1][3]) == res[0][4]                      # the union of the hop sets is the oracle's


@pytest.mark.parametrize("name", ["sage_mean", "gcn_wsum_3l", "gin_3l"])
def test_vertex_deletions_are_expanded_by_the_router(env, name):
    """The workers never see a vertex deletion: the router turns it into the deletions of the vertex's edges
    (cut edges reach both workers) and a zero feature row."""
    ripple, Oracle = env
    n, P = 700, 3
    model, L, src, dst, X, W, owner, Cluster, _ = setup(name, P, n, 5000, 6)
    orc = Oracle(n, src, dst, X, model, W)
    cl = Cluster(P, owner, src, dst, X, model, W, max_batch=4096)
    stream = I.UpdateStream(n, src, dst, model.dims[0], 6, mix=(0.38, 0.38, 0.2, 0.04))
    for b, bs in enumerate([1, 5, 20, 60, 20, 5, 40, 3]):
        ups, rows = stream.next_batch(bs)
        if b == 3:
            ups[10] = (I.OP_DEL_VERTEX, 0, 0)       # the hub whose out-edges cut every partition
        cl.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        for l in range(L + 1):
            assert np.array_equal(cl.affected(l), orc.affected(l)), (name, b, l)
    full = orc.full()
    for l in range(L + 1):
        assert max_err(cl.embeddings(l, n), full[l]) <= TOL, (name, l)
    cl.close()


@pytest.mark.parametrize("P", [2, 3])
def test_stored_edge_weights_across_partitions(env, P):
    """The weighted sum with a stored weight per edge (the paper's GC-W, which Sec. 6.3.1 runs distributed): a cut
    edge keeps its weight at both workers, messages into halo mailboxes are scaled by it."""
    ripple, Oracle = env
    from paper_2601_12347_b200.partitioned import Cluster
    n = 700
    model = I.graphconv_model([18, 36, 20, 10], I.AGG_WSUM_EDGE)
    src, dst = I.er_graph(n, 5000, 8)
    have = set(zip(src.tolist(), dst.tolist()))
    extra = [(0, int(v)) for v in range(1, 300) if (0, int(v)) not in have]
    src = np.concatenate([src, np.array([a for a, _ in extra], dtype=np.int32)])
    dst = np.concatenate([dst, np.array([b for _, b in extra], dtype=np.int32)])
    ew = I.edge_weights(src.size, 8)
    X = I.features(n, 18, 8)
    W = I.make_weights(model, 8, zero_bias=False)
    owner = np.random.default_rng(8).integers(0, P, size=n).astype(np.int32)
    orc = Oracle(n, src, dst, X, model, W, edge_weights=ew)
    cl = Cluster(P, owner, src, dst, X, model, W, edge_weights=ew)
    full = orc.full()
    for l in range(4):
        assert max_err(cl.embeddings(l, n), full[l]) <= TOL, f"bootstrap, layer {l}"
    stream = I.UpdateStream(n, src, dst, 18, 8)
    for b, bs in enumerate([1, 2, 7, 33, 100, 1, 64]):
        ups, rows, ow = stream.next_batch_weighted(bs)
        cl.apply_batch(ups, rows, ow)
        assert orc.apply_incremental(ups, rows, op_weights=ow) == 0
        for l in range(4):
            assert np.array_equal(cl.affected(l), orc.affected(l)), (P, b, l)
    full = orc.full()
    for l in range(4):
        assert max_err(cl.embeddings(l, n), full[l]) <= TOL, (P, l)
    # the stored weights themselves: every worker's copy of its edges, cut edges included
    rp_o, col_o = orc.export_csr()
    w_o = orc.export_weights()
    want = {(int(u), int(v)): float(a) for u, v, a in zip(np.repeat(np.arange(n), np.diff(rp_o)), col_o, w_o)}
    for r, wk in enumerate(cl.workers):
        gof = cl.router.global_ids(r, wk.n)
        rowptr, col, wts = wk.export_graph_weighted()
        su = np.repeat(np.arange(wk.n), np.diff(rowptr))
        for u, v, a in zip(gof[su].tolist(), gof[col].tolist(), wts.tolist()):
            assert want[(u, v)] == a
    cl.close()


@pytest.mark.parametrize("name", ["sage_mean", "gcn_wsum_3l", "gin_3l"])
def test_layer_wise_inference_can_be_run_again_between_batches(env, name):
    """The bootstrap call, run again after batches that added and deleted edges and created halo slots: every
    cached row is computed anew from the current graph, and the stream continues from that state."""
    ripple, Oracle = env
    n, P = 700, 3
    model, L, src, dst, X, W, owner, Cluster, _ = setup(name, P, n, 5000, 9)
    orc = Oracle(n, src, dst, X, model, W)
    cl = Cluster(P, owner, src, dst, X, model, W)
    stream = I.UpdateStream(n, src, dst, model.dims[0], 9)
    for rnd in range(3):
        for bs in [1, 40, 7, 150]:
            ups, rows = stream.next_batch(bs)
            cl.apply_batch(ups, rows)
            assert orc.apply_incremental(ups, rows) == 0
            for l in range(L + 1):
                assert np.array_equal(cl.affected(l), orc.affected(l)), (name, rnd, bs, l)
        before = [cl.embeddings(l, n) for l in range(L + 1)]
        cl.recompute_full()
        full = orc.full()
        for l in range(L + 1):
            got = cl.embeddings(l, n)
            assert max_err(got, full[l]) <= TOL, (name, rnd, l)
            assert max_err(got, before[l].astype(np.float64)) <= 2 * TOL    # and it agreed with the incremental state
    cl.close()


def test_recomputation_discards_the_rounding_of_an_unnormalised_sum_stack(env):
    """A partitioned context has no per-row rebuild (rows of remote in-neighbours are not resident), so on the
    GIN-sum stack of the skewed sparse graph, whose rows reach 1e6, the roundings of the incremental additions add
    up over the batches; the layer-wise inference run again brings every row back to within the bound that a fresh
    fp32 evaluation meets (tests/tolerances.py)."""
    from tolerances import GIN_ROW_SLACK
    ripple, Oracle = env
    from paper_2601_12347_b200.partitioned import Cluster
    w = I.workloads()["sparse-deep-gin"]
    src, dst = I.make_graph(w)
    X = I.features(w.n, w.model.dims[0], w.seed)
    W = I.make_weights(w.model, w.seed)
    L = len(w.model.layers)
    owner = np.random.default_rng(21).integers(0, 2, size=w.n).astype(np.int32)
    orc = Oracle(w.n, src, dst, X, w.model, W)
    cl = Cluster(2, owner, src, dst, X, w.model, W, max_batch=2048)
    stream = I.make_stream(w, src, dst, 21)
    for bs in [1000, 33, 1000, 257, 1000, 1000]:
        ups, rows = stream.next_batch(bs)
        cl.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        for l in range(L + 1):
            assert np.array_equal(cl.affected(l), orc.affected(l)), (bs, l)
    full = orc.full()
    drift = [G.max_err(cl.embeddings(l, w.n), full[l], GIN_ROW_SLACK) for l in range(L + 1)]
    cl.recompute_full()
    fresh = [G.max_err(cl.embeddings(l, w.n), full[l], GIN_ROW_SLACK) for l in range(L + 1)]
    assert max(fresh) <= TOL, fresh
    assert max(drift) <= 10 * TOL, drift          # a lost or doubled message would be O(1), not a few roundings
    cl.close()
