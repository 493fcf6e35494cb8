"""Parity at full size, in the launch configurations bench.py times.

Dense graph (2 449 029 vertices, 123 718 280 edges, 100 features):
  * 2-layer GraphSAGE-mean 100-256-47 at every batch size of the configuration: 100 consecutive
    batches of 10, 100 of 100, 20 of 1000 and 5 of 10 000, one after the other on the same context.
    While the oracle's incremental route can follow (batches of 10, 100 and the first batches of
    1000; it runs in pull form on all host cores) ALL rows of ALL layers are compared with it;
    after that the oracle follows the structure only and rows are checked one by one against the
    layer definition.
  * 3-layer model: ordinary stream, and the two hub-stress streams (feature-only, delete-heavy: every
    endpoint among the top-1 % out-degree vertices); 4-layer model.  Saturated hops rebuild their
    aggregates, wide layers run on the tensor-core update.
  * GraphConv-max against the oracle's hybrid route, all rows.
Ultra-dense second graph (232 965 vertices, 114.9 M edges, 602 features): 2- and 4-layer models.

Compared exactly after EVERY batch: every affected list A_l, the update counters, the number of
edges carrying a message at each hop, both degree arrays of all vertices.  The canonical CSR of the
whole graph is compared exactly at the end of every phase (exporting and sorting 124 M entries
after each of 225 batches would take longer than everything else together; a slot holding a wrong
neighbour shows there, a wrong count shows at once in the degrees).

Row check against the definition (Eq. 1-2): the oracle recomputes h^l_v in fp64 from the GPU's own
H^{l-1} over the oracle's current graph.  With H^0 bit-identical to the features, row-wise
agreement at every layer is the induction step of "equals full recomputation".  The sample always
holds every vertex of A_1 (up to 10 000), the 100 largest in- and out-degree hubs, the sinks that
lost at least half of their in-edges in the last batch (rebuilt from their in-lists by the library),
vertices from the start and the end of every affected list, vertices with an empty in-list, and
4 000 random vertices.
"""
import time

import numpy as np
import pytest

from paper_2601_12347_b200 import inputs as I
from tolerances import TOL

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2601_12347_b200 import build as B
    B.build_library()
    from paper_2601_12347_b200 import ripple
    from oracle.oracle import Oracle
    torch.cuda.set_device(0)
    return ripple, Oracle


_graphs = {}


def graph_of(wname):
    """Graphs are generated once per (kind, size, seed): the dense workloads all share one."""
    w = I.workloads()[wname]
    key = (w.graph, w.n, w.e, w.seed)
    if key not in _graphs:
        _graphs.clear()          # one large graph on the host at a time
        _graphs[key] = I.make_graph(w)
        # the generator still draws the graph whose checksum was recorded (tests/golden/generator_checksums.json)
        import importlib.util
        import json
        import os
        gold = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
        spec = importlib.util.spec_from_file_location("write_generator_checksums",
                                                      os.path.join(gold, "write_generator_checksums.py"))
        mod = importlib.util.module_from_spec(spec)
        spec.loader.exec_module(mod)
        want = json.load(open(os.path.join(gold, "generator_checksums.json")))
        for name, rec in want.items():
            wn = I.workloads()[name]
            if (wn.graph, wn.n, wn.e, wn.seed) == key:
                assert mod.graph_digest(*_graphs[key]) == rec["graph"], f"generator output of {name} changed"
    return w, _graphs[key]


def check_structure(rp, orc, L, tag):
    st = rp.stats()
    for l in range(L + 1):
        assert np.array_equal(rp.affected(l).cpu().numpy(), orc.affected(l)), f"{tag}: A_{l} differs"
    c = orc.counts()
    assert (st["n_added"], st["n_deleted"], st["n_noop_add"], st["n_noop_del"], st["n_superseded"]) == \
        (c["added"], c["deleted"], c["noop_add"], c["noop_del"], c["superseded"]), tag
    for l in range(1, L + 1):
        assert st["active_edges"][l] == orc.active_edges(l), f"{tag}: active edges of hop {l}"
    do, di = rp.degrees()
    odo, odi = orc.degrees()
    assert np.array_equal(do.cpu().numpy(), odo) and np.array_equal(di.cpu().numpy(), odi), f"{tag}: degrees"
    return st


def check_csr(rp, orc):
    rowptr, col = rp.export_graph()
    orp, ocol = orc.export_csr()
    assert np.array_equal(rowptr, orp) and np.array_equal(col, ocol)


def all_rows_err(rp, orc, L):
    """max over all layers, rows and columns of |got - ref| / (1 + |ref|), ref = the oracle's cached state"""
    worst = 0.0
    for l in range(L + 1):
        got = rp.embeddings(l).cpu().numpy()
        ref = orc.H(l)
        for i in range(0, got.shape[0], 1 << 18):
            r = ref[i:i + (1 << 18)]
            worst = max(worst, float(np.max(np.abs(got[i:i + (1 << 18)] - r) / (1.0 + np.abs(r)))))
    return worst


def sample_rows(rng, w, orc, L, last_ups):
    odo, odi = orc.degrees()
    s = set(rng.integers(0, w.n, size=4000).tolist())
    s |= set(np.argsort(odi)[-100:].tolist()) | set(np.argsort(odo)[-100:].tolist())
    s |= set(orc.affected(1)[:10000].tolist())
    for l in range(1, L + 1):
        s |= set(orc.affected(l)[:300].tolist()) | set(orc.affected(l)[-300:].tolist())
    s |= set(np.nonzero(odi == 0)[0][:50].tolist())
    dels = last_ups[last_ups["op"] == I.OP_DEL_EDGE]["v"]
    if dels.size:     # sinks that lost at least as many in-edges as they keep
        v, cnt = np.unique(dels, return_counts=True)
        s |= set(v[cnt >= odi[v]].tolist())
    return np.array(sorted(s), dtype=np.int32), odi


def check_sampled_rows(rp, orc, w, L, last_ups, tag):
    H = [np.ascontiguousarray(rp.embeddings(l).cpu().numpy()) for l in range(L + 1)]
    ids, odi = sample_rows(np.random.default_rng(0), w, orc, L, last_ups)
    worst = 0.0
    for l in range(1, L + 1):
        _, ref = orc.rows_from_prev(l, ids, H[l - 1])
        err = np.max(np.abs(H[l][ids].astype(np.float64) - ref) / (1.0 + np.abs(ref)), axis=1)
        i = int(np.argmax(err))
        assert err[i] <= TOL, f"{tag}: layer {l}, vertex {ids[i]} (in-degree {odi[ids[i]]}): err {err[i]}"
        worst = max(worst, float(err[i]))
    print(f"{tag}: {ids.size} sampled rows x {L} layers against the definition, worst err {worst:.2e}")
    return H


def test_dense_2l_every_batch_size_of_the_configuration(env):
    ripple, Oracle = env
    w, (src, dst) = graph_of("dense-2l")
    X = I.features(w.n, w.model.dims[0], w.seed)
    W = I.make_weights(w.model, w.seed)
    L = len(w.model.layers)
    rp = ripple.Ripple(w.n, src, dst, X, w.model, W, max_batch=10000)
    orc = Oracle(w.n, src, dst, X, w.model, W)
    stream = I.make_stream(w, src, dst)
    feat_now = {}

    def note_features(ups, rows):
        for r in ups[ups["op"] == I.OP_SET_FEATURE]:
            feat_now[int(r["u"])] = rows[int(r["v"])]

    t0 = time.time()
    # the oracle's incremental route follows: all rows of all layers
    for bsz, n_batches in ((10, 100), (100, 100), (1000, 5)):
        for b in range(n_batches):
            ups, rows = stream.next_batch(bsz)
            rp.apply_batch(ups, rows)
            assert orc.apply_incremental(ups, rows, pull=True) == 0
            check_structure(rp, orc, L, f"B={bsz} batch {b}")
            note_features(ups, rows)
        check_csr(rp, orc)
        worst = all_rows_err(rp, orc, L)
        print(f"dense-2l B={bsz}: {n_batches} batches, all rows of all layers, worst err {worst:.2e} "
              f"({time.time() - t0:.0f} s)")
        assert worst <= TOL, (bsz, worst)
    # from here on the oracle follows the structure only; rows are checked against the definition
    for bsz, n_batches in ((1000, 15), (10000, 5)):
        for b in range(n_batches):
            ups, rows = stream.next_batch(bsz)
            rp.apply_batch(ups, rows)
            assert orc.apply_structure(ups, rows.shape[0]) == 0
            st = check_structure(rp, orc, L, f"B={bsz} batch {b} (structure)")
            if bsz == 1000:
                assert list(st["scatter_pull"][1:L + 1]) == [0, 0]       # both hops push their deltas
            note_features(ups, rows)
        check_csr(rp, orc)
        H = check_sampled_rows(rp, orc, w, L, ups, f"dense-2l B={bsz} after {n_batches} batches")
    X_now = X.copy()
    for v, row in feat_now.items():
        X_now[v] = row
    assert np.array_equal(H[0], X_now)      # H^0 is the features with the replaced rows, bit for bit
    rp.close()
    orc.close()


def test_full_size_gcx_batches_against_the_hybrid_oracle(env):
    """GraphConv-max on the dense graph, batches of 1000: the oracle's hybrid-incremental route is fast
    enough to follow at full size, so every row of every layer is compared within tolerance, and the
    affected lists exactly where they are unique."""
    ripple, Oracle = env
    w, (src, dst) = graph_of("dense-gcx-2l")
    X = I.features(w.n, w.model.dims[0], w.seed)
    W = I.make_weights(w.model, w.seed)
    L = len(w.model.layers)
    rp = ripple.Ripple(w.n, src, dst, X, w.model, W, max_batch=1000)
    orc = Oracle(w.n, src, dst, X, w.model, W)
    stream = I.make_stream(w, src, dst)
    for b in range(3):
        ups, rows = stream.next_batch(1000)
        rp.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        st = rp.stats()
        # Affected is value-based here (a cached maximum changed).  Layer 0 and 1 depend on the fp32
        # features only and must agree exactly; from layer 2 on the two sides see embeddings that
        # differ by rounding, and a pre-activation within rounding of zero is an exact 0 after ReLU
        # on one side and a tiny positive number on the other, so a handful of vertices (measured: one
        # in 288 K) may be called changed by one side only: both lists are valid.
        for l in range(L + 1):
            a, o = rp.affected(l).cpu().numpy(), orc.affected(l)
            if l <= 1:
                assert np.array_equal(a, o), f"batch {b}: A_{l} differs"
            else:
                odd = np.setxor1d(a, o)
                assert odd.size <= max(4, 1e-4 * o.size), f"batch {b}: A_{l} differs in {odd.size} of {o.size}"
                print(f"batch {b}: |A_{l}| = {o.size}, {odd.size} vertices on one side only")
        assert st["active_edges"][1] == orc.active_edges(1)
    worst = all_rows_err(rp, orc, L)
    assert worst <= TOL, worst
    for l in range(1, L + 1):
        got = rp.aggregate(l)[0].cpu().numpy().astype(np.float64)
        assert float(np.max(np.abs(got - orc.S(l)) / (1.0 + np.abs(orc.S(l))))) <= TOL
    print(f"dense-gcx-2l: all rows, worst err {worst:.2e}")
    rp.close()
    orc.close()


# workload, batches, the form of each hop in the last batch (0 = delta messages pushed, 1 = delta messages gathered per
# sink: wide messages from few senders, chosen from the batch before; 2 = aggregates rebuilt)
DEEP_CASES = [
    ("dense-3l", 3, [0, 1, 2]),
    ("dense-3l-hub-feature", 5, [0, 2, 2]),
    ("dense-3l-hub-delete", 5, [0, 2, 2]),
    ("dense-4l", 2, [0, 1, 2, 2]),
    ("dense-gat-2l", 3, [0, 0]),        # attention layers never take the rebuilding form: recomputation is per vertex
    ("dense-gat-3l", 2, [0, 0, 0]),
    ("reddit-2l", 2, [0, 2]),
    ("reddit-4l", 2, [0, 2, 2, 2]),
]


@pytest.mark.parametrize("wname,n_batches,forms", DEEP_CASES, ids=[c[0] for c in DEEP_CASES])
def test_full_size_batches_of_1000_structure_and_sampled_rows(env, wname, n_batches, forms):
    ripple, Oracle = env
    w, (src, dst) = graph_of(wname)
    X = I.features(w.n, w.model.dims[0], w.seed)
    W = I.make_weights(w.model, w.seed)
    L = len(w.model.layers)
    rp = ripple.Ripple(w.n, src, dst, X, w.model, W, max_batch=1000)
    orc = Oracle(w.n, src, dst, X, w.model, W, bootstrap=False)
    stream = I.make_stream(w, src, dst)
    feat_now = {}
    for b in range(n_batches):
        ups, rows = stream.next_batch(1000)
        rp.apply_batch(ups, rows)
        assert orc.apply_structure(ups, rows.shape[0]) == 0
        st = check_structure(rp, orc, L, f"{wname} batch {b}")
        for r in ups[ups["op"] == I.OP_SET_FEATURE]:
            feat_now[int(r["u"])] = rows[int(r["v"])]
    assert list(st["scatter_pull"][1:L + 1]) == forms, st["scatter_pull"]
    check_csr(rp, orc)
    H = check_sampled_rows(rp, orc, w, L, ups, f"{wname} after {n_batches} batches of 1000")
    X_now = X.copy()
    for v, row in feat_now.items():
        X_now[v] = row
    assert np.array_equal(H[0], X_now)
    rp.close()
    orc.close()


def test_full_size_two_workers_of_the_partitioned_execution(env):
    """dense-2l split over two workers (uniformly random owners: the worst cut) on the one GPU: hop sets
    exact against the oracle's structure route after every batch, sampled rows of the gathered embeddings
    against the definition."""
    ripple, Oracle = env
    from paper_2601_12347_b200.partitioned import Cluster
    wname = "dense-2l"
    w, (src, dst) = graph_of(wname)
    X = I.features(w.n, w.model.dims[0], w.seed)
    W = I.make_weights(w.model, w.seed)
    L = len(w.model.layers)
    owner = np.random.default_rng(w.seed).integers(0, 2, size=w.n).astype(np.int32)
    cl = Cluster(2, owner, src, dst, X, w.model, W, max_batch=1000)
    orc = Oracle(w.n, src, dst, X, w.model, W, bootstrap=False)
    stream = I.make_stream(w, src, dst)
    for b in range(3):
        ups, rows = stream.next_batch(1000)
        cl.apply_batch(ups, rows)
        assert orc.apply_structure(ups, rows.shape[0]) == 0
        for l in range(L + 1):
            assert np.array_equal(cl.affected(l), orc.affected(l)), f"batch {b}: A_{l} differs"
    sent = cl.rows_sent()
    assert sent[L] > 100_000, sent
    H = [np.ascontiguousarray(cl.embeddings(l, w.n)) for l in range(L + 1)]
    ids, odi = sample_rows(np.random.default_rng(0), w, orc, L, ups)
    worst = 0.0
    for l in range(1, L + 1):
        _, ref = orc.rows_from_prev(l, ids, H[l - 1])
        err = np.max(np.abs(H[l][ids].astype(np.float64) - ref) / (1.0 + np.abs(ref)), axis=1)
        i = int(np.argmax(err))
        assert err[i] <= TOL, f"layer {l}, vertex {ids[i]} (in-degree {odi[ids[i]]}): err {err[i]}"
        worst = max(worst, float(err[i]))
    print(f"dense-2l over 2 workers after 3 batches of 1000: {ids.size} sampled rows x {L} layers, worst err {worst:.2e}, "
          f"halo rows sent in the last batch {sent[1:]}")
    cl.close()
    orc.close()


def test_mid_size_every_row_of_every_layer_through_pushed_gathered_and_rebuilt_hops(env):
    """The 3-layer configuration on the graph of a million vertices, where the oracle's incremental route still
    follows batches of 1000: after every batch ALL rows of all layers against it (not a sample), hop sets and counters
    exact.  From the second batch on hop 1 pushes its messages, hop 2 gathers them per sink (wide messages from few
    senders) and hop 3 rebuilds; the last layer's products run on the update kernel for narrow outputs."""
    import test_gpu_parity as G
    ripple, Oracle = env
    w, (src, dst) = graph_of("mid-3l")
    X = I.features(w.n, w.model.dims[0], w.seed)
    W = I.make_weights(w.model, w.seed)
    L = len(w.model.layers)
    rp = ripple.Ripple(w.n, src, dst, X, w.model, W, max_batch=1000)
    orc = Oracle(w.n, src, dst, X, w.model, W)
    stream = I.make_stream(w, src, dst, 77)
    worst = 0.0
    for b, bsz in enumerate([1000, 1000, 300]):
        ups, rows = stream.next_batch(bsz)
        rp.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows, pull=True) == 0
        G.check_frontiers(rp, orc, L)
        worst = max(worst, G.check_values(rp, [orc.H(l) for l in range(L + 1)], L))
        if b >= 1:
            assert list(rp.stats()["scatter_pull"][1:L + 1]) == [0, 1, 2]
    G.check_graph(rp, orc)
    print(f"mid-3l, 3 batches, every row of {L + 1} layers: worst err {worst:.2e}")
    rp.close()
    orc.close()
