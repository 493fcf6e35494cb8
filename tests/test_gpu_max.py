"""Monotonic (max, min) aggregation on the GPU against the oracle: Sec. 3.4.2, hybrid-incremental
propagation with pruning.  Graph state, affected sets (= vertices whose cached maximum changed) and
counters are compared exactly; embeddings and cached maxima within 1e-4 (1 + |ref|)."""
import os
import sys

import numpy as np
import pytest

sys.path.insert(0, os.path.dirname(__file__))
import test_gpu_parity as G  # noqa: E402
from test_gpu_parity import env  # noqa: E402,F401
from test_oracle_vertex_ops import random_batch  # noqa: E402

from paper_2601_12347_b200 import inputs as I  # noqa: E402

pytestmark = pytest.mark.gpu


def run(env, n, src, dst, model, seed, batches, **kw):
    ripple, Oracle = env
    L = len(model.layers)
    d0 = model.dims[0]
    X = I.features(n, d0, seed)
    W = I.make_weights(model, seed, zero_bias=False)
    rp = ripple.Ripple(n, src, dst, X, model, W, **kw)
    orc = Oracle(n, src, dst, X, model, W)
    G.check_values(rp, orc.full(), L, [None] + [orc.full_S(l) for l in range(1, L + 1)])   # bootstrap
    pruned = 0
    for b, (ups, rows) in enumerate(batches(orc)):
        rp.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        G.check_graph(rp, orc)
        G.check_frontiers(rp, orc, L)
        st = rp.stats()
        assert all(st["senders"][l] <= st["affected"][l] for l in range(L))
        # messages that changed no cached maximum: sinks reached but not affected
        pruned += sum(max(0, min(st["active_edges"][l], n) - st["affected"][l]) for l in range(1, L + 1))
        G.check_values(rp, [orc.H(l) for l in range(L + 1)], L, [None] + [orc.S(l) for l in range(1, L + 1)])
    G.check_values(rp, orc.full(), L, [None] + [orc.full_S(l) for l in range(1, L + 1)])
    rp.close()
    return pruned


@pytest.mark.parametrize("agg", [I.AGG_MAX, I.AGG_MIN], ids=["max", "min"])
@pytest.mark.parametrize("dims", [[18, 36, 10], [18, 36, 20, 10], [7, 5], [40, 16, 24]])
@pytest.mark.parametrize("graphs", [True, False], ids=["replayed", "direct"])
def test_small_models_with_every_update_type(env, dims, graphs, agg):
    model = I.graphconv_model(dims, agg)
    n, m = 600, 5000
    src, dst = I.er_graph(n, m, 7)
    stream = I.UpdateStream(n, src, dst, dims[0], 7)
    rng = np.random.default_rng(7)

    def batches(orc):
        for b, bs in enumerate([1, 3, 40, 1, 200, 3, 1, 3, 120, 1, 3]):   # repeated sizes: captured at the second, replayed from the third
            if b % 3 == 2:   # colliding operations, vertex deletions included
                rowptr, col = orc.export_csr()
                edges = {(u, int(col[j])) for u in range(n) for j in range(rowptr[u], rowptr[u + 1])}
                yield G.ups_array(random_batch(rng, n, edges, bs, 6, p_vertex=0.05)), I.features(6, dims[0], 300 + b)
            else:
                yield stream.next_batch(bs)

    run(env, n, src, dst, model, 7, batches, graphs=graphs)


@pytest.mark.parametrize("agg", [I.AGG_MAX, I.AGG_MIN], ids=["max", "min"])
def test_pruning_wide_layers_and_long_in_lists(env, agg):
    """256-column layers (tensor-core update with old rows kept for the messages), two sinks whose
    in-lists are recomputed by a whole block, and a hub whose out-list reaches half the graph."""
    model = I.graphconv_model([24, 256, 256, 12], agg)
    n = 9000
    src, dst = I.er_graph(n, 45000, 3)
    have = set(zip(src.tolist(), dst.tolist()))
    extra = [(u, 7) for u in range(100, 6100) if (u, 7) not in have]
    extra += [(u, 9) for u in range(0, 4600) if (u, 9) not in have and u != 9]
    extra += [(7, v) for v in range(200, 4700) if (7, v) not in have]
    src = np.concatenate([src, np.array([a for a, _ in extra], dtype=np.int32)])
    dst = np.concatenate([dst, np.array([b for _, b in extra], dtype=np.int32)])
    stream = I.UpdateStream(n, src, dst, 24, 3)

    def batches(orc):
        for b, bs in enumerate([1, 50, 1000, 10, 400, 2000]):
            ups, rows = stream.next_batch(bs)
            if b == 3:
                if rows.shape[0] == 0:
                    rows = I.features(1, 24, 5)
                ups = np.concatenate([ups, G.ups_array([(I.OP_SET_FEATURE, 7, 0), (I.OP_DEL_VERTEX, 9, 0)])])
            yield ups, rows

    pruned = run(env, n, src, dst, model, 3, batches, max_batch=8192)
    assert pruned > 0     # some messages changed no cached maximum and were not propagated


def test_gin_layers_are_refused(env):
    ripple, _ = env
    model = I.gin_model(8, 8, 2)
    model.agg = I.AGG_MAX
    src, dst = I.er_graph(50, 200, 1)
    with pytest.raises(ripple.RippleError) as ei:
        ripple.Ripple(50, src, dst, I.features(50, 8, 1), model, I.make_weights(model, 1))
    assert ei.value.status == ripple.ERR_INVALID_ARG


@pytest.mark.parametrize("agg", [I.AGG_MAX, I.AGG_MIN], ids=["max", "min"])
@pytest.mark.parametrize("dims", [[18, 36, 10], [18, 36, 20, 10], [24, 256, 12]])
def test_self_term_with_a_monotonic_aggregator(env, dims, agg):
    """SAGE layers with max / min pooling: affected = cached row changed, or own input row changed."""
    model = I.sage_model(dims, agg)
    n, m = 2500, 20000
    src, dst = I.er_graph(n, m, 11)
    stream = I.UpdateStream(n, src, dst, dims[0], 11)
    rng = np.random.default_rng(11)

    def batches(orc):
        for b, bs in enumerate([1, 3, 40, 7, 400, 1, 64, 1500, 120]):
            if b % 3 == 2:
                rowptr, col = orc.export_csr()
                edges = {(u, int(col[j])) for u in range(n) for j in range(rowptr[u], rowptr[u + 1])}
                yield G.ups_array(random_batch(rng, n, edges, bs, 6, p_vertex=0.05)), I.features(6, dims[0], 300 + b)
            else:
                yield stream.next_batch(bs)

    run(env, n, src, dst, model, 11, batches, max_batch=4096)


@pytest.mark.parametrize("batch", [100, 1000])
def test_sparse_gcx_100_consecutive_batches(env, batch):
    """The GC-X workload on the sparse graph: 100 consecutive batches, affected lists and counters
    exact after every batch, embeddings and cached maxima within tolerance every 25 batches."""
    ripple, Oracle = env
    w = I.workloads()["sparse-gcx"]
    src, dst = I.make_graph(w)
    X = I.features(w.n, w.model.dims[0], w.seed)
    W = I.make_weights(w.model, w.seed)
    L = len(w.model.layers)
    rp = ripple.Ripple(w.n, src, dst, X, w.model, W)
    orc = Oracle(w.n, src, dst, X, w.model, W)
    stream = I.make_stream(w, src, dst)
    for b in range(100):
        ups, rows = stream.next_batch(batch)
        rp.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        G.check_frontiers(rp, orc, L)
        if b % 25 == 24:
            G.check_graph(rp, orc)
            G.check_values(rp, [orc.H(l) for l in range(L + 1)], L, [None] + [orc.S(l) for l in range(1, L + 1)])
    G.check_values(rp, orc.full(), L, [None] + [orc.full_S(l) for l in range(1, L + 1)])
    rp.close()
