"""Parity of the CUDA path for the weighted sum with a stored weight per edge (the GC-W workload of
Sec. 6.1.1) against the oracle's route for it: graph AND weights bit-exact after every batch (the
weights travel with their entries through deletion, tail packing, row moves and appends), affected
sets and counters bit-exact, embeddings within 1e-4 (1 + |ref|)."""
import numpy as np
import pytest

from paper_2601_12347_b200 import inputs as I
from tolerances import GIN_ROW_SLACK, TOL

import test_gpu_parity as G

pytestmark = pytest.mark.gpu

env = G.env


def check_graph_and_weights(rp, orc):
    rowptr, col, w = rp.export_graph_weighted()
    orp, ocol = orc.export_csr()
    assert np.array_equal(rowptr, orp) and np.array_equal(col, ocol)
    assert np.array_equal(w, orc.export_weights()), "stored edge weights differ"
    do, di = rp.degrees()
    odo, odi = orc.degrees()
    assert np.array_equal(do.cpu().numpy(), odo) and np.array_equal(di.cpu().numpy(), odi)


def weighted_models():
    return {
        "gc_2l": I.graphconv_model([18, 36, 10], I.AGG_WSUM_EDGE),
        "gc_3l": I.graphconv_model([18, 36, 20, 10], I.AGG_WSUM_EDGE),
        "sage_2l": I.sage_model([18, 36, 10], I.AGG_WSUM_EDGE),
        "gc_47": I.graphconv_model([18, 64, 47], I.AGG_WSUM_EDGE),     # messages of 48 and 40 floats take the
        "gc_40": I.graphconv_model([18, 64, 40], I.AGG_WSUM_EDGE),     # lane-packed form of the push
    }


@pytest.mark.parametrize("name", list(weighted_models().keys()))
@pytest.mark.parametrize("mode", ["auto", "pull", "push-notransform", "regather", "auto-mixed"])
def test_small_weighted_graphs_every_scatter_form(env, name, mode):
    ripple, Oracle = env
    model = weighted_models()[name]
    L = len(model.layers)
    n, m = 700, 6000
    src, dst = I.er_graph(n, m, 3)
    have = set(zip(src.tolist(), dst.tolist()))
    extra = [(0, int(v)) for v in range(1, 400) if (0, int(v)) not in have]        # a long out-list
    extra += [(int(u), 9) for u in range(100, 500) if (int(u), 9) not in have]      # and a long in-list
    src = np.concatenate([src, np.array([a for a, _ in extra], dtype=np.int32)])
    dst = np.concatenate([dst, np.array([b for _, b in extra], dtype=np.int32)])
    w = I.edge_weights(src.size, 3)
    X = I.features(n, model.dims[0], 3)
    W = I.make_weights(model, 3, zero_bias=False)
    sm = {"auto": ripple.SCATTER_AUTO, "pull": ripple.SCATTER_PULL, "push-notransform": ripple.SCATTER_PUSH,
          "regather": ripple.SCATTER_REGATHER, "auto-mixed": ripple.SCATTER_AUTO}[mode]
    rp = ripple.Ripple(n, src, dst, X, model, W, scatter_mode=sm, pre_transform=mode != "push-notransform",
                       regather_threshold=0.05 if mode == "auto-mixed" else 0.0, slack=0.05, edge_weights=w)
    orc = Oracle(n, src, dst, X, model, W, edge_weights=w)
    check_graph_and_weights(rp, orc)
    G.check_values(rp, orc.full(), L, [None] + [orc.full_S(l) for l in range(1, L + 1)])
    stream = I.UpdateStream(n, src, dst, model.dims[0], 3, mix=(0.45, 0.35, 0.18, 0.02))
    for b, bs in enumerate([1, 1, 2, 7, 33, 100, 1, 250, 64, 5] * 2):
        ups, rows, ow = stream.next_batch_weighted(bs)
        rp.apply_batch(ups, rows, ow)
        assert orc.apply_incremental(ups, rows, op_weights=ow) == 0
        check_graph_and_weights(rp, orc)
        G.check_frontiers(rp, orc, L)
        if b % 5 == 4:
            G.check_values(rp, orc.full(), L, [None] + [orc.full_S(l) for l in range(1, L + 1)])
    rp.close()


def test_existing_edges_keep_their_weight_and_missing_weights_are_ones(env):
    ripple, Oracle = env
    model = weighted_models()["gc_2l"]
    n, src, dst, X, _, _ = G._small(seed=41)
    W = I.make_weights(model, 41, zero_bias=False)
    w = I.edge_weights(src.size, 41)
    rp = ripple.Ripple(n, src, dst, X, model, W, edge_weights=w)
    orc = Oracle(n, src, dst, X, model, W, edge_weights=w)
    eu, ev = int(src[0]), int(dst[0])
    missing = next((a, b) for a in range(n) for b in range(n) if a != b and (a, b) not in set(zip(src.tolist(), dst.tolist())))
    ups = G.ups_array([(I.OP_DEL_EDGE, eu, ev), (I.OP_ADD_EDGE, eu, ev), (I.OP_ADD_EDGE, missing[0], missing[1])])
    ow = np.array([5.0, 6.0, 0.5], dtype=np.float32)
    rp.apply_batch(ups, None, ow)
    assert orc.apply_incremental(ups, None, op_weights=ow) == 0
    check_graph_and_weights(rp, orc)
    G.check_frontiers(rp, orc, 2)
    assert rp.stats()["n_noop_add"] == 1 and rp.stats()["n_added"] == 1
    # a batch without weights: new edges get weight 1
    other = next((a, b) for a in range(n) for b in range(n) if a != b and a > 3 and (a, b) not in set(zip(src.tolist(), dst.tolist())))
    ups = G.ups_array([(I.OP_ADD_EDGE, other[0], other[1])])
    rp.apply_batch(ups)
    assert orc.apply_incremental(ups) == 0
    check_graph_and_weights(rp, orc)
    G.check_values(rp, orc.full(), 2)
    rp.close()


def test_device_resident_weighted_inputs(env):
    import torch
    ripple, Oracle = env
    model = weighted_models()["gc_2l"]
    n, m = 500, 4000
    src, dst = I.er_graph(n, m, 9)
    w = I.edge_weights(m, 9)
    X = I.features(n, model.dims[0], 9)
    W = I.make_weights(model, 9)
    rp = ripple.Ripple(n, torch.from_numpy(src).cuda(), torch.from_numpy(dst).cuda(), torch.from_numpy(X).cuda(),
                       model, W, edge_weights=torch.from_numpy(w).cuda())
    orc = Oracle(n, src, dst, X, model, W, edge_weights=w)
    stream = I.UpdateStream(n, src, dst, model.dims[0], 9)
    for _ in range(5):
        ups, rows, ow = stream.next_batch_weighted(50)
        dev_ups = torch.from_numpy(np.stack([ups["op"], ups["u"], ups["v"]], axis=1).astype(np.int32)).cuda()
        rp.apply_batch(dev_ups, torch.from_numpy(rows).cuda(), torch.from_numpy(ow).cuda())
        assert orc.apply_incremental(ups, rows, op_weights=ow) == 0
    check_graph_and_weights(rp, orc)
    G.check_frontiers(rp, orc, 2)
    G.check_values(rp, orc.full(), 2)
    rp.close()


@pytest.mark.parametrize("batch", [100, 1000])
def test_sparse_gcw_100_consecutive_batches(env, batch):
    ripple, Oracle = env
    wl = I.workloads()["sparse-gcw"]
    src, dst = I.make_graph(wl)
    w = I.edge_weights(src.size, wl.seed)
    X = I.features(wl.n, wl.model.dims[0], wl.seed)
    W = I.make_weights(wl.model, wl.seed)
    L = len(wl.model.layers)
    rp = ripple.Ripple(wl.n, src, dst, X, wl.model, W, edge_weights=w)
    orc = Oracle(wl.n, src, dst, X, wl.model, W, edge_weights=w)
    stream = I.make_stream(wl, src, dst)
    for b in range(100):
        ups, rows, ow = stream.next_batch_weighted(batch)
        rp.apply_batch(ups, rows, ow)
        assert orc.apply_incremental(ups, rows, pull=True, op_weights=ow) == 0
        G.check_frontiers(rp, orc, L)
        if b % 50 == 49:
            check_graph_and_weights(rp, orc)
            G.check_values(rp, [orc.H(l) for l in range(L + 1)], L, row_slack=GIN_ROW_SLACK)
    # an unnormalised sum on the skewed graph: rows of 1e4 at layer 2, so the bound carries the same multiple of
    # the fp32 floor as the GIN-sum stack (tests/tolerances.py, measured in tests/test_fp32_floor.py)
    G.check_values(rp, orc.full(), L, [None] + [orc.full_S(l) for l in range(1, L + 1)], row_slack=GIN_ROW_SLACK)
    rp.close()
