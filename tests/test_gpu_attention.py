"""Parity of the CUDA path for attention layers (Sec. 3.4.1, Eq. 3) against the oracle's
hybrid-incremental route: graph, hop sets and counters bit-exact after every batch; embeddings within
1e-4 (1 + |ref|) of the oracle's full recomputation; the cached numerator / denominator rows within
the same bound scaled by sqrt(in-degree) (they are fp32 sums of that many terms)."""
import numpy as np
import pytest

from paper_2601_12347_b200 import inputs as I
from tolerances import TOL

import test_gpu_parity as G

pytestmark = pytest.mark.gpu

env = G.env


def cached_rows(orc, L):
    """[numerator | denominator] per layer, as the library lays them out."""
    return [None] + [np.concatenate([orc.S(l), orc.Den(l)[:, None]], axis=1) for l in range(1, L + 1)]


def check_graph(rp, orc):
    rowptr, col = rp.export_graph()
    orp, ocol = orc.export_csr()
    assert np.array_equal(rowptr, orp) and np.array_equal(col, ocol)


def hub_graph(n, m, seed):
    src, dst = I.er_graph(n, m, seed)
    have = set(zip(src.tolist(), dst.tolist()))
    extra = [(0, int(v)) for v in range(1, 400) if (0, int(v)) not in have]        # a long out-list
    extra += [(int(u), 9) for u in range(100, 700) if (int(u), 9) not in have]      # and a long in-list (3 chunks)
    src = np.concatenate([src, np.array([a for a, _ in extra], dtype=np.int32)])
    dst = np.concatenate([dst, np.array([b for _, b in extra], dtype=np.int32)])
    return src, dst


MODELS = {
    "d18_2l": dict(d=18, n_layers=2, d_att=8, slope=1.0),
    "d18_3l_leaky": dict(d=18, n_layers=3, d_att=8, slope=0.2),
    "d64_2l_leaky": dict(d=64, n_layers=2, d_att=16, slope=0.2),
    "d130_2l": dict(d=130, n_layers=2, d_att=4, slope=0.2),       # the denominator shares the last 16-byte piece of the row
    "d300_2l_relu": dict(d=300, n_layers=2, d_att=8, slope=0.2, act=I.ACT_RELU),
}


@pytest.mark.parametrize("name", list(MODELS.keys()))
def test_small_graphs_every_batch(env, name):
    ripple, Oracle = env
    model = I.gat_model(**MODELS[name])
    L = len(model.layers)
    n = 900
    src, dst = hub_graph(n, 7000, 3)
    X = I.features(n, model.dims[0], 3)
    W = I.make_weights(model, 3)
    rp = ripple.Ripple(n, src, dst, X, model, W, slack=0.05)
    orc = Oracle(n, src, dst, X, model, W)
    G.check_values(rp, orc.full(), L, cached_rows(orc, L))
    stream = I.UpdateStream(n, src, dst, model.dims[0], 3, mix=(0.45, 0.35, 0.18, 0.02))
    for b, bs in enumerate([1, 1, 2, 7, 33, 100, 1, 250, 64, 5] * 2):
        ups, rows = stream.next_batch(bs)
        rp.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        check_graph(rp, orc)
        G.check_frontiers(rp, orc, L)
        if b % 3 == 2:
            G.check_values(rp, orc.full(), L, cached_rows(orc, L))
    G.check_values(rp, orc.full(), L, cached_rows(orc, L))
    rp.close()


def test_single_updates_of_each_kind(env):
    ripple, Oracle = env
    model = I.gat_model(20, 2, d_att=8, slope=0.2)
    n, src, dst, X, _, _ = G._small(seed=41)
    X = I.features(n, 20, 41)
    W = I.make_weights(model, 41)
    rp = ripple.Ripple(n, src, dst, X, model, W)
    orc = Oracle(n, src, dst, X, model, W)
    have = set(zip(src.tolist(), dst.tolist()))
    missing = next((a, b) for a in range(n) for b in range(n) if a != b and (a, b) not in have)
    row = I.features(1, 20, 77)
    cases = [
        (G.ups_array([(I.OP_ADD_EDGE, missing[0], missing[1])]), None),
        (G.ups_array([(I.OP_DEL_EDGE, int(src[5]), int(dst[5]))]), None),
        (G.ups_array([(I.OP_SET_FEATURE, int(src[7]), 0)]), row),
        (G.ups_array([(I.OP_DEL_VERTEX, int(dst[11]), 0)]), None),
        (G.ups_array([(I.OP_SET_FEATURE, int(src[9]), 0), (I.OP_DEL_EDGE, int(src[9]), int(dst[9])),
                      (I.OP_ADD_EDGE, int(dst[9]), int(src[9]))]), row),
        (np.zeros(0, dtype=I.UPDATE_DTYPE), None),
    ]
    for ups, rows in cases:
        rp.apply_batch(ups, rows)
        assert orc.apply_incremental(ups, rows) == 0
        check_graph(rp, orc)
        G.check_frontiers(rp, orc, 2)
        G.check_values(rp, orc.full(), 2, cached_rows(orc, 2))
    rp.close()


def test_rows_outside_the_hop_sets_keep_their_bits(env):
    ripple, Oracle = env
    model = I.gat_model(24, 3, d_att=8, slope=0.2)
    n = 3000
    src, dst = I.er_graph(n, 9000, 8)
    X = I.features(n, 24, 8)
    W = I.make_weights(model, 8)
    rp = ripple.Ripple(n, src, dst, X, model, W)
    stream = I.UpdateStream(n, src, dst, 24, 8)
    for _ in range(4):
        before = [rp.embeddings(l).clone() for l in range(4)]
        ups, rows = stream.next_batch(3)
        rp.apply_batch(ups, rows)
        for l in range(4):
            keep = np.setdiff1d(np.arange(n), rp.affected(l).cpu().numpy())
            assert bool((rp.embeddings(l)[keep] == before[l][keep]).all())
    rp.close()


def test_long_stream_stays_within_tolerance_and_budget_gathers_rows_anew(env):
    ripple, Oracle = env
    model = I.gat_model(32, 2, d_att=8, slope=0.2)
    n = 1500
    src, dst = hub_graph(n, 12000, 5)
    X = I.features(n, 32, 5)
    W = I.make_weights(model, 5)
    rebuilt = {}
    for budget in (0.0, 1.5):     # the default, and one so tight that rows come due within the stream
        rp = ripple.Ripple(n, src, dst, X, model, W, rebuild_budget=budget)
        orc = Oracle(n, src, dst, X, model, W)
        stream = I.UpdateStream(n, src, dst, 32, 5)
        total = 0
        for b in range(60):
            ups, rows = stream.next_batch(40)
            rp.apply_batch(ups, rows)
            assert orc.apply_incremental(ups, rows) == 0
            total += sum(rp.stats()["rows_rebuilt"])
            if b % 20 == 19:
                G.check_frontiers(rp, orc, 2)
                G.check_values(rp, orc.full(), 2, cached_rows(orc, 2))
        rebuilt[budget] = total
        rp.close()
    assert rebuilt[1.5] > 0 and rebuilt[1.5] > rebuilt[0.0]


def test_recompute_full_and_device_resident_inputs(env):
    import torch
    ripple, Oracle = env
    model = I.gat_model(16, 2, d_att=4, slope=1.0)
    n, m = 500, 4000
    src, dst = I.er_graph(n, m, 9)
    X = I.features(n, 16, 9)
    W = I.make_weights(model, 9)
    rp = ripple.Ripple(n, torch.from_numpy(src).cuda(), torch.from_numpy(dst).cuda(), torch.from_numpy(X).cuda(), model, W)
    orc = Oracle(n, src, dst, X, model, W)
    stream = I.UpdateStream(n, src, dst, 16, 9)
    for _ in range(6):     # the same size again and again: the launch chain is captured and replayed
        ups, rows = stream.next_batch(50)
        dev_ups = torch.from_numpy(np.stack([ups["op"], ups["u"], ups["v"]], axis=1).astype(np.int32)).cuda()
        rp.apply_batch(dev_ups, torch.from_numpy(rows).cuda())
        assert orc.apply_incremental(ups, rows) == 0
        G.check_frontiers(rp, orc, 2)
    G.check_values(rp, orc.full(), 2, cached_rows(orc, 2))
    rp.recompute_full()
    G.check_values(rp, orc.full(), 2, cached_rows(orc, 2))
    rp.close()


def test_bad_attention_layers_are_refused(env):
    ripple, Oracle = env
    n, src, dst, X, _, _ = G._small(seed=41)
    X = I.features(n, 12, 1)
    model = I.gat_model(12, 2, d_att=4)
    W = I.make_weights(model, 1)
    model.agg = I.AGG_MEAN
    with pytest.raises(Exception):
        ripple.Ripple(n, src, dst, X, model, W)
    model = I.gat_model(12, 2, d_att=4)
    model.layers[1].d_out = 8
    with pytest.raises(Exception):
        ripple.Ripple(n, src, dst, X, model, I.make_weights(I.gat_model(12, 2, d_att=4), 1))
