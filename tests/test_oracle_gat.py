"""Pins for the oracle's attention layers (Sec. 3.4.1, Eq. 3) and their hybrid-incremental route.

The oracle is checked against things other than itself:
  * Eq. 3 as dense masked-softmax algebra (scipy.special.softmax over an explicit n x n matrix),
  * closed forms: a = 0 gives the mean of the in-neighbours; one in-neighbour gives that row back;
    with a linear logit the sink half of a cancels; every output lies between the column-wise
    minimum and maximum of the in-neighbour rows; two in-neighbours give a logistic blend,
  * the invariant of the method: after every batch the hybrid-incremental result, the scoped
    recomputation and full recomputation agree at every layer, for every kind of update,
  * the hop sets against a structural brute force (computation-tree signatures with a self term),
  * the cached numerator / denominator against their definition.
"""
import numpy as np
import pytest
from scipy.special import softmax

from oracle.oracle import Oracle
from paper_2601_12347_b200 import inputs as I


def dense_gat(n, src, dst, X, model, weights):
    """h'_v = sum_u softmax_u(z_uv) h_u over in-neighbours, z_uv = lrelu(a_s.(W h_u) + a_d.(W h_v))."""
    mask = np.zeros((n, n), dtype=bool)     # mask[v, u]: u -> v is an edge
    mask[dst, src] = True
    H = [X.astype(np.float64)]
    for ly, w in zip(model.layers, weights):
        Wh = H[-1] @ w["Wa"].astype(np.float64)
        s = Wh @ w["ba"].astype(np.float64)
        t = Wh @ w["bb"].astype(np.float64)
        z = t[:, None] + s[None, :]
        z = np.where(z < 0, ly.eps * z, z)
        z = np.where(mask, z, -np.inf)
        has = mask.any(axis=1)
        alpha = np.zeros((n, n))
        alpha[has] = softmax(z[has], axis=1)
        Z = alpha @ H[-1]
        H.append(np.maximum(Z, 0.0) if ly.act == I.ACT_RELU else Z)
    return H


def rel_err(a, b):
    return float(np.max(np.abs(a - b) / (1.0 + np.abs(b)))) if a.size else 0.0


def _setup(n=40, m=140, d=6, L=3, d_att=4, slope=1.0, seed=5, act=I.ACT_IDENTITY):
    model = I.gat_model(d, L, d_att=d_att, slope=slope, act=act)
    src, dst = I.er_graph(n, m, seed)
    X = I.features(n, d, seed)
    W = I.make_weights(model, seed)
    return model, src, dst, X, W


@pytest.mark.parametrize("slope", [1.0, 0.2])
@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("act", [I.ACT_IDENTITY, I.ACT_RELU])
def test_full_matches_dense_masked_softmax(slope, seed, act):
    model, src, dst, X, W = _setup(slope=slope, seed=seed, act=act)
    o = Oracle(40, src, dst, X, model, W)
    ref = dense_gat(40, src, dst, X, model, W)
    full = o.full()
    for l in range(len(ref)):
        assert rel_err(full[l], ref[l]) < 1e-12, l
        assert rel_err(o.H(l), ref[l]) < 1e-12, l     # the bootstrap state


def test_zero_attention_vector_is_the_mean_of_in_neighbours():
    model, src, dst, X, W = _setup(L=1)
    W[0]["ba"][:] = 0
    W[0]["bb"][:] = 0
    o = Oracle(40, src, dst, X, model, W)
    for v in range(40):
        nb = src[dst == v]
        want = X[nb].astype(np.float64).mean(axis=0) if nb.size else np.zeros(6)
        assert np.allclose(o.H(1)[v], want, rtol=1e-13, atol=1e-13)


def test_single_in_neighbour_returns_its_row_and_none_returns_zeros():
    n, d = 5, 3
    src = np.array([0, 1, 2], dtype=np.int32)
    dst = np.array([1, 2, 2], dtype=np.int32)       # 1 <- 0;  2 <- {1, 2 is not its own neighbour}
    src[2], dst[2] = 3, 2                            # 2 <- {1, 3}
    model = I.gat_model(d, 1, d_att=2)
    W = I.make_weights(model, 3)
    X = I.features(n, d, 3)
    o = Oracle(n, src, dst, X, model, W)
    assert np.allclose(o.H(1)[1], X[0].astype(np.float64), rtol=0, atol=1e-15)
    assert np.all(o.H(1)[0] == 0) and np.all(o.H(1)[4] == 0)
    # two in-neighbours: a logistic blend of the two rows with the difference of the source logits
    Wa, a_s = W[0]["Wa"].astype(np.float64), W[0]["ba"].astype(np.float64)
    s = X.astype(np.float64) @ Wa @ a_s
    p = 1.0 / (1.0 + np.exp(s[3] - s[1]))            # weight of vertex 1
    want = p * X[1].astype(np.float64) + (1 - p) * X[3].astype(np.float64)
    assert np.allclose(o.H(1)[2], want, rtol=1e-13, atol=1e-14)


def test_direction_sink_attends_over_in_neighbours_not_out_neighbours():
    # 0 -> 2, 1 -> 2, 2 -> 3: vertex 2's output mixes rows 0 and 1 only; vertex 3's is row 2
    src = np.array([0, 1, 2], dtype=np.int32)
    dst = np.array([2, 2, 3], dtype=np.int32)
    model = I.gat_model(2, 1, d_att=2)
    W = I.make_weights(model, 9)
    X = np.array([[1, 0], [0, 1], [5, 5], [7, 7]], dtype=np.float32)
    o = Oracle(4, src, dst, X, model, W)
    h = o.H(1)
    assert abs(h[2].sum() - 1.0) < 1e-14 and np.all(h[2] > 0) and np.all(h[2] < 1)
    assert np.allclose(h[3], [5, 5])
    assert np.all(h[0] == 0) and np.all(h[1] == 0)


def test_linear_logit_makes_the_sink_half_irrelevant_and_leaky_one_does_not():
    model, src, dst, X, W = _setup(slope=1.0, L=2)
    a = Oracle(40, src, dst, X, model, W).full()
    W2 = [dict(w) for w in W]
    for w in W2:
        w["bb"] = (w["bb"] * -3.0 + 0.5).astype(np.float32)
    b = Oracle(40, src, dst, X, model, W2).full()
    assert rel_err(a[2], b[2]) < 1e-12
    model2 = I.gat_model(6, 2, d_att=4, slope=0.2)
    c = Oracle(40, src, dst, X, model2, W).full()
    d = Oracle(40, src, dst, X, model2, W2).full()
    assert rel_err(c[2], d[2]) > 1e-3


def test_output_lies_in_the_hull_of_the_in_neighbour_rows():
    model, src, dst, X, W = _setup(slope=0.2, L=1, n=60, m=300)
    o = Oracle(60, src, dst, X, model, W)
    X64 = X.astype(np.float64)
    for v in range(60):
        nb = src[dst == v]
        if nb.size:
            assert np.all(o.H(1)[v] <= X64[nb].max(axis=0) + 1e-12)
            assert np.all(o.H(1)[v] >= X64[nb].min(axis=0) - 1e-12)


def _cached_sums(o, l, n, src, dst, model, W):
    """Numerator and denominator of Eq. 3 from the oracle's own H^{l-1}, by the definition."""
    ly, w = model.layers[l - 1], W[l - 1]
    Hp = o.H(l - 1)
    Wh = Hp @ w["Wa"].astype(np.float64)
    s, t = Wh @ w["ba"].astype(np.float64), Wh @ w["bb"].astype(np.float64)
    num, den = np.zeros_like(Hp), np.zeros(n)
    for u, v in zip(src.tolist(), dst.tolist()):
        z = s[u] + t[v]
        e = np.exp(ly.eps * z if z < 0 else z)
        num[v] += e * Hp[u]
        den[v] += e
    return num, den


@pytest.mark.parametrize("slope", [1.0, 0.2])
@pytest.mark.parametrize("mix", [(0.4, 0.4, 0.2, 0.0), (0.3, 0.3, 0.2, 0.2), (0.0, 0.0, 1.0, 0.0),
                                 (0.5, 0.5, 0.0, 0.0)], ids=["mixed", "vdel", "feat", "edges"])
def test_hybrid_incremental_equals_full_and_scoped_every_batch(slope, mix):
    n = 60
    model, src, dst, X, W = _setup(n=n, m=240, slope=slope, seed=11)
    o = Oracle(n, src, dst, X, model, W)
    rc = Oracle(n, src, dst, X, model, W)
    stream = I.UpdateStream(n, src, dst, 6, 11, mix=mix)
    for b in range(12):
        ups, rows = stream.next_batch(1 + 3 * (b % 4))
        assert o.apply_incremental(ups, rows) == 0
        assert rc.apply_scoped(ups, rows) == 0
        full = o.full()
        for l in range(4):
            assert rel_err(o.H(l), full[l]) < 1e-10, (b, l)
            assert rel_err(rc.H(l), full[l]) < 1e-12, (b, l)
            assert np.array_equal(o.affected(l), rc.affected(l))
        rp, col = o.export_csr()
        s2 = np.repeat(np.arange(n, dtype=np.int32), np.diff(rp))
        for l in range(1, 4):
            num, den = _cached_sums(o, l, n, s2, col, model, W)
            assert rel_err(o.S(l), num) < 1e-10, (b, l)
            assert rel_err(o.Den(l), den) < 1e-10, (b, l)


def _signatures(n, edges, fver, L):
    ins = {v: [] for v in range(n)}
    for (u, v) in edges:
        ins[v].append(u)
    sig = [[("x", v, fver[v]) for v in range(n)]]
    for _ in range(L):
        prev = sig[-1]
        sig.append([hash((prev[v], frozenset((u, prev[u]) for u in ins[v]))) for v in range(n)])
    return sig


def test_hop_sets_match_structural_brute_force_with_self_term():
    n, L = 40, 3
    model, src, dst, X, W = _setup(n=n, m=100, L=L, seed=21)
    o = Oracle(n, src, dst, X, model, W)
    stream = I.UpdateStream(n, src, dst, 6, 21)
    edges = set(zip(src.tolist(), dst.tolist()))
    fver = [0] * n
    for b in range(10):
        ups, rows = stream.next_batch(1 + b % 4)
        old = _signatures(n, edges, fver, L)
        for r in ups:
            if r["op"] == I.OP_ADD_EDGE:
                edges.add((int(r["u"]), int(r["v"])))
            elif r["op"] == I.OP_DEL_EDGE:
                edges.discard((int(r["u"]), int(r["v"])))
            else:
                fver[int(r["u"])] += 1
        new = _signatures(n, edges, fver, L)
        assert o.apply_incremental(ups, rows) == 0
        for l in range(L + 1):
            want = np.array([v for v in range(n) if old[l][v] != new[l][v]], dtype=np.int32)
            assert np.array_equal(o.affected(l), want), (b, l)


def test_rows_outside_the_hop_sets_keep_their_bits():
    n = 50
    model, src, dst, X, W = _setup(n=n, m=120, slope=0.2, seed=4)
    o = Oracle(n, src, dst, X, model, W)
    stream = I.UpdateStream(n, src, dst, 6, 4)
    for b in range(6):
        before = [o.H(l).copy() for l in range(4)]
        ups, rows = stream.next_batch(2)
        assert o.apply_incremental(ups, rows) == 0
        for l in range(4):
            keep = np.setdiff1d(np.arange(n), o.affected(l))
            assert np.array_equal(o.H(l)[keep], before[l][keep])


def test_row_from_prev_matches_full_for_attention_layers():
    n = 40
    model, src, dst, X, W = _setup(n=n, slope=0.2)
    o = Oracle(n, src, dst, X, model, W)
    full = o.full()
    for l in (1, 2, 3):
        prev = full[l - 1].astype(np.float32)
        for v in (0, 7, 39):
            S, h = o.row_from_prev(l, v, prev)
            ref = dense_gat(n, src, dst, prev, I.gat_model(6, 1, d_att=4, slope=0.2), [W[l - 1]])[1][v]
            assert np.allclose(h, ref, rtol=1e-12, atol=1e-13)


def test_monotonic_aggregation_is_refused_for_attention_layers():
    model, src, dst, X, W = _setup()
    model.agg = I.AGG_MAX
    o = Oracle(40, src, dst, X, model, W, bootstrap=False)
    ups = np.zeros(1, dtype=I.UPDATE_DTYPE)
    ups[0] = (I.OP_ADD_EDGE, 0, 1)
    assert o.apply_incremental(ups, None) == -3


def test_worked_example_of_the_attention_section():
    """Sec. 3.4.1's example: D aggregates over A and C; when C's features change, the only parts of D's
    numerator and denominator that move are C's terms, by exp(z_new) h_new - exp(z_old) h_old and
    exp(z_new) - exp(z_old) (the paper writes the message as old minus new; the sink subtracts it)."""
    A, B, C, D = 0, 1, 2, 3
    src = np.array([A, C, B], dtype=np.int32)
    dst = np.array([D, D, A], dtype=np.int32)
    model = I.gat_model(3, 1, d_att=2, slope=1.0)
    W = I.make_weights(model, 5)
    X = I.features(4, 3, 5)
    o = Oracle(4, src, dst, X, model, W)
    num0, den0 = o.S(1)[D].copy(), float(o.Den(1)[D])
    new_row = I.features(1, 3, 6)
    ups = np.zeros(1, dtype=I.UPDATE_DTYPE)
    ups[0] = (I.OP_SET_FEATURE, C, 0)
    assert o.apply_incremental(ups, new_row) == 0
    Wa, a_s, a_d = (W[0][k].astype(np.float64) for k in ("Wa", "ba", "bb"))
    t_D = X[D].astype(np.float64) @ Wa @ a_d
    z_old = X[C].astype(np.float64) @ Wa @ a_s + t_D
    z_new = new_row[0].astype(np.float64) @ Wa @ a_s + t_D
    assert np.allclose(o.S(1)[D] - num0, np.exp(z_new) * new_row[0] - np.exp(z_old) * X[C], rtol=1e-12, atol=1e-13)
    assert np.isclose(o.Den(1)[D] - den0, np.exp(z_new) - np.exp(z_old), rtol=1e-12, atol=1e-13)
    assert o.affected(1).tolist() == [C, D]      # C was in the tree at hop 0, so it is at hop 1 (it recomputes); D by the message
    z_A = X[A].astype(np.float64) @ Wa @ a_s + t_D
    want = (np.exp(z_A) * X[A] + np.exp(z_new) * new_row[0]) / (np.exp(z_A) + np.exp(z_new))
    assert np.allclose(o.H(1)[D], want, rtol=1e-12, atol=1e-13)
