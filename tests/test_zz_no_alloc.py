"""The export entry point that allocates no device memory.

Some callers cannot let this library call cudaMalloc: the process may already have handed all
device memory to a framework's caching allocator, or it may be on a latency budget that rules out
the synchronisation an allocation can imply.  For them ripple_export_graph_static stages through
fixed device arrays inside the library instead of freshly allocated buffers.  It must return
exactly what ripple_export_graph returns, on every call (the fixed arrays are shared and keep the
previous call's contents), and must refuse graphs beyond its stated limits.

This file is named so that pytest collects it last: a run that stops at the first failure has
then already run every other test.
"""
import numpy as np
import pytest

from paper_2601_12347_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ripple():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2601_12347_b200 import build as B
    B.build_library()
    from paper_2601_12347_b200 import ripple as R
    torch.cuda.set_device(0)
    return R


def test_static_export_equals_allocating_export_on_consecutive_calls(ripple):
    model = I.sage_model([12, 16, 4], I.AGG_MEAN)
    n, m = 3000, 40000
    src, dst = I.er_graph(n, m, 13)
    X = I.features(n, 12, 13)
    W = I.make_weights(model, 13)
    rp = ripple.Ripple(n, src, dst, X, model, W)
    stream = I.UpdateStream(n, src, dst, 12, 13)
    # first call: a larger graph state; second call: a smaller one, so stale contents of the
    # shared arrays from the first call would show up if any were read back
    for round_, mix in enumerate([(0.9, 0.05, 0.05), (0.0, 1.0, 0.0)]):
        st = I.UpdateStream(n, src, dst, 12, 13 + round_, mix=mix) if round_ == 0 else stream
        if round_ == 1:
            st = I.UpdateStream(n, *[a.copy() for a in (want_src, want_dst)], 12, 99, mix=mix)
        for _ in range(3):
            ups, rows = st.next_batch(500)
            rp.apply_batch(ups, rows)
        want_rp, want_col = rp.export_graph()
        got_rp, got_col = rp.export_graph_static()
        assert np.array_equal(got_rp, want_rp)
        assert np.array_equal(got_col, want_col)
        # from the second call on nothing may be allocated on the device: not by the library, and not
        # behind its back by the CUDA runtime on its behalf (the first call may have paid one-time
        # costs of the context, such as loading the kernel)
        import torch
        free_before, _ = torch.cuda.mem_get_info()
        again_rp, again_col = rp.export_graph_static()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before, "the allocation-free export changed the amount of free device memory"
        assert np.array_equal(again_rp, want_rp) and np.array_equal(again_col, want_col)
        want_src = np.repeat(np.arange(n, dtype=np.int32), np.diff(want_rp)).astype(np.int32)
        want_dst = want_col.astype(np.int32)
    assert want_col.size < m   # the second state really is smaller than the first
    rp.close()


def test_static_export_rejects_graphs_beyond_its_limit(ripple):
    model = I.sage_model([4, 4], I.AGG_SUM)
    n = (1 << 18) + 1
    src = np.arange(0, 1000, dtype=np.int32)
    dst = np.arange(1, 1001, dtype=np.int32)
    X = np.zeros((n, 4), dtype=np.float32)
    W = I.make_weights(model, 0)
    rp = ripple.Ripple(n, src, dst, X, model, W)
    with pytest.raises(ripple.RippleError) as ei:
        rp.export_graph_static()
    assert ei.value.status == ripple.ERR_CAPACITY
    assert "262144" in str(ei.value) and "vertices" in str(ei.value)
    rowptr, col = rp.export_graph()     # the allocating entry point still serves it
    assert rowptr[-1] == 1000
    rp.close()


def test_static_export_rejects_too_many_edges_on_a_small_vertex_set(ripple):
    """The second limit: few enough vertices, but more edges than the fixed column array holds."""
    model = I.sage_model([4, 4], I.AGG_SUM)
    n = 4096
    u = np.repeat(np.arange(2048, dtype=np.int32), 1100)
    v = np.tile(np.arange(1100, dtype=np.int32), 2048)
    keep = u != v
    src, dst = u[keep], v[keep]
    assert n <= (1 << 18) and src.size > (1 << 21)
    X = np.zeros((n, 4), dtype=np.float32)
    W = I.make_weights(model, 0)
    rp = ripple.Ripple(n, src, dst, X, model, W)
    with pytest.raises(ripple.RippleError) as ei:
        rp.export_graph_static()
    assert ei.value.status == ripple.ERR_CAPACITY
    assert "2097152" in str(ei.value) and "edges" in str(ei.value)
    rowptr, col = rp.export_graph()
    assert rowptr[-1] == src.size
    rp.close()
