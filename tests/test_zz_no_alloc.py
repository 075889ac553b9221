"""The allocation-free epoch (ampnet_run_epoch_static) against the ordinary one, through the C ABI.

Some users of the library may not allocate device memory while they train (all free memory already handed to
another pool, or a loop that cannot afford cudaMalloc's device-wide synchronisation).  For them the library
offers the same training epoch with its queues and caches in a fixed array inside the library image.  This test
runs two epochs in a row through each entry point, from identical parameters, and expects the same losses and
parameters within the tolerances the parity tests use.  It is collected last on purpose.
"""
import numpy as np
import pytest

from workloads import ir, data, params as wp

pytestmark = pytest.mark.gpu


def test_static_scratch_epoch_matches_the_allocating_epoch_twice_in_a_row():
    import paper_1705_09786_b200 as amp
    g = ir.rnn()
    inst = data.list_instances(n=150)
    p = wp.init_params(g)
    a, b = amp.Engine(g), amp.Engine(g)
    for e in (a, b):
        e.load_instances(inst)
        e.set_params(p)
    order = np.random.default_rng(3).permutation(inst.n)
    for call in range(2):
        od = None if call == 0 else order          # the second call also carries an epoch order (part of the size check)
        sa, la = a.run_epoch(mak=16, muf=50, lr=0.05, deterministic=True, timeout_s=60, order=od)
        calls = (b.alloc_calls, b.free_calls, len(b._blocks))
        sb, lb = b.run_epoch(mak=16, muf=50, lr=0.05, deterministic=True, timeout_s=60, static_scratch=True, order=od)
        assert (b.alloc_calls, b.free_calls, len(b._blocks)) == calls, "the static epoch went to the allocator"
        assert (sb.node_messages, sb.ppt_messages, sb.rounds, sb.route_hash) == \
               (sa.node_messages, sa.ppt_messages, sa.rounds, sa.route_hash), call
        np.testing.assert_allclose(lb, la, rtol=1e-5, atol=2e-6)
        pa, pb = a.get_params(), b.get_params()
        for k in pa:
            scale = np.abs(pa[k]).max() + 1e-30
            assert np.abs(pb[k] - pa[k]).max() / scale <= 1e-4, (call, k)
        for n in g.ppt_nodes():
            np.testing.assert_array_equal(b.update_log(n), a.update_log(n))
    # the handle's own memory is untouched by the static call: an ordinary epoch still works afterwards
    sb, lb = b.run_epoch(mak=16, muf=50, lr=0.05, deterministic=True, timeout_s=60)
    sa, la = a.run_epoch(mak=16, muf=50, lr=0.05, deterministic=True, timeout_s=60)
    np.testing.assert_allclose(lb, la, rtol=1e-5, atol=2e-6)
    a.close()
    b.close()


def test_static_scratch_never_allocates_near_its_size_limit():
    """Runs whose scratch lands just under and just over the fixed array's size: the first must run without a single
    allocator call, the second must be refused before anything runs (never served from allocator memory)."""
    import paper_1705_09786_b200 as amp
    g = ir.rnn()
    inst = data.list_instances(n=40)
    fits, refused = 0, 0
    for mak in (256, 512, 768, 1024, 1280, 1536, 2048, 3072):      # scratch grows with the keys in flight
        e = amp.Engine(g)
        e.load_instances(inst)
        calls = (e.alloc_calls, e.free_calls, len(e._blocks))
        try:
            st, _ = e.run_epoch(mak=mak, muf=50, lr=0.05, timeout_s=60, static_scratch=True)
            assert st.instances == inst.n
            fits += 1
        except amp.AmpnetError as err:
            assert err.status == 1 and "bytes" in str(err)
            refused += 1
        assert (e.alloc_calls, e.free_calls, len(e._blocks)) == calls, mak
        e.close()
    assert fits >= 1 and refused >= 1


def test_static_scratch_refuses_runs_that_do_not_fit():
    import paper_1705_09786_b200 as amp
    g = ir.tree()                                   # 20,000 x 300 embedding accumulator alone is 24 MB
    e = amp.Engine(g)
    e.load_instances(data.tree_instances(n=30))
    with pytest.raises(amp.AmpnetError) as ei:
        e.run_epoch(mak=64, muf=100, lr=0.05, static_scratch=True)
    assert ei.value.status == 1 and "bytes" in str(ei.value)
    st, loss = e.run_epoch(mak=64, muf=100, lr=0.05, timeout_s=60)      # the ordinary entry point is unaffected
    assert st.instances == 30 and np.isfinite(loss).all()
    e.close()
