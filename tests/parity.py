"""Shared comparison of the CUDA engine with the CPU oracle on the same seeded inputs (deterministic schedule)."""
import numpy as np


def run_both(oracle_mod, graph, inst, params, mak, muf, lr, order=None, timeout_s=60.0, payload_bf16=False, optimizer=None, **engine_kw):
    import paper_1705_09786_b200 as amp
    o = oracle_mod.Oracle(graph, payload_bf16=payload_bf16)
    o.load_instances(inst)
    o.set_params(params)
    if optimizer:
        o.set_optimizer(**optimizer)
    ost, oloss = o.run_epoch(mak=mak, muf=muf, lr=lr, order=order)
    e = amp.Engine(graph, payload_bf16=payload_bf16)
    e.load_instances(inst)
    e.set_params(params)
    if optimizer:
        e.set_optimizer(**optimizer)
    est, eloss = e.run_epoch(mak=mak, muf=muf, lr=lr, deterministic=True, order=order, timeout_s=timeout_s, **engine_kw)
    return o, ost, oloss, e, est, eloss


def assert_parity(graph, o, ost, oloss, e, est, eloss, param_rtol=1e-4, loss_rtol=1e-5, loss_atol=2e-6, param_floor=1e-30):
    """Integer bookkeeping bit-exact; parameters within max relative error 1e-4 (relative to the largest
    magnitude of the tensor, with elementwise slack for entries near zero); per-instance losses within 1e-5."""
    # routing, key bookkeeping, update counts: exact
    assert est.node_messages == ost.node_messages
    assert est.ppt_messages == ost.ppt_messages
    assert est.route_hash == ost.route_hash, "routed (node, direction, state) multiset differs"
    assert est.rounds == ost.rounds
    assert est.max_active_observed == ost.max_active_observed
    assert est.max_staleness == ost.max_staleness
    for a, b in zip(e.key_log(), o.key_log()):
        np.testing.assert_array_equal(a, b)
    for i in range(len(graph.names)):
        es, os_ = e.node_stats(i), o.node_stats(i)
        assert (es["fwd_msgs"], es["bwd_msgs"]) == (os_["fwd_msgs"], os_["bwd_msgs"]), graph.names[i]
    for i in graph.ppt_nodes():
        es, os_ = e.node_stats(i), o.node_stats(i)
        assert es["n_updates"] == os_["n_updates"], graph.names[i]
        assert es["n_grads_applied"] == os_["n_grads_applied"], graph.names[i]
        np.testing.assert_array_equal(es["staleness_hist"], os_["staleness_hist"])
        np.testing.assert_array_equal(e.update_log(i), o.update_log(i))
    assert e.leftover_cache_entries() == 0
    # floating point
    np.testing.assert_allclose(eloss, oloss, rtol=loss_rtol, atol=loss_atol)
    worst = 0.0
    ep, op = e.get_params(), o.get_params()
    for k in op:
        scale = max(np.abs(op[k]).max(), param_floor)
        err = np.abs(ep[k].astype(np.float64) - op[k]).max() / scale
        worst = max(worst, err)
        assert err <= param_rtol, (graph.names[k[0]], k[1], err)
    return worst
