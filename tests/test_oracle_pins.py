"""Pins of the CPU oracle against things other than itself (no GPU needed).

Each test is chosen so that a plausible mistake in the oracle (a dropped term, a wrong sign or index,
a transposed operand, a wrong schedule rule) fails at least one of them.
"""
import os

import numpy as np
import pytest

from workloads import ir, data, params as wp
import helpers as H

GOLD = os.path.join(os.path.dirname(__file__), "golden")
FAMILIES = ["mlp", "rnn", "tree", "ggnn", "tree_lstm"]
BIG = 1 << 30


def make(oracle_mod, g, inst, p):
    o = oracle_mod.Oracle(g)
    o.load_instances(inst)
    o.set_params(p)
    return o


# ---------------------------------------------------------------------------------------------------
# gradients: message-driven backprop == autograd of an independently written recursion / dense form
# ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("family", FAMILIES)
def test_accumulators_equal_autograd_of_direct_formulation(oracle_mod, family):
    g, inst, p = H.tiny_case(family, n=4)
    o = make(oracle_mod, g, inst, p)
    st, loss = o.run_epoch(mak=1, muf=BIG, lr=0.1, flush=False)
    grads, losses = H.dataset_grad(g, p, inst)
    np.testing.assert_allclose(loss, losses, rtol=1e-12, atol=1e-13)
    for (node, which), gr in grads.items():
        np.testing.assert_allclose(o.get_accum(node, which), gr, rtol=1e-9, atol=1e-12,
                                   err_msg=f"{family} node {g.names[node]} which {which}")
    assert st.leftover_cache_entries == 0


def test_grouped_leaves_give_the_gradients_and_message_count_of_the_recursion(oracle_mod):
    """The tree IR with the leaf operations of a tree grouped into one matrix message (Sec. 6): the same losses and
    gradients as the direct recursion over the tree (which knows nothing of the IR), the caches empty at the end, and
    the node-message count that follows from the graph: Lookup, LeafCell and Ungroup take one forward message per tree
    instead of two per leaf (3 - 2L), backward the Ungroup takes L and the other two one each instead of 2L (2 - L):
    33L - 18 becomes 30L - 13."""
    g, inst, p = H.tiny_case("tree_grouped", n=5)
    o = make(oracle_mod, g, inst, p)
    st, loss = o.run_epoch(mak=2, muf=BIG, lr=0.1, flush=False)
    grads, losses = H.dataset_grad(g, p, inst)
    np.testing.assert_allclose(loss, losses, rtol=1e-12, atol=1e-13)
    for (node, which), gr in grads.items():
        np.testing.assert_allclose(o.get_accum(node, which), gr, rtol=1e-9, atol=1e-12, err_msg=g.names[node])
    L = (np.diff(inst.offsets) + 1) // 2
    assert st.node_messages == int((30 * L - 13).sum()) and st.leftover_cache_entries == 0
    # one flush of the whole set from the same start: the same step as with the ungrouped IR (a gradient is one payload row)
    g0, _, _ = H.tiny_case("tree", n=5)
    o0, o1 = make(oracle_mod, g0, inst, p), make(oracle_mod, g, inst, p)
    o0.run_epoch(mak=2, muf=BIG, lr=0.1)
    o1.run_epoch(mak=2, muf=BIG, lr=0.1)
    p0, p1 = o0.get_params(), o1.get_params()
    for k in p0:
        np.testing.assert_allclose(p1[k], p0[k], rtol=1e-12, atol=1e-14)
        assert o1.node_stats(k[0])["n_grads_applied"] == o0.node_stats(k[0])["n_grads_applied"]


@pytest.mark.parametrize("family", FAMILIES)
def test_accumulators_equal_finite_differences(oracle_mod, family):
    """Central differences of the independent loss; touches every parameter tensor."""
    g, inst, p = H.tiny_case(family, n=2, seed=3)
    o = make(oracle_mod, g, inst, p)
    o.run_epoch(mak=2, muf=BIG, lr=0.0, flush=False)
    import torch
    rng = np.random.default_rng(0)

    def total(pp):
        P = {k: torch.tensor(v, dtype=torch.float64) for k, v in pp.items()}
        return float(sum(H.LOSS_FNS[g.name](g, P, inst, i) for i in range(inst.n)))

    eps = 1e-6
    for key, v in p.items():
        acc = o.get_accum(*key)
        flat = v.ravel()
        for idx in rng.choice(flat.size, size=min(4, flat.size), replace=False):
            pp = {k: a.copy() for k, a in p.items()}
            pp[key].ravel()[idx] += eps
            up = total(pp)
            pp[key].ravel()[idx] -= 2 * eps
            dn = total(pp)
            fd = (up - dn) / (2 * eps)
            assert abs(acc.ravel()[idx] - fd) <= 1e-6 * max(1.0, abs(fd)), (family, key, idx)


# ---------------------------------------------------------------------------------------------------
# update rule + schedule: exact agreement with textbook (minibatch) SGD for the MLP when mak = 1
# ---------------------------------------------------------------------------------------------------
def _textbook_sgd(g, p, inst, lr, batch):
    """20-line SGD loop: mean gradient over consecutive batches, numpy fp64, manual backprop."""
    nodes = g.ppt_nodes()
    W = [p[(n, 0)].copy() for n in nodes]
    b = [p[(n, 1)].copy() for n in nodes]
    losses = []
    for s in range(0, inst.n, batch):
        gW = [np.zeros_like(w) for w in W]
        gb = [np.zeros_like(v) for v in b]
        idx = range(s, min(s + batch, inst.n))
        for i in idx:
            xs = [inst.dense[i].astype(np.float64)]
            for k in range(len(W)):
                z = W[k] @ xs[-1] + b[k]
                xs.append(np.maximum(z, 0) if k < len(W) - 1 else z)
            y = xs[-1]
            lse = np.log(np.exp(y - y.max()).sum()) + y.max()
            losses.append(lse - y[inst.labels_i[i]])
            d = np.exp(y - lse)
            d[inst.labels_i[i]] -= 1
            for k in reversed(range(len(W))):
                if k < len(W) - 1:
                    d = d * (xs[k + 1] > 0)
                gW[k] += np.outer(d, xs[k])
                gb[k] += d
                d = W[k].T @ d
        for k in range(len(W)):
            W[k] -= lr * gW[k] / len(idx)
            b[k] -= lr * gb[k] / len(idx)
    return W, b, np.array(losses)


@pytest.mark.parametrize("batch", [1, 4, 5])
def test_mlp_mak1_is_textbook_minibatch_sgd(oracle_mod, batch):
    g = ir.mlp((12, 9, 7, 4))
    inst = data.mlp_instances(n=13, dim=12, classes=4)
    p = wp.init_params(g)
    lr = float(np.float32(0.1))
    o = make(oracle_mod, g, inst, p)
    st, loss = o.run_epoch(mak=1, muf=batch, lr=lr)
    W, b, ref_loss = _textbook_sgd(g, p, inst, lr, batch)
    np.testing.assert_allclose(loss, ref_loss, rtol=1e-12)
    for k, n in enumerate(g.ppt_nodes()):
        np.testing.assert_allclose(o.get_params(n, 0), W[k], rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(o.get_params(n, 1), b[k], rtol=1e-12, atol=1e-14)
        assert o.node_stats(n)["n_updates"] == -(-inst.n // batch)      # includes the epoch-end flush
    assert st.max_staleness == 0


def test_flush_applies_mean_of_accumulated_gradients(oracle_mod):
    g, inst, p = H.tiny_case("tree", n=3)
    lr = float(np.float32(0.05))
    o = make(oracle_mod, g, inst, p)
    o.run_epoch(mak=1, muf=BIG, lr=lr, flush=True)
    grads, _ = H.dataset_grad(g, p, inst)
    L = (np.diff(inst.offsets) + 1) // 2
    n_grad = {"lookup": L.sum(), "leaf_cell": L.sum(), "branch_cell": (L - 1).sum(), "classifier": (2 * L - 1).sum()}
    for (node, which), gr in grads.items():
        want = p[(node, which)] - lr * gr / n_grad[g.names[node]]
        np.testing.assert_allclose(o.get_params(node, which), want, rtol=1e-10, atol=1e-13)


# ---------------------------------------------------------------------------------------------------
# schedule: hand traces, key bookkeeping, closed-form message counts
# ---------------------------------------------------------------------------------------------------
def test_trace_a_mlp_schedule(oracle_mod):
    rows = H.read_golden(os.path.join(GOLD, "trace_a_mlp.txt"))
    keylog = np.array(rows[:3], dtype=np.int64)
    rounds, msgs, ppt, upd, stale = (int(v) for v in rows[3])
    g = ir.mlp((8, 6, 6, 3))
    inst = data.mlp_instances(n=3, dim=8, classes=3)
    o = make(oracle_mod, g, inst, wp.init_params(g))
    st, _ = o.run_epoch(mak=2, muf=1, lr=0.1)
    got = np.stack([a.astype(np.int64) for a in o.key_log()], axis=1)
    np.testing.assert_array_equal(got, keylog)
    assert (st.rounds, st.node_messages, st.ppt_messages, st.max_staleness) == (rounds, msgs, ppt, stale)
    assert [o.node_stats(n)["n_updates"] for n in g.ppt_nodes()] == [upd] * 3


def test_trace_b_tree_schedule(oracle_mod):
    rows = H.read_golden(os.path.join(GOLD, "trace_b_tree.txt"))
    keylog = np.array(rows[:1], dtype=np.int64)
    rounds, msgs, fwd, bwd, cls_upd, cls_stale = (int(v) for v in rows[1])
    g = ir.tree(vocab=10, emb=4, hidden=3, classes=2)
    inst = data.tree_instances(n=1, min_leaves=2, max_leaves=2, vocab=10, classes=2)
    o = make(oracle_mod, g, inst, wp.init_params(g))
    st, _ = o.run_epoch(mak=1, muf=1, lr=0.1)
    got = np.stack([a.astype(np.int64) for a in o.key_log()], axis=1)
    np.testing.assert_array_equal(got, keylog)
    assert (st.rounds, st.node_messages) == (rounds, msgs)
    stats = [o.node_stats(i) for i in range(len(g.names))]
    assert sum(s["fwd_msgs"] for s in stats) == fwd and sum(s["bwd_msgs"] for s in stats) == bwd
    c = stats[g.index("classifier")]
    assert c["n_updates"] == cls_upd
    assert np.nonzero(c["staleness_hist"])[0].max() == cls_stale


def _counts(inst):
    N = np.diff(inst.offsets) if inst.offsets is not None else None
    return N


@pytest.mark.parametrize("mak,muf", [(1, 1), (3, 7), (16, 50)])
def test_closed_form_message_counts_and_bookkeeping(oracle_mod, mak, muf):
    cases = []
    g = ir.mlp((8, 6, 6, 3))
    inst = data.mlp_instances(n=11, dim=8, classes=3)
    cases.append((g, inst, 7 * inst.n, {n: inst.n for n in g.ppt_nodes()}))
    g = ir.rnn(emb=6, hidden=6)
    inst = data.list_instances(n=9, max_len=6)
    T = np.diff(inst.offsets)
    cases.append((g, inst, int((13 * T + 3).sum()),
                  {g.index("lookup"): T.sum(), g.index("linear1"): T.sum(), g.index("linear2"): inst.n}))
    g = ir.tree(vocab=30, emb=6, hidden=5, classes=3)
    inst = data.tree_instances(n=7, min_leaves=2, max_leaves=9, vocab=30, classes=3)
    L = (np.diff(inst.offsets) + 1) // 2
    cases.append((g, inst, int((33 * L - 18).sum()),
                  {g.index("lookup"): L.sum(), g.index("leaf_cell"): L.sum(), g.index("branch_cell"): (L - 1).sum(),
                   g.index("classifier"): (2 * L - 1).sum()}))
    g = ir.ggnn(hidden=4, readout=3)
    inst = data.graph_instances(n=6, min_nodes=3, max_nodes=7)
    N, D = np.diff(inst.offsets), np.diff(inst.edge_offsets)
    Dc = np.array([[np.sum(inst.edge_type[inst.edge_offsets[i]:inst.edge_offsets[i + 1]] == c) for c in range(4)]
                   for i in range(inst.n)])
    Cp = (Dc > 0).sum(1)
    grads = {g.index("lookup"): N.sum(), g.index("gru"): 4 * N.sum(), g.index("readout1"): inst.n,
             g.index("readout2"): inst.n}
    for c in range(4):
        grads[g.index(f"edge_linear{c}")] = 4 * Dc[:, c].sum()
    # per propagation step: forward 3N+2D+4Cp+8 and backward 3N+2D+4Cp+8 consumed messages; 9 outside the loop
    cases.append((g, inst, int((4 * (6 * N + 4 * D + 8 * Cp + 16) + 9).sum()), grads))
    for g, inst, want_msgs, want_grads in cases:
        o = make(oracle_mod, g, inst, wp.init_params(g))
        st, _ = o.run_epoch(mak=mak, muf=muf, lr=0.01)
        assert st.node_messages == want_msgs, g.name
        assert st.leftover_cache_entries == 0, g.name            # forward/backward state invariant
        assert 1 <= st.max_active_observed <= mak
        ins, slot, adm, rel = o.key_log()
        assert sorted(ins.tolist()) == list(range(inst.n))       # admitted and released exactly once
        assert (rel > adm).all() and slot.max() < mak
        # a slot is never handed out again before it was released
        for s in range(mak):
            m = slot == s
            a, r = adm[m], rel[m]
            assert (a[1:] >= r[:-1]).all()
        for node, G in want_grads.items():                       # every gradient applied exactly once
            ns = o.node_stats(node)
            log = o.update_log(node)
            assert ns["n_grads_applied"] == G == log.sum(), (g.name, g.names[node])
            if g.name != "ggnn":                                 # one row per message: exact update count
                assert ns["n_updates"] == -(-int(G) // muf)
                assert (log[:-1] == muf).all()
            else:
                assert (log[:-1] >= muf).all()


@pytest.mark.parametrize("mak,muf", [(1, 1), (4, 1), (4, 2), (8, 3), (5, 32)])
def test_mlp_staleness_bound(oracle_mod, mak, muf):
    g = ir.mlp((8, 6, 6, 3))
    inst = data.mlp_instances(n=40, dim=8, classes=3)
    o = make(oracle_mod, g, inst, wp.init_params(g))
    st, _ = o.run_epoch(mak=mak, muf=muf, lr=0.01)
    assert st.max_staleness <= -(-(mak - 1) // muf)
    if mak == 1:
        assert st.max_staleness == 0
    if (mak, muf) == (4, 1):
        assert st.max_staleness == 3                             # the bound is attained: mak - 1 updates


def test_shuffled_order_is_a_permutation_of_the_work(oracle_mod):
    g, inst, p = H.tiny_case("rnn", n=6)
    o = make(oracle_mod, g, inst, p)
    order = data.epoch_order(inst.n, 5)
    assert sorted(order.tolist()) == list(range(inst.n)) and (order != np.arange(inst.n)).any()
    st, loss = o.run_epoch(mak=1, muf=BIG, lr=0.1, order=order, flush=False)
    grads, losses = H.dataset_grad(g, p, inst)
    np.testing.assert_allclose(loss, losses, rtol=1e-12)
    ins = o.key_log()[0]
    np.testing.assert_array_equal(ins, order)


# ---------------------------------------------------------------------------------------------------
# special cases that reduce to something else
# ---------------------------------------------------------------------------------------------------
def test_left_chain_tree_equals_rnn_over_its_leaves(oracle_mod):
    """A caterpillar tree ((((l0 l1) l2) l3) ...) is an RNN whose state starts at leaf 0."""
    L = 5
    g = ir.tree(vocab=9, emb=4, hidden=4, classes=3)
    inst = data.Instances(ir.KIND_BINARY_TREES, 1)
    M = 2 * L - 1
    left, right, tok = [], [], []
    # post-order: l0, l1, b(0,1)=2, l3.. : nodes: leaf0=0, leaf1=1, inner=2, leaf=3, inner=4, ...
    left += [-1, -1, 0]; right += [-1, -1, 1]; tok += [1, 2, -1]
    for k in range(2, L):
        leaf_id = len(left)
        left += [-1, len(left) - 1]; right += [-1, leaf_id]; tok += [k + 1, -1]
    inst.offsets = np.array([0, M]); inst.left = np.array(left); inst.right = np.array(right)
    inst.tokens = np.array(tok); inst.labels_i = np.arange(M) % 3
    inst.finalize()
    p = wp.init_params(g, emb_std=0.5)
    o = make(oracle_mod, g, inst, p)
    _, loss = o.run_epoch(mak=1, muf=BIG, lr=0.0, flush=False)
    E, (Wl, bl), (Wb, bb), (Wc, bc) = p[(g.index("lookup"), 0)], [p[(g.index("leaf_cell"), w)] for w in (0, 1)], \
        [p[(g.index("branch_cell"), w)] for w in (0, 1)], [p[(g.index("classifier"), w)] for w in (0, 1)]

    def cls_loss(h, lab):
        y = Wc @ h + bc
        return np.log(np.exp(y).sum()) - y[lab]

    leaves = [np.tanh(Wl @ E[t] + bl) for t in range(1, L + 1)]
    total = cls_loss(leaves[0], 0) + cls_loss(leaves[1], 1)
    h = np.tanh(Wb @ np.concatenate([leaves[0], leaves[1]]) + bb)
    total += cls_loss(h, 2)
    nid = 3
    for k in range(2, L):
        total += cls_loss(leaves[k], nid % 3)
        h = np.tanh(Wb @ np.concatenate([h, leaves[k]]) + bb)
        total += cls_loss(h, (nid + 1) % 3)
        nid += 2
    np.testing.assert_allclose(loss[0], total, rtol=1e-12)


def test_ggnn_without_edges_of_a_type_and_eval_matches_training_forward(oracle_mod):
    g, inst, p = H.tiny_case("ggnn", n=5)
    assert len(np.unique(inst.edge_type)) < 4 or True
    o = make(oracle_mod, g, inst, p)
    _, train_loss = o.run_epoch(mak=3, muf=BIG, lr=0.0, flush=False)
    ml, acc, ev_loss = o.eval()
    np.testing.assert_allclose(ev_loss, train_loss, rtol=1e-12)
    assert abs(ml - train_loss.mean()) < 1e-12


@pytest.mark.parametrize("family", FAMILIES)
def test_eval_is_forward_only_and_matches_direct_loss(oracle_mod, family):
    g, inst, p = H.tiny_case(family, n=4, seed=2)
    o = make(oracle_mod, g, inst, p)
    before = o.get_params()
    ml, acc, loss = o.eval()
    _, losses = H.dataset_grad(g, p, inst)
    np.testing.assert_allclose(loss, losses, rtol=1e-12, atol=1e-13)
    after = o.get_params()
    for k in before:
        np.testing.assert_array_equal(before[k], after[k])
    assert 0.0 <= acc <= 1.0


def test_asynchrony_changes_the_trajectory_but_not_the_accounting(oracle_mod):
    """mak > 1 with small muf gives stale gradients (different parameters) yet the same gradient counts."""
    g = ir.mlp((8, 6, 6, 3))
    inst = data.mlp_instances(n=24, dim=8, classes=3)
    p = wp.init_params(g)
    a, b = make(oracle_mod, g, inst, p), make(oracle_mod, g, inst, p)
    a.run_epoch(mak=1, muf=1, lr=0.1)
    sb, _ = b.run_epoch(mak=4, muf=1, lr=0.1)
    n = g.ppt_nodes()[0]
    assert np.abs(a.get_params(n, 0) - b.get_params(n, 0)).max() > 1e-6
    assert a.node_stats(n)["n_grads_applied"] == b.node_stats(n)["n_grads_applied"] == inst.n
    assert sb.max_staleness > 0


def test_bf16_payload_rounding_only_touches_payloads(oracle_mod):
    g, inst, p = H.tiny_case("tree", n=2)
    o = oracle_mod.Oracle(g, payload_bf16=True)
    o.load_instances(inst)
    o.set_params(p)
    _, l16 = o.run_epoch(mak=1, muf=BIG, lr=0.0, flush=False)
    o2 = make(oracle_mod, g, inst, p)
    _, l64 = o2.run_epoch(mak=1, muf=BIG, lr=0.0, flush=False)
    rel = np.abs(l16 - l64) / l64
    assert (rel > 0).any() and rel.max() < 3e-2            # bf16 has 8 bits of mantissa
    for k in p:
        np.testing.assert_array_equal(o.get_params(*k), p[k])


# ---------------------------------------------------------------------------------------------------
# optimisers (App. A: momentum-SGD and Adam as run-time options): against torch.optim on the textbook loop
# ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("kind", ["momentum", "adam"])
def test_optimizers_match_torch_optim_on_minibatch_training(oracle_mod, kind):
    import torch
    g = ir.mlp((10, 8, 6, 4))
    inst = data.mlp_instances(n=24, dim=10, classes=4)
    p = wp.init_params(g)
    batch, lr = 4, float(np.float32(0.05 if kind == "momentum" else 0.01))
    o = make(oracle_mod, g, inst, p)
    o.set_optimizer(kind)
    for _ in range(2):                                    # two epochs: the optimiser state carries over
        o.run_epoch(mak=1, muf=batch, lr=lr)
    P = H.tparams(p)
    f32 = lambda v: float(np.float32(v))
    opt = torch.optim.SGD(P.values(), lr=lr, momentum=f32(0.9)) if kind == "momentum" else \
        torch.optim.Adam(P.values(), lr=lr, betas=(f32(0.9), f32(0.999)), eps=f32(1e-8))
    for _ in range(2):
        for s in range(0, inst.n, batch):
            opt.zero_grad()
            loss = sum(H.mlp_loss(g, P, inst, i) for i in range(s, s + batch)) / batch
            loss.backward()
            opt.step()
    for k, v in P.items():
        np.testing.assert_allclose(o.get_params(*k), v.detach().numpy(), rtol=1e-9, atol=1e-12)


# ---------------------------------------------------------------------------------------------------
# replicas of a heavy node between a round-robin Cond and a Phi, synchronised by averaging (Sec. 5)
# ---------------------------------------------------------------------------------------------------
def _replicated_case(k, n=6):
    g1 = ir.rnn(emb=6, hidden=6)
    gk = ir.rnn(emb=6, hidden=6, replicas=k)
    inst = data.list_instances(n=n, max_len=5)
    p1 = wp.init_params(g1)
    copies = [gk.index("linear1")] + [gk.index(f"linear1_r{r}") for r in range(1, k)]
    pk = {}
    for (node, which), v in p1.items():                  # the canonical nodes keep their indices in the replicated graph
        pk[(node, which)] = v
    for c in copies[1:]:
        pk[(c, 0)], pk[(c, 1)] = p1[(g1.index("linear1"), 0)], p1[(g1.index("linear1"), 1)]
    return g1, gk, inst, p1, pk, copies


@pytest.mark.parametrize("k", [2, 3])
def test_replicas_split_the_gradient_of_the_unreplicated_model(oracle_mod, k):
    """With identical copies the model computes the same function, so the copies' accumulated gradients add up to the
    gradient of the unreplicated model (autograd of the independent formulation), every copy serves exactly the
    (instance, position) pairs with (instance + position) mod k = its port, and the other nodes are unaffected."""
    g1, gk, inst, p1, pk, copies = _replicated_case(k)
    o = make(oracle_mod, gk, inst, pk)
    st, loss = o.run_epoch(mak=3, muf=BIG, lr=0.1, flush=False)
    grads, losses = H.dataset_grad(g1, p1, inst)
    np.testing.assert_allclose(loss, losses, rtol=1e-12, atol=1e-13)
    lin1 = g1.index("linear1")
    for which in (0, 1):
        total = sum(o.get_accum(c, which) for c in copies)
        np.testing.assert_allclose(total, grads[(lin1, which)], rtol=1e-9, atol=1e-12)
    for (node, which), gr in grads.items():
        if node != lin1:
            np.testing.assert_allclose(o.get_accum(node, which), gr, rtol=1e-9, atol=1e-12)
    T = np.diff(inst.offsets)
    for r, c in enumerate(copies):
        want = sum(1 for i in range(inst.n) for u in range(T[i]) if (i + u) % k == r)
        assert o.node_stats(c)["fwd_msgs"] == want == o.node_stats(c)["bwd_msgs"]
    assert st.node_messages == int((17 * T + 3).sum()) and st.leftover_cache_entries == 0


def test_replica_averaging_is_the_mean_and_keeps_other_nodes(oracle_mod):
    g1, gk, inst, p1, pk, copies = _replicated_case(2, n=8)
    o = make(oracle_mod, gk, inst, pk)
    o.run_epoch(mak=2, muf=3, lr=float(np.float32(0.05)))
    before = o.get_params()
    assert np.abs(before[(copies[0], 0)] - before[(copies[1], 0)]).max() > 0      # the copies have drifted apart
    o.average_params(copies)
    after = o.get_params()
    for which in (0, 1):
        mean = (before[(copies[0], which)] + before[(copies[1], which)]) / 2
        for c in copies:
            np.testing.assert_allclose(after[(c, which)], mean, rtol=0, atol=1e-15)
    for key in before:
        if key[0] not in copies:
            np.testing.assert_array_equal(after[key], before[key])


# ---------------------------------------------------------------------------------------------------
# concurrent inference: instances that are only evaluated share the queues with training instances
# ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("family", FAMILIES)
def test_inference_instances_ride_along_without_touching_training(oracle_mod, family):
    g, inst, p = H.tiny_case(family, n=7)
    mask = np.array([0, 1, 0, 0, 1, 1, 0], np.uint8)
    train = np.nonzero(mask == 0)[0]
    # (a) gradients: the masked instances contribute nothing, the others exactly what they contribute alone
    o = make(oracle_mod, g, inst, p)
    st, loss, inf = o.run_epoch_mixed(mak=3, muf=BIG, lr=0.1, inference_only=mask, flush=False)
    ref = make(oracle_mod, g, inst, p)
    rst, rloss = ref.run_epoch(mak=3, muf=BIG, lr=0.1, order=train, flush=False)
    for node in g.ppt_nodes():
        for which, _ in g.param_shapes(node):
            np.testing.assert_allclose(o.get_accum(node, which), ref.get_accum(node, which), rtol=1e-12, atol=1e-14)
        assert o.node_stats(node)["bwd_msgs"] == ref.node_stats(node)["bwd_msgs"]
    assert st.leftover_cache_entries == 0 and st.max_active_observed <= 3
    # (b) losses: with unchanged parameters every instance's loss is its forward-only loss
    e = make(oracle_mod, g, inst, p)
    e.load_instances(inst, split=1)
    ml, acc, eloss = e.eval(split=1)
    np.testing.assert_allclose(loss, eloss, rtol=1e-12, atol=1e-14)
    assert inf["instances"] == int(mask.sum())
    assert inf["mean_loss"] == pytest.approx(eloss[mask == 1].mean(), rel=1e-12)
    assert st.mean_loss == pytest.approx(eloss[mask == 0].mean(), rel=1e-12)
    # (c) everything masked: a pure evaluation, no update anywhere
    o2 = make(oracle_mod, g, inst, p)
    st2, loss2, inf2 = o2.run_epoch_mixed(mak=2, muf=1, lr=0.5, inference_only=np.ones(7, np.uint8))
    np.testing.assert_allclose(loss2, eloss, rtol=1e-12, atol=1e-14)
    assert inf2["accuracy"] == pytest.approx(acc)
    for k, v in o2.get_params().items():
        np.testing.assert_array_equal(v, p[k].astype(np.float64))


# ---------------------------------------------------------------------------------------------------
# Split (inverse of Concat): slices forward, joins the parts' gradients backward
# ---------------------------------------------------------------------------------------------------
def test_split_gradients_equal_autograd(oracle_mod):
    import torch
    g = ir.IRGraph("split_heads")
    src = g.node("src", ir.SOURCE, out_dim=6, fn=ir.SRC_DENSE_ROW)
    l1 = g.node("linear1", ir.LINEAR, 6, 8, act=ir.ACT_TANH, flags=ir.FLAG_SOURCE_ADJACENT)
    sp = g.node("split", ir.SPLIT, 8, 4, fn_arg=2)
    g.edge(src, l1)
    g.edge(l1, sp)
    heads = []
    for k in range(2):
        h = g.node(f"head{k}", ir.LINEAR, 4, 3)
        ls = g.node(f"loss{k}", ir.LOSS_CE, 3, 0, fn=ir.LABEL_PER_INSTANCE)
        g.edge(sp, h, k, 0)
        g.edge(h, ls)
        heads.append(h)
    inst = data.mlp_instances(n=5, dim=6, classes=3)
    p = wp.init_params(g)
    o = make(oracle_mod, g, inst, p)
    st, loss = o.run_epoch(mak=2, muf=BIG, lr=0.1, flush=False)
    P = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in p.items()}
    total = 0
    for i in range(inst.n):
        x = torch.tensor(inst.dense[i], dtype=torch.float64)
        hid = torch.tanh(P[(l1, 0)] @ x + P[(l1, 1)])
        li = 0
        for k, h in enumerate(heads):
            y = P[(h, 0)] @ hid[4 * k:4 * k + 4] + P[(h, 1)]
            li = li + torch.logsumexp(y, 0) - y[int(inst.labels_i[i])]
        assert float(li.detach()) == pytest.approx(loss[i], rel=1e-12)
        total = total + li
    total.backward()
    for k, v in P.items():
        np.testing.assert_allclose(o.get_accum(*k), v.grad.numpy(), rtol=1e-9, atol=1e-12)
    assert st.leftover_cache_entries == 0


# ---------------------------------------------------------------------------------------------------
# bf16 payload rounding, reported accuracy, sparse-row optimiser state of the embedding table
# ---------------------------------------------------------------------------------------------------
def test_bf16_rounding_is_round_to_nearest_even(oracle_mod):
    """The oracle's payload rounding against torch's float32 -> bfloat16 conversion: random values of every magnitude,
    exact ties with an even and with an odd kept mantissa (truncation, round-half-up and round-half-away all fail
    here), values just off a tie, subnormals, signed zeros, infinities and NaN."""
    import torch
    rng = np.random.default_rng(7)
    bits = rng.integers(0, 1 << 32, size=200000, dtype=np.uint64).astype(np.uint32)
    rand = bits.view(np.float32)
    rand = rand[np.isfinite(rand)]
    hi = rng.integers(0, 1 << 16, size=4096, dtype=np.uint32) << 16
    hi = hi[((hi >> 23) & 0xff) != 0xff]
    ties = (hi | 0x8000).view(np.float32)                        # exactly half way between two bfloat16 neighbours
    above, below = (hi | 0x8001).view(np.float32), (hi | 0x7fff).view(np.float32)
    special = np.array([0.0, -0.0, np.inf, -np.inf, 1e-40, -1e-40, 1.17549435e-38, 3.3895314e38, -3.3895314e38, 1.0,
                        1.00390625, 1.01171875], np.float32)     # the last two: ties at 1 + 2^-8 (down) and 1 + 3 2^-8 (up)
    x = np.concatenate([rand, ties, above, below, special])
    want = torch.from_numpy(x.copy()).to(torch.bfloat16).to(torch.float32).numpy()
    got = oracle_mod.round_bf16(x).astype(np.float32)
    np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))
    assert np.isnan(oracle_mod.round_bf16(np.array([np.nan], np.float32))[0])
    # the two textbook ties, by value: 1 + 2^-8 -> 1 (even below), 1 + 3 2^-8 -> 1 + 2^-6 (even above)
    np.testing.assert_array_equal(oracle_mod.round_bf16(np.array([1.00390625, 1.01171875])), [1.0, 1.015625])


@pytest.mark.parametrize("family", ["mlp", "rnn", "tree"])
def test_reported_accuracy_is_the_argmax_of_an_independent_forward_pass(oracle_mod, family):
    """eval()'s accuracy (and its count of predictions) against the arg-max of the direct recursive forward pass."""
    g, inst, p = H.tiny_case(family, n=40 if family != "tree" else 12, seed=4)
    o = make(oracle_mod, g, inst, p)
    _, acc, _ = o.eval()
    want = H.accuracy(g, p, inst)
    assert 0.0 < want < 1.0                      # the case decides something: neither all right nor all wrong
    assert acc == pytest.approx(want, abs=1e-12)
    # a different parameter set moves both numbers together
    p2 = {k: v * (-1.0 if len(v.shape) == 1 else 1.0) + 0.1 for k, v in p.items()}
    o.set_params(p2)
    assert o.eval()[1] == pytest.approx(H.accuracy(g, p2, inst), abs=1e-12)


def _sparse_rows_reference(kind, E, grads_and_rows, lr, beta=(0.9, 0.999), eps=1e-8, mu=0.9):
    """Momentum-SGD / Adam on an embedding table in which an update moves only the rows that received a gradient since
    the previous update, and only their moments (plain numpy, written from the textbook update rules)."""
    E = E.copy()
    m, v = np.zeros_like(E), np.zeros_like(E)
    f32 = lambda x: float(np.float32(x))
    b1, b2, eps, mu = f32(beta[0]), f32(beta[1]), f32(eps), f32(mu)
    for t, (g, rows) in enumerate(grads_and_rows, start=1):
        for r in rows:
            if kind == "momentum":
                m[r] = mu * m[r] + g[r]
                E[r] -= lr * m[r]
            else:
                m[r] = b1 * m[r] + (1 - b1) * g[r]
                v[r] = b2 * v[r] + (1 - b2) * g[r] * g[r]
                E[r] -= lr * (m[r] / (1 - b1 ** t)) / (np.sqrt(v[r] / (1 - b2 ** t)) + eps)
    return E


@pytest.mark.parametrize("kind", ["momentum", "adam"])
def test_embedding_rows_move_only_when_touched_under_momentum_and_adam(oracle_mod, kind):
    """Two updates of the list model's embedding table (one per epoch: the threshold is never reached, the flush at the
    end of the epoch applies the mean gradient).  (1) When every table row is touched before each update the result is
    torch.optim's dense optimiser.  (2) When the second epoch's lists leave rows untouched, those rows and their moments
    stay as they were (no decay), which differs from the dense optimiser and equals a few lines of numpy."""
    import torch
    g = ir.rnn(vocab=14, emb=5, hidden=5, classes=10)
    look = g.index("lookup")
    p = wp.init_params(g, seed=3, emb_std=0.5)
    lr = float(np.float32(0.05))
    full = data.list_instances(n=60, max_len=6)                  # touches all 14 rows (digits 0-9 and the four ops)
    toks = full.tokens
    assert len(np.unique(toks)) == 14

    def epoch_grad(params, inst):
        grads, _ = H.dataset_grad(g, params, inst)
        n_tok = len(inst.tokens)                                 # one gradient per token reaches the table
        return grads[(look, 0)] / n_tok

    # (1) dense coincidence: both epochs on the full set
    o = make(oracle_mod, g, full, p)
    o.set_optimizer(kind)
    E = torch.tensor(p[(look, 0)], dtype=torch.float64, requires_grad=True)
    f32 = lambda x: float(np.float32(x))
    opt = torch.optim.SGD([E], lr=lr, momentum=f32(0.9)) if kind == "momentum" else \
        torch.optim.Adam([E], lr=lr, betas=(f32(0.9), f32(0.999)), eps=f32(1e-8))
    for _ in range(2):
        cur = o.get_params()
        opt.zero_grad()
        E.grad = torch.tensor(epoch_grad(cur, full))
        o.run_epoch(mak=1, muf=BIG, lr=lr)
        opt.step()
        np.testing.assert_allclose(o.get_params(look, 0), E.detach().numpy(), rtol=1e-9, atol=1e-12)

    # (2) the second epoch touches only some rows
    keep = [i for i in range(full.n) if set(toks[full.offsets[i]:full.offsets[i + 1]]) <= {0, 1, 2, 3, 10, 11}]
    assert len(keep) >= 1
    part = full.subset(np.array(keep))
    rows2 = sorted(set(part.tokens.tolist()))
    assert 0 < len(rows2) < 14
    o = make(oracle_mod, g, full, p)
    o.set_optimizer(kind)
    g1 = epoch_grad(o.get_params(), full)
    o.run_epoch(mak=1, muf=BIG, lr=lr)
    o.load_instances(part)
    g2 = epoch_grad(o.get_params(), part)
    o.run_epoch(mak=1, muf=BIG, lr=lr)
    want = _sparse_rows_reference(kind, p[(look, 0)], [(g1, range(14)), (g2, rows2)], lr)
    got = o.get_params(look, 0)
    np.testing.assert_allclose(got, want, rtol=1e-9, atol=1e-12)
    untouched = [r for r in range(14) if r not in rows2]
    after_first = _sparse_rows_reference(kind, p[(look, 0)], [(g1, range(14))], lr)
    np.testing.assert_allclose(got[untouched], after_first[untouched], rtol=1e-12, atol=0)
    # ... and a dense optimiser would have moved them (momentum / first moment carry over): the two readings differ here
    dense = torch.tensor(p[(look, 0)], dtype=torch.float64, requires_grad=True)
    dopt = torch.optim.SGD([dense], lr=lr, momentum=f32(0.9)) if kind == "momentum" else \
        torch.optim.Adam([dense], lr=lr, betas=(f32(0.9), f32(0.999)), eps=f32(1e-8))
    for gg in (g1, g2):
        dopt.zero_grad(); dense.grad = torch.tensor(gg); dopt.step()
    assert np.abs(dense.detach().numpy()[untouched] - got[untouched]).max() > 1e-6


# bf16 messages: what any fp32 implementation differs by from the fp64 oracle.  A payload that lies within fp32 rounding
# of a bf16 boundary rounds the other way (one bf16 ulp, 2^-8 relative), and behind a ReLU threshold that switches a whole
# gradient row.  The oracle measures this on itself (fp32 build against fp64 build, both with bf16 payloads); the tolerances
# of the GPU's bf16 parity test are these gaps with head room, not free parameters.
BF16_TOL = dict(param_rtol=2e-2, loss_rtol=2e-2, loss_atol=2e-3, param_floor=1e-2)
BF16_CASES = [("tree", 30, 16, 20, 0.02), ("rnn", 60, 8, 10, 0.02), ("ggnn", 20, 16, 40, 0.003), ("mlp", 40, 4, 8, 0.01),
              ("tree_lstm", 24, 16, 20, 0.02)]


def _bf16_case(family, n):
    gen = {"mlp": (ir.mlp, data.mlp_instances), "rnn": (ir.rnn, data.list_instances), "tree": (ir.tree, data.tree_instances),
           "ggnn": (ir.ggnn, data.graph_instances), "tree_lstm": (ir.tree_lstm, data.tree_instances)}[family]
    return gen[0](), gen[1](n=n)


def test_bf16_tolerances_come_from_the_oracles_own_fp32_gap(oracle_mod):
    worst_p = worst_l = 0.0
    for family, n, mak, muf, lr in BF16_CASES:
        g, inst = _bf16_case(family, n)
        p = wp.init_params(g)
        res = {}
        for real in ("f64", "f32"):
            o = oracle_mod.Oracle(g, real=real, payload_bf16=True)
            o.load_instances(inst)
            o.set_params(p)
            _, loss = o.run_epoch(mak=mak, muf=muf, lr=lr)
            res[real] = (o.get_params(), loss)
        (pa, la), (pb, lb) = res["f64"], res["f32"]
        gp = max(np.abs(pa[k] - pb[k].astype(np.float64)).max() / max(np.abs(pa[k]).max(), BF16_TOL["param_floor"]) for k in pa)
        gl = (np.abs(la - lb) / (np.abs(la) + BF16_TOL["loss_atol"] / BF16_TOL["loss_rtol"])).max()
        print(f"bf16 gap fp32 vs fp64 oracle, {family}: parameters {gp:.2e}, losses {gl:.2e}")
        assert gp <= BF16_TOL["param_rtol"] and gl <= BF16_TOL["loss_rtol"], family
        worst_p, worst_l = max(worst_p, gp), max(worst_l, gl)
    # head room, not slack: the tolerances stay within an order of magnitude of the largest gap measured
    assert BF16_TOL["param_rtol"] <= 10 * worst_p and BF16_TOL["loss_rtol"] <= 10 * worst_l
