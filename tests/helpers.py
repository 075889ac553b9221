"""Independent restatements used to pin the oracle (plain numpy / PyTorch CPU autograd, fp64).

Nothing here is shared with the oracle or with the CUDA path: these are textbook formulations written
directly over the list / tree / graph structure (recursion, dense adjacency), not over messages.
"""
import numpy as np
import torch

from workloads import ir


def read_golden(path):
    rows = []
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def tparams(params):
    return {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in params.items()}


def act(a, v):
    return {ir.ACT_NONE: lambda x: x, ir.ACT_RELU: torch.relu, ir.ACT_TANH: torch.tanh,
            ir.ACT_SIGMOID: torch.sigmoid}[a](v)


def ce(logits, label):
    return torch.logsumexp(logits, 0) - logits[label]


def mlp_loss(g, P, inst, i):
    x = torch.tensor(inst.dense[i], dtype=torch.float64)
    for n in g.ppt_nodes():
        x = act(int(g.nodes[n][3]), P[(n, 0)] @ x + P[(n, 1)])
    return ce(x, int(inst.labels_i[i]))


def rnn_loss(g, P, inst, i):
    look, l1, l2 = g.index("lookup"), g.index("linear1"), g.index("linear2")
    toks = inst.tokens[inst.offsets[i]:inst.offsets[i + 1]]
    h = torch.zeros(P[(l1, 0)].shape[0], dtype=torch.float64)
    a = int(g.nodes[l1][3])
    for t in toks:
        h = act(a, P[(l1, 0)] @ torch.cat([P[(look, 0)][int(t)], h]) + P[(l1, 1)])
    return ce(P[(l2, 0)] @ h + P[(l2, 1)], int(inst.labels_i[i]))


def tree_loss(g, P, inst, i):
    look, leaf, br, cls = (g.index(k) for k in ("lookup", "leaf_cell", "branch_cell", "classifier"))
    o = int(inst.offsets[i])
    m = int(inst.offsets[i + 1]) - o
    total = 0.0

    def rec(u):
        nonlocal total
        if inst.left[o + u] < 0:
            h = torch.tanh(P[(leaf, 0)] @ P[(look, 0)][int(inst.tokens[o + u])] + P[(leaf, 1)])
        else:
            h = torch.tanh(P[(br, 0)] @ torch.cat([rec(int(inst.left[o + u])), rec(int(inst.right[o + u]))])
                           + P[(br, 1)])
        total = total + ce(P[(cls, 0)] @ h + P[(cls, 1)], int(inst.labels_i[o + u]))
        return h

    rec(m - 1)
    return total


def tree_lstm_loss(g, P, inst, i):
    """Binary Tree-LSTM (Tai et al., N = 2) with separate leaf and branch cells; classifier on h at every node."""
    look, leaf, br, cls = (g.index(k) for k in ("lookup", "leaf_gates", "branch_gates", "classifier"))
    o = int(inst.offsets[i])
    m = int(inst.offsets[i + 1]) - o
    total = 0.0

    def rec(u):
        nonlocal total
        if inst.left[o + u] < 0:
            pi, po, pu = torch.chunk(P[(leaf, 0)] @ P[(look, 0)][int(inst.tokens[o + u])] + P[(leaf, 1)], 3)
            c = torch.sigmoid(pi) * torch.tanh(pu)
        else:
            (hl, cl), (hr, cr) = rec(int(inst.left[o + u])), rec(int(inst.right[o + u]))
            pi, pfl, pfr, po, pu = torch.chunk(P[(br, 0)] @ torch.cat([hl, hr]) + P[(br, 1)], 5)
            c = torch.sigmoid(pi) * torch.tanh(pu) + torch.sigmoid(pfl) * cl + torch.sigmoid(pfr) * cr
        h = torch.sigmoid(po) * torch.tanh(c)
        total = total + ce(P[(cls, 0)] @ h + P[(cls, 1)], int(inst.labels_i[o + u]))
        return h, c

    rec(m - 1)
    return total


def ggnn_loss(g, P, inst, i, steps=4):
    """Dense-adjacency formulation: a = sum_c A_c H W_c^T with A_c[dst, src] = #edges of type c."""
    look, gru, r1, r2 = (g.index(k) for k in ("lookup", "gru", "readout1", "readout2"))
    lins = [g.index(f"edge_linear{c}") for c in range(4)]
    o, o1 = int(inst.offsets[i]), int(inst.offsets[i + 1])
    eo, eo1 = int(inst.edge_offsets[i]), int(inst.edge_offsets[i + 1])
    n = o1 - o
    A = torch.zeros(4, n, n, dtype=torch.float64)
    for e in range(eo, eo1):
        A[int(inst.edge_type[e]), int(inst.edge_dst[e]), int(inst.edge_src[e])] += 1
    H = P[(look, 0)][torch.tensor(inst.tokens[o:o1].astype(np.int64))]
    for _ in range(steps):
        a = torch.zeros_like(H)
        for c in range(4):
            if A[c].sum() > 0:      # an absent edge type sends no message (and so adds no bias either)
                present = (A[c].sum(1, keepdim=True))
                a = a + A[c] @ (H @ P[(lins[c], 0)].T) + present * P[(lins[c], 1)]
        x = torch.cat([a, H], 1)
        z = torch.sigmoid(x @ P[(gru, 0)].T + P[(gru, 3)])
        r = torch.sigmoid(x @ P[(gru, 1)].T + P[(gru, 4)])
        c_ = torch.tanh(torch.cat([a, r * H], 1) @ P[(gru, 2)].T + P[(gru, 5)])
        H = (1 - z) * H + z * c_
    pooled = H.sum(0)
    y = P[(r2, 0)] @ torch.relu(P[(r1, 0)] @ pooled + P[(r1, 1)]) + P[(r2, 1)]
    return (y[0] - float(inst.labels_f[i])) ** 2


LOSS_FNS = {"mlp": mlp_loss, "rnn": rnn_loss, "tree": tree_loss, "tree_grouped": tree_loss, "ggnn": ggnn_loss, "tree_lstm": tree_lstm_loss}


def dataset_grad(g, params, inst):
    """Gradient of the summed loss over the whole dataset, and the per-instance losses."""
    P = tparams(params)
    losses = [LOSS_FNS[g.name](g, P, inst, i) for i in range(inst.n)]
    tot = sum(losses)
    tot.backward()
    grads = {k: (v.grad.numpy() if v.grad is not None else np.zeros(v.shape)) for k, v in P.items()}
    return grads, np.array([float(l.detach()) for l in losses])


def tiny_case(family, n=3, seed=0):
    """(graph, instances, params) small enough for finite differences."""
    from workloads import data, params as wp
    if family == "mlp":
        g = ir.mlp((7, 5, 4, 3))
        inst = data.mlp_instances(n=n, dim=7, classes=3)
    elif family == "rnn":
        g = ir.rnn(vocab=14, emb=5, hidden=5, classes=10)
        inst = data.list_instances(n=n, max_len=4)
    elif family == "tree":
        g = ir.tree(vocab=12, emb=5, hidden=4, classes=3)
        inst = data.tree_instances(n=n, min_leaves=2, max_leaves=5, vocab=12, classes=3)
    elif family == "tree_grouped":
        g = ir.tree(vocab=12, emb=5, hidden=4, classes=3, grouped_leaves=True)
        inst = data.tree_instances(n=n, min_leaves=2, max_leaves=5, vocab=12, classes=3)
    elif family == "tree_lstm":
        g = ir.tree_lstm(vocab=12, emb=5, hidden=4, classes=3)
        inst = data.tree_instances(n=n, min_leaves=2, max_leaves=5, vocab=12, classes=3)
    else:
        g = ir.ggnn(n_node_types=15, hidden=4, steps=4, readout=3)
        inst = data.graph_instances(n=n, min_nodes=3, max_nodes=6)
    p = wp.init_params(g, seed=seed + 1, emb_std=0.5)
    # non-zero biases so that a dropped bias term cannot hide
    rng = np.random.default_rng(seed + 5)
    for k in p:
        if p[k].ndim == 1:
            p[k] = rng.uniform(-0.3, 0.3, size=p[k].shape)
    return g, inst, p


# ---- predictions of the independent forward passes (for the accuracy the oracle reports) -----------------------
def _logit_rows(g, P, inst, i):
    """Every (logits, label) pair the model's classification loss sees for instance i, by direct recursion."""
    name = g.name
    if name == "mlp":
        x = torch.tensor(inst.dense[i], dtype=torch.float64)
        for n in g.ppt_nodes():
            x = act(int(g.nodes[n][3]), P[(n, 0)] @ x + P[(n, 1)])
        return [(x, int(inst.labels_i[i]))]
    if name == "rnn":
        look, l1, l2 = g.index("lookup"), g.index("linear1"), g.index("linear2")
        h = torch.zeros(P[(l1, 0)].shape[0], dtype=torch.float64)
        for t in inst.tokens[inst.offsets[i]:inst.offsets[i + 1]]:
            h = act(int(g.nodes[l1][3]), P[(l1, 0)] @ torch.cat([P[(look, 0)][int(t)], h]) + P[(l1, 1)])
        return [(P[(l2, 0)] @ h + P[(l2, 1)], int(inst.labels_i[i]))]
    assert name in ("tree", "tree_grouped")
    look, leaf, br, cls = (g.index(k) for k in ("lookup", "leaf_cell", "branch_cell", "classifier"))
    o = int(inst.offsets[i])
    rows = []

    def rec(u):
        if inst.left[o + u] < 0:
            h = torch.tanh(P[(leaf, 0)] @ P[(look, 0)][int(inst.tokens[o + u])] + P[(leaf, 1)])
        else:
            h = torch.tanh(P[(br, 0)] @ torch.cat([rec(int(inst.left[o + u])), rec(int(inst.right[o + u]))]) + P[(br, 1)])
        rows.append((P[(cls, 0)] @ h + P[(cls, 1)], int(inst.labels_i[o + u])))
        return h

    rec(int(inst.offsets[i + 1]) - o - 1)
    return rows


def accuracy(g, params, inst):
    """Fraction of classification decisions (arg-max, lowest index on ties) that hit the label, over the dataset."""
    P = {k: torch.tensor(v, dtype=torch.float64) for k, v in params.items()}
    hit = n = 0
    for i in range(inst.n):
        for logits, label in _logit_rows(g, P, inst, i):
            hit += int(int(torch.argmax(logits)) == label)
            n += 1
    return hit / n
