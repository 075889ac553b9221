"""Seeded synthetic instance generators for the four workload families.

Each generator returns an `Instances` object of flat, C-contiguous numpy arrays
(CSR-style), the format both implementations load.  The labels come from fixed
random "teacher" functions that are part of the data recipe only; they are not
the trained model and share no code with either implementation.

The data stand in for MNIST, the list-reduction set, the Stanford Sentiment
Treebank and QM9: they take those sets' shapes and sizes, none of their items.
"""
import numpy as np

from . import ir

MASTER_SEED = 20170509


def _rng(config_index, stream=0):
    return np.random.default_rng([MASTER_SEED, config_index, stream])


class Instances:
    """Flat arrays describing n instances of one kind.

    offsets      int64 [n+1]   tokens / tree nodes / graph nodes per instance
    tokens       int32 [total] token id / leaf token id (-1 at inner tree nodes) / graph node type
    left, right  int32 [total] trees: local child ids, -1 at leaves; children precede parents, root is last
    edge_offsets int64 [n+1], edge_src/dst/type int32 [E]: graphs, local node ids, directed edges
    dense        float32 [n, d]
    labels_i     int32 [n] or [total] (one label per tree node)
    labels_f     float32 [n]
    """

    def __init__(self, kind, n):
        self.kind = kind
        self.n = int(n)
        self.offsets = None
        self.tokens = None
        self.left = None
        self.right = None
        self.edge_offsets = None
        self.edge_src = None
        self.edge_dst = None
        self.edge_type = None
        self.dense = None
        self.labels_i = None
        self.labels_f = None

    def finalize(self):
        def c(a, dt):
            return None if a is None else np.ascontiguousarray(a, dtype=dt)
        self.offsets = c(self.offsets, np.int64)
        self.edge_offsets = c(self.edge_offsets, np.int64)
        for k in ("tokens", "left", "right", "edge_src", "edge_dst", "edge_type", "labels_i"):
            setattr(self, k, c(getattr(self, k), np.int32))
        self.dense = c(self.dense, np.float32)
        self.labels_f = c(self.labels_f, np.float32)
        return self

    def subset(self, idx):
        """Instances idx (in that order) as a new object."""
        idx = np.asarray(idx, dtype=np.int64)
        out = Instances(self.kind, len(idx))
        if self.dense is not None:
            out.dense = self.dense[idx]
        if self.labels_f is not None:
            out.labels_f = self.labels_f[idx]
        per_node_labels = self.labels_i is not None and self.offsets is not None and \
            len(self.labels_i) == int(self.offsets[-1]) and self.kind == ir.KIND_BINARY_TREES
        if self.labels_i is not None and not per_node_labels:
            out.labels_i = self.labels_i[idx]
        if self.offsets is not None:
            lens = (self.offsets[1:] - self.offsets[:-1])[idx]
            out.offsets = np.concatenate([[0], np.cumsum(lens)])
            sel = np.concatenate([np.arange(self.offsets[i], self.offsets[i + 1]) for i in idx]) \
                if len(idx) else np.zeros(0, np.int64)
            for k in ("tokens", "left", "right"):
                a = getattr(self, k)
                if a is not None:
                    setattr(out, k, a[sel])
            if per_node_labels:
                out.labels_i = self.labels_i[sel]
        if self.edge_offsets is not None:
            lens = (self.edge_offsets[1:] - self.edge_offsets[:-1])[idx]
            out.edge_offsets = np.concatenate([[0], np.cumsum(lens)])
            sel = np.concatenate([np.arange(self.edge_offsets[i], self.edge_offsets[i + 1]) for i in idx]) \
                if len(idx) else np.zeros(0, np.int64)
            for k in ("edge_src", "edge_dst", "edge_type"):
                setattr(out, k, getattr(self, k)[sel])
        return out.finalize()

    def head(self, n):
        return self.subset(np.arange(min(n, self.n)))


# ---------------------------------------------------------------------------
# C1: dense rows, 10-class labels from a linear teacher
# ---------------------------------------------------------------------------
def mlp_instances(n=2048, dim=784, classes=10, split=0):
    rng = _rng(1, split)
    teacher = _rng(1, 100).standard_normal((classes, dim))
    x = rng.random((n, dim), dtype=np.float64).astype(np.float32)
    # The teacher sees centred inputs: with x ~ U[0,1] uncentred, the teacher's row sums would decide
    # almost every label and the classes would collapse onto one or two.
    y = np.argmax((x.astype(np.float64) - 0.5) @ teacher.T, axis=1)
    out = Instances(ir.KIND_DENSE_ROWS, n)
    out.dense = x
    out.labels_i = y
    return out.finalize()


# ---------------------------------------------------------------------------
# C2: list reduction; tokens = [op, d_1 .. d_len]
# ---------------------------------------------------------------------------
def list_instances(n=20000, max_len=10, split=0):
    rng = _rng(2, split)
    lens = rng.integers(1, max_len + 1, size=n)
    ops = rng.integers(0, 4, size=n)
    offsets = np.concatenate([[0], np.cumsum(lens + 1)])
    tokens = np.empty(int(offsets[-1]), np.int32)
    labels = np.empty(n, np.int32)
    digits = rng.integers(0, 10, size=int(lens.sum()))
    p = 0
    for i in range(n):
        d = digits[p:p + lens[i]]
        p += lens[i]
        o = offsets[i]
        tokens[o] = 10 + ops[i]
        tokens[o + 1:o + 1 + lens[i]] = d
        if ops[i] == 0:
            labels[i] = int(d.sum()) % 10
        elif ops[i] == 1:
            labels[i] = int(d.max())
        elif ops[i] == 2:
            labels[i] = int(d.min())
        else:
            labels[i] = int(d[0])
    out = Instances(ir.KIND_SEQUENCES, n)
    out.offsets = offsets
    out.tokens = tokens
    out.labels_i = labels
    return out.finalize()


# ---------------------------------------------------------------------------
# C3 / C5: random binary trees, Zipf leaf tokens, per-node labels from a teacher tree net
# ---------------------------------------------------------------------------
def _zipf_tokens(rng, size, vocab, s=1.1):
    p = np.arange(1, vocab + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(p / p.sum())
    return np.minimum(np.searchsorted(cdf, rng.random(size)), vocab - 1).astype(np.int32)


def _random_tree(rng, n_leaves, left, right, base):
    """Post-order numbering of a tree built by recursive uniform splits; writes local child ids into
    left/right starting at index `base`; returns the number of nodes written (2*n_leaves - 1)."""
    # iterative to avoid deep recursion: stack of (n, phase)
    nxt = 0
    result = []      # stack of finished subtree root ids
    stack = [(n_leaves, 0, 0)]
    while stack:
        n, phase, k = stack.pop()
        if n == 1:
            left[base + nxt] = -1
            right[base + nxt] = -1
            result.append(nxt)
            nxt += 1
        elif phase == 0:
            k = int(rng.integers(1, n))
            stack.append((n, 1, k))
            stack.append((n - k, 0, 0))   # right subtree is built second ...
            stack.append((k, 0, 0))       # ... left first
        else:
            r = result.pop()
            l = result.pop()
            left[base + nxt] = l
            right[base + nxt] = r
            result.append(nxt)
            nxt += 1
    return nxt


def tree_instances(n=8544, min_leaves=2, max_leaves=50, vocab=20000, classes=5, split=0, config_index=3):
    rng = _rng(config_index, split)
    L = rng.integers(min_leaves, max_leaves + 1, size=n)
    M = 2 * L - 1
    offsets = np.concatenate([[0], np.cumsum(M)])
    total = int(offsets[-1])
    left = np.empty(total, np.int32)
    right = np.empty(total, np.int32)
    for i in range(n):
        m = _random_tree(rng, int(L[i]), left, right, int(offsets[i]))
        assert m == M[i]
    is_leaf = left < 0
    tokens = np.full(total, -1, np.int32)
    tokens[is_leaf] = _zipf_tokens(rng, int(is_leaf.sum()), vocab)
    labels = _tree_teacher_labels(offsets, left, right, tokens, vocab, classes, config_index)
    out = Instances(ir.KIND_BINARY_TREES, n)
    out.offsets, out.left, out.right, out.tokens, out.labels_i = offsets, left, right, tokens, labels
    return out.finalize()


def _tree_teacher_labels(offsets, left, right, tokens, vocab, classes, config_index, width=32):
    """Labels = argmax of a fixed random tanh tree net of width 32, evaluated level by level."""
    t = _rng(config_index, 100)
    emb = t.standard_normal((vocab, width))
    w_leaf = t.standard_normal((width, width)) / np.sqrt(width)
    w_branch = t.standard_normal((width, 2 * width)) / np.sqrt(2 * width) * 2.0
    w_cls = t.standard_normal((classes, width))
    total = len(left)
    base = np.repeat(offsets[:-1], np.diff(offsets))
    gl = np.where(left >= 0, left + base, -1)
    gr = np.where(right >= 0, right + base, -1)
    h = np.zeros((total, width))
    height = np.zeros(total, np.int64)
    # children precede parents, so one ordered pass gives the heights
    for i in np.nonzero(left >= 0)[0]:
        height[i] = 1 + max(height[gl[i]], height[gr[i]])
    leaves = np.nonzero(left < 0)[0]
    h[leaves] = np.tanh(emb[tokens[leaves]] @ w_leaf.T)
    for lev in range(1, int(height.max()) + 1 if total else 1):
        idx = np.nonzero(height == lev)[0]
        h[idx] = np.tanh(np.concatenate([h[gl[idx]], h[gr[idx]]], axis=1) @ w_branch.T)
    return np.argmax(h @ w_cls.T, axis=1).astype(np.int32)


# ---------------------------------------------------------------------------
# C4: molecule-like typed graphs, scalar target from a teacher graph net
# ---------------------------------------------------------------------------
def graph_instances(n=130000, min_nodes=9, max_nodes=29, n_node_types=15, steps=4, split=0):
    rng = _rng(4, split)
    N = rng.integers(min_nodes, max_nodes + 1, size=n)
    offsets = np.concatenate([[0], np.cumsum(N)])
    total = int(offsets[-1])
    # node types: Zipf-like over 15 symbols
    p = np.arange(1, n_node_types + 1, dtype=np.float64) ** (-1.5)
    tokens = np.minimum(np.searchsorted(np.cumsum(p / p.sum()), rng.random(total)), n_node_types - 1)
    n_bonds = np.maximum(N - 1, np.rint(1.05 * N).astype(np.int64))
    bond_p = np.cumsum([0.75, 0.12, 0.03, 0.10])
    e_off = np.concatenate([[0], np.cumsum(2 * n_bonds)])
    E = int(e_off[-1])
    src = np.empty(E, np.int32)
    dst = np.empty(E, np.int32)
    typ = np.empty(E, np.int32)
    u_parent = rng.random(total)
    for i in range(n):
        nn = int(N[i])
        bonds = set()
        pairs = []
        for v in range(1, nn):
            a = int(u_parent[offsets[i] + v] * v)
            pairs.append((a, v))
            bonds.add((a, v))
        tries = 0
        while len(pairs) < n_bonds[i] and tries < 64:
            tries += 1
            a, b = (int(x) for x in rng.integers(0, nn, size=2))
            if a == b:
                continue
            a, b = min(a, b), max(a, b)
            if (a, b) in bonds:
                continue
            bonds.add((a, b))
            pairs.append((a, b))
        assert len(pairs) == n_bonds[i]
        bt = np.searchsorted(bond_p, rng.random(len(pairs)))
        bt = np.minimum(bt, 3)
        o = int(e_off[i])
        pa = np.asarray(pairs, np.int32)
        src[o:o + 2 * len(pairs):2] = pa[:, 0]
        dst[o:o + 2 * len(pairs):2] = pa[:, 1]
        src[o + 1:o + 2 * len(pairs):2] = pa[:, 1]
        dst[o + 1:o + 2 * len(pairs):2] = pa[:, 0]
        typ[o:o + 2 * len(pairs):2] = bt
        typ[o + 1:o + 2 * len(pairs):2] = bt
    out = Instances(ir.KIND_TYPED_GRAPHS, n)
    out.offsets, out.tokens = offsets, tokens
    out.edge_offsets, out.edge_src, out.edge_dst, out.edge_type = e_off, src, dst, typ
    out.labels_f = _graph_teacher_targets(offsets, tokens, e_off, src, dst, typ, n_node_types, steps)
    return out.finalize()


def _graph_teacher_targets(offsets, tokens, e_off, src, dst, typ, n_node_types, steps, width=16):
    """Scalar target = fixed random gated graph net of width 16 (dataset-wide vectorised), standardised."""
    t = _rng(4, 100)
    emb = t.standard_normal((n_node_types, width))
    w_e = t.standard_normal((4, width, width)) / np.sqrt(width)
    w_z, w_r, w_c = (t.standard_normal((width, 2 * width)) / np.sqrt(2 * width) for _ in range(3))
    w_o = t.standard_normal(width) / np.sqrt(width)
    nbase = np.repeat(offsets[:-1], np.diff(offsets))
    ebase = np.repeat(offsets[:-1], np.diff(e_off))
    gs, gd = src + ebase, dst + ebase
    h = emb[tokens]
    sig = lambda v: 1.0 / (1.0 + np.exp(-v))
    for _ in range(steps):
        a = np.zeros_like(h)
        for c in range(4):
            m = typ == c
            np.add.at(a, gd[m], h[gs[m]] @ w_e[c].T)
        x = np.concatenate([a, h], axis=1)
        z, r = sig(x @ w_z.T), sig(x @ w_r.T)
        cnd = np.tanh(np.concatenate([a, r * h], axis=1) @ w_c.T)
        h = (1 - z) * h + z * cnd
    pooled = np.add.reduceat(h, offsets[:-1].astype(np.int64), axis=0) if len(h) else np.zeros((0, width))
    y = np.tanh(pooled / 8.0) @ w_o
    del nbase
    return ((y - y.mean()) / (y.std() + 1e-12)).astype(np.float32) if len(y) > 1 else y.astype(np.float32)


def epoch_order(n, shuffle_seed):
    """Instance order of one epoch: dataset order for seed 0, else a seeded permutation (host generated and
    handed to both implementations)."""
    if shuffle_seed == 0:
        return np.arange(n, dtype=np.int64)
    return np.random.default_rng([MASTER_SEED, 7, int(shuffle_seed)]).permutation(n).astype(np.int64)
