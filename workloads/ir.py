"""IR description format (integer codes) and the canonical IR graphs, as data.

An IR graph (paper Sec. 4) is a table of nodes and a table of edges.

nodes : int32 [n_nodes, 8]  columns = (type, in_dim, out_dim, act, fn, fn_arg,
                                       muf_override, flags)
edges : int32 [n_edges, 4]  columns = (src_node, src_port, dst_node, dst_port)

`src_port` is the index of the successor slot of the source node (Bcast and
Cond have several), `dst_port` the index of the predecessor slot of the
destination node (Phi and edge-wise Concat have several).

The message state is the integer tuple (inst, seq, slot, it, u, port): instance
index, admission sequence number, key slot, outer-iteration counter, position
(time step / tree-node id / graph-node id / edge id / edge type) and port.
State functions of Cond / Isu / Group / Ungroup / Flatmap are an enumerated
set (`fn`) evaluated against the instance's structure tables.
"""
import numpy as np

# ---- node types -----------------------------------------------------------
SOURCE, LINEAR, LOOKUP, GRUCELL, LOSS_CE, LOSS_MSE, NPT_SUMROWS, COND, PHI, ISU, \
    CONCAT, SPLIT, BCAST, GROUP, UNGROUP, FLATMAP, SINK, NPT_LSTM = range(18)
TYPE_NAMES = ["SOURCE", "LINEAR", "LOOKUP", "GRUCELL", "LOSS_CE", "LOSS_MSE", "NPT_SUMROWS",
              "COND", "PHI", "ISU", "CONCAT", "SPLIT", "BCAST", "GROUP", "UNGROUP", "FLATMAP", "SINK", "NPT_LSTM"]
PPT_TYPES = (LINEAR, LOOKUP, GRUCELL)

# NPT_LSTM.fn: which LSTM gate combination the parameter-free node applies to the gate pre-activations on port 0
LSTM_LEAF = 1          # [pi, po, pu] (3H): c = s(pi) tanh(pu), h = s(po) tanh(c); output [h; c]
LSTM_BRANCH = 2        # [pi, pfL, pfR, po, pu] (5H) and the children's cells [cL; cR] on port 1:
                       # c = s(pi) tanh(pu) + s(pfL) cL + s(pfR) cR, h = s(po) tanh(c)

# ---- activations fused into a PPT node -------------------------------------
ACT_NONE, ACT_RELU, ACT_TANH, ACT_SIGMOID = range(4)

# ---- state functions --------------------------------------------------------
# SOURCE.fn: what the controller pumps for one admitted instance
SRC_DENSE_ROW = 1      # one message, payload = the instance's dense feature row
SRC_TOKENS = 2         # one message per token position u = 0..T-1 (payload = token id)
SRC_ZERO_STATE = 3     # one message, zero payload of width out_dim (initial hidden state)
SRC_TREE_LEAVES = 4    # one message per leaf u of the tree (payload = leaf token id)
SRC_GRAPH_NODES = 5    # one message with N rows (payload = node type ids)
SRC_TREE_LEAVES_GROUPED = 6   # one message with L rows: the tokens of the tree's leaves in leaf order (Sec. 6: grouped leaf operations)
# COND.fn: successor index as a function of the state
COND_SEQ_END = 1       # u < T ? 0 : 1          (T = number of tokens of the instance)
COND_TREE_ROOT = 2     # u is the root ? 0 : 1
COND_BY_U = 3          # successor = u
COND_IT_LT = 4         # it < fn_arg ? 0 : 1
COND_ROUND_ROBIN = 5   # successor = (instance + u) mod number of successors   (replicas, Sec. 5)
# ISU.fn: invertible state update
ISU_U_INC = 1          # u -> u + 1
ISU_TREE_PARENT = 2    # (u, port) -> (parent(u), child slot of u); inverse picks the child
ISU_IT_INC = 3         # it -> it + 1
# CONCAT.fn: where the input port comes from; fn_arg = number of ports, in_dim = width per port
CONCAT_BY_EDGE = 1
CONCAT_BY_STATE_PORT = 2
# GROUP.fn: (group key, member index, expected count) from the incoming state
GROUP_EDGES_BY_TYPE = 1   # u = edge id -> key = type(e), member = rank of e within its type
GROUP_EDGES_BY_DST = 2    # u = edge id -> key = dst(e),  member = rank of e among in-edges of dst
GROUP_ALL_NODES = 3       # u = node id -> key = 0,       member = u, count = N
# UNGROUP.fn: state of row i of an incoming matrix message
UNGROUP_NODES = 1         # row i -> u = i
UNGROUP_TYPE_EDGES = 2    # u = type c, row i -> u = id of the i-th edge of type c
UNGROUP_LEAVES = 3        # row i -> u = position of the tree's i-th leaf
# FLATMAP.fn
FLATMAP_OUT_EDGES = 1     # u = node v -> one message per out-edge e of v, u = e
# LOSS.fn: where the label comes from
LABEL_PER_INSTANCE = 1
LABEL_PER_TREE_NODE = 2

# ---- node flags ---------------------------------------------------------------
FLAG_SOURCE_ADJACENT = 1   # PPT directly fed by a SOURCE: no input gradient, retire instead

# ---- instance kinds -------------------------------------------------------------
KIND_DENSE_ROWS, KIND_SEQUENCES, KIND_BINARY_TREES, KIND_TYPED_GRAPHS = range(4)

# ---- parameter selectors ("which") ---------------------------------------------
# LINEAR: 0 = W [out,in], 1 = b [out];  LOOKUP: 0 = E [V,d]
# GRUCELL (x = [a; h], in_dim = 2H): 0 = Wz, 1 = Wr, 2 = Wc (each [H, 2H]), 3 = bz, 4 = br, 5 = bc
N_EDGE_TYPES = 4


class IRGraph:
    def __init__(self, name):
        self.name = name
        self._nodes = []
        self._edges = []
        self.names = []

    def node(self, name, type_, in_dim=0, out_dim=0, act=ACT_NONE, fn=0, fn_arg=0, muf=0, flags=0):
        self._nodes.append((type_, in_dim, out_dim, act, fn, fn_arg, muf, flags))
        self.names.append(name)
        return len(self._nodes) - 1

    def edge(self, src, dst, src_port=0, dst_port=0):
        self._edges.append((src, src_port, dst, dst_port))

    @property
    def nodes(self):
        return np.asarray(self._nodes, dtype=np.int32).reshape(-1, 8)

    @property
    def edges(self):
        return np.asarray(self._edges, dtype=np.int32).reshape(-1, 4)

    def index(self, name):
        return self.names.index(name)

    def ppt_nodes(self):
        return [i for i, n in enumerate(self._nodes) if n[0] in PPT_TYPES]

    def param_shapes(self, i):
        """[(which, shape)] of node i's parameters."""
        t, din, dout = self._nodes[i][:3]
        if t == LINEAR:
            return [(0, (dout, din)), (1, (dout,))]
        if t == LOOKUP:
            return [(0, (din, dout))]
        if t == GRUCELL:
            return [(0, (dout, din)), (1, (dout, din)), (2, (dout, din)), (3, (dout,)), (4, (dout,)), (5, (dout,))]
        return []


def mlp(dims=(784, 256, 256, 10)):
    """Source -> Linear(ReLU) ... -> Linear -> softmax-CE.  7 node-messages per instance for 3 layers."""
    g = IRGraph("mlp")
    src = g.node("src", SOURCE, out_dim=dims[0], fn=SRC_DENSE_ROW)
    prev = src
    for k in range(len(dims) - 1):
        last = k == len(dims) - 2
        lin = g.node(f"linear{k + 1}", LINEAR, dims[k], dims[k + 1], act=ACT_NONE if last else ACT_RELU,
                     flags=FLAG_SOURCE_ADJACENT if k == 0 else 0)
        g.edge(prev, lin)
        prev = lin
    loss = g.node("loss", LOSS_CE, dims[-1], 0, fn=LABEL_PER_INSTANCE)
    g.edge(prev, loss)
    return g


def rnn(vocab=14, emb=128, hidden=128, classes=10, act=ACT_TANH, replicas=1):
    """Variable-length RNN (paper Fig. 2): Lookup -> Concat(with h from Phi) -> Linear-1 -> Isu(t+1)
    -> Cond(end?) -> Phi loop | Linear-2 -> Loss.  13T+3 node-messages for T tokens.
    replicas > 1: Linear-1 is replicated in full between a Cond (round robin over instance + position) and a Phi
    (Sec. 5); the copies are "linear1", "linear1_r1", ...; 17T+3 node-messages."""
    assert emb == hidden, "Concat ports have one common width"
    g = IRGraph("rnn")
    s_tok = g.node("src_tokens", SOURCE, fn=SRC_TOKENS)
    look = g.node("lookup", LOOKUP, vocab, emb, flags=FLAG_SOURCE_ADJACENT)
    s_h0 = g.node("src_h0", SOURCE, out_dim=hidden, fn=SRC_ZERO_STATE)
    phi = g.node("phi", PHI, hidden, hidden)
    cat = g.node("concat", CONCAT, emb, emb + hidden, fn=CONCAT_BY_EDGE, fn_arg=2)
    lin1 = g.node("linear1", LINEAR, emb + hidden, hidden, act=act)
    isu = g.node("isu", ISU, hidden, hidden, fn=ISU_U_INC)
    cond = g.node("cond", COND, hidden, hidden, fn=COND_SEQ_END)
    lin2 = g.node("linear2", LINEAR, hidden, classes)
    loss = g.node("loss", LOSS_CE, classes, 0, fn=LABEL_PER_INSTANCE)
    g.edge(s_tok, look)
    g.edge(look, cat, 0, 0)
    g.edge(s_h0, phi, 0, 0)
    g.edge(phi, cat, 0, 1)
    if replicas > 1:            # appended after the canonical nodes, so that those keep their indices
        cond_r = g.node("cond_replica", COND, emb + hidden, emb + hidden, fn=COND_ROUND_ROBIN)
        phi_r = g.node("phi_replica", PHI, hidden, hidden)
        copies = [lin1] + [g.node(f"linear1_r{k}", LINEAR, emb + hidden, hidden, act=act) for k in range(1, replicas)]
        g.edge(cat, cond_r)
        for k, c in enumerate(copies):
            g.edge(cond_r, c, k, 0)
            g.edge(c, phi_r, 0, k)
        g.edge(phi_r, isu)
    else:
        g.edge(cat, lin1)
        g.edge(lin1, isu)
    g.edge(isu, cond)
    g.edge(cond, phi, 0, 1)     # loop
    g.edge(cond, lin2, 1, 0)    # exit
    g.edge(lin2, loss)
    return g


def tree_lstm(vocab=20000, emb=300, hidden=150, classes=5):
    """Binary Tree-LSTM split into a leaf and a branch cell (Sec. 6, sentiment model).  A cell is an ordinary Linear node that
    produces the gate pre-activations (leaf: emb -> 3H, branch: [hL; hR] -> 5H) followed by a parameter-free gate node;
    a cell's output [h; c] is split into an h stream (classifier at every node, parent's [hL; hR]) and a c stream
    (parent's [cL; cR]); both streams end in a Sink at the root."""
    g = IRGraph("tree_lstm")
    H = hidden
    src = g.node("src_leaves", SOURCE, fn=SRC_TREE_LEAVES)
    look = g.node("lookup", LOOKUP, vocab, emb, flags=FLAG_SOURCE_ADJACENT)
    leaf = g.node("leaf_gates", LINEAR, emb, 3 * H)
    leaf_g = g.node("leaf_lstm", NPT_LSTM, 3 * H, 2 * H, fn=LSTM_LEAF)
    phi = g.node("phi", PHI, 2 * H, 2 * H)
    sp = g.node("split_hc", SPLIT, 2 * H, H, fn_arg=2)
    bc = g.node("bcast", BCAST, H, H, fn_arg=2)
    cls = g.node("classifier", LINEAR, H, classes)
    loss = g.node("loss", LOSS_CE, classes, 0, fn=LABEL_PER_TREE_NODE)
    cond_h = g.node("cond_root_h", COND, H, H, fn=COND_TREE_ROOT)
    sink_h = g.node("sink_h", SINK, H, 0)
    isu_h = g.node("isu_parent_h", ISU, H, H, fn=ISU_TREE_PARENT)
    cat_h = g.node("concat_h", CONCAT, H, 2 * H, fn=CONCAT_BY_STATE_PORT, fn_arg=2)
    br = g.node("branch_gates", LINEAR, 2 * H, 5 * H)
    cond_c = g.node("cond_root_c", COND, H, H, fn=COND_TREE_ROOT)
    sink_c = g.node("sink_c", SINK, H, 0)
    isu_c = g.node("isu_parent_c", ISU, H, H, fn=ISU_TREE_PARENT)
    cat_c = g.node("concat_c", CONCAT, H, 2 * H, fn=CONCAT_BY_STATE_PORT, fn_arg=2)
    br_g = g.node("branch_lstm", NPT_LSTM, 5 * H, 2 * H, fn=LSTM_BRANCH)
    g.edge(src, look)
    g.edge(look, leaf)
    g.edge(leaf, leaf_g)
    g.edge(leaf_g, phi, 0, 0)
    g.edge(br_g, phi, 0, 1)
    g.edge(phi, sp)
    g.edge(sp, bc, 0, 0)            # h
    g.edge(bc, cls, 0, 0)
    g.edge(cls, loss)
    g.edge(bc, cond_h, 1, 0)
    g.edge(cond_h, sink_h, 0, 0)
    g.edge(cond_h, isu_h, 1, 0)
    g.edge(isu_h, cat_h)
    g.edge(cat_h, br)
    g.edge(br, br_g, 0, 0)
    g.edge(sp, cond_c, 1, 0)        # c
    g.edge(cond_c, sink_c, 0, 0)
    g.edge(cond_c, isu_c, 1, 0)
    g.edge(isu_c, cat_c)
    g.edge(cat_c, br_g, 0, 1)
    return g


def tree(vocab=20000, emb=300, hidden=150, classes=5, grouped_leaves=False):
    """Binary tree RNN: Lookup -> LeafCell -> Phi <- BranchCell; Phi -> Bcast -> {Classifier -> Loss,
    Cond(root ? Sink : Isu(parent) -> Concat(left,right) -> BranchCell)}.  33L-18 node-messages for L leaves.
    grouped_leaves (Sec. 6: the leaf operations of a tree grouped into one call): the controller pumps one message whose
    rows are the tokens of the tree's leaves, Lookup and LeafCell work on that matrix, and an Ungroup in front of the
    Phi hands every leaf its row (backward: it collects the leaves' gradients into one matrix message)."""
    g = IRGraph("tree_grouped" if grouped_leaves else "tree")
    src = g.node("src_leaves", SOURCE, fn=SRC_TREE_LEAVES_GROUPED if grouped_leaves else SRC_TREE_LEAVES)
    look = g.node("lookup", LOOKUP, vocab, emb, flags=FLAG_SOURCE_ADJACENT)
    leaf = g.node("leaf_cell", LINEAR, emb, hidden, act=ACT_TANH)
    phi = g.node("phi", PHI, hidden, hidden)
    bc = g.node("bcast", BCAST, hidden, hidden, fn_arg=2)
    cls = g.node("classifier", LINEAR, hidden, classes)
    loss = g.node("loss", LOSS_CE, classes, 0, fn=LABEL_PER_TREE_NODE)
    cond = g.node("cond_root", COND, hidden, hidden, fn=COND_TREE_ROOT)
    sink = g.node("sink", SINK, hidden, 0)
    isu = g.node("isu_parent", ISU, hidden, hidden, fn=ISU_TREE_PARENT)
    cat = g.node("concat", CONCAT, hidden, 2 * hidden, fn=CONCAT_BY_STATE_PORT, fn_arg=2)
    br = g.node("branch_cell", LINEAR, 2 * hidden, hidden, act=ACT_TANH)
    g.edge(src, look)
    g.edge(look, leaf)
    if grouped_leaves:
        ung = g.node("ungroup_leaves", UNGROUP, hidden, hidden, fn=UNGROUP_LEAVES)
        g.edge(leaf, ung)
        g.edge(ung, phi, 0, 0)
    else:
        g.edge(leaf, phi, 0, 0)
    g.edge(br, phi, 0, 1)
    g.edge(phi, bc)
    g.edge(bc, cls, 0, 0)
    g.edge(cls, loss)
    g.edge(bc, cond, 1, 0)
    g.edge(cond, sink, 0, 0)
    g.edge(cond, isu, 1, 0)
    g.edge(isu, cat)
    g.edge(cat, br)
    return g


def ggnn(n_node_types=15, hidden=100, steps=4, n_edge_types=N_EDGE_TYPES, readout=100):
    """Gated graph neural network (paper Fig. 3a): Lookup -> Phi_loop -> Bcast -> {Concat port 1 (h),
    Ungroup -> Flatmap(out-edges) -> Group(by type) -> Cond -> Linear_c -> Phi -> Ungroup -> Group(by dst)
    -> sum -> Group(all) -> Concat port 0 (a)} -> GRUCell -> Isu(it+1) -> Cond(it < steps) -> loop | sum-pool
    -> Linear(ReLU) -> Linear -> MSE."""
    g = IRGraph("ggnn")
    H = hidden
    src = g.node("src_graph", SOURCE, fn=SRC_GRAPH_NODES)
    look = g.node("lookup", LOOKUP, n_node_types, H, flags=FLAG_SOURCE_ADJACENT)
    phi_loop = g.node("phi_loop", PHI, H, H)
    bc = g.node("bcast", BCAST, H, H, fn_arg=2)
    ung_n = g.node("ungroup_nodes", UNGROUP, H, H, fn=UNGROUP_NODES)
    fm = g.node("flatmap_edges", FLATMAP, H, H, fn=FLATMAP_OUT_EDGES)
    grp_t = g.node("group_by_type", GROUP, H, H, fn=GROUP_EDGES_BY_TYPE)
    cond_t = g.node("cond_type", COND, H, H, fn=COND_BY_U)
    lins = [g.node(f"edge_linear{c}", LINEAR, H, H) for c in range(n_edge_types)]
    phi_t = g.node("phi_type", PHI, H, H)
    ung_e = g.node("ungroup_edges", UNGROUP, H, H, fn=UNGROUP_TYPE_EDGES)
    grp_d = g.node("group_by_dst", GROUP, H, H, fn=GROUP_EDGES_BY_DST)
    summ = g.node("sum_incoming", NPT_SUMROWS, H, H)
    grp_a = g.node("group_all", GROUP, H, H, fn=GROUP_ALL_NODES)
    cat = g.node("concat", CONCAT, H, 2 * H, fn=CONCAT_BY_EDGE, fn_arg=2)
    gru = g.node("gru", GRUCELL, 2 * H, H)
    isu = g.node("isu_it", ISU, H, H, fn=ISU_IT_INC)
    cond_it = g.node("cond_it", COND, H, H, fn=COND_IT_LT, fn_arg=steps)
    pool = g.node("sum_pool", NPT_SUMROWS, H, H)
    r1 = g.node("readout1", LINEAR, H, readout, act=ACT_RELU)
    r2 = g.node("readout2", LINEAR, readout, 1)
    loss = g.node("loss", LOSS_MSE, 1, 0, fn=LABEL_PER_INSTANCE)
    g.edge(src, look)
    g.edge(look, phi_loop, 0, 0)
    g.edge(phi_loop, bc)
    g.edge(bc, cat, 0, 1)
    g.edge(bc, ung_n, 1, 0)
    g.edge(ung_n, fm)
    g.edge(fm, grp_t)
    g.edge(grp_t, cond_t)
    for c, lin in enumerate(lins):
        g.edge(cond_t, lin, c, 0)
        g.edge(lin, phi_t, 0, c)
    g.edge(phi_t, ung_e)
    g.edge(ung_e, grp_d)
    g.edge(grp_d, summ)
    g.edge(summ, grp_a)
    g.edge(grp_a, cat, 0, 0)
    g.edge(cat, gru)
    g.edge(gru, isu)
    g.edge(isu, cond_it)
    g.edge(cond_it, phi_loop, 0, 1)
    g.edge(cond_it, pool, 1, 0)
    g.edge(pool, r1)
    g.edge(r1, r2)
    g.edge(r2, loss)
    return g
