// Host helpers that emit the IR descriptions of the four canonical model families (Sec. 2, Sec. 4 of the paper):
// multi-layer perceptron, variable-length RNN (Fig. 2), binary tree RNN, gated graph neural network (Fig. 3a).
// Plain host code: no device is needed to call them.
#include <vector>

#include "../../include/ampnet.h"

namespace {

struct Builder {
  std::vector<ampnet_node_desc_t> nodes;
  std::vector<ampnet_edge_desc_t> edges;
  int node(int type, int in_dim = 0, int out_dim = 0, int act = 0, int fn = 0, int fn_arg = 0, int flags = 0) {
    ampnet_node_desc_t d{type, in_dim, out_dim, act, fn, fn_arg, 0, flags};
    nodes.push_back(d);
    return (int)nodes.size() - 1;
  }
  void edge(int src, int dst, int src_port = 0, int dst_port = 0) { edges.push_back(ampnet_edge_desc_t{src, src_port, dst, dst_port}); }
  ampnet_status_t emit(ampnet_node_desc_t* n, int32_t cap_n, int32_t* n_n, ampnet_edge_desc_t* e, int32_t cap_e, int32_t* n_e) const {
    if (!n_n || !n_e) return AMPNET_EINVAL;
    *n_n = (int32_t)nodes.size();
    *n_e = (int32_t)edges.size();
    if (!n || !e || cap_n < *n_n || cap_e < *n_e) return AMPNET_EOVERFLOW;   // the counts say how much room is needed
    for (size_t i = 0; i < nodes.size(); i++) n[i] = nodes[i];
    for (size_t i = 0; i < edges.size(); i++) e[i] = edges[i];
    return AMPNET_OK;
  }
};

}  // namespace

extern "C" {

ampnet_status_t ampnet_ir_mlp(const int32_t* dims, int32_t n_dims, ampnet_node_desc_t* nodes, int32_t cap_nodes,
                              int32_t* n_nodes, ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges) {
  if (!dims || n_dims < 2) return AMPNET_EINVAL;
  for (int i = 0; i < n_dims; i++) if (dims[i] < 1) return AMPNET_EINVAL;
  Builder b;
  int prev = b.node(AMPNET_SOURCE, 0, dims[0], 0, AMPNET_SRC_DENSE_ROW);
  for (int k = 0; k + 1 < n_dims; k++) {
    const bool last = k == n_dims - 2;
    int lin = b.node(AMPNET_LINEAR, dims[k], dims[k + 1], last ? AMPNET_ACT_NONE : AMPNET_ACT_RELU, 0, 0,
                     k == 0 ? AMPNET_FLAG_SOURCE_ADJACENT : 0);
    b.edge(prev, lin);
    prev = lin;
  }
  int loss = b.node(AMPNET_LOSS_CE, dims[n_dims - 1], 0, 0, AMPNET_LABEL_PER_INSTANCE);
  b.edge(prev, loss);
  return b.emit(nodes, cap_nodes, n_nodes, edges, cap_edges, n_edges);
}

ampnet_status_t ampnet_ir_rnn(int32_t vocab, int32_t emb, int32_t hidden, int32_t classes, int32_t act,
                              ampnet_node_desc_t* nodes, int32_t cap_nodes, int32_t* n_nodes,
                              ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges) {
  return ampnet_ir_rnn_replicated(vocab, emb, hidden, classes, act, 1, nodes, cap_nodes, n_nodes, edges, cap_edges, n_edges);
}

ampnet_status_t ampnet_ir_rnn_replicated(int32_t vocab, int32_t emb, int32_t hidden, int32_t classes, int32_t act, int32_t replicas,
                                         ampnet_node_desc_t* nodes, int32_t cap_nodes, int32_t* n_nodes,
                                         ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges) {
  if (vocab < 1 || emb < 1 || hidden < 1 || classes < 1 || emb != hidden) return AMPNET_EINVAL;   // one width per Concat port
  if (replicas < 1 || replicas > 8) return AMPNET_EINVAL;                                          // a Cond has at most 8 ports
  Builder b;
  int s_tok = b.node(AMPNET_SOURCE, 0, 0, 0, AMPNET_SRC_TOKENS);
  int look = b.node(AMPNET_LOOKUP, vocab, emb, 0, 0, 0, AMPNET_FLAG_SOURCE_ADJACENT);
  int s_h0 = b.node(AMPNET_SOURCE, 0, hidden, 0, AMPNET_SRC_ZERO_STATE);
  int phi = b.node(AMPNET_PHI, hidden, hidden);
  int cat = b.node(AMPNET_CONCAT, emb, emb + hidden, 0, AMPNET_CONCAT_BY_EDGE, 2);
  int lin1 = b.node(AMPNET_LINEAR, emb + hidden, hidden, act);
  int isu = b.node(AMPNET_ISU, hidden, hidden, 0, AMPNET_ISU_U_INC);
  int cond = b.node(AMPNET_COND, hidden, hidden, 0, AMPNET_COND_SEQ_END);
  int lin2 = b.node(AMPNET_LINEAR, hidden, classes);
  int loss = b.node(AMPNET_LOSS_CE, classes, 0, 0, AMPNET_LABEL_PER_INSTANCE);
  b.edge(s_tok, look);
  b.edge(look, cat, 0, 0);
  b.edge(s_h0, phi, 0, 0);
  b.edge(phi, cat, 0, 1);
  if (replicas > 1) {      // the copies go between a round-robin Cond and a Phi, after the canonical nodes
    int cond_r = b.node(AMPNET_COND, emb + hidden, emb + hidden, 0, AMPNET_COND_ROUND_ROBIN);
    int phi_r = b.node(AMPNET_PHI, hidden, hidden);
    b.edge(cat, cond_r);
    b.edge(cond_r, lin1, 0, 0);
    b.edge(lin1, phi_r, 0, 0);
    for (int k = 1; k < replicas; k++) {
      int c = b.node(AMPNET_LINEAR, emb + hidden, hidden, act);
      b.edge(cond_r, c, k, 0);
      b.edge(c, phi_r, 0, k);
    }
    b.edge(phi_r, isu);
  } else {
    b.edge(cat, lin1);
    b.edge(lin1, isu);
  }
  b.edge(isu, cond);
  b.edge(cond, phi, 0, 1);
  b.edge(cond, lin2, 1, 0);
  b.edge(lin2, loss);
  return b.emit(nodes, cap_nodes, n_nodes, edges, cap_edges, n_edges);
}

static ampnet_status_t tree_ir(bool grouped, int32_t vocab, int32_t emb, int32_t hidden, int32_t classes,
                               ampnet_node_desc_t* nodes, int32_t cap_nodes, int32_t* n_nodes,
                               ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges) {
  if (vocab < 1 || emb < 1 || hidden < 1 || classes < 1) return AMPNET_EINVAL;
  Builder b;
  int src = b.node(AMPNET_SOURCE, 0, 0, 0, grouped ? AMPNET_SRC_TREE_LEAVES_GROUPED : AMPNET_SRC_TREE_LEAVES);
  int look = b.node(AMPNET_LOOKUP, vocab, emb, 0, 0, 0, AMPNET_FLAG_SOURCE_ADJACENT);
  int leaf = b.node(AMPNET_LINEAR, emb, hidden, AMPNET_ACT_TANH);
  int phi = b.node(AMPNET_PHI, hidden, hidden);
  int bc = b.node(AMPNET_BCAST, hidden, hidden, 0, 0, 2);
  int cls = b.node(AMPNET_LINEAR, hidden, classes);
  int loss = b.node(AMPNET_LOSS_CE, classes, 0, 0, AMPNET_LABEL_PER_TREE_NODE);
  int cond = b.node(AMPNET_COND, hidden, hidden, 0, AMPNET_COND_TREE_ROOT);
  int sink = b.node(AMPNET_SINK, hidden, 0);
  int isu = b.node(AMPNET_ISU, hidden, hidden, 0, AMPNET_ISU_TREE_PARENT);
  int cat = b.node(AMPNET_CONCAT, hidden, 2 * hidden, 0, AMPNET_CONCAT_BY_STATE_PORT, 2);
  int br = b.node(AMPNET_LINEAR, 2 * hidden, hidden, AMPNET_ACT_TANH);
  b.edge(src, look);
  b.edge(look, leaf);
  if (grouped) {                       // (the extra node comes last, so that the other nodes keep their indices)
    int ung = b.node(AMPNET_UNGROUP, hidden, hidden, 0, AMPNET_UNGROUP_LEAVES);
    b.edge(leaf, ung);
    b.edge(ung, phi, 0, 0);
  } else b.edge(leaf, phi, 0, 0);
  b.edge(br, phi, 0, 1);
  b.edge(phi, bc);
  b.edge(bc, cls, 0, 0);
  b.edge(cls, loss);
  b.edge(bc, cond, 1, 0);
  b.edge(cond, sink, 0, 0);
  b.edge(cond, isu, 1, 0);
  b.edge(isu, cat);
  b.edge(cat, br);
  return b.emit(nodes, cap_nodes, n_nodes, edges, cap_edges, n_edges);
}

ampnet_status_t ampnet_ir_tree(int32_t vocab, int32_t emb, int32_t hidden, int32_t classes,
                               ampnet_node_desc_t* nodes, int32_t cap_nodes, int32_t* n_nodes,
                               ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges) {
  return tree_ir(false, vocab, emb, hidden, classes, nodes, cap_nodes, n_nodes, edges, cap_edges, n_edges);
}

ampnet_status_t ampnet_ir_tree_grouped(int32_t vocab, int32_t emb, int32_t hidden, int32_t classes,
                                       ampnet_node_desc_t* nodes, int32_t cap_nodes, int32_t* n_nodes,
                                       ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges) {
  return tree_ir(true, vocab, emb, hidden, classes, nodes, cap_nodes, n_nodes, edges, cap_edges, n_edges);
}

ampnet_status_t ampnet_ir_tree_lstm(int32_t vocab, int32_t emb, int32_t hidden, int32_t classes,
                                    ampnet_node_desc_t* nodes, int32_t cap_nodes, int32_t* n_nodes,
                                    ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges) {
  if (vocab < 1 || emb < 1 || hidden < 1 || classes < 1) return AMPNET_EINVAL;
  Builder b;
  const int H = hidden;
  int src = b.node(AMPNET_SOURCE, 0, 0, 0, AMPNET_SRC_TREE_LEAVES);
  int look = b.node(AMPNET_LOOKUP, vocab, emb, 0, 0, 0, AMPNET_FLAG_SOURCE_ADJACENT);
  int leaf = b.node(AMPNET_LINEAR, emb, 3 * H);                                   // leaf cell: gate pre-activations i, o, u
  int leaf_g = b.node(AMPNET_NPT_LSTM, 3 * H, 2 * H, 0, AMPNET_LSTM_LEAF);
  int phi = b.node(AMPNET_PHI, 2 * H, 2 * H);
  int sp = b.node(AMPNET_SPLIT, 2 * H, H, 0, 0, 2);                               // [h; c] -> h stream, c stream
  int bc = b.node(AMPNET_BCAST, H, H, 0, 0, 2);
  int cls = b.node(AMPNET_LINEAR, H, classes);
  int loss = b.node(AMPNET_LOSS_CE, classes, 0, 0, AMPNET_LABEL_PER_TREE_NODE);
  int cond_h = b.node(AMPNET_COND, H, H, 0, AMPNET_COND_TREE_ROOT);
  int sink_h = b.node(AMPNET_SINK, H, 0);
  int isu_h = b.node(AMPNET_ISU, H, H, 0, AMPNET_ISU_TREE_PARENT);
  int cat_h = b.node(AMPNET_CONCAT, H, 2 * H, 0, AMPNET_CONCAT_BY_STATE_PORT, 2);
  int br = b.node(AMPNET_LINEAR, 2 * H, 5 * H);                                   // branch cell: i, fL, fR, o, u from [hL; hR]
  int cond_c = b.node(AMPNET_COND, H, H, 0, AMPNET_COND_TREE_ROOT);
  int sink_c = b.node(AMPNET_SINK, H, 0);
  int isu_c = b.node(AMPNET_ISU, H, H, 0, AMPNET_ISU_TREE_PARENT);
  int cat_c = b.node(AMPNET_CONCAT, H, 2 * H, 0, AMPNET_CONCAT_BY_STATE_PORT, 2);
  int br_g = b.node(AMPNET_NPT_LSTM, 5 * H, 2 * H, 0, AMPNET_LSTM_BRANCH);
  b.edge(src, look);
  b.edge(look, leaf);
  b.edge(leaf, leaf_g);
  b.edge(leaf_g, phi, 0, 0);
  b.edge(br_g, phi, 0, 1);
  b.edge(phi, sp);
  b.edge(sp, bc, 0, 0);
  b.edge(bc, cls, 0, 0);
  b.edge(cls, loss);
  b.edge(bc, cond_h, 1, 0);
  b.edge(cond_h, sink_h, 0, 0);
  b.edge(cond_h, isu_h, 1, 0);
  b.edge(isu_h, cat_h);
  b.edge(cat_h, br);
  b.edge(br, br_g, 0, 0);
  b.edge(sp, cond_c, 1, 0);
  b.edge(cond_c, sink_c, 0, 0);
  b.edge(cond_c, isu_c, 1, 0);
  b.edge(isu_c, cat_c);
  b.edge(cat_c, br_g, 0, 1);
  return b.emit(nodes, cap_nodes, n_nodes, edges, cap_edges, n_edges);
}

ampnet_status_t ampnet_ir_ggnn(int32_t n_node_types, int32_t hidden, int32_t steps, int32_t n_edge_types, int32_t readout,
                               ampnet_node_desc_t* nodes, int32_t cap_nodes, int32_t* n_nodes,
                               ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges) {
  if (n_node_types < 1 || hidden < 1 || steps < 1 || n_edge_types < 1 || n_edge_types > 8 || readout < 1) return AMPNET_EINVAL;
  Builder b;
  const int H = hidden;
  int src = b.node(AMPNET_SOURCE, 0, 0, 0, AMPNET_SRC_GRAPH_NODES);
  int look = b.node(AMPNET_LOOKUP, n_node_types, H, 0, 0, 0, AMPNET_FLAG_SOURCE_ADJACENT);
  int phi_loop = b.node(AMPNET_PHI, H, H);
  int bc = b.node(AMPNET_BCAST, H, H, 0, 0, 2);
  int ung_n = b.node(AMPNET_UNGROUP, H, H, 0, AMPNET_UNGROUP_NODES);
  int fm = b.node(AMPNET_FLATMAP, H, H, 0, AMPNET_FLATMAP_OUT_EDGES);
  int grp_t = b.node(AMPNET_GROUP, H, H, 0, AMPNET_GROUP_EDGES_BY_TYPE);
  int cond_t = b.node(AMPNET_COND, H, H, 0, AMPNET_COND_BY_U);
  std::vector<int> lins;
  for (int c = 0; c < n_edge_types; c++) lins.push_back(b.node(AMPNET_LINEAR, H, H));
  int phi_t = b.node(AMPNET_PHI, H, H);
  int ung_e = b.node(AMPNET_UNGROUP, H, H, 0, AMPNET_UNGROUP_TYPE_EDGES);
  int grp_d = b.node(AMPNET_GROUP, H, H, 0, AMPNET_GROUP_EDGES_BY_DST);
  int summ = b.node(AMPNET_NPT_SUMROWS, H, H);
  int grp_a = b.node(AMPNET_GROUP, H, H, 0, AMPNET_GROUP_ALL_NODES);
  int cat = b.node(AMPNET_CONCAT, H, 2 * H, 0, AMPNET_CONCAT_BY_EDGE, 2);
  int gru = b.node(AMPNET_GRUCELL, 2 * H, H);
  int isu = b.node(AMPNET_ISU, H, H, 0, AMPNET_ISU_IT_INC);
  int cond_it = b.node(AMPNET_COND, H, H, 0, AMPNET_COND_IT_LT, steps);
  int pool = b.node(AMPNET_NPT_SUMROWS, H, H);
  int r1 = b.node(AMPNET_LINEAR, H, readout, AMPNET_ACT_RELU);
  int r2 = b.node(AMPNET_LINEAR, readout, 1);
  int loss = b.node(AMPNET_LOSS_MSE, 1, 0, 0, AMPNET_LABEL_PER_INSTANCE);
  b.edge(src, look);
  b.edge(look, phi_loop, 0, 0);
  b.edge(phi_loop, bc);
  b.edge(bc, cat, 0, 1);
  b.edge(bc, ung_n, 1, 0);
  b.edge(ung_n, fm);
  b.edge(fm, grp_t);
  b.edge(grp_t, cond_t);
  for (int c = 0; c < n_edge_types; c++) { b.edge(cond_t, lins[c], c, 0); b.edge(lins[c], phi_t, 0, c); }
  b.edge(phi_t, ung_e);
  b.edge(ung_e, grp_d);
  b.edge(grp_d, summ);
  b.edge(summ, grp_a);
  b.edge(grp_a, cat, 0, 0);
  b.edge(cat, gru);
  b.edge(gru, isu);
  b.edge(isu, cond_it);
  b.edge(cond_it, phi_loop, 0, 1);
  b.edge(cond_it, pool, 1, 0);
  b.edge(pool, r1);
  b.edge(r1, r2);
  b.edge(r2, loss);
  return b.emit(nodes, cap_nodes, n_nodes, edges, cap_edges, n_edges);
}

}  // extern "C"
