// AMPNet CPU oracle -- TEST INFRASTRUCTURE, not part of the product path.
//
// A plain, slow, single-threaded restatement of asynchronous model-parallel (AMP) training of an IR
// graph (paper Sec. 3, Sec. 4, App. A), used only to check the CUDA implementation and as a timed CPU
// baseline.  It shares no code with the CUDA path.  Only tests, the smoke check and the benchmark's
// CPU-baseline leg may load it.
//
// What it follows:
//   * Sec. 3: forward/backward messages; every parameterised node accumulates gradients locally and,
//     once min_update_frequency (muf) gradients have arrived, applies a local update and clears the
//     accumulator; max_active_keys (mak) bounds the instances in flight; staleness of a gradient = number
//     of updates of the node between the gradient's forward and backward computation.
//   * Sec. 4: message = payload + state; node semantics of PPT (Linear, Lookup, GRU cell), NPT (row sum),
//     Loss, Cond, Phi, Isu, Concat, Split, Bcast, Group, Ungroup, Flatmap; the invariant that every forward
//     message is answered by a backward message with the same state (checked: all caches empty at the end).
//   * App. A: backward messages take priority over forward messages.
//
// Readings where the paper is silent (all listed in the design notes of the repository):
//   update trigger n >= muf; one gradient per payload row; update = mean of accumulated gradients,
//   theta -= lr * A / n; leftovers flushed at epoch end; backward uses the current W and the cached forward
//   activations; a canonical round schedule (below) replaces the timing-dependent runtime; lowest free key
//   slot; sums and concatenations are done in member/port/edge index order at completion; GRU in the form
//   h' = (1-z)*h + z*c with the reset gate applied to h before W_c; loss over a tree = plain sum over nodes.
//
// Canonical schedule.  Only PPT nodes hold order-sensitive state, every other node fires eagerly the moment
// its inputs are complete.  Round r: (1) the controller processes the retire notices of round r-1, then
// admits instances while active < mak (lowest free slot) and pumps their source messages, which land in the
// PPT inboxes of round r; (2) every PPT node sorts its inbox by (backward first, admission seq, it, u, port)
// and processes it one message at a time (an update takes effect before the next message); what it emits
// lands in the inboxes of round r+1.
//
// Parity pins (tests, -m "not gpu"): finite differences in fp64 for every family, exact agreement with a
// textbook SGD / minibatch-SGD loop, autograd of independently written recursions for RNN / tree / graph
// nets, closed-form message counts, hand traces of the schedule, exactly-once gradient accounting.
// Unpinned by design: the convergence figures of the paper's Table 1 (they need the paper's datasets) and
// asynchronous trajectories (timing dependent).

#include <algorithm>
#include <array>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <map>
#include <memory>
#include <string>
#include <tuple>
#include <vector>

#ifndef ORACLE_REAL
#define ORACLE_REAL double
#endif
typedef ORACLE_REAL real;

namespace {

enum { LSTM_LEAF = 1, LSTM_BRANCH = 2 };
enum NodeType { SOURCE, LINEAR, LOOKUP, GRUCELL, LOSS_CE, LOSS_MSE, NPT_SUMROWS, COND, PHI, ISU, CONCAT, SPLIT,
                BCAST, GROUP, UNGROUP, FLATMAP, SINK, NPT_LSTM, N_TYPES };
enum Act { ACT_NONE, ACT_RELU, ACT_TANH, ACT_SIGMOID };
enum { SRC_DENSE_ROW = 1, SRC_TOKENS, SRC_ZERO_STATE, SRC_TREE_LEAVES, SRC_GRAPH_NODES, SRC_TREE_LEAVES_GROUPED };
enum { COND_SEQ_END = 1, COND_TREE_ROOT, COND_BY_U, COND_IT_LT, COND_ROUND_ROBIN };
enum { ISU_U_INC = 1, ISU_TREE_PARENT, ISU_IT_INC };
enum { CONCAT_BY_EDGE = 1, CONCAT_BY_STATE_PORT };
enum { GROUP_EDGES_BY_TYPE = 1, GROUP_EDGES_BY_DST, GROUP_ALL_NODES };
enum { UNGROUP_NODES = 1, UNGROUP_TYPE_EDGES, UNGROUP_LEAVES };
enum { FLATMAP_OUT_EDGES = 1 };
enum { LABEL_PER_INSTANCE = 1, LABEL_PER_TREE_NODE };
enum { FLAG_SOURCE_ADJACENT = 1 };
enum { KIND_DENSE_ROWS, KIND_SEQUENCES, KIND_BINARY_TREES, KIND_TYPED_GRAPHS };
enum Dir { FWD = 0, BWD = 1 };

struct State { int inst = 0, seq = 0, slot = 0, it = 0, u = 0, port = 0; };
typedef std::tuple<int, int, int> Key;
static Key key_of(const State& s) { return Key(s.slot, s.it, s.u); }

struct Msg {
  int dir = FWD;
  bool eval = false;
  State s;
  int rows = 0, dim = 0;
  std::vector<real> p;       // row-major [rows x dim]
};

// Per-instance structure tables ("reference to the graph structure" carried by the state, Sec. 4).
struct Structure {
  int n_pos = 0;                          // tokens / tree nodes / graph nodes
  std::vector<int> tokens;
  std::vector<int> left, right, parent, child_slot;
  int root = -1;
  std::vector<int> leaves;
  std::vector<int> esrc, edst, etype;
  std::vector<std::vector<int>> out_edges, in_edges, type_edges;   // edge ids in increasing order
  std::vector<int> rank_out, rank_in, rank_type;
  const float* dense = nullptr;
  std::vector<int> labels;                // per instance (size 1) or per tree node
  double target = 0;
};

struct Dataset {
  int kind = -1;
  int dense_dim = 0;
  std::vector<Structure> inst;
  std::vector<float> dense;
};

static uint64_t mix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}
// Order-independent fingerprint of one routed message (summed mod 2^64 over all deliveries).
static uint64_t msg_hash(int node, int dir, int aport, const State& s) {
  uint64_t a = (uint64_t)node | ((uint64_t)dir << 16) | ((uint64_t)(aport & 0xff) << 20) | ((uint64_t)(s.port & 0xff) << 28);
  uint64_t b = ((uint64_t)(uint32_t)s.inst << 32) | ((uint64_t)(s.it & 0xff) << 24) | (uint64_t)(s.u & 0xffffff);
  return mix64(mix64(a) ^ (b * 0x9E3779B97F4A7C15ull));
}

static real round_bf16(real v) {
  float f = (float)v;
  uint32_t b;
  std::memcpy(&b, &f, 4);
  if ((b & 0x7f800000u) == 0x7f800000u) return v;
  uint32_t r = b + 0x7fffu + ((b >> 16) & 1u);
  r &= 0xffff0000u;
  std::memcpy(&f, &r, 4);
  return (real)f;
}

static real act_fwd(int a, real v) {
  switch (a) {
    case ACT_RELU: return v > 0 ? v : 0;
    case ACT_TANH: return std::tanh(v);
    case ACT_SIGMOID: return 1 / (1 + std::exp(-v));
    default: return v;
  }
}
static real act_grad_from_y(int a, real y) {
  switch (a) {
    case ACT_RELU: return y > 0 ? 1 : 0;
    case ACT_TANH: return 1 - y * y;
    case ACT_SIGMOID: return y * (1 - y);
    default: return 1;
  }
}

struct Engine;

struct NodeStats {
  int64_t fwd_msgs = 0, bwd_msgs = 0, n_updates = 0, n_grads_applied = 0;
  int64_t stale_hist[64] = {0};
  int max_staleness = 0;
  std::vector<int> update_log;
};

struct Node {
  Engine* E = nullptr;
  int id = 0, type = 0, in_dim = 0, out_dim = 0, act = 0, fn = 0, fn_arg = 0, muf_override = 0, flags = 0;
  NodeStats st;
  virtual ~Node() {}
  virtual void forward(Msg& m, int in_port) = 0;
  virtual void backward(Msg& m, int from_succ) = 0;
  virtual size_t cache_size() const { return 0; }
  virtual bool is_ppt() const { return false; }
  // PPT interface
  virtual int n_params() const { return 0; }
  virtual std::vector<real>* param(int) { return nullptr; }
  virtual std::vector<real>* accum(int) { return nullptr; }
  virtual void flush() {}
  virtual void reset_run() {}
};

struct Engine {
  std::vector<std::unique_ptr<Node>> nodes;
  std::vector<std::vector<std::pair<int, int>>> succ, pred;   // [node][port] -> (other node, other port)
  Dataset data[2];
  Dataset* cur = nullptr;
  bool bf16 = false;
  std::string err;
  // run configuration
  int mak = 1, muf = 1;
  real lr = 0;
  // optimiser applied at a local update (App. A: SGD, momentum-SGD, Adam): 0 SGD, 1 momentum, 2 Adam
  int opt = 0;
  real mu = 0.9, beta1 = 0.9, beta2 = 0.999, eps = 1e-8;
  // schedule state
  std::vector<std::vector<Msg>> inbox_a, inbox_b;
  std::vector<std::vector<Msg>>* target = nullptr;
  std::vector<int> retire_notices;       // slots
  std::vector<int> inflight_eval;        // per slot: forward-only messages of the slot's instance waiting in PPT inboxes
  std::vector<double> loss;              // per instance
  std::vector<int> correct, n_pred;      // eval accuracy bookkeeping
  int64_t node_messages = 0, ppt_messages = 0;
  uint64_t route_hash = 0;

  const Structure& S(const State& s) const { return cur->inst[s.inst]; }

  void deliver(int node, int aport, Msg& m) {
    Node* n = nodes[node].get();
    if (n->type == SOURCE) {               // the controller: a source message came home
      if (m.dir == BWD) retire_notices.push_back(m.s.slot);
      return;
    }
    node_messages++;
    route_hash += msg_hash(node, m.dir, aport, m.s);
    if (m.dir == FWD) n->st.fwd_msgs++; else n->st.bwd_msgs++;
    if (n->is_ppt()) {
      if (m.eval && !inflight_eval.empty()) inflight_eval[m.s.slot]++;
      (*target)[node].push_back(m);
      return;
    }
    if (m.dir == FWD) n->forward(m, aport); else n->backward(m, aport);
  }
  void round_payload(Msg& m) { if (bf16) for (auto& v : m.p) v = round_bf16(v); }
  void emit_fwd(int node, int out_port, Msg& m) {
    m.dir = FWD;
    auto& e = succ[node][out_port];
    deliver(e.first, e.second, m);
  }
  void emit_bwd(int node, int in_port, Msg& m) {
    m.dir = BWD;
    auto& e = pred[node][in_port];
    deliver(e.first, e.second, m);
  }
};

// ------------------------------------------------------------------------------------------------
// PPT nodes (Sec. 4, "Payload transformations")
// ------------------------------------------------------------------------------------------------
struct PPTBase : Node {
  int n_acc = 0, version = 0;
  bool is_ppt() const override { return true; }
  int muf() const { return muf_override > 0 ? muf_override : E->muf; }
  virtual void apply(real inv_n) = 0;     // theta <- optimiser step on the mean gradient A * inv_n; A = 0
  // Optimiser state per parameter tensor, kept across epochs; opt_t counts this node's updates (Adam bias correction).
  std::vector<std::vector<real>> mom, var;
  long long opt_t = 0;
  void reset_optimizer() { mom.clear(); var.clear(); opt_t = 0; }
  void opt_step(std::vector<real>& P, std::vector<real>& A, int w, size_t k, real inv_n) {
    const real g = A[k] * inv_n;
    A[k] = 0;
    if (E->opt == 0) { P[k] -= E->lr * g; return; }
    if ((int)mom.size() <= w) { mom.resize(w + 1); var.resize(w + 1); }
    if (mom[w].size() != P.size()) { mom[w].assign(P.size(), 0); var[w].assign(P.size(), 0); }
    if (E->opt == 1) {                       // v <- mu v + g; theta <- theta - lr v
      real& v = mom[w][k];
      v = E->mu * v + g;
      P[k] -= E->lr * v;
    } else {                                 // Adam with bias correction, t = number of updates of this node
      real& m = mom[w][k];
      real& v = var[w][k];
      m = E->beta1 * m + (1 - E->beta1) * g;
      v = E->beta2 * v + (1 - E->beta2) * g * g;
      const real mh = m / (1 - std::pow(E->beta1, (real)opt_t));
      const real vh = v / (1 - std::pow(E->beta2, (real)opt_t));
      P[k] -= E->lr * mh / (std::sqrt(vh) + E->eps);
    }
  }
  void record_staleness(int v_fwd) {
    int s = version - v_fwd;
    st.stale_hist[std::min(s, 63)]++;
    st.max_staleness = std::max(st.max_staleness, s);
  }
  // Sec. 3: once the number of accumulated gradients reaches the threshold, update locally and clear.
  void maybe_update() { if (n_acc >= muf()) do_update(); }
  void do_update() {
    if (n_acc == 0) return;
    opt_t++;
    apply((real)1 / (real)n_acc);
    st.n_updates++;
    st.n_grads_applied += n_acc;
    st.update_log.push_back(n_acc);
    n_acc = 0;
    version++;
  }
  void flush() override { do_update(); }
  void reset_run() override {
    n_acc = 0; version = 0; st = NodeStats();
    for (int w = 0; w < n_params(); w++) std::fill(accum(w)->begin(), accum(w)->end(), (real)0);
  }
};

struct Linear : PPTBase {
  std::vector<real> W, b, AW, Ab;
  struct Entry { std::vector<real> x, y; int rows, version; };
  std::map<Key, Entry> cache;
  void init() { W.assign((size_t)out_dim * in_dim, 0); b.assign(out_dim, 0); AW.assign(W.size(), 0); Ab.assign(out_dim, 0); }
  int n_params() const override { return 2; }
  std::vector<real>* param(int w) override { return w == 0 ? &W : w == 1 ? &b : nullptr; }
  std::vector<real>* accum(int w) override { return w == 0 ? &AW : w == 1 ? &Ab : nullptr; }
  size_t cache_size() const override { return cache.size(); }

  void forward(Msg& m, int) override {
    Msg o; o.eval = m.eval; o.s = m.s; o.rows = m.rows; o.dim = out_dim; o.p.assign((size_t)m.rows * out_dim, 0);
    for (int r = 0; r < m.rows; r++)
      for (int j = 0; j < out_dim; j++) {
        real acc = b[j];
        for (int i = 0; i < in_dim; i++) acc += W[(size_t)j * in_dim + i] * m.p[(size_t)r * in_dim + i];
        o.p[(size_t)r * out_dim + j] = act_fwd(act, acc);
      }
    E->round_payload(o);
    if (!m.eval) cache[key_of(m.s)] = Entry{m.p, o.p, m.rows, version};
    E->emit_fwd(id, 0, o);
  }
  void backward(Msg& m, int) override {
    auto it = cache.find(key_of(m.s));
    if (it == cache.end()) { E->err = "Linear: backward without cached activation"; return; }
    Entry e = std::move(it->second);
    cache.erase(it);
    record_staleness(e.version);
    std::vector<real> dpre((size_t)e.rows * out_dim);
    for (size_t k = 0; k < dpre.size(); k++) dpre[k] = m.p[k] * act_grad_from_y(act, e.y[k]);
    Msg o; o.s = m.s; o.rows = e.rows; o.dim = in_dim;
    if (!(flags & FLAG_SOURCE_ADJACENT)) {
      // input gradient with the CURRENT weights (no weight stashing)
      o.p.assign((size_t)e.rows * in_dim, 0);
      for (int r = 0; r < e.rows; r++)
        for (int j = 0; j < out_dim; j++) {
          real d = dpre[(size_t)r * out_dim + j];
          for (int i = 0; i < in_dim; i++) o.p[(size_t)r * in_dim + i] += W[(size_t)j * in_dim + i] * d;
        }
      E->round_payload(o);
    } else { o.rows = 0; o.dim = 0; }
    for (int r = 0; r < e.rows; r++)
      for (int j = 0; j < out_dim; j++) {
        real d = dpre[(size_t)r * out_dim + j];
        Ab[j] += d;
        for (int i = 0; i < in_dim; i++) AW[(size_t)j * in_dim + i] += d * e.x[(size_t)r * in_dim + i];
      }
    n_acc += e.rows;
    maybe_update();
    E->emit_bwd(id, 0, o);
  }
  void apply(real inv_n) override {
    for (size_t k = 0; k < W.size(); k++) opt_step(W, AW, 0, k, inv_n);
    for (size_t k = 0; k < b.size(); k++) opt_step(b, Ab, 1, k, inv_n);
  }
};

struct Lookup : PPTBase {        // in_dim = vocabulary, out_dim = embedding width
  std::vector<real> Emb, AE;
  std::vector<char> touched;
  std::vector<int> touched_list;
  struct Entry { std::vector<int> ids; int version; };
  std::map<Key, Entry> cache;
  void init() { Emb.assign((size_t)in_dim * out_dim, 0); AE.assign(Emb.size(), 0); touched.assign(in_dim, 0); }
  int n_params() const override { return 1; }
  std::vector<real>* param(int w) override { return w == 0 ? &Emb : nullptr; }
  std::vector<real>* accum(int w) override { return w == 0 ? &AE : nullptr; }
  size_t cache_size() const override { return cache.size(); }
  void reset_run() override {
    PPTBase::reset_run();
    std::fill(touched.begin(), touched.end(), 0);
    touched_list.clear();
  }

  void forward(Msg& m, int) override {         // payload = token ids, one per row
    Msg o; o.eval = m.eval; o.s = m.s; o.rows = m.rows; o.dim = out_dim; o.p.resize((size_t)m.rows * out_dim);
    Entry e; e.version = version;
    for (int r = 0; r < m.rows; r++) {
      int idx = (int)m.p[r];
      if (idx < 0 || idx >= in_dim) { E->err = "Lookup: id out of range"; return; }
      e.ids.push_back(idx);
      for (int j = 0; j < out_dim; j++) o.p[(size_t)r * out_dim + j] = Emb[(size_t)idx * out_dim + j];
    }
    E->round_payload(o);
    if (!m.eval) cache[key_of(m.s)] = e;
    E->emit_fwd(id, 0, o);
  }
  void backward(Msg& m, int) override {
    auto it = cache.find(key_of(m.s));
    if (it == cache.end()) { E->err = "Lookup: backward without cached ids"; return; }
    Entry e = std::move(it->second);
    cache.erase(it);
    record_staleness(e.version);
    for (size_t r = 0; r < e.ids.size(); r++) {
      int idx = e.ids[r];
      if (!touched[idx]) { touched[idx] = 1; touched_list.push_back(idx); }
      for (int j = 0; j < out_dim; j++) AE[(size_t)idx * out_dim + j] += m.p[r * out_dim + j];
    }
    n_acc += (int)e.ids.size();
    maybe_update();
    Msg o; o.s = m.s;                 // no input gradient: the message goes home to the controller
    E->emit_bwd(id, 0, o);
  }
  void apply(real inv_n) override {   // touched rows only (their moments too: untouched rows do not decay)
    for (int idx : touched_list) {
      for (int j = 0; j < out_dim; j++) opt_step(Emb, AE, 0, (size_t)idx * out_dim + j, inv_n);
      touched[idx] = 0;
    }
    touched_list.clear();
  }
};

struct GRUCell : PPTBase {       // x = [a; h], in_dim = 2H, out_dim = H
  std::vector<real> Wz, Wr, Wc, bz, br, bc, AWz, AWr, AWc, Abz, Abr, Abc;
  struct Entry { std::vector<real> x, z, r, c; int rows, version; };
  std::map<Key, Entry> cache;
  void init() {
    size_t n = (size_t)out_dim * in_dim;
    for (auto* v : {&Wz, &Wr, &Wc, &AWz, &AWr, &AWc}) v->assign(n, 0);
    for (auto* v : {&bz, &br, &bc, &Abz, &Abr, &Abc}) v->assign(out_dim, 0);
  }
  int n_params() const override { return 6; }
  std::vector<real>* param(int w) override {
    std::vector<real>* t[6] = {&Wz, &Wr, &Wc, &bz, &br, &bc};
    return w >= 0 && w < 6 ? t[w] : nullptr;
  }
  std::vector<real>* accum(int w) override {
    std::vector<real>* t[6] = {&AWz, &AWr, &AWc, &Abz, &Abr, &Abc};
    return w >= 0 && w < 6 ? t[w] : nullptr;
  }
  size_t cache_size() const override { return cache.size(); }

  void forward(Msg& m, int) override {
    const int H = out_dim, I = in_dim;
    Entry e; e.rows = m.rows; e.version = version; e.x = m.p;
    e.z.resize((size_t)m.rows * H); e.r.resize(e.z.size()); e.c.resize(e.z.size());
    Msg o; o.eval = m.eval; o.s = m.s; o.rows = m.rows; o.dim = H; o.p.resize(e.z.size());
    std::vector<real> xc(I);
    for (int row = 0; row < m.rows; row++) {
      const real* x = &m.p[(size_t)row * I];      // x[0..H) = a, x[H..2H) = h
      for (int j = 0; j < H; j++) {
        real az = bz[j], ar = br[j];
        for (int i = 0; i < I; i++) { az += Wz[(size_t)j * I + i] * x[i]; ar += Wr[(size_t)j * I + i] * x[i]; }
        e.z[(size_t)row * H + j] = act_fwd(ACT_SIGMOID, az);
        e.r[(size_t)row * H + j] = act_fwd(ACT_SIGMOID, ar);
      }
      for (int i = 0; i < H; i++) { xc[i] = x[i]; xc[H + i] = e.r[(size_t)row * H + i] * x[H + i]; }
      for (int j = 0; j < H; j++) {
        real ac = bc[j];
        for (int i = 0; i < I; i++) ac += Wc[(size_t)j * I + i] * xc[i];
        real c = std::tanh(ac), z = e.z[(size_t)row * H + j];
        e.c[(size_t)row * H + j] = c;
        o.p[(size_t)row * H + j] = (1 - z) * x[H + j] + z * c;
      }
    }
    E->round_payload(o);
    if (!m.eval) cache[key_of(m.s)] = std::move(e);
    E->emit_fwd(id, 0, o);
  }
  void backward(Msg& m, int) override {
    const int H = out_dim, I = in_dim;
    auto it = cache.find(key_of(m.s));
    if (it == cache.end()) { E->err = "GRUCell: backward without cached activation"; return; }
    Entry e = std::move(it->second);
    cache.erase(it);
    record_staleness(e.version);
    Msg o; o.s = m.s; o.rows = e.rows; o.dim = I; o.p.assign((size_t)e.rows * I, 0);
    std::vector<real> dpc(H), dpz(H), dpr(H), dq(H), xc(I);
    for (int row = 0; row < e.rows; row++) {
      const real* x = &e.x[(size_t)row * I];
      const real *z = &e.z[(size_t)row * H], *r = &e.r[(size_t)row * H], *c = &e.c[(size_t)row * H];
      const real* g = &m.p[(size_t)row * H];
      real* dx = &o.p[(size_t)row * I];             // dx[0..H) = da, dx[H..2H) = dh
      for (int j = 0; j < H; j++) {
        real dc = g[j] * z[j], dz = g[j] * (c[j] - x[H + j]);
        dx[H + j] = g[j] * (1 - z[j]);
        dpc[j] = dc * (1 - c[j] * c[j]);
        dpz[j] = dz * z[j] * (1 - z[j]);
      }
      // [da_c; dq] = Wc^T dpc
      std::fill(dq.begin(), dq.end(), 0);
      for (int j = 0; j < H; j++)
        for (int i = 0; i < H; i++) { dx[i] += Wc[(size_t)j * I + i] * dpc[j]; dq[i] += Wc[(size_t)j * I + H + i] * dpc[j]; }
      for (int i = 0; i < H; i++) {
        real dr = dq[i] * x[H + i];
        dx[H + i] += dq[i] * r[i];
        dpr[i] = dr * r[i] * (1 - r[i]);
      }
      for (int j = 0; j < H; j++)
        for (int i = 0; i < I; i++) dx[i] += Wz[(size_t)j * I + i] * dpz[j] + Wr[(size_t)j * I + i] * dpr[j];
      for (int i = 0; i < H; i++) { xc[i] = x[i]; xc[H + i] = r[i] * x[H + i]; }
      for (int j = 0; j < H; j++) {
        Abz[j] += dpz[j]; Abr[j] += dpr[j]; Abc[j] += dpc[j];
        for (int i = 0; i < I; i++) {
          AWz[(size_t)j * I + i] += dpz[j] * x[i];
          AWr[(size_t)j * I + i] += dpr[j] * x[i];
          AWc[(size_t)j * I + i] += dpc[j] * xc[i];
        }
      }
    }
    E->round_payload(o);
    n_acc += e.rows;
    maybe_update();
    E->emit_bwd(id, 0, o);
  }
  void apply(real inv_n) override {
    std::vector<real>* P[6] = {&Wz, &Wr, &Wc, &bz, &br, &bc};
    std::vector<real>* A[6] = {&AWz, &AWr, &AWc, &Abz, &Abr, &Abc};
    for (int t = 0; t < 6; t++)
      for (size_t k = 0; k < P[t]->size(); k++) opt_step(*P[t], *A[t], t, k, inv_n);
  }
};

// ------------------------------------------------------------------------------------------------
// Loss layer: receives the prediction, reads the label the controller pumped for this state, records the
// loss and initiates backward propagation (Sec. 4).
// ------------------------------------------------------------------------------------------------
struct Loss : Node {
  void forward(Msg& m, int) override {
    const Structure& S = E->S(m.s);
    Msg o; o.s = m.s; o.rows = m.rows; o.dim = in_dim; o.p.resize(m.p.size());
    double l = 0;
    if (type == LOSS_CE) {
      int label = fn == LABEL_PER_TREE_NODE ? S.labels[m.s.u] : S.labels[0];
      real mx = m.p[0];
      int arg = 0;
      for (int j = 1; j < in_dim; j++) if (m.p[j] > mx) { mx = m.p[j]; arg = j; }
      real sum = 0;
      for (int j = 0; j < in_dim; j++) sum += std::exp(m.p[j] - mx);
      real lse = mx + std::log(sum);
      l = (double)(lse - m.p[label]);
      for (int j = 0; j < in_dim; j++) o.p[j] = std::exp(m.p[j] - lse) - (j == label ? 1 : 0);
      E->correct[m.s.inst] += arg == label;
      E->n_pred[m.s.inst] += 1;
    } else {
      real d = m.p[0] - (real)S.target;
      l = (double)(d * d);
      o.p[0] = 2 * d;
      E->n_pred[m.s.inst] += 1;
    }
    E->loss[m.s.inst] += l;
    if (m.eval) return;
    E->round_payload(o);
    E->emit_bwd(id, 0, o);
  }
  void backward(Msg&, int) override {}
};

// Sink: closes the root's upward path so that the forward message is answered (zero gradient).
struct Sink : Node {
  void forward(Msg& m, int) override {
    if (m.eval) return;
    Msg o; o.s = m.s; o.rows = m.rows; o.dim = m.dim; o.p.assign(m.p.size(), 0);
    E->emit_bwd(id, 0, o);
  }
  void backward(Msg&, int) override {}
};

// ------------------------------------------------------------------------------------------------
// Control flow (Sec. 4, "Loops, state, and control flow")
// ------------------------------------------------------------------------------------------------
struct Cond : Node {            // routes on the state only; stateless
  void forward(Msg& m, int) override {
    const Structure& S = E->S(m.s);
    int k = 0;
    switch (fn) {
      case COND_SEQ_END: k = m.s.u < S.n_pos ? 0 : 1; break;
      case COND_TREE_ROOT: k = m.s.u == S.root ? 0 : 1; break;
      case COND_BY_U: k = m.s.u; break;
      case COND_IT_LT: k = m.s.it < fn_arg ? 0 : 1; break;
      case COND_ROUND_ROBIN: k = (int)((m.s.inst + m.s.u) % (long long)E->succ[id].size()); break;   // replicas (Sec. 5)
      default: E->err = "Cond: unknown fn";
    }
    E->emit_fwd(id, k, m);
  }
  void backward(Msg& m, int) override { E->emit_bwd(id, 0, m); }
};

struct Phi : Node {             // records the origin keyed on the state; backpropagates to it
  std::map<Key, int> origin;
  size_t cache_size() const override { return origin.size(); }
  void forward(Msg& m, int in_port) override {
    if (!m.eval) origin[key_of(m.s)] = in_port;
    E->emit_fwd(id, 0, m);
  }
  void backward(Msg& m, int) override {
    auto it = origin.find(key_of(m.s));
    if (it == origin.end()) { E->err = "Phi: backward without recorded origin"; return; }
    int p = it->second;
    origin.erase(it);
    E->emit_bwd(id, p, m);
  }
};

struct Isu : Node {             // invertible state update
  void forward(Msg& m, int) override {
    const Structure& S = E->S(m.s);
    switch (fn) {
      case ISU_U_INC: m.s.u += 1; break;
      case ISU_TREE_PARENT: m.s.port = S.child_slot[m.s.u]; m.s.u = S.parent[m.s.u]; break;
      case ISU_IT_INC: m.s.it += 1; break;
      default: E->err = "Isu: unknown fn";
    }
    E->emit_fwd(id, 0, m);
  }
  void backward(Msg& m, int) override {
    const Structure& S = E->S(m.s);
    switch (fn) {
      case ISU_U_INC: m.s.u -= 1; break;
      case ISU_TREE_PARENT: m.s.u = m.s.port == 0 ? S.left[m.s.u] : S.right[m.s.u]; m.s.port = 0; break;
      case ISU_IT_INC: m.s.it -= 1; break;
      default: E->err = "Isu: unknown fn";
    }
    E->emit_bwd(id, 0, m);
  }
};

// ------------------------------------------------------------------------------------------------
// Aggregation / disaggregation (Sec. 4, "Aggregation and disaggregation")
// ------------------------------------------------------------------------------------------------
struct Bcast : Node {           // fn_arg = k successors
  struct Part { std::vector<std::vector<real>> g; int got = 0; int rows = 0; };
  std::map<Key, Part> part;
  size_t cache_size() const override { return part.size(); }
  void forward(Msg& m, int) override {
    for (int k = 0; k < fn_arg; k++) { Msg c = m; E->emit_fwd(id, k, c); }
  }
  void backward(Msg& m, int from) override {
    Part& p = part[key_of(m.s)];
    if (p.g.empty()) p.g.resize(fn_arg);
    p.g[from] = m.p; p.got++; p.rows = m.rows;
    if (p.got < fn_arg) return;
    Msg o; o.s = m.s; o.rows = p.rows; o.dim = in_dim; o.p.assign(p.g[0].size(), 0);
    for (int k = 0; k < fn_arg; k++)               // successor-index order
      for (size_t i = 0; i < o.p.size(); i++) o.p[i] += p.g[k][i];
    part.erase(key_of(m.s));
    E->round_payload(o);
    E->emit_bwd(id, 0, o);
  }
};

struct Concat : Node {          // fn_arg = k ports of width in_dim each
  struct Part { std::vector<std::vector<real>> x; int got = 0; int rows = 0; };
  std::map<Key, Part> part;
  size_t cache_size() const override { return part.size(); }
  void forward(Msg& m, int in_port) override {
    int port = fn == CONCAT_BY_STATE_PORT ? m.s.port : in_port;
    State os = m.s; os.port = 0;                   // keyed on the state of the OUTPUT message
    Part& p = part[key_of(os)];
    if (p.x.empty()) p.x.resize(fn_arg);
    p.x[port] = m.p; p.got++; p.rows = m.rows;
    if (p.got < fn_arg) return;
    Msg o; o.eval = m.eval; o.s = os; o.rows = p.rows; o.dim = out_dim; o.p.resize((size_t)p.rows * out_dim);
    for (int r = 0; r < p.rows; r++)
      for (int k = 0; k < fn_arg; k++)
        for (int i = 0; i < in_dim; i++) o.p[(size_t)r * out_dim + k * in_dim + i] = p.x[k][(size_t)r * in_dim + i];
    part.erase(key_of(os));
    E->emit_fwd(id, 0, o);
  }
  void backward(Msg& m, int) override {
    for (int k = 0; k < fn_arg; k++) {
      Msg o; o.s = m.s; o.rows = m.rows; o.dim = in_dim; o.p.resize((size_t)m.rows * in_dim);
      for (int r = 0; r < m.rows; r++)
        for (int i = 0; i < in_dim; i++) o.p[(size_t)r * in_dim + i] = m.p[(size_t)r * out_dim + k * in_dim + i];
      if (fn == CONCAT_BY_STATE_PORT) { o.s.port = k; E->emit_bwd(id, 0, o); }
      else E->emit_bwd(id, k, o);
    }
  }
};

struct Split : Node {           // inverse of Concat: fn_arg = k successors of width out_dim each
  struct Part { std::vector<std::vector<real>> g; int got = 0; int rows = 0; };
  std::map<Key, Part> part;
  size_t cache_size() const override { return part.size(); }
  void forward(Msg& m, int) override {
    for (int k = 0; k < fn_arg; k++) {
      Msg o; o.eval = m.eval; o.s = m.s; o.rows = m.rows; o.dim = out_dim; o.p.resize((size_t)m.rows * out_dim);
      for (int r = 0; r < m.rows; r++)
        for (int i = 0; i < out_dim; i++) o.p[(size_t)r * out_dim + i] = m.p[(size_t)r * in_dim + k * out_dim + i];
      E->emit_fwd(id, k, o);
    }
  }
  void backward(Msg& m, int from) override {
    Part& p = part[key_of(m.s)];
    if (p.g.empty()) p.g.resize(fn_arg);
    p.g[from] = m.p; p.got++; p.rows = m.rows;
    if (p.got < fn_arg) return;
    Msg o; o.s = m.s; o.rows = p.rows; o.dim = in_dim; o.p.resize((size_t)p.rows * in_dim);
    for (int r = 0; r < p.rows; r++)
      for (int k = 0; k < fn_arg; k++)
        for (int i = 0; i < out_dim; i++) o.p[(size_t)r * in_dim + k * out_dim + i] = p.g[k][(size_t)r * out_dim + i];
    part.erase(key_of(m.s));
    E->emit_bwd(id, 0, o);
  }
};

struct GroupInfo { int gkey, member, count; };

struct Group : Node {
  struct Part { std::vector<std::vector<real>> rows; std::vector<State> states; int got = 0; };
  std::map<Key, Part> part;            // forward assembly, keyed on the NEW state
  std::map<Key, std::vector<State>> members;   // original states, restored in the backward phase
  size_t cache_size() const override { return part.size() + members.size(); }
  GroupInfo info(const State& s) const {
    const Structure& S = E->S(s);
    switch (fn) {
      case GROUP_EDGES_BY_TYPE: { int c = S.etype[s.u]; return {c, S.rank_type[s.u], (int)S.type_edges[c].size()}; }
      case GROUP_EDGES_BY_DST: { int v = S.edst[s.u]; return {v, S.rank_in[s.u], (int)S.in_edges[v].size()}; }
      case GROUP_ALL_NODES: return {0, s.u, S.n_pos};
    }
    return {0, 0, 1};
  }
  void forward(Msg& m, int) override {
    GroupInfo gi = info(m.s);
    State os = m.s; os.u = gi.gkey;
    Part& p = part[key_of(os)];
    if (p.rows.empty()) { p.rows.resize(gi.count); p.states.resize(gi.count); }
    p.rows[gi.member] = m.p; p.states[gi.member] = m.s; p.got++;
    if (p.got < gi.count) return;
    Msg o; o.eval = m.eval; o.s = os; o.rows = gi.count; o.dim = in_dim; o.p.resize((size_t)gi.count * in_dim);
    for (int r = 0; r < gi.count; r++)             // member-index order, not arrival order
      for (int i = 0; i < in_dim; i++) o.p[(size_t)r * in_dim + i] = p.rows[r][i];
    if (!m.eval) members[key_of(os)] = p.states;
    part.erase(key_of(os));
    E->emit_fwd(id, 0, o);
  }
  void backward(Msg& m, int) override {
    auto it = members.find(key_of(m.s));
    if (it == members.end()) { E->err = "Group: backward without cached member states"; return; }
    std::vector<State> st = std::move(it->second);
    members.erase(it);
    for (size_t r = 0; r < st.size(); r++) {
      Msg o; o.s = st[r]; o.rows = 1; o.dim = in_dim;
      o.p.assign(m.p.begin() + r * in_dim, m.p.begin() + (r + 1) * in_dim);
      E->emit_bwd(id, 0, o);
    }
  }
};

struct Ungroup : Node {
  struct Orig { State s; int rows; };
  struct Part { std::vector<std::vector<real>> rows; int got = 0; };
  std::map<Key, Orig> orig;
  std::map<Key, Part> part;
  size_t cache_size() const override { return orig.size() + part.size(); }
  int row_u(const State& s, int i) const {
    const Structure& S = E->S(s);
    if (fn == UNGROUP_LEAVES) return S.leaves[i];            // Sec. 6, grouped leaf operations: row i is the tree's i-th leaf
    return fn == UNGROUP_TYPE_EDGES ? S.type_edges[s.u][i] : i;
  }
  std::pair<int, int> inverse(const State& s) const {      // (group u, row)
    const Structure& S = E->S(s);
    if (fn == UNGROUP_TYPE_EDGES) return {S.etype[s.u], S.rank_type[s.u]};
    if (fn == UNGROUP_LEAVES) {
      for (size_t k = 0; k < S.leaves.size(); k++) if (S.leaves[k] == s.u) return {0, (int)k};
      return {0, -1};
    }
    return {0, s.u};
  }
  void forward(Msg& m, int) override {
    if (!m.eval) orig[key_of(m.s)] = Orig{m.s, m.rows};
    for (int r = 0; r < m.rows; r++) {
      Msg o; o.eval = m.eval; o.s = m.s; o.s.u = row_u(m.s, r); o.rows = 1; o.dim = in_dim;
      o.p.assign(m.p.begin() + (size_t)r * in_dim, m.p.begin() + (size_t)(r + 1) * in_dim);
      E->emit_fwd(id, 0, o);
    }
  }
  void backward(Msg& m, int) override {
    auto gr = inverse(m.s);
    State gs = m.s; gs.u = gr.first;
    auto it = orig.find(key_of(gs));
    if (it == orig.end()) { E->err = "Ungroup: backward without cached state"; return; }
    Part& p = part[key_of(gs)];
    if (p.rows.empty()) p.rows.resize(it->second.rows);
    p.rows[gr.second] = m.p; p.got++;
    if (p.got < it->second.rows) return;
    Msg o; o.s = it->second.s; o.rows = it->second.rows; o.dim = in_dim; o.p.resize((size_t)o.rows * in_dim);
    for (int r = 0; r < o.rows; r++)
      for (int i = 0; i < in_dim; i++) o.p[(size_t)r * in_dim + i] = p.rows[r][i];
    part.erase(key_of(gs));
    orig.erase(it);
    E->emit_bwd(id, 0, o);
  }
};

struct Flatmap : Node {
  struct Orig { State s; int count; };
  struct Part { std::vector<std::vector<real>> g; int got = 0; };
  std::map<Key, Orig> orig;            // keyed on the incoming state
  std::map<Key, Part> part;
  size_t cache_size() const override { return orig.size() + part.size(); }
  void forward(Msg& m, int) override {
    const Structure& S = E->S(m.s);
    const std::vector<int>& out = S.out_edges[m.s.u];
    if (!m.eval) orig[key_of(m.s)] = Orig{m.s, (int)out.size()};
    for (int e : out) { Msg o = m; o.s.u = e; E->emit_fwd(id, 0, o); }
  }
  void backward(Msg& m, int) override {
    const Structure& S = E->S(m.s);
    State is = m.s; is.u = S.esrc[m.s.u];
    auto it = orig.find(key_of(is));
    if (it == orig.end()) { E->err = "Flatmap: backward without cached state"; return; }
    Part& p = part[key_of(is)];
    if (p.g.empty()) p.g.resize(it->second.count);
    p.g[S.rank_out[m.s.u]] = m.p; p.got++;
    if (p.got < it->second.count) return;
    Msg o; o.s = it->second.s; o.rows = 1; o.dim = in_dim; o.p.assign(in_dim, 0);
    for (int k = 0; k < it->second.count; k++)      // edge-index order
      for (int i = 0; i < in_dim; i++) o.p[i] += p.g[k][i];
    part.erase(key_of(is));
    orig.erase(it);
    E->round_payload(o);
    E->emit_bwd(id, 0, o);
  }
};

struct SumRows : Node {         // non-parameterised payload transform: sum of the rows
  std::map<Key, int> rows;
  size_t cache_size() const override { return rows.size(); }
  void forward(Msg& m, int) override {
    Msg o; o.eval = m.eval; o.s = m.s; o.rows = 1; o.dim = in_dim; o.p.assign(in_dim, 0);
    for (int r = 0; r < m.rows; r++)
      for (int i = 0; i < in_dim; i++) o.p[i] += m.p[(size_t)r * in_dim + i];
    if (!m.eval) rows[key_of(m.s)] = m.rows;
    E->round_payload(o);
    E->emit_fwd(id, 0, o);
  }
  void backward(Msg& m, int) override {
    auto it = rows.find(key_of(m.s));
    if (it == rows.end()) { E->err = "SumRows: backward without cached row count"; return; }
    int n = it->second;
    rows.erase(it);
    Msg o; o.s = m.s; o.rows = n; o.dim = in_dim; o.p.resize((size_t)n * in_dim);
    for (int r = 0; r < n; r++) for (int i = 0; i < in_dim; i++) o.p[(size_t)r * in_dim + i] = m.p[i];
    E->emit_bwd(id, 0, o);
  }
};

// LSTM gate combination (Sec. 6: the Tree-LSTM is split into a leaf and a branch cell).  Parameter-free: the gate
// pre-activations come from an ordinary Linear node on port 0, the children's cell states [cL; cR] on port 1 (branch).
//   leaf:   i = s(pi), o = s(po), u = tanh(pu);                 c = i u;                 h = o tanh(c)
//   branch: i, fL, fR, o = s(.), u = tanh(pu);                  c = i u + fL cL + fR cR;  h = o tanh(c)
// Output payload [h; c]; H = out_dim / 2.  The inputs are cached keyed on the state for the backward pass.
struct LstmGate : Node {
  struct In { std::vector<real> pre, cells; int got = 0; };
  std::map<Key, In> in;
  size_t cache_size() const override { return in.size(); }
  static real sg(real x) { return (real)1 / ((real)1 + std::exp(-x)); }
  void forward(Msg& m, int port) override {
    const int H = out_dim / 2, need = fn == LSTM_BRANCH ? 2 : 1;
    In& c = in[key_of(m.s)];
    if (port == 0) c.pre = m.p; else c.cells = m.p;
    if (++c.got < need) return;
    Msg o; o.eval = m.eval; o.s = m.s; o.rows = 1; o.dim = out_dim; o.p.assign(out_dim, 0);
    for (int j = 0; j < H; j++) {
      real cj, oj;
      if (fn == LSTM_LEAF) { cj = sg(c.pre[j]) * std::tanh(c.pre[2 * H + j]); oj = sg(c.pre[H + j]); }
      else {
        cj = sg(c.pre[j]) * std::tanh(c.pre[4 * H + j]) + sg(c.pre[H + j]) * c.cells[j] + sg(c.pre[2 * H + j]) * c.cells[H + j];
        oj = sg(c.pre[3 * H + j]);
      }
      o.p[j] = oj * std::tanh(cj);
      o.p[H + j] = cj;
    }
    if (m.eval) in.erase(key_of(m.s)); else c.got = 0;
    E->round_payload(o);
    E->emit_fwd(id, 0, o);
  }
  void backward(Msg& m, int) override {
    const int H = out_dim / 2;
    auto it = in.find(key_of(m.s));
    if (it == in.end()) { E->err = "LstmGate: backward without cached inputs"; return; }
    const In c = it->second;
    in.erase(it);
    Msg dp; dp.s = m.s; dp.rows = 1; dp.dim = in_dim; dp.p.assign(in_dim, 0);
    Msg dc; dc.s = m.s; dc.rows = 1; dc.dim = out_dim; dc.p.assign(out_dim, 0);
    for (int j = 0; j < H; j++) {
      const real gh = m.p[j], gc = m.p[H + j];
      if (fn == LSTM_LEAF) {
        const real i = sg(c.pre[j]), o = sg(c.pre[H + j]), u = std::tanh(c.pre[2 * H + j]);
        const real cj = i * u, tc = std::tanh(cj), d = gc + gh * o * (1 - tc * tc);
        dp.p[j] = d * u * i * (1 - i);
        dp.p[H + j] = gh * tc * o * (1 - o);
        dp.p[2 * H + j] = d * i * (1 - u * u);
      } else {
        const real i = sg(c.pre[j]), fl = sg(c.pre[H + j]), fr = sg(c.pre[2 * H + j]), o = sg(c.pre[3 * H + j]), u = std::tanh(c.pre[4 * H + j]);
        const real cl = c.cells[j], cr = c.cells[H + j];
        const real cj = i * u + fl * cl + fr * cr, tc = std::tanh(cj), d = gc + gh * o * (1 - tc * tc);
        dp.p[j] = d * u * i * (1 - i);
        dp.p[H + j] = d * cl * fl * (1 - fl);
        dp.p[2 * H + j] = d * cr * fr * (1 - fr);
        dp.p[3 * H + j] = gh * tc * o * (1 - o);
        dp.p[4 * H + j] = d * i * (1 - u * u);
        dc.p[j] = d * fl;
        dc.p[H + j] = d * fr;
      }
    }
    E->round_payload(dp);
    E->emit_bwd(id, 0, dp);
    if (fn == LSTM_BRANCH) { E->round_payload(dc); E->emit_bwd(id, 1, dc); }
  }
};

struct SourceNode : Node {
  void forward(Msg&, int) override {}
  void backward(Msg&, int) override {}
};

// ------------------------------------------------------------------------------------------------
// Controller loop + canonical round schedule
// ------------------------------------------------------------------------------------------------
struct KeyLogEntry { int64_t inst; int slot; int64_t admit, release; };

struct RunStats {
  int64_t instances, node_messages, ppt_messages, rounds;
  double seconds, mean_loss;
  int32_t max_staleness;
  int64_t max_active_observed;
  uint64_t route_hash;
  int64_t leftover_cache_entries;
};

struct Oracle {
  Engine E;
  std::vector<KeyLogEntry> key_log;

  int pump_sources(int inst, int seq, int slot, bool eval) {    // returns #source messages emitted
    const Structure& S = E.cur->inst[inst];
    int emitted = 0;
    for (auto& np : E.nodes) {
      Node* n = np.get();
      if (n->type != SOURCE) continue;
      auto send = [&](int u, int rows, int dim, std::vector<real> payload) {
        Msg m; m.eval = eval; m.s.inst = inst; m.s.seq = seq; m.s.slot = slot; m.s.u = u;
        m.rows = rows; m.dim = dim; m.p = std::move(payload);
        E.emit_fwd(n->id, 0, m);
        emitted++;
      };
      switch (n->fn) {
        case SRC_DENSE_ROW: {
          std::vector<real> x(E.cur->dense_dim);
          for (int i = 0; i < E.cur->dense_dim; i++) x[i] = (real)S.dense[i];
          send(0, 1, E.cur->dense_dim, x);
        } break;
        case SRC_TOKENS:
          for (int t = 0; t < S.n_pos; t++) send(t, 1, 1, std::vector<real>(1, (real)S.tokens[t]));
          break;
        case SRC_ZERO_STATE: send(0, 1, n->out_dim, std::vector<real>(n->out_dim, 0)); break;
        case SRC_TREE_LEAVES:
          for (int u : S.leaves) send(u, 1, 1, std::vector<real>(1, (real)S.tokens[u]));
          break;
        case SRC_GRAPH_NODES: {
          std::vector<real> ids(S.n_pos);
          for (int v = 0; v < S.n_pos; v++) ids[v] = (real)S.tokens[v];
          send(0, S.n_pos, 1, ids);
        } break;
        case SRC_TREE_LEAVES_GROUPED: {                      // one matrix message: the leaves' tokens in leaf order
          std::vector<real> ids(S.leaves.size());
          for (size_t k = 0; k < S.leaves.size(); k++) ids[k] = (real)S.tokens[S.leaves[k]];
          send(0, (int)S.leaves.size(), 1, ids);
        } break;
        default: E.err = "Source: unknown fn";
      }
    }
    return emitted;
  }

  void process_ppt_inboxes(std::vector<std::vector<Msg>>& cur) {
    for (size_t i = 0; i < cur.size(); i++) {
      auto& box = cur[i];
      if (box.empty()) continue;
      std::stable_sort(box.begin(), box.end(), [](const Msg& a, const Msg& b) {
        return std::make_tuple(-a.dir, a.s.seq, a.s.it, a.s.u, a.s.port) <
               std::make_tuple(-b.dir, b.s.seq, b.s.it, b.s.u, b.s.port);
      });
      Node* n = E.nodes[i].get();
      for (auto& m : box) {
        E.ppt_messages++;
        if (m.dir == FWD) n->forward(m, 0); else n->backward(m, 0);
        if (m.eval && !E.inflight_eval.empty()) E.inflight_eval[m.s.slot]--;      // after its successors were emitted
      }
      box.clear();
    }
  }
  static bool all_empty(const std::vector<std::vector<Msg>>& v) {
    for (auto& b : v) if (!b.empty()) return false;
    return true;
  }

  // inference_only (may be null): per instance, != 0 marks an instance that is only evaluated (forward messages, nothing
  // cached, no gradients) while the others train: concurrent inference in the same queues (Sec. 1, Sec. 6).  Such an
  // instance is finished, and its key released in the next round, once none of its messages is left anywhere.
  int run_epoch(int split, int mak, int muf, double lr, const int64_t* order, int64_t n_order, int flush,
                RunStats* out, double* per_instance_loss, const uint8_t* inference_only = nullptr, double* inf_out = nullptr) {
    E.cur = &E.data[split];
    const int64_t n_inst = (int64_t)E.cur->inst.size();
    E.mak = mak; E.muf = muf; E.lr = (real)lr; E.err.clear();
    E.inbox_a.assign(E.nodes.size(), {}); E.inbox_b.assign(E.nodes.size(), {});
    E.retire_notices.clear();
    E.loss.assign(n_inst, 0); E.correct.assign(n_inst, 0); E.n_pred.assign(n_inst, 0);
    E.node_messages = E.ppt_messages = 0; E.route_hash = 0;
    for (auto& n : E.nodes) { n->reset_run(); n->st = NodeStats(); }
    key_log.clear();
    std::vector<int> slot_inst(mak, -1), outstanding(mak, 0), slot_log(mak, -1);
    std::vector<char> slot_eval(mak, 0);
    E.inflight_eval.assign(inference_only ? mak : 0, 0);
    int active = 0; int64_t next = 0, max_active = 0, r = 0;
    auto* cur = &E.inbox_a; auto* nxt = &E.inbox_b;
    for (;; r++) {
      // (1) controller: retirements of the previous round, then admission
      for (int slot : E.retire_notices)
        if (--outstanding[slot] == 0) {
          key_log[slot_log[slot]].release = r;
          slot_inst[slot] = -1; active--;
        }
      E.retire_notices.clear();
      E.target = cur;
      while (active < mak && next < n_order) {
        int slot = 0;
        while (slot_inst[slot] >= 0) slot++;              // lowest free slot
        int inst = (int)order[next];
        slot_inst[slot] = inst; active++;
        slot_log[slot] = (int)key_log.size();
        key_log.push_back(KeyLogEntry{inst, slot, r, -1});
        slot_eval[slot] = inference_only && inference_only[inst];
        outstanding[slot] = pump_sources(inst, (int)next, slot, slot_eval[slot] != 0);
        if (slot_eval[slot]) outstanding[slot] = 1;            // one notice: "nothing of this instance is left"
        next++;
      }
      max_active = std::max<int64_t>(max_active, active);
      if (next == n_order && active == 0 && all_empty(*cur)) break;
      if (!E.err.empty()) return 1;
      // (2) every PPT node processes its inbox of this round; emissions land in the next round's inboxes
      E.target = nxt;
      process_ppt_inboxes(*cur);
      std::swap(cur, nxt);
      for (int sl = 0; sl < mak && inference_only; sl++)
        if (slot_inst[sl] >= 0 && slot_eval[sl] && outstanding[sl] == 1 && E.inflight_eval[sl] == 0) E.retire_notices.push_back(sl);
      if (!E.err.empty()) return 1;
      if (r > (int64_t)4e9) { E.err = "schedule did not terminate"; return 1; }
    }
    if (flush) for (auto& n : E.nodes) n->flush();
    int64_t leftover = 0;
    int max_stale = 0;
    for (auto& n : E.nodes) { leftover += (int64_t)n->cache_size(); max_stale = std::max(max_stale, n->st.max_staleness); }
    double tot = 0, itot = 0; int64_t n_train = 0, n_inf = 0, ic = 0, ip = 0;
    for (int64_t i = 0; i < n_order; i++) {
      const int64_t k = order[i];
      if (inference_only && inference_only[k]) { itot += E.loss[k]; n_inf++; ic += E.correct[k]; ip += E.n_pred[k]; }
      else { tot += E.loss[k]; n_train++; }
    }
    if (inf_out) { inf_out[0] = (double)n_inf; inf_out[1] = n_inf ? itot / n_inf : 0; inf_out[2] = ip ? (double)ic / (double)ip : 0; }
    if (per_instance_loss) for (int64_t i = 0; i < n_inst; i++) per_instance_loss[i] = E.loss[i];
    if (out) {
      out->instances = n_order; out->node_messages = E.node_messages; out->ppt_messages = E.ppt_messages;
      out->rounds = r + 1; out->seconds = 0; out->mean_loss = n_train ? tot / n_train : 0;
      out->max_staleness = max_stale; out->max_active_observed = max_active; out->route_hash = E.route_hash;
      out->leftover_cache_entries = leftover;
    }
    return 0;
  }

  // Forward-only pass over a split, one instance at a time, nothing cached.
  int eval(int split, double* mean_loss, double* accuracy, double* per_instance_loss) {
    E.cur = &E.data[split];
    const int64_t n_inst = (int64_t)E.cur->inst.size();
    E.err.clear();
    E.inbox_a.assign(E.nodes.size(), {}); E.inbox_b.assign(E.nodes.size(), {});
    E.loss.assign(n_inst, 0); E.correct.assign(n_inst, 0); E.n_pred.assign(n_inst, 0);
    E.inflight_eval.clear();
    auto* cur = &E.inbox_a; auto* nxt = &E.inbox_b;
    for (int64_t i = 0; i < n_inst; i++) {
      E.target = cur;
      pump_sources((int)i, (int)i, 0, true);
      while (!all_empty(*cur)) {
        E.target = nxt;
        process_ppt_inboxes(*cur);
        std::swap(cur, nxt);
        if (!E.err.empty()) return 1;
      }
    }
    double tot = 0; int64_t c = 0, p = 0;
    for (int64_t i = 0; i < n_inst; i++) { tot += E.loss[i]; c += E.correct[i]; p += E.n_pred[i]; }
    if (mean_loss) *mean_loss = n_inst ? tot / n_inst : 0;
    if (accuracy) *accuracy = p ? (double)c / (double)p : 0;
    if (per_instance_loss) for (int64_t i = 0; i < n_inst; i++) per_instance_loss[i] = E.loss[i];
    return 0;
  }
};

template <class T> static Node* make(Engine* E) { T* t = new T(); t->E = E; return t; }

}  // namespace

// ------------------------------------------------------------------------------------------------
// C interface (ctypes)
// ------------------------------------------------------------------------------------------------
extern "C" {

typedef RunStats oracle_stats_t;

int oracle_real_bytes() { return (int)sizeof(real); }

void* oracle_create(const int32_t* nodes, int n_nodes, const int32_t* edges, int n_edges, int payload_bf16) {
  Oracle* O = new Oracle();
  Engine& E = O->E;
  E.bf16 = payload_bf16 != 0;
  for (int i = 0; i < n_nodes; i++) {
    const int32_t* d = nodes + 8 * i;
    Node* n = nullptr;
    switch (d[0]) {
      case SOURCE: n = make<SourceNode>(&E); break;
      case LINEAR: n = make<Linear>(&E); break;
      case LOOKUP: n = make<Lookup>(&E); break;
      case GRUCELL: n = make<GRUCell>(&E); break;
      case LOSS_CE: case LOSS_MSE: n = make<Loss>(&E); break;
      case NPT_SUMROWS: n = make<SumRows>(&E); break;
      case NPT_LSTM: n = make<LstmGate>(&E); break;
      case COND: n = make<Cond>(&E); break;
      case PHI: n = make<Phi>(&E); break;
      case ISU: n = make<Isu>(&E); break;
      case CONCAT: n = make<Concat>(&E); break;
      case SPLIT: n = make<Split>(&E); break;
      case BCAST: n = make<Bcast>(&E); break;
      case GROUP: n = make<Group>(&E); break;
      case UNGROUP: n = make<Ungroup>(&E); break;
      case FLATMAP: n = make<Flatmap>(&E); break;
      case SINK: n = make<Sink>(&E); break;
      default: delete O; return nullptr;
    }
    n->id = i; n->type = d[0]; n->in_dim = d[1]; n->out_dim = d[2]; n->act = d[3]; n->fn = d[4]; n->fn_arg = d[5];
    n->muf_override = d[6]; n->flags = d[7];
    if (n->type == LINEAR) static_cast<Linear*>(n)->init();
    if (n->type == LOOKUP) static_cast<Lookup*>(n)->init();
    if (n->type == GRUCELL) static_cast<GRUCell*>(n)->init();
    E.nodes.emplace_back(n);
  }
  E.succ.assign(n_nodes, {}); E.pred.assign(n_nodes, {});
  for (int k = 0; k < n_edges; k++) {
    const int32_t* e = edges + 4 * k;
    int s = e[0], sp = e[1], d = e[2], dp = e[3];
    if (s < 0 || s >= n_nodes || d < 0 || d >= n_nodes || sp < 0 || dp < 0) { delete O; return nullptr; }
    if ((int)E.succ[s].size() <= sp) E.succ[s].resize(sp + 1, {-1, -1});
    if ((int)E.pred[d].size() <= dp) E.pred[d].resize(dp + 1, {-1, -1});
    E.succ[s][sp] = {d, dp};
    E.pred[d][dp] = {s, sp};
  }
  return O;
}

void oracle_destroy(void* h) { delete static_cast<Oracle*>(h); }

const char* oracle_last_error(void* h) { return static_cast<Oracle*>(h)->E.err.c_str(); }

int oracle_load_instances(void* h, int split, int kind, int64_t n, const int64_t* offsets, const int32_t* tokens,
                          const int32_t* left, const int32_t* right, const int64_t* edge_offsets,
                          const int32_t* esrc, const int32_t* edst, const int32_t* etype, const float* dense,
                          int dense_dim, const int32_t* labels_i, const float* labels_f) {
  Oracle* O = static_cast<Oracle*>(h);
  Dataset& D = O->E.data[split];
  D = Dataset();
  D.kind = kind; D.dense_dim = dense_dim;
  if (dense) D.dense.assign(dense, dense + (size_t)n * dense_dim);
  D.inst.resize(n);
  for (int64_t i = 0; i < n; i++) {
    Structure& S = D.inst[i];
    if (kind == KIND_DENSE_ROWS) {
      S.n_pos = 1; S.dense = D.dense.data() + (size_t)i * dense_dim;
      if (labels_i) S.labels.assign(1, labels_i[i]);
      if (labels_f) S.target = labels_f[i];
      continue;
    }
    int64_t o = offsets[i];
    S.n_pos = (int)(offsets[i + 1] - o);
    S.tokens.assign(tokens + o, tokens + o + S.n_pos);
    if (kind == KIND_SEQUENCES) {
      if (labels_i) S.labels.assign(1, labels_i[i]);
    } else if (kind == KIND_BINARY_TREES) {
      S.left.assign(left + o, left + o + S.n_pos);
      S.right.assign(right + o, right + o + S.n_pos);
      S.parent.assign(S.n_pos, -1); S.child_slot.assign(S.n_pos, 0);
      for (int u = 0; u < S.n_pos; u++) {
        if (S.left[u] >= 0) { S.parent[S.left[u]] = u; S.child_slot[S.left[u]] = 0;
                              S.parent[S.right[u]] = u; S.child_slot[S.right[u]] = 1; }
        else S.leaves.push_back(u);
      }
      for (int u = 0; u < S.n_pos; u++) if (S.parent[u] < 0) S.root = u;
      if (labels_i) S.labels.assign(labels_i + o, labels_i + o + S.n_pos);
    } else if (kind == KIND_TYPED_GRAPHS) {
      int64_t eo = edge_offsets[i]; int ne = (int)(edge_offsets[i + 1] - eo);
      S.esrc.assign(esrc + eo, esrc + eo + ne); S.edst.assign(edst + eo, edst + eo + ne);
      S.etype.assign(etype + eo, etype + eo + ne);
      S.out_edges.assign(S.n_pos, {}); S.in_edges.assign(S.n_pos, {});
      int nt = 0;
      for (int e = 0; e < ne; e++) nt = std::max(nt, S.etype[e] + 1);
      S.type_edges.assign(std::max(nt, 1), {});
      S.rank_out.resize(ne); S.rank_in.resize(ne); S.rank_type.resize(ne);
      for (int e = 0; e < ne; e++) {
        S.rank_out[e] = (int)S.out_edges[S.esrc[e]].size(); S.out_edges[S.esrc[e]].push_back(e);
        S.rank_in[e] = (int)S.in_edges[S.edst[e]].size(); S.in_edges[S.edst[e]].push_back(e);
        S.rank_type[e] = (int)S.type_edges[S.etype[e]].size(); S.type_edges[S.etype[e]].push_back(e);
      }
      if (labels_f) S.target = labels_f[i];
      if (labels_i) S.labels.assign(1, labels_i[i]);
    }
  }
  return 0;
}

int64_t oracle_param_count(void* h, int node, int which) {
  Oracle* O = static_cast<Oracle*>(h);
  if (node < 0 || node >= (int)O->E.nodes.size()) return -1;
  auto* p = O->E.nodes[node]->param(which);
  return p ? (int64_t)p->size() : -1;
}
int oracle_set_params(void* h, int node, int which, const double* src, int64_t n) {
  auto* p = static_cast<Oracle*>(h)->E.nodes[node]->param(which);
  if (!p || (int64_t)p->size() != n) return 1;
  for (int64_t i = 0; i < n; i++) (*p)[i] = (real)src[i];
  return 0;
}
int oracle_get_params(void* h, int node, int which, double* dst, int64_t n) {
  auto* p = static_cast<Oracle*>(h)->E.nodes[node]->param(which);
  if (!p || (int64_t)p->size() != n) return 1;
  for (int64_t i = 0; i < n; i++) dst[i] = (double)(*p)[i];
  return 0;
}
int oracle_get_accum(void* h, int node, int which, double* dst, int64_t n) {
  auto* p = static_cast<Oracle*>(h)->E.nodes[node]->accum(which);
  if (!p || (int64_t)p->size() != n) return 1;
  for (int64_t i = 0; i < n; i++) dst[i] = (double)(*p)[i];
  return 0;
}

int oracle_run_epoch(void* h, int split, int mak, int muf, double lr, const int64_t* order, int64_t n_order,
                     int flush, oracle_stats_t* out, double* per_instance_loss) {
  if (mak < 1 || muf < 1) return 1;
  return static_cast<Oracle*>(h)->run_epoch(split, mak, muf, lr, order, n_order, flush, out, per_instance_loss);
}

// inf_out: {inference instances, their mean loss, their accuracy}
int oracle_run_epoch_mixed(void* h, int split, int mak, int muf, double lr, const int64_t* order, int64_t n_order,
                           int flush, const uint8_t* inference_only, oracle_stats_t* out, double* per_instance_loss, double* inf_out) {
  if (mak < 1 || muf < 1) return 1;
  return static_cast<Oracle*>(h)->run_epoch(split, mak, muf, lr, order, n_order, flush, out, per_instance_loss, inference_only, inf_out);
}

// kind: 0 SGD, 1 momentum-SGD (v <- mu v + g, theta -= lr v), 2 Adam (bias-corrected); state is kept across epochs.
int oracle_set_optimizer(void* h, int kind, double mu, double beta1, double beta2, double eps, int reset_state) {
  Oracle* O = static_cast<Oracle*>(h);
  if (kind < 0 || kind > 2) return 1;
  O->E.opt = kind; O->E.mu = (real)mu; O->E.beta1 = (real)beta1; O->E.beta2 = (real)beta2; O->E.eps = (real)eps;
  if (reset_state)
    for (auto& n : O->E.nodes) if (n->is_ppt()) static_cast<PPTBase*>(n.get())->reset_optimizer();
  return 0;
}

int oracle_eval(void* h, int split, double* mean_loss, double* accuracy, double* per_instance_loss) {
  return static_cast<Oracle*>(h)->eval(split, mean_loss, accuracy, per_instance_loss);
}

int oracle_get_node_stats(void* h, int node, int64_t* n_updates, int64_t* n_grads_applied, int64_t* stale_hist,
                          int64_t* fwd_msgs, int64_t* bwd_msgs) {
  Oracle* O = static_cast<Oracle*>(h);
  if (node < 0 || node >= (int)O->E.nodes.size()) return 1;
  const NodeStats& s = O->E.nodes[node]->st;
  if (n_updates) *n_updates = s.n_updates;
  if (n_grads_applied) *n_grads_applied = s.n_grads_applied;
  if (stale_hist) std::memcpy(stale_hist, s.stale_hist, sizeof(s.stale_hist));
  if (fwd_msgs) *fwd_msgs = s.fwd_msgs;
  if (bwd_msgs) *bwd_msgs = s.bwd_msgs;
  return 0;
}

int64_t oracle_get_update_log(void* h, int node, int32_t* n_per_update, int64_t cap) {
  const NodeStats& s = static_cast<Oracle*>(h)->E.nodes[node]->st;
  int64_t n = (int64_t)s.update_log.size();
  for (int64_t i = 0; i < std::min(n, cap); i++) n_per_update[i] = s.update_log[i];
  return n;
}

int64_t oracle_get_key_log(void* h, int64_t* inst, int32_t* slot, int64_t* admit, int64_t* release, int64_t cap) {
  Oracle* O = static_cast<Oracle*>(h);
  int64_t n = (int64_t)O->key_log.size();
  for (int64_t i = 0; i < std::min(n, cap); i++) {
    inst[i] = O->key_log[i].inst; slot[i] = O->key_log[i].slot;
    admit[i] = O->key_log[i].admit; release[i] = O->key_log[i].release;
  }
  return n;
}

// The bf16 rounding applied to emitted payloads, exposed so that a test can pin it against an independent conversion.
void oracle_round_bf16(const double* in, double* out, int64_t n) {
  for (int64_t i = 0; i < n; i++) out[i] = (double)round_bf16((real)in[i]);
}

}  // extern "C"
