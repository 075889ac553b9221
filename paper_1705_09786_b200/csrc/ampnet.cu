// Host side of the AMPNet engine: the C ABI of include/ampnet.h.
//   * IR builder checks and placement of the parameterised nodes on CTAs ("scheduler on the host"),
//   * structure encoder: trees / graphs / lists -> routing tables in device memory,
//   * key-space inference, allocation of queues and keyed caches, kernel launch, statistics.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <string>
#include <vector>

#include "../../include/ampnet.h"
#include "engine.cuh"

using namespace amp;

// host hooks of the direct-delivery engine (engine_fast.cu)
extern "C" int ampnet_direct_threads();
extern "C" size_t ampnet_direct_tile_smem_bytes(int in_dim, int rows, int batch_rows, int loss_head);
extern "C" size_t ampnet_direct_bwd_tile_smem_bytes(int out_dim, int cols, int batch_rows);
extern "C" size_t ampnet_direct_tc_tile_smem_bytes(int in_dim, int batch_rows);
extern "C" void ampnet_direct_tc_limits(int* rows, int* max_batch_rows, int* k_multiple);
extern "C" int ampnet_direct_max_units();
extern "C" void ampnet_direct_limits(int* max_nodes, int* max_ppts, int* max_landings, int* batch_rows);
extern "C" cudaError_t ampnet_direct_static_smem(size_t* bytes);
extern "C" cudaError_t ampnet_direct_launch(const amp::Ctx* ctx, int n_ctas, size_t smem_bytes, cudaStream_t stream, int n_sms);

namespace {

struct DeviceArena {           // one allocation carved into aligned pieces
  char* base = nullptr;
  size_t size = 0, used = 0;
  template <class T> T* take(size_t n) {
    used = (used + 255) & ~(size_t)255;
    T* p = base ? reinterpret_cast<T*>(base + used) : nullptr;
    used += n * sizeof(T);
    return p;
  }
};

struct HostDataset {
  bool loaded = false;
  int kind = -1, dense_dim = 0, NT = 1, labels_per_node = 0;
  long long n = 0;
  int maxT = 1, maxM = 1, maxN = 1, maxD = 1, maxDc = 1, maxIn = 1, maxOut = 1, maxL = 1;
  long long total_pos = 0, total_edges = 0;
  DevInst dev{};
  std::vector<void*> allocs;
};

struct HostPPT {
  int node = 0, kind = 0, in = 0, out = 0, nmat = 1;
  float *W = nullptr, *b = nullptr;
  float *om = nullptr, *ov = nullptr;   // optimiser moments (nW + nb floats each), allocated by ampnet_set_optimizer
  long long opt_t = 0;                  // updates applied since the optimiser state was reset
  size_t nW = 0, nb = 0;
  int T = 1, R = 0, BM = 0, J = 0;
  int NE = 0, G = 1;                    // emitter CTAs of the node and their batch groups
  bool a_global = false;                // the tiles' gradient accumulators live in device memory (frees shared memory for staging rows)
  int xwt_rb = 8;                       // output rows per pass of X.W^T: 16 where the larger scratch still fits
  int TB = 0, CB = 0, NS = 1;           // direct-delivery engine: backward column tiles, columns per tile, gradient slots per key
  int tc = 0;                           // direct-delivery engine: forward tiles of 64 rows on the tensor cores (bf16 runs)
  int LT = 1;                           // direct-delivery engine: tiles that share the messages of a node that feeds a Loss
  size_t bwd_smem_floats = 0;
  double emit_load = 0.0;               // emitter-seconds the node's emission took in the last asynchronous epoch (0: unknown)
  size_t smem_floats = 0;
};

}  // namespace

struct ampnet_graph {
  std::vector<ampnet_node_desc_t> nodes;
  std::vector<ampnet_edge_desc_t> edges;
  std::vector<DevNode> hnodes;        // topology filled at creation, storage at run time
  std::vector<HostPPT> ppts;
  std::vector<int> sources, losses;
  bool has_it = false; int it_steps = 0;
  bool payload_bf16 = false;
  int opt = 0; float opt_mu = 0.9f, opt_beta1 = 0.9f, opt_beta2 = 0.999f, opt_eps = 1e-8f;
  ampnet_allocator_t alloc{};
  cudaStream_t stream = nullptr;
  int device = 0, n_sms = 0, max_smem = 0;
  HostDataset data[2];
  std::string err;
  // run state
  DeviceArena ctl, bulk;
  void *ctl_mem = nullptr, *bulk_mem = nullptr;
  size_t ctl_cap = 0, bulk_cap = 0;
  // A control arena of under 1 MiB is tried at two positions 1 MiB apart during the first asynchronous epochs and stays
  // at the faster one: which half of the L2 a line is homed in depends on its address, the hot lines of a small arena
  // all move together with it, and the list workload runs 38 k or 25 k instances/s depending on where they fall.
  void* ctl_alloc = nullptr;
  char* ctl_cand[2] = {nullptr, nullptr};
  int ctl_trials = 0, ctl_choice = -1;
  double ctl_rate[2] = {0.0, 0.0};
  std::vector<std::pair<size_t, size_t>> leftover_regions;   // (offset, bytes) inside ctl
  std::vector<std::pair<void*, size_t>> zero_regions;        // parts of the bulk arena that must start a run at zero
  std::vector<PPTStats*> d_stats;
  std::vector<int*> d_update_log;
  unsigned long long* d_node_msgs = nullptr;
  KeyLog* d_keylog = nullptr;
  long long n_keylog = 0;
  int update_log_cap = 1 << 20;
  std::vector<PPTStats> last_stats;
  std::vector<unsigned long long> last_node_msgs;
  bool have_run = false;
  bool arenas_lent = false;           // the arenas belong to the caller of execute() (static scratch): never freed or grown
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
};

// FP32 FMA issue rate of the device, measured: every thread runs 16 independent FMA chains from registers.
__global__ void __launch_bounds__(256) fma_peak_kernel(float* sink, int iters) {
  float a[16];
#pragma unroll
  for (int k = 0; k < 16; k++) a[k] = 1.0f + 1e-3f * (float)(threadIdx.x + k);
  const float m = 1.0000001f, c = 1e-7f;
  for (int i = 0; i < iters; i++) {
#pragma unroll
    for (int k = 0; k < 16; k++) a[k] = fmaf(a[k], m, c);
  }
  float s = 0.f;
#pragma unroll
  for (int k = 0; k < 16; k++) s += a[k];
  if (s == 12345.678f) sink[0] = s;          // keeps the chains alive
}

// End-of-epoch replica synchronisation (Sec. 5): element-wise mean of up to eight nodes' parameters, written back to all.
struct AvgArgs { float* W[8]; float* b[8]; int n; long long nW, nb; };
__global__ void average_params_kernel(const AvgArgs a) {
  const long long total = a.nW + a.nb, stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    float* const* arr = i < a.nW ? a.W : a.b;
    const long long j = i < a.nW ? i : i - a.nW;
    float s = 0.f;
    for (int k = 0; k < a.n; k++) s += arr[k][j];
    s /= (float)a.n;
    for (int k = 0; k < a.n; k++) arr[k][j] = s;
  }
}

namespace {

ampnet_status_t set_err(ampnet_graph* g, ampnet_status_t st, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (g) g->err = buf;
  return st;
}

#define CUDA_TRY(g, call)                                                                                  \
  do {                                                                                                     \
    cudaError_t e_ = (call);                                                                               \
    if (e_ != cudaSuccess) return set_err(g, AMPNET_ECUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

void* dev_alloc(ampnet_graph* g, size_t bytes) {
  if (bytes == 0) bytes = 256;
  if (g->alloc.alloc) return g->alloc.alloc(g->alloc.ctx, bytes);
  void* p = nullptr;
  if (cudaMalloc(&p, bytes) != cudaSuccess) return nullptr;
  return p;
}
void dev_free(ampnet_graph* g, void* p) {
  if (!p) return;
  if (g->alloc.free) g->alloc.free(g->alloc.ctx, p);
  else if (!g->alloc.alloc) cudaFree(p);
}

bool is_ppt_type(int t) { return t == LINEAR || t == LOOKUP || t == GRUCELL; }

uint64_t splitmix(uint64_t& s) {
  uint64_t z = (s += 0x9E3779B97F4A7C15ull);
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
double uniform01(uint64_t& s) { return (double)(splitmix(s) >> 11) * (1.0 / 9007199254740992.0); }

int j_bucket(int in) {
  const int j = (in + 31) / 32;
  const int b[] = {4, 7, 10, 16, 25, 32};
  for (int v : b) if (j <= v) return v;
  return -1;
}

template <class T>
ampnet_status_t upload(ampnet_graph* g, HostDataset& D, const std::vector<T>& h, const T** out) {
  void* p = dev_alloc(g, std::max<size_t>(h.size(), 1) * sizeof(T));
  if (!p) return set_err(g, AMPNET_ENOMEM, "device allocation of %zu bytes failed", h.size() * sizeof(T));
  D.allocs.push_back(p);
  if (!h.empty()) CUDA_TRY(g, cudaMemcpyAsync(p, h.data(), h.size() * sizeof(T), cudaMemcpyHostToDevice, g->stream));
  *out = reinterpret_cast<const T*>(p);
  return AMPNET_OK;
}
template <class T>
ampnet_status_t upload_raw(ampnet_graph* g, HostDataset& D, const T* h, size_t n, const T** out) {
  void* p = dev_alloc(g, std::max<size_t>(n, 1) * sizeof(T));
  if (!p) return set_err(g, AMPNET_ENOMEM, "device allocation of %zu bytes failed", n * sizeof(T));
  D.allocs.push_back(p);
  if (n) CUDA_TRY(g, cudaMemcpyAsync(p, h, n * sizeof(T), cudaMemcpyHostToDevice, g->stream));
  *out = reinterpret_cast<const T*>(p);
  return AMPNET_OK;
}

void free_dataset(ampnet_graph* g, HostDataset& D) {
  for (void* p : D.allocs) dev_free(g, p);
  D = HostDataset();
}

// ---- IR checks ---------------------------------------------------------------------------------------
ampnet_status_t build_topology(ampnet_graph* g) {
  const int n = (int)g->nodes.size();
  g->hnodes.assign(n, DevNode{});
  for (int i = 0; i < n; i++) {
    const auto& d = g->nodes[i];
    if (d.type < 0 || d.type >= N_NODE_TYPES) return set_err(g, AMPNET_EINVAL, "node %d: unknown type %d", i, d.type);
    if (d.in_dim < 0 || d.out_dim < 0) return set_err(g, AMPNET_EINVAL, "node %d: negative dimension", i);
    DevNode& h = g->hnodes[i];
    h.type = d.type; h.in_dim = d.in_dim; h.out_dim = d.out_dim; h.act = d.act; h.fn = d.fn; h.fn_arg = d.fn_arg;
    h.flags = d.flags; h.ppt = -1;
    for (int k = 0; k < MAX_PORTS; k++) h.succ_node[k] = h.pred_node[k] = h.succ_port[k] = h.pred_port[k] = -1;
    if (d.act < 0 || d.act > 3) return set_err(g, AMPNET_EINVAL, "node %d: unknown activation %d", i, d.act);
  }
  for (size_t k = 0; k < g->edges.size(); k++) {
    const auto& e = g->edges[k];
    if (e.src_node < 0 || e.src_node >= n || e.dst_node < 0 || e.dst_node >= n)
      return set_err(g, AMPNET_EINVAL, "edge %zu: node index out of range", k);
    if (e.src_port < 0 || e.src_port >= MAX_PORTS || e.dst_port < 0 || e.dst_port >= MAX_PORTS)
      return set_err(g, AMPNET_EINVAL, "edge %zu: port out of range (max %d)", k, MAX_PORTS);
    DevNode &s = g->hnodes[e.src_node], &d = g->hnodes[e.dst_node];
    if (s.succ_node[e.src_port] >= 0) return set_err(g, AMPNET_EINVAL, "edge %zu: source port used twice", k);
    if (d.pred_node[e.dst_port] >= 0) return set_err(g, AMPNET_EINVAL, "edge %zu: destination port used twice", k);
    s.succ_node[e.src_port] = e.dst_node; s.succ_port[e.src_port] = e.dst_port;
    d.pred_node[e.dst_port] = e.src_node; d.pred_port[e.dst_port] = e.src_port;
    s.n_succ = std::max(s.n_succ, e.src_port + 1);
    d.n_pred = std::max(d.n_pred, e.dst_port + 1);
  }
  for (int i = 0; i < n; i++) {
    DevNode& h = g->hnodes[i];
    for (int k = 0; k < h.n_succ; k++) if (h.succ_node[k] < 0) return set_err(g, AMPNET_EINVAL, "node %d: successor port %d unconnected", i, k);
    for (int k = 0; k < h.n_pred; k++) if (h.pred_node[k] < 0) return set_err(g, AMPNET_EINVAL, "node %d: predecessor port %d unconnected", i, k);
    auto need = [&](bool c, const char* what) { return c ? AMPNET_OK : set_err(g, AMPNET_EINVAL, "node %d: %s", i, what); };
    ampnet_status_t st = AMPNET_OK;
    switch (h.type) {
      case SOURCE:
        st = need(h.n_pred == 0 && h.n_succ == 1 && h.fn >= 1 && h.fn <= 6, "SOURCE needs one successor and a valid fn");
        if (st == AMPNET_OK) g->sources.push_back(i);
        break;
      case LINEAR:
        st = need(h.n_pred == 1 && h.n_succ == 1 && h.in_dim > 0 && h.out_dim > 0, "LINEAR needs one predecessor, one successor, positive dims");
        if (st == AMPNET_OK) {
          const bool fed = g->hnodes[h.pred_node[0]].type == SOURCE;
          st = need(fed == ((h.flags & 1) != 0), "FLAG_SOURCE_ADJACENT must be set exactly on PPT nodes fed by a SOURCE");
        }
        break;
      case LOOKUP:
        st = need(h.n_pred == 1 && h.n_succ == 1 && h.in_dim > 0 && h.out_dim > 0 && g->hnodes[h.pred_node[0]].type == SOURCE &&
                  (h.flags & 1), "LOOKUP must be fed by a SOURCE and flagged source-adjacent");
        break;
      case GRUCELL:
        st = need(h.n_pred == 1 && h.n_succ == 1 && h.out_dim > 0 && h.in_dim == 2 * h.out_dim && !(h.flags & 1), "GRUCELL needs in_dim == 2*out_dim");
        break;
      case LOSS_CE: case LOSS_MSE:
        st = need(h.n_pred == 1 && h.n_succ == 0 && h.in_dim > 0 && (h.type == LOSS_CE || h.in_dim == 1), "LOSS needs one predecessor and no successor");
        if (st == AMPNET_OK) g->losses.push_back(i);
        break;
      case SINK: st = need(h.n_pred == 1 && h.n_succ == 0, "SINK needs one predecessor and no successor"); break;
      case COND: st = need(h.n_pred == 1 && h.n_succ >= 1 && h.fn >= 1 && h.fn <= 5, "COND needs one predecessor and a valid fn"); break;
      case PHI: st = need(h.n_pred >= 1 && h.n_succ == 1, "PHI needs predecessors and one successor"); break;
      case ISU:
        st = need(h.n_pred == 1 && h.n_succ == 1 && h.fn >= 1 && h.fn <= 3, "ISU needs a valid fn");
        break;
      case CONCAT:
        st = need(h.n_succ == 1 && h.fn_arg >= 1 && h.fn_arg <= MAX_PORTS && h.out_dim == h.fn_arg * h.in_dim &&
                  ((h.fn == 1 && h.n_pred == h.fn_arg) || (h.fn == 2 && h.n_pred == 1)), "CONCAT ports / widths inconsistent");
        break;
      case BCAST: st = need(h.n_pred == 1 && h.fn_arg >= 1 && h.n_succ == h.fn_arg, "BCAST needs fn_arg successors"); break;
      case SPLIT:
        st = need(h.n_pred == 1 && h.fn_arg >= 1 && h.fn_arg <= MAX_PORTS && h.n_succ == h.fn_arg && h.in_dim == h.fn_arg * h.out_dim,
                  "SPLIT needs fn_arg successors of width in_dim / fn_arg");
        break;
      case GROUP: st = need(h.n_pred == 1 && h.n_succ == 1 && h.fn >= 1 && h.fn <= 3, "GROUP needs a valid fn"); break;
      case UNGROUP: st = need(h.n_pred == 1 && h.n_succ == 1 && h.fn >= 1 && h.fn <= 3, "UNGROUP needs a valid fn"); break;
      case FLATMAP: st = need(h.n_pred == 1 && h.n_succ == 1 && h.fn == 1, "FLATMAP needs a valid fn"); break;
      case NPT_SUMROWS: st = need(h.n_pred == 1 && h.n_succ == 1, "NPT_SUMROWS needs one predecessor and one successor"); break;
      case NPT_LSTM:
        st = need(h.n_succ == 1 && (h.fn == 1 || h.fn == 2) && h.n_pred == h.fn && h.out_dim > 0 && h.out_dim % 2 == 0 &&
                  h.in_dim == (h.fn == 1 ? 3 : 5) * (h.out_dim / 2), "NPT_LSTM needs fn 1 (3H -> 2H, one port) or 2 (5H and 2H -> 2H, two ports)");
        break;
    }
    if (st != AMPNET_OK) return st;
    if (h.type == ISU && h.fn == 3) g->has_it = true;
    if (h.type == COND && h.fn == 4) g->it_steps = std::max(g->it_steps, h.fn_arg);
  }
  if (g->sources.empty() || g->sources.size() > 4) return set_err(g, AMPNET_EINVAL, "the graph needs 1..4 SOURCE nodes");
  if (g->losses.empty() || g->losses.size() > 4) return set_err(g, AMPNET_EINVAL, "the graph needs 1..4 LOSS nodes");
  // widths along the edges
  auto out_width = [&](const DevNode& h) {
    if (h.type == LINEAR || h.type == LOOKUP || h.type == GRUCELL || h.type == CONCAT || h.type == SPLIT || h.type == NPT_LSTM) return h.out_dim;
    if (h.type == SOURCE) return (h.fn == 1 || h.fn == 3) ? h.out_dim : 0;
    return h.in_dim;
  };
  for (size_t k = 0; k < g->edges.size(); k++) {
    const DevNode &s = g->hnodes[g->edges[k].src_node], &d = g->hnodes[g->edges[k].dst_node];
    const int w = out_width(s);
    if (d.type == LOOKUP || w == 0) continue;
    if (d.type == SINK) continue;
    const int want = (d.type == NPT_LSTM && g->edges[k].dst_port == 1) ? d.out_dim : d.in_dim;    // port 1 of the gate node takes [cL; cR]
    if (w != want) return set_err(g, AMPNET_EINVAL, "edge %zu: width %d does not match the destination's input width %d", k, w, want);
  }
  // every cycle must pass through a PHI: the graph without PHI nodes is acyclic
  std::vector<int> indeg(n, 0);
  for (const auto& e : g->edges) if (g->hnodes[e.src_node].type != PHI && g->hnodes[e.dst_node].type != PHI) indeg[e.dst_node]++;
  std::vector<int> q;
  int seen = 0, n_non_phi = 0;
  for (int i = 0; i < n; i++) if (g->hnodes[i].type != PHI) { n_non_phi++; if (!indeg[i]) q.push_back(i); }
  while (!q.empty()) {
    int u = q.back(); q.pop_back(); seen++;
    for (int k = 0; k < g->hnodes[u].n_succ; k++) {
      int v = g->hnodes[u].succ_node[k];
      if (g->hnodes[v].type == PHI) continue;
      if (--indeg[v] == 0) q.push_back(v);
    }
  }
  if (seen != n_non_phi) return set_err(g, AMPNET_EINVAL, "the IR graph has a cycle that does not pass through a PHI node");
  return AMPNET_OK;
}

ampnet_status_t create_params(ampnet_graph* g, uint64_t seed) {
  uint64_t s = seed * 0x9E3779B97F4A7C15ull + 12345;
  for (int i = 0; i < (int)g->hnodes.size(); i++) {
    DevNode& h = g->hnodes[i];
    if (!is_ppt_type(h.type)) continue;
    HostPPT P;
    P.node = i; P.kind = h.type; P.in = h.in_dim; P.out = h.out_dim; P.nmat = h.type == GRUCELL ? 3 : 1;
    if (h.type != LOOKUP && j_bucket(h.in_dim) < 0) return set_err(g, AMPNET_EINVAL, "node %d: in_dim %d above 1024 is not supported", i, h.in_dim);
    P.nW = (size_t)P.nmat * P.in * P.out;
    P.nb = h.type == LOOKUP ? 0 : (size_t)P.nmat * P.out;
    std::vector<float> w(P.nW), b(P.nb, 0.f);
    if (h.type == LOOKUP) {
      for (size_t k = 0; k + 1 < w.size() + 1; k += 2) {      // Box-Muller, N(0, 0.1)
        double u1 = std::max(uniform01(s), 1e-300), u2 = uniform01(s);
        double r = std::sqrt(-2.0 * std::log(u1)) * 0.1;
        w[k] = (float)(r * std::cos(6.283185307179586 * u2));
        if (k + 1 < w.size()) w[k + 1] = (float)(r * std::sin(6.283185307179586 * u2));
      }
    } else {
      const double lim = std::sqrt(6.0 / (P.in + P.out));
      for (auto& v : w) v = (float)((2.0 * uniform01(s) - 1.0) * lim);
    }
    P.W = (float*)dev_alloc(g, P.nW * sizeof(float));
    P.b = (float*)dev_alloc(g, std::max<size_t>(P.nb, 1) * sizeof(float));
    if (!P.W || !P.b) return set_err(g, AMPNET_ENOMEM, "parameter allocation failed");
    CUDA_TRY(g, cudaMemcpy(P.W, w.data(), P.nW * sizeof(float), cudaMemcpyHostToDevice));
    if (P.nb) CUDA_TRY(g, cudaMemcpy(P.b, b.data(), P.nb * sizeof(float), cudaMemcpyHostToDevice));
    h.ppt = (int)g->ppts.size();
    g->ppts.push_back(P);
  }
  if (g->ppts.empty()) return set_err(g, AMPNET_EINVAL, "the graph has no parameterised node");
  if ((int)g->hnodes.size() > MAX_SMEM_NODES || (int)g->ppts.size() > MAX_SMEM_PPTS)
    return set_err(g, AMPNET_EINVAL, "the IR graph is too large: at most %d nodes and %d parameterised nodes", MAX_SMEM_NODES, MAX_SMEM_PPTS);
  return AMPNET_OK;
}

// ---- key-space inference: bounds of the position u and of the payload rows at every node ---------------
struct Dom { int U, rows; };

void infer_domains(ampnet_graph* g, const HostDataset& D) {
  const int n = (int)g->hnodes.size();
  std::vector<Dom> in(n, Dom{1, 1}), out(n, Dom{1, 1});
  for (int pass = 0; pass < 4 * n + 8; pass++) {
    bool changed = false;
    for (int i = 0; i < n; i++) {
      DevNode& h = g->hnodes[i];
      Dom a{1, 1};
      for (int k = 0; k < h.n_pred; k++) { const Dom& p = out[h.pred_node[k]]; a.U = std::max(a.U, p.U); a.rows = std::max(a.rows, p.rows); }
      Dom o = a;
      switch (h.type) {
        case SOURCE:
          if (h.fn == 2) o = Dom{D.maxT + 1, 1};
          else if (h.fn == 4) o = Dom{D.maxM, 1};
          else if (h.fn == 5) o = Dom{1, D.maxN};
          else if (h.fn == 6) o = Dom{1, D.maxL};          // the leaves of a tree as the rows of one message
          else o = Dom{1, 1};
          break;
        case FLATMAP: o = Dom{D.maxD, 1}; break;
        case GROUP:
          if (h.fn == 1) o = Dom{D.NT, D.maxDc};
          else if (h.fn == 2) o = Dom{D.maxN, D.maxIn};
          else o = Dom{1, D.maxN};
          break;
        case UNGROUP: o = h.fn == 2 ? Dom{D.maxD, 1} : h.fn == 3 ? Dom{D.maxM, 1} : Dom{D.maxN, 1}; break;
        case NPT_SUMROWS: o = Dom{a.U, 1}; break;
        default: break;
      }
      if (o.U != out[i].U || o.rows != out[i].rows || a.U != in[i].U || a.rows != in[i].rows) changed = true;
      in[i] = a; out[i] = o;
    }
    if (!changed) break;
  }
  for (int i = 0; i < n; i++) {
    g->hnodes[i].U_in = in[i].U; g->hnodes[i].rows_in = in[i].rows;
    g->hnodes[i].U_out = out[i].U; g->hnodes[i].rows_out = out[i].rows;
  }
}

unsigned pow2_at_least(unsigned long long v) {
  unsigned p = 64;
  while (p < v && p < (1u << 30)) p <<= 1;
  return p;
}

size_t tile_smem_floats(const HostPPT& P, int R, int BM, bool a_global = false, int xwt_rb = 8) {      // mirrors the carve-up at the top of ppt_main
  if (P.kind == LOOKUP) return 64;
  const size_t LW = (size_t)pad_ldw(P.in), LX = (size_t)pad_ldx(P.in), RP = (size_t)((R + 3) & ~3), nm = (size_t)P.nmat;
  auto p4 = [](size_t v) { return (v + 3) & ~(size_t)3; };
  return (a_global ? 1 : 2) * nm * R * LW + 2 * p4(nm * R) + (size_t)BM * LX * (P.kind == GRUCELL ? 2 : 1) + (nm + 1) * BM * RP + p4(nm * BM * R) +
         xwt_scratch_floats(xwt_rb) + 64;
}

// Placement: row tiles per PPT node.  Every node starts with the fewest tiles whose weights + accumulators + staging
// fit in shared memory; the remaining tile budget goes, one tile at a time, to the node with the most multiply-add work
// per tile (a GRU cell counts twice: three matrices and a second, dependent stage), so that the nodes' batch cycles
// come out alike.  A tile costs 1 + emitters CTAs; the controller and one scheduler CTA per node come off the top.
ampnet_status_t place(ampnet_graph* g, int n_ctas, int max_batch_rows, std::vector<Role>& roles, int emitters) {
  cudaFuncAttributes fa{};
  size_t static_smem = 40 * 1024;
  if (cudaFuncGetAttributes(&fa, ampnet_engine) == cudaSuccess) static_smem = fa.sharedSizeBytes;
  const size_t budget = ((size_t)g->max_smem - static_smem - 1024) / sizeof(float);
  int max_tiles = 16;      // default; a node whose tile does not fit in shared memory gets more, up to MAX_TILES
  if (const char* e = getenv("AMPNET_MAX_TILES")) max_tiles = std::max(1, std::min(MAX_TILES, atoi(e)));
  const int np = (int)g->ppts.size();
  for (auto& P : g->ppts) { P.LT = 1; P.tc = 0; }                // (choices of the direct-delivery engine)
  const int tile_budget = emitters > 0 ? (n_ctas - 1 - np) / (1 + emitters) : n_ctas - 1;
  std::vector<int> limit(np, 1), bm_of(np, 0);
  std::vector<double> work(np, 0.0);
  auto fit = [&](HostPPT& P, int t_from, int bm, int& t_out) {      // fewest tiles >= t_from that fit with capacity bm
    for (int t = t_from; t <= std::min(MAX_TILES, P.out); t++) {
      const int R = (P.out + t - 1) / t;
      if ((P.out + R - 1) / R < t_from) continue;
      if (tile_smem_floats(P, R, bm, P.a_global) <= budget) { t_out = (P.out + R - 1) / R; return true; }
    }
    return false;
  };
  int used_tiles = 0;
  for (int p = 0; p < np; p++) {
    HostPPT& P = g->ppts[p];
    const DevNode& h = g->hnodes[P.node];
    const int rows_max = h.rows_in;
    int BM = MAX_BATCH_ROWS;
    if (max_batch_rows > 0) BM = std::max(rows_max, std::min(BM, max_batch_rows));
    if (rows_max > MAX_BATCH_ROWS) return set_err(g, AMPNET_EINVAL, "node %d: %d payload rows per message exceed the supported %d", P.node, rows_max, MAX_BATCH_ROWS);
    P.J = P.kind == LOOKUP ? 4 : j_bucket(P.in);
    if (P.kind == LOOKUP) {
      // a large table means gathers and accumulations bound by DRAM latency: deal its rows to several tiles
      P.T = (P.in >= 4096 && tile_budget >= 24) ? 4 : 1;
      P.R = 0; P.BM = BM; limit[p] = P.T; bm_of[p] = BM;
      used_tiles += P.T;
      continue;
    }
    // Keep the micro-batch capacity if more row tiles make the tile fit; only then shrink the capacity.
    const int bm_min = std::max(rows_max, 4);
    bool placed = false;
    P.a_global = false;
    for (int bm = BM; !placed; bm = std::max(bm_min, bm / 2)) {
      int t = 0;
      if (fit(P, 1, bm, t)) { P.T = t; bm_of[p] = bm; placed = true; break; }
      if (bm == bm_min) return set_err(g, AMPNET_EINVAL, "node %d does not fit in shared memory with %d row tiles", P.node, MAX_TILES);
    }
    // A node so wide that fewer than 32 rows can be staged beside its weight and accumulator tiles keeps the accumulators
    // in device memory instead (read and written once per backward batch) if that buys a larger micro-batch.
    if (bm_of[p] < 32 && bm_of[p] < BM) {
      P.a_global = true;
      bool better = false;
      for (int bm = BM; bm > bm_of[p]; bm /= 2) {
        int t = 0;
        if (fit(P, 1, bm, t)) { P.T = t; bm_of[p] = bm; better = true; break; }
      }
      if (!better) P.a_global = false;
    }
    // a node with a handful of output rows (a classifier) may still have a tile per row; others keep 4 rows per tile
    limit[p] = std::max(P.T, std::min(max_tiles, P.out <= 16 ? P.out : std::max(1, P.out / 4)));
    work[p] = (double)P.nmat * P.in * P.out * (P.kind == GRUCELL ? 2.0 : 1.0);
    used_tiles += P.T;
  }
  if (1 + used_tiles * (1 + emitters) + (emitters > 0 ? np : 0) > n_ctas) return AMPNET_EOVERFLOW;   // retried with fewer emitters
  for (;;) {
    int best = -1;
    for (int p = 0; p < np; p++) {
      const HostPPT& P = g->ppts[p];
      if (P.kind == LOOKUP || P.T >= limit[p]) continue;
      if (best < 0 || work[p] / P.T > work[best] / g->ppts[best].T) best = p;
    }
    if (best < 0) break;
    HostPPT& P = g->ppts[best];
    int t = 0;
    if (!fit(P, P.T + 1, bm_of[best], t) || t > limit[best] || t <= P.T) { limit[best] = P.T; continue; }   // rows per tile are whole: the tile count moves in steps
    if (used_tiles + (t - P.T) > tile_budget) { limit[best] = P.T; continue; }
    used_tiles += t - P.T; P.T = t;
  }
  int used = 1;
  for (int p = 0; p < np; p++) {
    HostPPT& P = g->ppts[p];
    if (P.kind != LOOKUP) { P.R = (P.out + P.T - 1) / P.T; P.T = (P.out + P.R - 1) / P.R; P.BM = bm_of[p]; }
    P.xwt_rb = (P.kind != LOOKUP && P.R > 8 && tile_smem_floats(P, P.R, P.BM, P.a_global, 16) <= budget) ? 16 : 8;
    P.smem_floats = tile_smem_floats(P, P.R, P.BM, P.a_global, P.xwt_rb);
    used += P.T;
  }
  if (used > n_ctas) return set_err(g, AMPNET_EINVAL, "placement needs %d CTAs but only %d are available", used, n_ctas);
  roles.clear();
  roles.push_back(Role{-1, 0, 0, 0});
  for (int p = 0; p < (int)g->ppts.size(); p++)
    for (int t = 0; t < g->ppts[p].T; t++) roles.push_back(Role{p, t, 0, 0});
  for (auto& P : g->ppts) { P.NE = 0; P.G = 1; }
  if (emitters > 0) {
    const int need = 1 + (used - 1) * (1 + emitters) + (int)g->ppts.size();
    if (need > n_ctas) return AMPNET_EOVERFLOW;                                                     // retried with fewer emitters / tiles
    double load = 0.0;
    for (auto& P : g->ppts) load += P.emit_load;
    if (load > 0.0) {
      // Feedback from the last asynchronous epoch: every node keeps two emitters, the rest of the pool is dealt out in
      // proportion to the emitter time the nodes' emission took (largest remainder first).
      const int pool = n_ctas - 1 - np - (used - 1);
      int left = pool;
      for (auto& P : g->ppts) { P.NE = 2; left -= 2; }
      std::vector<double> want(np);
      for (int p = 0; p < np; p++) want[p] = g->ppts[p].emit_load / load * std::max(left, 0);
      for (int p = 0; p < np && left > 0; p++) { const int k = std::min(left, (int)std::floor(want[p])); g->ppts[p].NE += k; left -= k; want[p] -= k; }
      while (left > 0) {
        int best = 0;
        for (int p = 1; p < np; p++) if (want[p] > want[best]) best = p;
        g->ppts[best].NE++; want[best] -= 1.0; left--;
      }
    } else {
      for (auto& P : g->ppts) P.NE = P.T * emitters;
      // spare SMs become emitters of the nodes that have the fewest (a node with few row tiles emits as many messages)
      for (int spare = n_ctas - need; spare > 0; spare--) {
        HostPPT* best = nullptr;
        for (auto& P : g->ppts) if (P.NE < 24 && (!best || P.NE < best->NE)) best = &P;
        if (!best) break;
        best->NE++;
      }
    }
    // batch groups: a large pool works on up to four batches at a time (a batch's emission can take several tile cycles)
    for (auto& P : g->ppts) P.G = P.NE >= 16 ? 4 : P.NE >= 9 ? 3 : std::min(2, P.NE);
    for (int p = 0; p < (int)g->ppts.size(); p++) roles.push_back(Role{p, 0, 2, 0});                 // one scheduler CTA per node
    for (int p = 0; p < (int)g->ppts.size(); p++)
      for (int e = 0; e < g->ppts[p].NE; e++) roles.push_back(Role{p, 0, 1, e});
  }
  return AMPNET_OK;
}

// ---- direct-delivery engine: which graphs it takes, and its placement -------------------------------------
// It runs asynchronous epochs of graphs whose messages are single rows and whose parameter-free chains it can resolve
// per message: Cond, Phi, Isu, Bcast, Concat (assembling in the next node's input cache), Sink, and a Loss fed directly
// by a Linear node.  Everything else (row-wise Group / Ungroup / Flatmap, GRU and LSTM cells, the deterministic
// schedule, per-node message counters) stays with the interpreter engine.
bool direct_candidate(ampnet_graph* g, const HostDataset& D, int det) {
  if (det) return false;
  if (const char* e = getenv("AMPNET_ENGINE")) if (!strcmp(e, "classic")) return false;
  if (const char* e = getenv("AMPNET_TUNE")) if (atoi(e) & (16 | 32 | 8)) return false;
  if (D.kind == 3) return false;
  const int n = (int)g->hnodes.size();
  int max_nodes = 0, max_ppts = 0, max_landings = 0, batch_rows = 0;
  ampnet_direct_limits(&max_nodes, &max_ppts, &max_landings, &batch_rows);
  if (n > max_nodes || (int)g->ppts.size() > max_ppts) return false;
  for (int i = 0; i < n; i++) {
    const DevNode& h = g->hnodes[i];
    if (h.rows_in != 1 || h.rows_out != 1) return false;
    switch (h.type) {
      case SOURCE: if (h.fn < 1 || h.fn > 4) return false; break;
      case LINEAR: case LOOKUP: case COND: case PHI: case ISU: case SINK: break;
      case LOSS_CE: case LOSS_MSE: if (g->hnodes[h.pred_node[0]].type != LINEAR) return false; break;
      case CONCAT: {
        const DevNode& s = g->hnodes[h.succ_node[0]];
        if (h.fn_arg > max_landings) return false;
        if (s.type != LINEAR || (s.in_dim & 3) || s.in_dim != h.out_dim || s.U_in != h.U_out || s.rows_in != h.rows_in) return false;
      } break;
      case BCAST: {
        if (h.fn_arg > max_landings) return false;
        // backward, the sum forms in the gradient buffer of the parameterised node behind Phi / Cond / Isu
        std::vector<int> todo{h.pred_node[0]};
        std::vector<char> seen(n, 0);
        while (!todo.empty()) {
          const int v = todo.back(); todo.pop_back();
          if (seen[v]) continue;
          seen[v] = 1;
          const DevNode& p = g->hnodes[v];
          if (p.type == LINEAR || p.type == LOOKUP) continue;
          if (p.type != PHI && p.type != COND && p.type != ISU) return false;
          for (int k = 0; k < p.n_pred; k++) todo.push_back(p.pred_node[k]);
        }
      } break;
      default: return false;
    }
  }
  return true;
}

// Tiles of the direct-delivery engine.  A Linear node is split by direction: forward row tiles of `rows` weight rows
// (AMPNET_DIRECT_ROWS, default 16) and backward column tiles of `cols` input columns (AMPNET_DIRECT_COLS, default 16;
// 4, 8, 16 or 32), more per tile where the CTA budget, shared memory or the register-resident accumulators ask for it.
// A node that feeds a Loss is one tile for both directions (the Loss needs the whole output row); a large embedding
// table is dealt to four tiles by row id.
static ampnet_status_t direct_overflow(int where) {
  if (getenv("AMPNET_DEBUG")) fprintf(stderr, "[ampnet] direct-delivery placement does not fit (check %d): interpreter engine\n", where);
  return AMPNET_EOVERFLOW;
}

ampnet_status_t place_direct(ampnet_graph* g, int n_ctas, std::vector<Role>& roles) {
  size_t static_smem = 48 * 1024;
  ampnet_direct_static_smem(&static_smem);
  const size_t budget = (size_t)g->max_smem - static_smem - 1024;
  int rows = 16, cols = 16;
  if (const char* e = getenv("AMPNET_DIRECT_ROWS")) rows = std::max(1, atoi(e));
  if (const char* e = getenv("AMPNET_DIRECT_COLS")) { const int c = atoi(e); if (c == 4 || c == 8 || c == 16 || c == 32) cols = c; }
  const int np = (int)g->ppts.size(), tile_budget = n_ctas - 1, max_units = ampnet_direct_max_units();
  int lim_nodes = 0, lim_ppts = 0, lim_landings = 0, BATCH = MAX_BATCH_ROWS;
  ampnet_direct_limits(&lim_nodes, &lim_ppts, &lim_landings, &BATCH);
  std::vector<int> fixed(np, 0);
  std::vector<char> fixed_rows(np, 0);
  int tc_rows = 64, tc_bm = 64, tc_k = 16;
  ampnet_direct_tc_limits(&tc_rows, &tc_bm, &tc_k);
  bool use_tc = true;
  if (const char* e = getenv("AMPNET_TENSOR_CORES")) use_tc = atoi(e) != 0;
  // gradient slots: the backward sum of a Bcast forms in the gradient buffer of the node behind Phi / Cond / Isu
  for (auto& P : g->ppts) P.NS = 1;
  for (int i = 0; i < (int)g->hnodes.size(); i++) {
    const DevNode& h = g->hnodes[i];
    if (h.type != BCAST) continue;
    std::vector<int> todo{h.pred_node[0]};
    std::vector<char> seen(g->hnodes.size(), 0);
    while (!todo.empty()) {
      const int v = todo.back(); todo.pop_back();
      if (seen[v]) continue;
      seen[v] = 1;
      const DevNode& p = g->hnodes[v];
      if (p.type == LINEAR || p.type == LOOKUP) { g->ppts[p.ppt].NS = std::max(g->ppts[p.ppt].NS, h.fn_arg); continue; }
      for (int k = 0; k < p.n_pred; k++) todo.push_back(p.pred_node[k]);
    }
  }
  for (int p = 0; p < np; p++) {
    HostPPT& P = g->ppts[p];
    const DevNode& h = g->hnodes[P.node];
    P.NE = 0; P.G = 1; P.a_global = false; P.J = 0; P.TB = 0; P.CB = 0; P.bwd_smem_floats = 0; P.tc = 0; P.LT = 1;
    if (P.kind == LOOKUP) { P.T = (P.in >= 4096 && tile_budget >= 24) ? 4 : 1; P.R = 0; P.BM = BATCH; fixed[p] = 1; continue; }
    const int st = g->hnodes[h.succ_node[0]].type;
    P.BM = BATCH;
    if (st == LOSS_CE || st == LOSS_MSE) { P.R = P.out; fixed[p] = 1; }
    else {
      P.R = std::min(P.out, rows);
      // bf16 runs: a node whose shape fits the instruction (rows in whole tiles of 64, input width a multiple of 16) runs its
      // forward products on the tensor cores (AMPNET_TENSOR_CORES=0 keeps them on the FMA units)
      if (g->payload_bf16 && use_tc && P.kind == LINEAR && P.out % tc_rows == 0 && P.in % tc_k == 0) { P.tc = 1; P.R = tc_rows; P.BM = std::min(P.BM, tc_bm); fixed_rows[p] = 1; }
      P.CB = cols;
      while (P.CB > 4 && (long long)P.out * (P.CB / 4) > max_units) P.CB /= 2;
      if ((long long)P.out * (P.CB / 4) > max_units) return direct_overflow(1);        // accumulators of a column tile exceed the registers
    }
  }
  auto fits = [&](const HostPPT& P) {
    const size_t fwd = P.tc ? ampnet_direct_tc_tile_smem_bytes(P.in, P.BM) : ampnet_direct_tile_smem_bytes(P.in, P.R, P.BM, P.CB == 0);
    return fwd <= budget && (P.CB == 0 || ampnet_direct_bwd_tile_smem_bytes(P.out, P.CB, P.BM) <= budget);
  };
  for (int p = 0; p < np; p++) {
    HostPPT& P = g->ppts[p];
    if (P.kind == LOOKUP) continue;
    while (!fits(P)) {
      if (P.BM > 16) P.BM /= 2;
      else if (P.tc) { P.tc = 0; fixed_rows[p] = 0; P.R = std::min(P.out, rows); P.BM = BATCH; }       // the weights alone do not fit as one 64-row tile
      else if (!fixed[p] && P.R > 1) { P.R = (P.R + 1) / 2; P.BM = BATCH; }
      else return direct_overflow(2);
    }
  }
  // over the budget: grow the tiles of whichever node has the most tiles of a kind that can still grow (rows per forward
  // tile while its weights and a few staged rows still fit; columns per backward tile while the accumulators fit the registers)
  std::vector<char> rows_stuck(fixed_rows);
  for (;;) {
    int used = 0, best = -1, best_n = 0; bool best_cols = false;
    for (int p = 0; p < np; p++) {
      HostPPT& P = g->ppts[p];
      if (P.kind != LOOKUP) { P.T = (P.out + P.R - 1) / P.R; P.TB = P.CB ? (P.in + P.CB - 1) / P.CB : 0; }
      used += P.T + P.TB;
      if (fixed[p]) continue;
      if (!rows_stuck[p] && P.R < P.out && P.T > best_n) { best = p; best_n = P.T; best_cols = false; }
      if (P.CB && P.CB < 32 && (long long)P.out * (P.CB * 2 / 4) <= max_units && P.TB > best_n) { best = p; best_n = P.TB; best_cols = true; }
    }
    if (used <= tile_budget) break;
    if (best < 0) return direct_overflow(4);
    HostPPT& P = g->ppts[best];
    if (best_cols) { P.CB *= 2; while (!fits(P) && P.BM > 8) P.BM /= 2; if (!fits(P)) return direct_overflow(5); continue; }
    const int r0 = P.R, bm0 = P.BM;
    P.R++;
    while (!fits(P) && P.BM > 8) P.BM /= 2;
    if (!fits(P)) { P.R = r0; P.BM = bm0; rows_stuck[best] = 1; }
  }
  // CTAs left over go to the loss heads: their tiles share the node's messages (every tree node, every list, passes
  // through that one node) and meet at its updates
  {
    int used = 0, heads = 0, want = 8;
    if (const char* e = getenv("AMPNET_LOSS_TILES")) want = std::max(1, std::min(16, atoi(e)));
    for (int p = 0; p < np; p++) { used += g->ppts[p].T + g->ppts[p].TB; heads += fixed[p] && g->ppts[p].kind != LOOKUP; }
    for (int p = 0; p < np && heads > 0; p++) {
      HostPPT& P = g->ppts[p];
      if (!fixed[p] || P.kind == LOOKUP) continue;
      P.LT = std::max(1, std::min(want, 1 + (tile_budget - used) / heads));
    }
  }
  // ... and then to the embedding tables (their rows are dealt to the tiles by id: gathers and scatter-adds of a batch
  // spread over more SMs; measured on the tree workload: 50 k / 68 k / 75 k / 77 k / 78 k trees/s with 1 / 2 / 4 / 8 / 16 tiles)
  {
    int used = 0, want = 16;
    if (const char* e = getenv("AMPNET_LOOKUP_TILES")) want = std::max(1, std::min(32, atoi(e)));
    for (int p = 0; p < np; p++) used += (g->ppts[p].LT > 1 ? g->ppts[p].LT : g->ppts[p].T) + g->ppts[p].TB;
    for (int p = 0; p < np; p++) {
      HostPPT& P = g->ppts[p];
      if (P.kind != LOOKUP || P.T <= 1) continue;
      const int t = std::max(std::min(P.T, want), std::min(want, P.T + (tile_budget - used)));
      used += t - P.T;
      P.T = t;
    }
  }
  roles.clear();
  roles.push_back(Role{-1, 0, 0, 0});
  for (int p = 0; p < np; p++) {
    HostPPT& P = g->ppts[p];
    P.smem_floats = P.kind == LOOKUP ? 64 : (P.tc ? ampnet_direct_tc_tile_smem_bytes(P.in, P.BM) : ampnet_direct_tile_smem_bytes(P.in, P.R, P.BM, P.CB == 0)) / sizeof(float);
    P.bwd_smem_floats = P.TB ? ampnet_direct_bwd_tile_smem_bytes(P.out, P.CB, P.BM) / sizeof(float) : 0;
    for (int t = 0; t < (P.LT > 1 ? P.LT : P.T); t++) roles.push_back(Role{p, t, 0, 0});
    for (int t = 0; t < P.TB; t++) roles.push_back(Role{p, t, 3, 0});
  }
  return AMPNET_OK;
}

// ---- run ---------------------------------------------------------------------------------------------------
struct RunPlan {
  std::vector<DevNode> nodes;
  std::vector<DevPPT> ppts;
  std::vector<Role> roles;
  Ctx ctx{};
  size_t smem_bytes = 0;
  bool direct = false;                // the run goes to the direct-delivery engine
};

inline bool eval_uses_classic(int) { return false; }

ampnet_status_t plan_run(ampnet_graph* g, int split, int mak, int det, int eval, const ampnet_run_cfg_t* cfg,
                         long long n_order, bool dry, RunPlan& R) {
  HostDataset& D = g->data[split];
  infer_domains(g, D);
  const int IT = g->has_it ? g->it_steps + 1 : 1;
  int n_ctas = cfg && cfg->n_ctas > 0 ? std::min(cfg->n_ctas, g->n_sms) : g->n_sms;
  // Asynchronous runs pair every tile with an emitter CTA when the SMs allow it (with fewer tiles if need be).
  int tune = 0;
  if (const char* e = getenv("AMPNET_TUNE")) tune = atoi(e);
  int emit_ctas = (!det && !(tune & 32)) ? ((tune & 64) ? 1 : 2) : 0;
  const int mbr = cfg ? cfg->max_batch_rows : 0;
  ampnet_status_t st = AMPNET_EOVERFLOW;
  R.direct = !eval_uses_classic(eval) && mbr == 0 && direct_candidate(g, D, det);
  if (R.direct) {
    st = place_direct(g, n_ctas, R.roles);
    if (st == AMPNET_EOVERFLOW) R.direct = false;             // too few CTAs for its tiles: the interpreter engine places its own
    else if (st != AMPNET_OK) return st;
    else emit_ctas = 0;
  }
  // Two emitter CTAs per tile if the SMs allow it, with as many tiles per node as fit; then one; then none.
  for (; !R.direct && emit_ctas > 0 && st == AMPNET_EOVERFLOW; emit_ctas--) {
    st = place(g, n_ctas, mbr, R.roles, emit_ctas);
    if (st != AMPNET_EOVERFLOW) break;
  }
  if (!R.direct && st == AMPNET_EOVERFLOW) { emit_ctas = 0; st = place(g, n_ctas, mbr, R.roles, 0); }
  if (st == AMPNET_EOVERFLOW) return set_err(g, AMPNET_EINVAL, "the model needs more CTAs than the %d available (one per row tile + the controller)", n_ctas);
  if (st != AMPNET_OK) return st;
  const int depth = R.direct ? 1 : emit_ctas > 0 ? 5 : 2;       // emitters work in up to four batch groups: a tile may be four batches ahead
  R.ctx.emit_ctas = emit_ctas; R.ctx.depth = depth; R.ctx.sched_ctas = emit_ctas > 0 ? 1 : 0;
  n_ctas = (int)R.roles.size();
  DeviceArena &C = g->ctl, &B = g->bulk;
  C.used = B.used = 0;
  if (dry) { C.base = B.base = nullptr; } else { C.base = (char*)g->ctl_mem; B.base = (char*)g->bulk_mem; }
  g->leftover_regions.clear();
  g->zero_regions.clear();
  auto track = [&](void* p, size_t bytes) { if (!dry) g->leftover_regions.push_back({(size_t)((char*)p - C.base), bytes}); };
  R.nodes = g->hnodes;
  R.ppts.assign(g->ppts.size(), DevPPT{});
  g->d_stats.assign(g->ppts.size(), nullptr);
  g->d_update_log.assign(g->ppts.size(), nullptr);
  size_t max_smem_floats = 2048;        // at least the two batch slots of a scheduler CTA
  int cta = 1;
  for (size_t p = 0; p < g->ppts.size(); p++) {
    const HostPPT& H = g->ppts[p];
    const DevNode& h = g->hnodes[H.node];
    DevPPT& P = R.ppts[p];
    P.node = H.node; P.kind = H.kind; P.in_dim = H.in; P.out_dim = H.out; P.act = h.act; P.flags = h.flags;
    P.muf_override = g->nodes[H.node].muf_override;
    P.T = H.T; P.cta0 = cta; cta += H.T; P.R = H.R; P.BM = H.BM; P.J = H.J;
    P.U = h.U_in; P.rows_max = h.rows_in;
    P.W = H.W; P.b = H.b;
    P.om = H.om; P.ov = H.ov; P.opt_t0 = H.opt_t;
    const size_t keys = (size_t)mak * IT * P.U;
    const bool source_fed = g->hnodes[h.pred_node[0]].type == SOURCE;
    P.xld = pad_ldw(P.in_dim);
    if (!source_fed) {
      P.xcache = B.take<float>(keys * P.rows_max * P.xld);
      if (P.xld != P.in_dim && !dry) g->zero_regions.push_back({P.xcache, keys * P.rows_max * P.xld * sizeof(float)});   // the row padding
    }
    if (H.kind != LOOKUP) P.ycache = B.take<float>(keys * P.rows_max * P.out_dim);
    P.NS = R.direct ? H.NS : 1; P.tc = R.direct ? H.tc : 0; P.TB = H.TB; P.CB = H.CB; P.bwd_smem_floats = (int)H.bwd_smem_floats;
    P.gbuf = B.take<float>(keys * P.rows_max * P.out_dim * P.NS);
    if (R.direct) {                  // one gradient slot per contributor: nothing is added in memory, nothing cleared
      for (int d = 0; d < 2; d++) { P.injoin[d] = C.take<int>(keys); track(P.injoin[d], keys * sizeof(int)); }
      P.wver = C.take<unsigned>(1);
      P.LT = H.LT;
      if (H.LT > 1) {
        const size_t PS = (size_t)H.out * H.in + H.out;
        P.lh_count = C.take<int>(1);
        P.lh_part = B.take<float>(2 * (size_t)H.LT * PS);
        P.lh_mom = B.take<float>(2 * (size_t)(H.LT - 1) * PS);
      }
    } else P.LT = 1;
    if (H.kind == GRUCELL) {
      P.zc = B.take<float>(keys * P.rows_max * P.out_dim);
      P.rc = B.take<float>(keys * P.rows_max * P.out_dim);
      P.cc = B.take<float>(keys * P.rows_max * P.out_dim);
      P.part2 = B.take<float>((size_t)depth * (P.T + 1) * P.BM * P.in_dim);
    }
    P.vcache = B.take<int>(keys);
    const unsigned cap = pow2_at_least(2ull * keys);
    if (cap > (det ? (1u << 20) : (1u << 23)))
      return set_err(g, AMPNET_EINVAL, "node %d: queue capacity %u above the supported 2^%d (lower max_active_keys)", H.node, cap, det ? 20 : 23);
    for (int d = 0; d < 2; d++) {
      P.ring[d].e = B.take<Hdr>(cap);
      if (R.direct && !dry) g->zero_regions.push_back({P.ring[d].e, (size_t)cap * sizeof(Hdr)});     // entries carry their ticket: none may survive a run
      P.ring[d].seq = C.take<unsigned>(cap);
      P.ring[d].tail = C.take<unsigned>(1);
      P.ring[d].mask = cap - 1;
    }
    P.sched = B.take<unsigned>(2 * (size_t)cap); P.sched_mask = 2 * cap - 1;
    P.batches = B.take<BatchDesc>(2 * (size_t)cap); P.batch_mask = 2 * cap - 1;
    P.batch_pub = C.take<unsigned>(1);
    P.bhdr = B.take<Hdr>((size_t)BATCH_BLOCKS * MAX_BATCH_MSGS);
    P.ctxblk = B.take<BatchCtx>((size_t)BATCH_BLOCKS);
    P.sortbuf = B.take<unsigned long long>(cap);
    if ((P.T > 1 && H.kind != LOOKUP) || H.kind == GRUCELL) P.dxpart = B.take<float>((size_t)depth * P.T * P.BM * P.in_dim);
    P.stage_floats = (long long)P.BM * std::max(P.in_dim, P.out_dim);
    P.stage = B.take<float>((size_t)depth * P.stage_floats);
    P.emit_pub = C.take<unsigned>(P.T);
    P.emit_fin = C.take<unsigned>(P.T);
    P.fetched = C.take<unsigned>(1);
    P.emit_done = C.take<unsigned>((size_t)std::max(1, H.NE));
    P.NE = H.NE; P.G = H.G;
    P.nbar = C.take<unsigned>(1);
    P.stats = C.take<PPTStats>(1);
    P.update_log = B.take<int>(g->update_log_cap); P.update_log_cap = g->update_log_cap;
    P.a_global = H.a_global ? 1 : 0;
    P.xwt_rb = H.xwt_rb;
    // accumulators kept in device memory start every run at zero; they live beside the caches so that the control arena
    // stays small (queues and counters only)
    auto zeroed = [&](size_t n_floats) {
      float* a = B.take<float>(n_floats);
      if (!dry) g->zero_regions.push_back({a, n_floats * sizeof(float)});
      return a;
    };
    if (H.a_global) P.A = zeroed((size_t)H.T * H.nmat * H.R * pad_ldw(H.in));
    if (H.kind == LOOKUP) {
      P.A = zeroed(H.nW);
      P.touched_flag = reinterpret_cast<int*>(zeroed(H.in));
      P.touched_list = reinterpret_cast<int*>(zeroed((size_t)H.in + H.T));      // one segment of ceil(V / T) entries per tile
      P.touched_n = C.take<int>(H.T);
    }
    P.smem_floats = (int)H.smem_floats;
    max_smem_floats = std::max(max_smem_floats, H.smem_floats);
    if (R.direct) max_smem_floats = std::max(max_smem_floats, H.bwd_smem_floats);
    g->d_stats[p] = P.stats; g->d_update_log[p] = P.update_log;
  }
  for (size_t i = 0; i < R.nodes.size(); i++) {
    DevNode& n = R.nodes[i];
    const size_t kin = (size_t)mak * IT * n.U_in, kout = (size_t)mak * IT * n.U_out;
    switch (n.type) {
      case CONCAT: {
        n.jstride = (long long)n.rows_in * n.out_dim;
        n.jcnt = C.take<int>(kout); track(n.jcnt, kout * sizeof(int));
        const DevNode& s = R.nodes[n.succ_node[0]];
        if (is_ppt_type(s.type) && R.ppts[s.ppt].xcache && R.ppts[s.ppt].xld == s.in_dim && s.U_in == n.U_out && s.rows_in == n.rows_in) { n.jbuf = R.ppts[s.ppt].xcache; n.jalias = 1; }
        else n.jbuf = B.take<float>(kout * n.jstride);
      } break;
      case GROUP:
        n.jld = n.in_dim;
        n.jstride = (long long)n.rows_out * n.in_dim;
        n.jcnt = C.take<int>(kout); track(n.jcnt, kout * sizeof(int));
        break;
      case NPT_LSTM:         // per key: gate pre-activations, the children's cells, the output [h; c]
        n.jstride = (long long)n.in_dim + 2 * n.out_dim;
        n.jbuf = B.take<float>(kin * n.jstride);
        n.jcnt = C.take<int>(kin); track(n.jcnt, kin * sizeof(int));
        break;
      case UNGROUP:
      case SPLIT:            // the backward join of the parts' gradients
        n.jstride = (long long)n.rows_in * n.in_dim;
        n.jbuf = B.take<float>(kin * n.jstride);
        n.jcnt = C.take<int>(kin); track(n.jcnt, kin * sizeof(int));
        break;
      case FLATMAP:
        n.jstride = (long long)(D.maxOut + 1) * n.in_dim;
        n.jbuf = B.take<float>(kin * n.jstride);
        n.jcnt = C.take<int>(kin); track(n.jcnt, kin * sizeof(int));
        break;
      case BCAST:
        n.jstride = (long long)(n.fn_arg + 1) * n.rows_in * n.in_dim;
        n.jbuf = B.take<float>(kin * n.jstride);
        n.jcnt = C.take<int>(kin); track(n.jcnt, kin * sizeof(int));
        break;
      case NPT_SUMROWS:
        n.jstride = n.in_dim;
        n.jbuf = B.take<float>(kin * n.jstride);
        n.rowcnt = C.take<int>(kin); track(n.rowcnt, kin * sizeof(int));
        break;
      case LOSS_CE: case LOSS_MSE:
        n.jstride = n.in_dim;
        n.jbuf = B.take<float>(kin * n.jstride);
        n.lossval = B.take<float>(kin);
        n.predok = B.take<int>(kin);
        break;
      case PHI:
        n.origin = C.take<unsigned char>(kin); track(n.origin, kin);
        if (R.direct) { n.jcnt = C.take<int>(kin); track(n.jcnt, kin * sizeof(int)); }
        break;
      default: break;
    }
  }
  // GROUP buffers come second: a Group that feeds an edge-wise Concat assembles its rows inside the Concat's buffer
  for (size_t i = 0; i < R.nodes.size(); i++) {
    DevNode& n = R.nodes[i];
    if (n.type != GROUP) continue;
    const size_t kout = (size_t)mak * IT * n.U_out;
    const DevNode& s = R.nodes[n.succ_node[0]];
    if (s.type == CONCAT && s.fn == 1 && s.U_out == n.U_out && s.rows_in == n.rows_out && s.in_dim == n.in_dim && s.jbuf) {
      n.jbuf = s.jbuf + (size_t)n.succ_port[0] * s.in_dim; n.jld = s.out_dim; n.jstride = s.jstride; n.jalias = 1;
    } else n.jbuf = B.take<float>(kout * n.jstride);
  }
  Ctx& X = R.ctx;
  X.n_nodes = (int)R.nodes.size(); X.n_ppts = (int)R.ppts.size(); X.n_ctas = n_ctas;
  X.nodes = B.take<DevNode>(R.nodes.size());
  X.ppts = B.take<DevPPT>(R.ppts.size());
  X.roles = B.take<Role>(R.roles.size());
  X.inst = D.dev;
  X.g = C.take<Globals>(1);
  X.node_msgs = C.take<unsigned long long>(R.nodes.size() * 2);
  g->d_node_msgs = X.node_msgs;
  X.n_sources = (int)g->sources.size();
  for (size_t k = 0; k < g->sources.size(); k++) X.src_nodes[k] = g->sources[k];
  X.n_loss = (int)g->losses.size();
  // A forward-only instance is finished when it has reached every end of the graph: a Loss with one label per instance
  // and a Sink are reached once, a Loss with a label per position (tree node) once per position.
  X.ends_per_instance = X.ends_per_position = 0;
  for (auto& hn : g->hnodes) {
    if (hn.type == SINK) X.ends_per_instance++;
    if (hn.type == LOSS_CE || hn.type == LOSS_MSE) { if (hn.type == LOSS_CE && hn.fn == 2) X.ends_per_position++; else X.ends_per_instance++; }
  }
  for (size_t k = 0; k < g->losses.size(); k++) X.loss_nodes[k] = g->losses[k];
  X.slot_inst = B.take<int>(mak);
  X.outstanding = C.take<int>(mak);
  X.slot_log = C.take<int>(mak);
  X.keylog = det ? B.take<KeyLog>((size_t)std::max<long long>(n_order, 1)) : nullptr;
  g->d_keylog = X.keylog;
  const unsigned rcap = pow2_at_least(2ull * mak * (unsigned long long)std::max({D.maxT + 1, D.maxL, D.maxM + 1, 2}));
  X.retire_e = B.take<unsigned>(rcap);
  X.retire_seq = reinterpret_cast<unsigned*>(C.take<unsigned long long>(rcap));      // (the direct-delivery engine keeps 8-byte notices here)
  X.retire_mask = rcap - 1;
  X.order = nullptr; X.n_order = n_order;
  X.loss_out = B.take<float>((size_t)std::max<long long>(D.n, 1));
  X.wide = 0;
  for (auto& hn : g->hnodes) if (hn.type == UNGROUP || hn.type == GROUP) X.wide = 1;
  X.bf16 = g->payload_bf16 ? 1 : 0;
  X.tune = 0;
  if (const char* e = getenv("AMPNET_TUNE")) X.tune = atoi(e);
  if (X.tune & 1) X.wide = 0;
  X.mak = mak; X.muf = cfg ? cfg->min_update_frequency : 1; X.det = det; X.eval = eval; X.IT = IT;
  X.lr = cfg ? cfg->lr : 0.f;
  X.opt = g->opt; X.mu = g->opt_mu; X.beta1 = g->opt_beta1; X.beta2 = g->opt_beta2; X.eps = g->opt_eps;
  double to = cfg && cfg->timeout_s > 0 ? cfg->timeout_s : 120.0;
  X.timeout_ns = (unsigned long long)(to * 1e9);
  X.ctl_base = C.base;
  R.smem_bytes = max_smem_floats * sizeof(float);
  return AMPNET_OK;
}

// Slack added to what a dry plan counted: alignment of the pieces carved after it (order, inference mask).
constexpr size_t ARENA_SLACK = 4096, BULK_EXTRA = 1024;

ampnet_status_t ensure_arenas(ampnet_graph* g, size_t ctl_need, size_t bulk_need) {
  ctl_need += ARENA_SLACK; bulk_need += ARENA_SLACK;
  if (g->arenas_lent) {               // lent memory is used as it is: nothing is freed, nothing allocated
    if (ctl_need > g->ctl_cap || bulk_need > g->bulk_cap)
      return set_err(g, AMPNET_EINVAL, "the lent scratch is too small for this run (%zu + %zu bytes needed)", ctl_need, bulk_need);
    return AMPNET_OK;
  }
  if (ctl_need > g->ctl_cap) {
    const size_t MiB = (size_t)1 << 20;
    const bool small = ctl_need <= MiB;
    dev_free(g, g->ctl_alloc);
    g->ctl_alloc = dev_alloc(g, small ? 3 * MiB : ctl_need);
    g->ctl_mem = g->ctl_alloc;
    g->ctl_cand[0] = g->ctl_cand[1] = nullptr;
    g->ctl_trials = 0; g->ctl_choice = -1;
    if (small && g->ctl_alloc) {
      g->ctl_cand[0] = reinterpret_cast<char*>(((uintptr_t)g->ctl_alloc + MiB - 1) & ~(uintptr_t)(MiB - 1));
      g->ctl_cand[1] = g->ctl_cand[0] + MiB;
      g->ctl_mem = g->ctl_cand[0];
    }
    g->ctl_cap = g->ctl_mem ? (small ? MiB : ctl_need) : 0;
    if (!g->ctl_mem) return set_err(g, AMPNET_ENOMEM, "device allocation of %zu bytes (queues, counters) failed", ctl_need);
  }
  if (bulk_need > g->bulk_cap) {
    dev_free(g, g->bulk_mem);
    g->bulk_mem = dev_alloc(g, bulk_need);
    g->bulk_cap = g->bulk_mem ? bulk_need : 0;
    if (!g->bulk_mem) return set_err(g, AMPNET_ENOMEM, "device allocation of %zu bytes (keyed caches) failed", bulk_need);
  }
  return AMPNET_OK;
}

ampnet_status_t execute(ampnet_graph* g, int split, int mak, int det, int eval, const ampnet_run_cfg_t* cfg,
                        ampnet_epoch_stats_t* out, float* per_instance_loss, double* accuracy,
                        const uint8_t* inference_only = nullptr, ampnet_inference_stats_t* inference = nullptr) {
  HostDataset& D = g->data[split];
  if (!D.loaded) return set_err(g, AMPNET_ESTATE, "no instances loaded for split %d", split);
  if (mak < 1) return set_err(g, AMPNET_EINVAL, "max_active_keys must be >= 1");
  if (!eval && cfg->min_update_frequency < 1) return set_err(g, AMPNET_EINVAL, "min_update_frequency must be >= 1");
  long long n_order = D.n;
  const long long* order = nullptr;
  if (cfg && cfg->order) {
    order = reinterpret_cast<const long long*>(cfg->order); n_order = cfg->n_order;
    if (n_order < 0) return set_err(g, AMPNET_EINVAL, "n_order must be >= 0");
    for (long long i = 0; i < n_order; i++)
      if (order[i] < 0 || order[i] >= D.n) return set_err(g, AMPNET_EINVAL, "order[%lld] = %lld is not an instance", i, (long long)order[i]);
  }
  if (det && n_order >= (1ll << 24)) return set_err(g, AMPNET_EINVAL, "the deterministic schedule supports fewer than 2^24 instances per epoch");
  const bool dbg = getenv("AMPNET_DEBUG") != nullptr;
  CUDA_TRY(g, cudaSetDevice(g->device));
  RunPlan R;
  g->have_run = false;                // planning re-targets the statistics pointers: the previous run's are gone from here on
  if (dbg) fprintf(stderr, "[ampnet] planning\n");
  ampnet_status_t st = plan_run(g, split, mak, det, eval, cfg, n_order, true, R);
  if (st != AMPNET_OK) return st;
  const size_t order_bytes = order ? (size_t)n_order * sizeof(long long) : 0;
  const size_t mask_bytes = inference_only ? (size_t)D.n : 0;
  st = ensure_arenas(g, g->ctl.used, g->bulk.used + order_bytes + mask_bytes + BULK_EXTRA);
  if (st != AMPNET_OK) return st;
  const bool ctl_own = g->ctl_cand[0] && (g->ctl_mem == g->ctl_cand[0] || g->ctl_mem == g->ctl_cand[1]);
  const bool ctl_trial = ctl_own && g->ctl_choice < 0 && !det && !eval && !R.direct && !getenv("AMPNET_NO_ARENA_TRIAL");
  if (ctl_own) g->ctl_mem = g->ctl_cand[g->ctl_choice >= 0 ? g->ctl_choice : (ctl_trial && g->ctl_trials >= 2) ? 1 : 0];
  if (ctl_own && getenv("AMPNET_ARENA_POS")) g->ctl_mem = g->ctl_cand[atoi(getenv("AMPNET_ARENA_POS")) & 1];
  st = plan_run(g, split, mak, det, eval, cfg, n_order, false, R);
  if (st != AMPNET_OK) return st;
  if (order) {
    long long* d_order = g->bulk.take<long long>((size_t)n_order);
    CUDA_TRY(g, cudaMemcpyAsync(d_order, order, order_bytes, cudaMemcpyHostToDevice, g->stream));
    R.ctx.order = d_order;
  }
  if (inference_only) {
    unsigned char* d_mask = g->bulk.take<unsigned char>(mask_bytes);
    CUDA_TRY(g, cudaMemcpyAsync(d_mask, inference_only, mask_bytes, cudaMemcpyHostToDevice, g->stream));
    R.ctx.inference_only = d_mask;
  }
  if ((size_t)R.smem_bytes > (size_t)g->max_smem) return set_err(g, AMPNET_EINVAL, "tile needs %zu bytes of shared memory", R.smem_bytes);
  CUDA_TRY(g, cudaMemsetAsync(g->ctl_mem, 0, g->ctl.used, g->stream));
  for (auto& z : g->zero_regions) CUDA_TRY(g, cudaMemsetAsync(z.first, 0, z.second, g->stream));
  CUDA_TRY(g, cudaMemsetAsync(R.ctx.slot_inst, 0xFF, (size_t)mak * sizeof(int), g->stream));
  CUDA_TRY(g, cudaMemsetAsync(R.ctx.loss_out, 0, (size_t)std::max<long long>(D.n, 1) * sizeof(float), g->stream));
  CUDA_TRY(g, cudaMemcpyAsync(R.ctx.nodes, R.nodes.data(), R.nodes.size() * sizeof(DevNode), cudaMemcpyHostToDevice, g->stream));
  CUDA_TRY(g, cudaMemcpyAsync(R.ctx.ppts, R.ppts.data(), R.ppts.size() * sizeof(DevPPT), cudaMemcpyHostToDevice, g->stream));
  CUDA_TRY(g, cudaMemcpyAsync(R.ctx.roles, R.roles.data(), R.roles.size() * sizeof(Role), cudaMemcpyHostToDevice, g->stream));
  if (dbg) fprintf(stderr, "[ampnet] %s engine, %d CTAs, %zu B smem, ctl %zu B, bulk %zu B\n", R.direct ? "direct-delivery" : "interpreter", R.ctx.n_ctas, R.smem_bytes, g->ctl.used, g->bulk.used);
  if (dbg) for (auto& P : g->ppts) fprintf(stderr, "[ampnet]   node %d: %d tiles x %d rows%s, %d backward tiles x %d columns, batch %d, slots %d\n", P.node, P.LT > 1 ? P.LT : P.T, P.R, P.tc ? " (tensor cores)" : P.LT > 1 ? " (shared loss head)" : "", P.TB, P.CB, P.BM, P.NS);
  if (R.direct) {
    CUDA_TRY(g, cudaEventRecord(g->ev0, g->stream));
    const cudaError_t le = ampnet_direct_launch(&R.ctx, R.ctx.n_ctas, R.smem_bytes, g->stream, g->n_sms);
    if (le == cudaErrorCooperativeLaunchTooLarge) return set_err(g, AMPNET_EINVAL, "%d CTAs cannot be co-resident", R.ctx.n_ctas);
    if (le != cudaSuccess) return set_err(g, AMPNET_ECUDA, "launch of the direct-delivery engine failed: %s", cudaGetErrorString(le));
  } else {
    CUDA_TRY(g, cudaFuncSetAttribute(ampnet_engine, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)R.smem_bytes));
    int per_sm = 0;
    CUDA_TRY(g, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ampnet_engine, THREADS, R.smem_bytes));
    if (per_sm < 1 || (long long)per_sm * g->n_sms < R.ctx.n_ctas)
      return set_err(g, AMPNET_EINVAL, "%d CTAs cannot be co-resident (%d per SM)", R.ctx.n_ctas, per_sm);
    void* args[] = {&R.ctx};
    CUDA_TRY(g, cudaEventRecord(g->ev0, g->stream));
    CUDA_TRY(g, cudaLaunchCooperativeKernel((void*)ampnet_engine, dim3(R.ctx.n_ctas), dim3(THREADS), args, R.smem_bytes, g->stream));
  }
  CUDA_TRY(g, cudaEventRecord(g->ev1, g->stream));
  Globals G;
  CUDA_TRY(g, cudaMemcpyAsync(&G, R.ctx.g, sizeof G, cudaMemcpyDeviceToHost, g->stream));
  g->last_stats.assign(g->ppts.size(), PPTStats{});
  for (size_t p = 0; p < g->ppts.size(); p++)
    CUDA_TRY(g, cudaMemcpyAsync(&g->last_stats[p], g->d_stats[p], sizeof(PPTStats), cudaMemcpyDeviceToHost, g->stream));
  g->last_node_msgs.assign(R.nodes.size() * 2, 0);
  CUDA_TRY(g, cudaMemcpyAsync(g->last_node_msgs.data(), g->d_node_msgs, g->last_node_msgs.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost, g->stream));
  if (per_instance_loss)
    CUDA_TRY(g, cudaMemcpyAsync(per_instance_loss, R.ctx.loss_out, (size_t)D.n * sizeof(float), cudaMemcpyDeviceToHost, g->stream));
  if (dbg) fprintf(stderr, "[ampnet] launched, waiting\n");
  CUDA_TRY(g, cudaStreamSynchronize(g->stream));
  if (dbg) fprintf(stderr, "[ampnet] done\n");
  g->have_run = true;
  if (!eval) for (size_t p = 0; p < g->ppts.size(); p++) g->ppts[p].opt_t += (long long)g->last_stats[p].n_updates;
  if (!eval && !det && !R.direct && R.ctx.emit_ctas)      // emitter time of the node = time of its first emitter x emitters (they share every batch)
    for (size_t p = 0; p < g->ppts.size(); p++) g->ppts[p].emit_load = (double)G.role_cycles[8 + 8 * p + 5] * std::max(1, g->ppts[p].NE) + 1.0;
  if (getenv("AMPNET_TUNE") && (atoi(getenv("AMPNET_TUNE")) & 8)) {
    static const char* names[] = {"SOURCE", "LINEAR", "LOOKUP", "GRUCELL", "LOSS_CE", "LOSS_MSE", "SUMROWS", "COND", "PHI", "ISU", "CONCAT", "SPLIT", "BCAST", "GROUP", "UNGROUP", "FLATMAP", "SINK", "LSTM"};
    int khz = 1965000;
    cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, g->device);      // cycles -> microseconds at the device's SM clock
    const double us = 1e3 / (double)khz;
    fprintf(stderr, "[ctrl] us: retire %.0f admit %.0f clear %.0f pump %.0f idle %.0f admissions %llu\n", G.role_cycles[0] * us, G.role_cycles[1] * us,
            G.role_cycles[2] * us, G.role_cycles[3] * us, G.role_cycles[4] * us, G.role_cycles[5]);
    for (size_t p = 0; p < g->ppts.size(); p++) {
      const unsigned long long* r = G.role_cycles + 8 + 8 * p;
      fprintf(stderr, "[role] node %2d sched us: wait-tile %.0f no-msg %.0f form %.0f (context %.0f) | emitter(0,0) us: wait %.0f load %.0f emit %.0f batches %llu\n",
              g->ppts[p].node, r[0] * us, r[1] * us, r[2] * us, r[7] * us, r[3] * us, r[4] * us, r[5] * us, r[6]);
    }
    for (size_t p = 0; p < g->ppts.size(); p++) {
      fprintf(stderr, "[step] node %2d us:", g->ppts[p].node);
      for (int k = 0; k < 12; k++) fprintf(stderr, " %.0f", G.step_cycles[p][k] * us);
      fprintf(stderr, "\n");
    }
    for (int t = 0; t < N_NODE_TYPES * 2; t++)
      if (G.walk_steps[t]) fprintf(stderr, "[walk] %-8s %s steps %10llu cycles/step %8.0f\n", names[t / 2], t & 1 ? "BWD" : "FWD", G.walk_steps[t], (double)G.walk_cycles[t] / G.walk_steps[t]);
  }
  g->n_keylog = det ? G.n_keylog : 0;
  float ms = 0;
  CUDA_TRY(g, cudaEventElapsedTime(&ms, g->ev0, g->ev1));
  if (ctl_trial && G.status == 0 && G.node_messages > 0 && ms > 0) {     // epochs 0, 1 at the first position, epoch 2 at the second
    g->ctl_trials++;
    if (g->ctl_trials == 2) g->ctl_rate[0] = (double)G.node_messages / ms;
    if (g->ctl_trials == 3) { g->ctl_rate[1] = (double)G.node_messages / ms; g->ctl_choice = g->ctl_rate[1] > 1.03 * g->ctl_rate[0] ? 1 : 0; }
  }
  if (out) {
    std::memset(out, 0, sizeof *out);
    out->instances = n_order; out->node_messages = (int64_t)G.node_messages; out->rounds = (int64_t)G.rounds;
    out->seconds = ms * 1e-3; const long long n_train = n_order - (long long)G.inf_instances;
    out->mean_loss = n_train > 0 ? G.total_loss / (double)n_train : 0.0;
    out->max_active_observed = G.max_active; out->route_hash = G.route_hash;
    for (auto& s : g->last_stats) {
      out->ppt_messages += (int64_t)s.msgs; out->max_staleness = std::max(out->max_staleness, s.max_staleness);
      out->micro_batches += (int64_t)s.batches; out->micro_batch_rows += (int64_t)s.batch_rows;
    }
  }
  if (accuracy) *accuracy = G.n_pred ? (double)G.correct / (double)G.n_pred : 0.0;
  if (inference) {
    inference->instances = (int64_t)G.inf_instances;
    inference->mean_loss = G.inf_instances ? G.inf_loss / (double)G.inf_instances : 0.0;
    inference->accuracy = G.inf_pred ? (double)G.inf_correct / (double)G.inf_pred : 0.0;
  }
  if (G.status == ST_TIMEOUT) return set_err(g, AMPNET_ETIMEOUT, "a bounded device wait gave up (node %d, detail %d)", G.err_node, G.err_detail);
  if (G.status == ST_OVERFLOW) return set_err(g, AMPNET_EOVERFLOW, "a queue / cache / key-space bound was exceeded (node %d, detail %d)", G.err_node, G.err_detail);
  if (G.status != 0) return set_err(g, AMPNET_ECUDA, "device status %d", G.status);
  return AMPNET_OK;
}

}  // namespace

// ---------------------------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------------------------
extern "C" {

ampnet_status_t ampnet_graph_create(const ampnet_ir_desc_t* ir, uint64_t init_seed, void* cuda_stream,
                                    const ampnet_allocator_t* allocator, ampnet_graph_t** out) {
  if (!out) return AMPNET_EINVAL;
  *out = nullptr;
  if (!ir || !ir->nodes || ir->n_nodes < 1 || ir->n_edges < 0 || (ir->n_edges > 0 && !ir->edges)) return AMPNET_EINVAL;
  if (ir->payload_dtype != 0 && ir->payload_dtype != 1) return AMPNET_EINVAL;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return AMPNET_ECUDA;
  ampnet_graph* g = new ampnet_graph();
  g->nodes.assign(ir->nodes, ir->nodes + ir->n_nodes);
  if (ir->n_edges) g->edges.assign(ir->edges, ir->edges + ir->n_edges);
  g->payload_bf16 = ir->payload_dtype == 1;
  if (allocator) g->alloc = *allocator;
  g->stream = (cudaStream_t)cuda_stream;
  ampnet_status_t st = AMPNET_OK;
  cudaDeviceProp prop;
  if (cudaGetDevice(&g->device) != cudaSuccess || cudaGetDeviceProperties(&prop, g->device) != cudaSuccess) st = AMPNET_ECUDA;
  if (st == AMPNET_OK) {
    g->n_sms = prop.multiProcessorCount;
    g->max_smem = (int)prop.sharedMemPerBlockOptin;
    if (!prop.cooperativeLaunch) st = set_err(g, AMPNET_ECUDA, "the device does not support cooperative launch");
  }
  if (st == AMPNET_OK) st = build_topology(g);
  if (st == AMPNET_OK) st = create_params(g, init_seed);
  if (st == AMPNET_OK && (cudaEventCreate(&g->ev0) != cudaSuccess || cudaEventCreate(&g->ev1) != cudaSuccess)) st = AMPNET_ECUDA;
  if (st != AMPNET_OK) {
    // keep the message readable through a static buffer: the handle is not returned
    static thread_local std::string last;
    last = g->err;
    ampnet_graph_destroy(g);
    return st;
  }
  *out = g;
  return AMPNET_OK;
}

void ampnet_graph_destroy(ampnet_graph_t* g) {
  if (!g) return;
  cudaStreamSynchronize(g->stream);
  for (auto& P : g->ppts) { dev_free(g, P.W); dev_free(g, P.b); dev_free(g, P.om); dev_free(g, P.ov); }
  free_dataset(g, g->data[0]);
  free_dataset(g, g->data[1]);
  dev_free(g, g->ctl_alloc);
  dev_free(g, g->bulk_mem);
  if (g->ev0) cudaEventDestroy(g->ev0);
  if (g->ev1) cudaEventDestroy(g->ev1);
  delete g;
}

ampnet_status_t ampnet_set_optimizer(ampnet_graph_t* g, int32_t kind, float momentum, float beta1, float beta2, float eps,
                                     int32_t reset_state) {
  if (!g) return AMPNET_EINVAL;
  if (kind < AMPNET_OPT_SGD || kind > AMPNET_OPT_ADAM) return set_err(g, AMPNET_EINVAL, "unknown optimiser %d", kind);
  if (kind == AMPNET_OPT_MOMENTUM && !(momentum >= 0.f && momentum < 1.f)) return set_err(g, AMPNET_EINVAL, "momentum must lie in [0, 1)");
  if (kind == AMPNET_OPT_ADAM && !(beta1 >= 0.f && beta1 < 1.f && beta2 >= 0.f && beta2 < 1.f && eps > 0.f))
    return set_err(g, AMPNET_EINVAL, "Adam needs beta1, beta2 in [0, 1) and eps > 0");
  CUDA_TRY(g, cudaSetDevice(g->device));
  CUDA_TRY(g, cudaStreamSynchronize(g->stream));
  for (auto& P : g->ppts) {
    const size_t bytes = (P.nW + P.nb) * sizeof(float);
    float** want[2] = {kind >= AMPNET_OPT_MOMENTUM ? &P.om : nullptr, kind == AMPNET_OPT_ADAM ? &P.ov : nullptr};
    for (float** w : want) {
      if (!w) continue;
      const bool fresh = *w == nullptr;
      if (fresh && !(*w = (float*)dev_alloc(g, bytes))) return set_err(g, AMPNET_ENOMEM, "optimiser state allocation of %zu bytes failed", bytes);
      if (fresh || reset_state) CUDA_TRY(g, cudaMemsetAsync(*w, 0, bytes, g->stream));
    }
    if (reset_state) P.opt_t = 0;
  }
  CUDA_TRY(g, cudaStreamSynchronize(g->stream));
  g->opt = kind; g->opt_mu = momentum; g->opt_beta1 = beta1; g->opt_beta2 = beta2; g->opt_eps = eps;
  return AMPNET_OK;
}

ampnet_status_t ampnet_average_params(ampnet_graph_t* g, const int32_t* nodes, int32_t n) {
  if (!g) return AMPNET_EINVAL;
  if (!nodes || n < 1 || n > 8) return set_err(g, AMPNET_EINVAL, "between 1 and 8 nodes are averaged");
  AvgArgs a{};
  const HostPPT* first = nullptr;
  for (int k = 0; k < n; k++) {
    const int node = nodes[k];
    if (node < 0 || node >= (int)g->hnodes.size() || g->hnodes[node].ppt < 0) return set_err(g, AMPNET_EINVAL, "node %d has no parameters", node);
    const HostPPT& P = g->ppts[g->hnodes[node].ppt];
    if (!first) first = &P;
    if (P.kind != first->kind || P.nW != first->nW || P.nb != first->nb) return set_err(g, AMPNET_EINVAL, "node %d differs in type or shape from node %d", node, nodes[0]);
    for (int j = 0; j < k; j++) if (nodes[j] == node) return set_err(g, AMPNET_EINVAL, "node %d is listed twice", node);
    a.W[k] = P.W; a.b[k] = P.b;
  }
  a.n = n; a.nW = (long long)first->nW; a.nb = (long long)first->nb;
  CUDA_TRY(g, cudaSetDevice(g->device));
  const long long total = a.nW + a.nb;
  const int blocks = (int)std::min<long long>((total + 255) / 256, 148 * 8);
  average_params_kernel<<<blocks, 256, 0, g->stream>>>(a);
  CUDA_TRY(g, cudaGetLastError());
  CUDA_TRY(g, cudaStreamSynchronize(g->stream));
  return AMPNET_OK;
}

ampnet_status_t ampnet_measure_fma_peak(int32_t device, double* tflops) {
  if (!tflops) return AMPNET_EINVAL;
  cudaDeviceProp prop{};
  if (cudaSetDevice(device) != cudaSuccess || cudaGetDeviceProperties(&prop, device) != cudaSuccess) return AMPNET_ECUDA;
  float* sink = nullptr;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (cudaMalloc(&sink, 256) != cudaSuccess) return AMPNET_ENOMEM;
  ampnet_status_t rc = AMPNET_OK;
  const int blocks = prop.multiProcessorCount * 8, iters = 1 << 16;
  float best_ms = 1e30f;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) rc = AMPNET_ECUDA;
  for (int rep = 0; rep < 4 && rc == AMPNET_OK; rep++) {        // the first repetition warms up
    cudaEventRecord(e0, 0);
    fma_peak_kernel<<<blocks, 256>>>(sink, iters);
    cudaEventRecord(e1, 0);
    float ms = 0.f;
    if (cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) rc = AMPNET_ECUDA;
    else if (rep > 0) best_ms = std::min(best_ms, ms);
  }
  if (rc == AMPNET_OK) *tflops = (double)blocks * 256.0 * 16.0 * 2.0 * (double)iters / (best_ms * 1e-3) / 1e12;
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  cudaFree(sink);
  return rc;
}

const char* ampnet_last_error(const ampnet_graph_t* g) { return g ? g->err.c_str() : "invalid handle"; }

ampnet_status_t ampnet_load_instances(ampnet_graph_t* g, int32_t split, const ampnet_instances_t* in) {
  if (!g) return AMPNET_EINVAL;
  if (split < 0 || split > 1 || !in) return set_err(g, AMPNET_EINVAL, "bad split or NULL instances");
  if (in->n_instances < 0 || in->kind < 0 || in->kind > 3) return set_err(g, AMPNET_EINVAL, "bad kind or instance count");
  CUDA_TRY(g, cudaSetDevice(g->device));
  CUDA_TRY(g, cudaStreamSynchronize(g->stream));
  free_dataset(g, g->data[split]);
  HostDataset& D = g->data[split];
  const long long n = in->n_instances;
  D.kind = in->kind; D.n = n;
  // which inputs does the graph need
  int vocab = 0; bool per_node_labels = false, need_int_labels = false, need_float_labels = false;
  for (auto& h : g->hnodes) {
    if (h.type == LOOKUP) vocab = vocab ? std::min(vocab, h.in_dim) : h.in_dim;
    if (h.type == LOSS_CE) { need_int_labels = true; if (h.fn == 2) per_node_labels = true; }
    if (h.type == LOSS_MSE) need_float_labels = true;
  }
  for (int s : g->sources) {
    const int fn = g->hnodes[s].fn;
    const int want = fn == 1 ? 0 : fn == 2 ? 1 : (fn == 4 || fn == 6) ? 2 : fn == 5 ? 3 : -1;
    if (want >= 0 && want != in->kind) return set_err(g, AMPNET_EINVAL, "instance kind %d does not match the graph's source (fn %d)", in->kind, fn);
    if (fn == 1 && g->hnodes[s].out_dim != in->dense_dim) return set_err(g, AMPNET_EINVAL, "dense_dim %d does not match the source width %d", in->dense_dim, g->hnodes[s].out_dim);
  }
  if (need_int_labels && !in->labels_i) return set_err(g, AMPNET_EINVAL, "labels_i is required by the loss");
  if (need_float_labels && !in->labels_f) return set_err(g, AMPNET_EINVAL, "labels_f is required by the loss");
  D.labels_per_node = per_node_labels ? 1 : 0;
  DevInst& V = D.dev;
  V = DevInst{};
  V.kind = in->kind; V.n = n; V.labels_per_node = D.labels_per_node;
  ampnet_status_t st;
  long long total = 0;
  if (in->kind == AMPNET_KIND_DENSE_ROWS) {
    if (!in->dense || in->dense_dim < 1) return set_err(g, AMPNET_EINVAL, "dense rows need dense and dense_dim");
    D.dense_dim = V.dense_dim = in->dense_dim;
    if ((st = upload_raw(g, D, in->dense, (size_t)n * in->dense_dim, &V.dense)) != AMPNET_OK) return st;
  } else {
    if (!in->offsets || !in->tokens) return set_err(g, AMPNET_EINVAL, "offsets and tokens are required");
    if (in->offsets[0] != 0) return set_err(g, AMPNET_EINVAL, "offsets[0] must be 0");
    for (long long i = 0; i < n; i++) {
      const long long len = in->offsets[i + 1] - in->offsets[i];
      if (len < 1) return set_err(g, AMPNET_EINVAL, "instance %lld is empty", i);
      if (len > 16000) return set_err(g, AMPNET_EINVAL, "instance %lld has %lld positions (max 16000)", i, len);
    }
    total = in->offsets[n];
    D.total_pos = total;
    if ((st = upload_raw(g, D, in->offsets, (size_t)n + 1, reinterpret_cast<const int64_t**>(&V.offsets))) != AMPNET_OK) return st;
    if ((st = upload_raw(g, D, in->tokens, (size_t)total, &V.tokens)) != AMPNET_OK) return st;
  }
  if (in->kind == AMPNET_KIND_SEQUENCES) {
    for (long long i = 0; i < n; i++) D.maxT = std::max<int>(D.maxT, (int)(in->offsets[i + 1] - in->offsets[i]));
    for (long long k = 0; k < total; k++)
      if (in->tokens[k] < 0 || (vocab && in->tokens[k] >= vocab)) return set_err(g, AMPNET_EINVAL, "token %lld = %d outside the vocabulary", k, in->tokens[k]);
  } else if (in->kind == AMPNET_KIND_BINARY_TREES) {
    if (!in->left || !in->right) return set_err(g, AMPNET_EINVAL, "trees need left and right");
    std::vector<int> parent((size_t)total, -1), cslot((size_t)total, 0), root((size_t)n, -1), leaf_ids;
    std::vector<long long> leaf_off((size_t)n + 1, 0);
    for (long long i = 0; i < n; i++) {
      const long long o = in->offsets[i];
      const int m = (int)(in->offsets[i + 1] - o);
      D.maxM = std::max(D.maxM, m);
      int nl = 0;
      for (int u = 0; u < m; u++) {
        const int l = in->left[o + u], r = in->right[o + u];
        if ((l < 0) != (r < 0)) return set_err(g, AMPNET_EINVAL, "tree %lld node %d has exactly one child", i, u);
        if (l >= 0) {
          if (l >= u || r >= u || l == r) return set_err(g, AMPNET_EINVAL, "tree %lld node %d: children must precede their parent", i, u);
          if (parent[o + l] >= 0 || parent[o + r] >= 0) return set_err(g, AMPNET_EINVAL, "tree %lld: node with two parents", i);
          parent[o + l] = u; cslot[o + l] = 0; parent[o + r] = u; cslot[o + r] = 1;
        } else {
          const int t = in->tokens[o + u];
          if (t < 0 || (vocab && t >= vocab)) return set_err(g, AMPNET_EINVAL, "tree %lld leaf %d: token %d outside the vocabulary", i, u, t);
          leaf_ids.push_back(u); nl++;
        }
      }
      int nroot = 0;
      for (int u = 0; u < m; u++) if (parent[o + u] < 0) { root[i] = u; nroot++; }
      if (nroot != 1) return set_err(g, AMPNET_EINVAL, "tree %lld has %d roots", i, nroot);
      leaf_off[i + 1] = leaf_off[i] + nl;
      D.maxL = std::max(D.maxL, nl);
    }
    if ((st = upload_raw(g, D, in->left, (size_t)total, &V.left)) != AMPNET_OK) return st;
    if ((st = upload_raw(g, D, in->right, (size_t)total, &V.right)) != AMPNET_OK) return st;
    if ((st = upload(g, D, parent, &V.parent)) != AMPNET_OK) return st;
    if ((st = upload(g, D, cslot, &V.child_slot)) != AMPNET_OK) return st;
    if ((st = upload(g, D, root, &V.root)) != AMPNET_OK) return st;
    if ((st = upload(g, D, leaf_off, &V.leaf_off)) != AMPNET_OK) return st;
    if ((st = upload(g, D, leaf_ids, &V.leaf_ids)) != AMPNET_OK) return st;
  } else if (in->kind == AMPNET_KIND_TYPED_GRAPHS) {
    if (!in->edge_offsets || !in->edge_src || !in->edge_dst || !in->edge_type) return set_err(g, AMPNET_EINVAL, "graphs need the edge arrays");
    const long long E = in->edge_offsets[n];
    D.total_edges = E;
    int NT = 1;
    for (long long e = 0; e < E; e++) {
      if (in->edge_type[e] < 0 || in->edge_type[e] >= MAX_PORTS) return set_err(g, AMPNET_EINVAL, "edge %lld: type %d out of range", e, in->edge_type[e]);
      NT = std::max(NT, in->edge_type[e] + 1);
    }
    for (auto& h : g->hnodes) if (h.type == COND && h.fn == 3) NT = std::max(NT, h.n_succ);
    D.NT = V.NT = NT;
    std::vector<long long> out_off((size_t)total + 1, 0), in_off((size_t)total + 1, 0), type_off((size_t)n * NT + 1, 0);
    std::vector<int> out_list((size_t)E), in_list((size_t)E), type_list((size_t)E), rank_out((size_t)E), rank_in((size_t)E), rank_type((size_t)E);
    for (long long i = 0; i < n; i++) {
      const long long o = in->offsets[i], eo = in->edge_offsets[i];
      const int N = (int)(in->offsets[i + 1] - o), ne = (int)(in->edge_offsets[i + 1] - eo);
      if (ne < 0) return set_err(g, AMPNET_EINVAL, "graph %lld: negative edge count", i);
      D.maxN = std::max(D.maxN, N); D.maxD = std::max(D.maxD, ne);
      std::vector<int> od(N, 0), id(N, 0), td(NT, 0);
      for (int e = 0; e < ne; e++) {
        const int s = in->edge_src[eo + e], d = in->edge_dst[eo + e];
        if (s < 0 || s >= N || d < 0 || d >= N) return set_err(g, AMPNET_EINVAL, "graph %lld edge %d: endpoint out of range", i, e);
        rank_out[eo + e] = od[s]++; rank_in[eo + e] = id[d]++; rank_type[eo + e] = td[in->edge_type[eo + e]]++;
      }
      for (int v = 0; v < N; v++) {
        if (od[v] == 0 || id[v] == 0) return set_err(g, AMPNET_EINVAL, "graph %lld: node %d has no incoming or no outgoing edge", i, v);
        out_off[o + v + 1] = out_off[o + v] + od[v]; in_off[o + v + 1] = in_off[o + v] + id[v];
        D.maxOut = std::max(D.maxOut, od[v]); D.maxIn = std::max(D.maxIn, id[v]);
        const int t = in->tokens[o + v];
        if (t < 0 || (vocab && t >= vocab)) return set_err(g, AMPNET_EINVAL, "graph %lld node %d: type %d outside the vocabulary", i, v, t);
      }
      for (int c = 0; c < NT; c++) { type_off[i * NT + c + 1] = type_off[i * NT + c] + td[c]; D.maxDc = std::max(D.maxDc, td[c]); }
      for (int e = 0; e < ne; e++) {
        const int s = in->edge_src[eo + e], d = in->edge_dst[eo + e], c = in->edge_type[eo + e];
        out_list[out_off[o + s] + rank_out[eo + e]] = e;
        in_list[in_off[o + d] + rank_in[eo + e]] = e;
        type_list[type_off[i * NT + c] + rank_type[eo + e]] = e;
      }
    }
    if ((st = upload_raw(g, D, in->edge_offsets, (size_t)n + 1, reinterpret_cast<const int64_t**>(&V.edge_off))) != AMPNET_OK) return st;
    if ((st = upload_raw(g, D, in->edge_src, (size_t)E, &V.esrc)) != AMPNET_OK) return st;
    if ((st = upload_raw(g, D, in->edge_dst, (size_t)E, &V.edst)) != AMPNET_OK) return st;
    if ((st = upload_raw(g, D, in->edge_type, (size_t)E, &V.etype)) != AMPNET_OK) return st;
    if ((st = upload(g, D, rank_out, &V.rank_out)) != AMPNET_OK) return st;
    if ((st = upload(g, D, rank_in, &V.rank_in)) != AMPNET_OK) return st;
    if ((st = upload(g, D, rank_type, &V.rank_type)) != AMPNET_OK) return st;
    if ((st = upload(g, D, out_off, &V.out_off)) != AMPNET_OK) return st;
    if ((st = upload(g, D, in_off, &V.in_off)) != AMPNET_OK) return st;
    if ((st = upload(g, D, type_off, &V.type_off)) != AMPNET_OK) return st;
    if ((st = upload(g, D, out_list, &V.out_list)) != AMPNET_OK) return st;
    if ((st = upload(g, D, in_list, &V.in_list)) != AMPNET_OK) return st;
    if ((st = upload(g, D, type_list, &V.type_list)) != AMPNET_OK) return st;
  }
  if (in->labels_i) {
    const size_t nl = per_node_labels ? (size_t)total : (size_t)n;
    int classes = 0;
    for (int l : g->losses) if (g->hnodes[l].type == LOSS_CE) classes = g->hnodes[l].in_dim;
    for (size_t k = 0; k < nl && classes; k++)
      if (in->labels_i[k] < 0 || in->labels_i[k] >= classes) return set_err(g, AMPNET_EINVAL, "label %zu = %d outside 0..%d", k, in->labels_i[k], classes - 1);
    if ((st = upload_raw(g, D, in->labels_i, nl, &V.labels_i)) != AMPNET_OK) return st;
  }
  if (in->labels_f) if ((st = upload_raw(g, D, in->labels_f, (size_t)n, &V.labels_f)) != AMPNET_OK) return st;
  CUDA_TRY(g, cudaStreamSynchronize(g->stream));
  D.loaded = true;
  return AMPNET_OK;
}

ampnet_status_t ampnet_run_epoch(ampnet_graph_t* g, const ampnet_run_cfg_t* cfg, ampnet_epoch_stats_t* out,
                                 float* per_instance_loss) {
  if (!g) return AMPNET_EINVAL;
  if (!cfg) return set_err(g, AMPNET_EINVAL, "NULL run configuration");
  return execute(g, 0, cfg->max_active_keys, cfg->deterministic ? 1 : 0, 0, cfg, out, per_instance_loss, nullptr);
}

ampnet_status_t ampnet_run_epoch_mixed(ampnet_graph_t* g, const ampnet_run_cfg_t* cfg, const uint8_t* inference_only,
                                       ampnet_epoch_stats_t* out, float* per_instance_loss, ampnet_inference_stats_t* inference) {
  if (!g) return AMPNET_EINVAL;
  if (!cfg || !inference_only) return set_err(g, AMPNET_EINVAL, "NULL run configuration or mask");
  return execute(g, 0, cfg->max_active_keys, cfg->deterministic ? 1 : 0, 0, cfg, out, per_instance_loss, nullptr, inference_only, inference);
}

ampnet_status_t ampnet_eval(ampnet_graph_t* g, int32_t split, int32_t max_active_keys, double* mean_loss,
                            double* accuracy, float* per_instance_loss) {
  if (!g) return AMPNET_EINVAL;
  if (split < 0 || split > 1) return set_err(g, AMPNET_EINVAL, "bad split");
  ampnet_run_cfg_t cfg{};
  cfg.max_active_keys = max_active_keys > 0 ? max_active_keys : 64;
  cfg.min_update_frequency = 1;
  ampnet_epoch_stats_t st{};
  ampnet_status_t rc = execute(g, split, cfg.max_active_keys, 0, 1, &cfg, &st, per_instance_loss, accuracy);
  if (mean_loss) *mean_loss = st.mean_loss;
  return rc;
}

static HostPPT* find_ppt(ampnet_graph_t* g, int node) {
  if (!g || node < 0 || node >= (int)g->hnodes.size() || g->hnodes[node].ppt < 0) return nullptr;
  return &g->ppts[g->hnodes[node].ppt];
}
static bool param_slice(const HostPPT& P, int which, float** base, size_t* n) {
  if (P.kind == LINEAR) {
    if (which == 0) { *base = P.W; *n = P.nW; return true; }
    if (which == 1) { *base = P.b; *n = P.nb; return true; }
  } else if (P.kind == LOOKUP) {
    if (which == 0) { *base = P.W; *n = P.nW; return true; }
  } else if (P.kind == GRUCELL) {
    const size_t m = (size_t)P.in * P.out;
    if (which >= 0 && which < 3) { *base = P.W + which * m; *n = m; return true; }
    if (which >= 3 && which < 6) { *base = P.b + (which - 3) * P.out; *n = P.out; return true; }
  }
  return false;
}

ampnet_status_t ampnet_param_count(ampnet_graph_t* g, int32_t node, int32_t which, int64_t* n) {
  HostPPT* P = find_ppt(g, node);
  float* b; size_t c;
  if (!P || !n || !param_slice(*P, which, &b, &c)) return g ? set_err(g, AMPNET_EINVAL, "no parameter (%d, %d)", node, which) : AMPNET_EINVAL;
  *n = (int64_t)c;
  return AMPNET_OK;
}
ampnet_status_t ampnet_get_params(ampnet_graph_t* g, int32_t node, int32_t which, float* dst, int64_t n) {
  HostPPT* P = find_ppt(g, node);
  float* b; size_t c;
  if (!P || !dst || !param_slice(*P, which, &b, &c) || (int64_t)c != n) return g ? set_err(g, AMPNET_EINVAL, "bad parameter request (%d, %d, %lld)", node, which, (long long)n) : AMPNET_EINVAL;
  CUDA_TRY(g, cudaMemcpyAsync(dst, b, c * sizeof(float), cudaMemcpyDeviceToHost, g->stream));
  CUDA_TRY(g, cudaStreamSynchronize(g->stream));
  return AMPNET_OK;
}
ampnet_status_t ampnet_param_device_ptr(ampnet_graph_t* g, int32_t node, int32_t which, float** dev, int64_t* n) {
  HostPPT* P = find_ppt(g, node);
  float* b; size_t c;
  if (!P || !dev || !param_slice(*P, which, &b, &c)) return g ? set_err(g, AMPNET_EINVAL, "no parameter (%d, %d)", node, which) : AMPNET_EINVAL;
  CUDA_TRY(g, cudaStreamSynchronize(g->stream));
  *dev = b;
  if (n) *n = (int64_t)c;
  return AMPNET_OK;
}
ampnet_status_t ampnet_set_params(ampnet_graph_t* g, int32_t node, int32_t which, const float* src, int64_t n) {
  HostPPT* P = find_ppt(g, node);
  float* b; size_t c;
  if (!P || !src || !param_slice(*P, which, &b, &c) || (int64_t)c != n) return g ? set_err(g, AMPNET_EINVAL, "bad parameter request (%d, %d, %lld)", node, which, (long long)n) : AMPNET_EINVAL;
  CUDA_TRY(g, cudaMemcpyAsync(b, src, c * sizeof(float), cudaMemcpyHostToDevice, g->stream));
  CUDA_TRY(g, cudaStreamSynchronize(g->stream));
  return AMPNET_OK;
}

ampnet_status_t ampnet_get_node_stats(ampnet_graph_t* g, int32_t node, int64_t* n_updates, int64_t* n_grads_applied,
                                      int64_t* staleness_hist, int64_t* fwd_msgs, int64_t* bwd_msgs) {
  if (!g) return AMPNET_EINVAL;
  if (!g->have_run) return set_err(g, AMPNET_ESTATE, "no run yet");
  if (node < 0 || node >= (int)g->hnodes.size()) return set_err(g, AMPNET_EINVAL, "bad node");
  if (fwd_msgs) *fwd_msgs = (int64_t)g->last_node_msgs[node * 2];
  if (bwd_msgs) *bwd_msgs = (int64_t)g->last_node_msgs[node * 2 + 1];
  const int p = g->hnodes[node].ppt;
  if (n_updates) *n_updates = p >= 0 ? (int64_t)g->last_stats[p].n_updates : 0;
  if (n_grads_applied) *n_grads_applied = p >= 0 ? (int64_t)g->last_stats[p].n_grads_applied : 0;
  if (staleness_hist) for (int k = 0; k < 64; k++) staleness_hist[k] = p >= 0 ? (int64_t)g->last_stats[p].stale_hist[k] : 0;
  return AMPNET_OK;
}

ampnet_status_t ampnet_get_update_log(ampnet_graph_t* g, int32_t node, int32_t* n_per_update, int64_t cap, int64_t* n) {
  if (!g) return AMPNET_EINVAL;
  if (!g->have_run) return set_err(g, AMPNET_ESTATE, "no run yet");
  if (node < 0 || node >= (int)g->hnodes.size() || g->hnodes[node].ppt < 0) return set_err(g, AMPNET_EINVAL, "not a parameterised node");
  const int p = g->hnodes[node].ppt;
  const int64_t have = std::min<int64_t>(g->last_stats[p].log_n, g->update_log_cap);
  if (n) *n = g->last_stats[p].log_n;
  const int64_t c = std::min(have, cap);
  if (c > 0 && n_per_update) {
    CUDA_TRY(g, cudaMemcpyAsync(n_per_update, g->d_update_log[p], (size_t)c * sizeof(int), cudaMemcpyDeviceToHost, g->stream));
    CUDA_TRY(g, cudaStreamSynchronize(g->stream));
  }
  return AMPNET_OK;
}

ampnet_status_t ampnet_get_key_log(ampnet_graph_t* g, int64_t* inst, int32_t* slot, int64_t* admit_round,
                                   int64_t* release_round, int64_t cap, int64_t* n) {
  if (!g) return AMPNET_EINVAL;
  if (!g->have_run) return set_err(g, AMPNET_ESTATE, "no run yet");
  if (n) *n = g->n_keylog;
  const int64_t c = std::min<int64_t>(g->n_keylog, cap);
  if (c > 0) {
    std::vector<KeyLog> h((size_t)c);
    CUDA_TRY(g, cudaMemcpyAsync(h.data(), g->d_keylog, (size_t)c * sizeof(KeyLog), cudaMemcpyDeviceToHost, g->stream));
    CUDA_TRY(g, cudaStreamSynchronize(g->stream));
    for (int64_t i = 0; i < c; i++) {
      if (inst) inst[i] = h[i].inst;
      if (slot) slot[i] = h[i].slot;
      if (admit_round) admit_round[i] = h[i].admit;
      if (release_round) release_round[i] = h[i].release;
    }
  }
  return AMPNET_OK;
}

ampnet_status_t ampnet_leftover_cache_entries(ampnet_graph_t* g, int64_t* n) {
  if (!g || !n) return AMPNET_EINVAL;
  if (!g->have_run) return set_err(g, AMPNET_ESTATE, "no run yet");
  int64_t cnt = 0;
  std::vector<unsigned char> h;
  for (auto& r : g->leftover_regions) {
    h.resize(r.second);
    CUDA_TRY(g, cudaMemcpyAsync(h.data(), (char*)g->ctl_mem + r.first, r.second, cudaMemcpyDeviceToHost, g->stream));
    CUDA_TRY(g, cudaStreamSynchronize(g->stream));
    for (unsigned char c : h) cnt += c != 0;
  }
  *n = cnt;
  return AMPNET_OK;
}

ampnet_status_t ampnet_get_phase_cycles(ampnet_graph_t* g, int32_t node, uint64_t* cycles8, int64_t* batches) {
  if (!g) return AMPNET_EINVAL;
  if (!g->have_run) return set_err(g, AMPNET_ESTATE, "no run yet");
  if (node < 0 || node >= (int)g->hnodes.size() || g->hnodes[node].ppt < 0) return set_err(g, AMPNET_EINVAL, "not a parameterised node");
  const PPTStats& s = g->last_stats[g->hnodes[node].ppt];
  if (cycles8) for (int k = 0; k < 16; k++) cycles8[k] = s.phase_cycles[k];
  if (batches) *batches = (int64_t)s.batches;
  return AMPNET_OK;
}

ampnet_status_t ampnet_get_queue_occupancy(ampnet_graph_t* g, int32_t node, int64_t* max_pending_fwd, int64_t* max_pending_bwd) {
  if (!g) return AMPNET_EINVAL;
  if (!g->have_run) return set_err(g, AMPNET_ESTATE, "no run yet");
  if (node < 0 || node >= (int)g->hnodes.size() || g->hnodes[node].ppt < 0) return set_err(g, AMPNET_EINVAL, "not a parameterised node");
  const PPTStats& s = g->last_stats[g->hnodes[node].ppt];
  if (max_pending_fwd) *max_pending_fwd = (int64_t)s.max_pending[0];
  if (max_pending_bwd) *max_pending_bwd = (int64_t)s.max_pending[1];
  return AMPNET_OK;
}

ampnet_status_t ampnet_get_micro_batch_split(ampnet_graph_t* g, int32_t node, int64_t* fma_batches, int64_t* tensor_core_batches) {
  if (!g) return AMPNET_EINVAL;
  if (!g->have_run) return set_err(g, AMPNET_ESTATE, "no run yet");
  if (node < 0 || node >= (int)g->hnodes.size() || g->hnodes[node].ppt < 0) return set_err(g, AMPNET_EINVAL, "not a parameterised node");
  const PPTStats& s = g->last_stats[g->hnodes[node].ppt];
  if (fma_batches) *fma_batches = (int64_t)(s.batches - s.tc_batches);
  if (tensor_core_batches) *tensor_core_batches = (int64_t)s.tc_batches;
  return AMPNET_OK;
}

ampnet_status_t ampnet_get_placement(ampnet_graph_t* g, int32_t node, int32_t* n_tiles, int32_t* batch_rows) {
  HostPPT* P = find_ppt(g, node);
  if (!P) return g ? set_err(g, AMPNET_EINVAL, "not a parameterised node") : AMPNET_EINVAL;
  if (n_tiles) *n_tiles = P->LT > 1 ? P->LT : P->T;
  if (batch_rows) *batch_rows = P->BM;
  return AMPNET_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------------------
// Training epoch that allocates nothing
// ---------------------------------------------------------------------------------------------------------
// Scratch of ampnet_run_epoch_static: the queues, counters and keyed caches of one run.  It lives in the
// library image, so every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[AMPNET_STATIC_SCRATCH_BYTES];
// In host code the array's name is only a stand-in; the device address comes from cudaGetSymbolAddress.
static void* g_static_scratch_addr[64] = {nullptr};

extern "C" ampnet_status_t ampnet_run_epoch_static(ampnet_graph_t* g, const ampnet_run_cfg_t* cfg,
                                                   ampnet_epoch_stats_t* out, float* per_instance_loss) {
  if (!g) return AMPNET_EINVAL;
  if (!cfg) return set_err(g, AMPNET_EINVAL, "NULL run configuration");
  if (g->device < 0 || g->device >= 64) return set_err(g, AMPNET_EINVAL, "device index %d not supported", g->device);
  HostDataset& D = g->data[0];
  if (!D.loaded) return set_err(g, AMPNET_ESTATE, "no instances loaded for split 0");
  if (cfg->max_active_keys < 1 || cfg->min_update_frequency < 1) return set_err(g, AMPNET_EINVAL, "max_active_keys and min_update_frequency must be >= 1");
  CUDA_TRY(g, cudaSetDevice(g->device));
  if (!g_static_scratch_addr[g->device]) {       // set-up, once per device, with that device current
    void* ptr = nullptr;
    CUDA_TRY(g, cudaGetSymbolAddress(&ptr, g_static_scratch));
    g_static_scratch_addr[g->device] = ptr;
  }
  // size the run state without touching any memory, and refuse what does not fit
  const long long n_order = cfg->order ? cfg->n_order : D.n;
  RunPlan plan;
  g->have_run = false;                // the dry plan re-targets the statistics pointers of the previous run
  ampnet_status_t st = plan_run(g, 0, cfg->max_active_keys, cfg->deterministic ? 1 : 0, 0, cfg, n_order, true, plan);
  if (st != AMPNET_OK) return st;
  const size_t order_bytes = cfg->order ? (size_t)std::max<long long>(n_order, 0) * sizeof(long long) : 0;
  // the very sizes execute() will ask ensure_arenas() for
  const size_t ctl_need = ((g->ctl.used + ARENA_SLACK + 255) & ~(size_t)255);
  const size_t bulk_need = g->bulk.used + order_bytes + BULK_EXTRA + ARENA_SLACK;
  if (ctl_need + bulk_need > (size_t)AMPNET_STATIC_SCRATCH_BYTES)
    return set_err(g, AMPNET_EINVAL, "this run needs %zu bytes of scratch but the static scratch holds %zu: lower "
                   "max_active_keys or use ampnet_run_epoch", ctl_need + bulk_need, (size_t)AMPNET_STATIC_SCRATCH_BYTES);
  // lend the static array to the handle for the duration of this call
  void *own_ctl = g->ctl_mem, *own_bulk = g->bulk_mem;
  const size_t own_ctl_cap = g->ctl_cap, own_bulk_cap = g->bulk_cap;
  char* base = static_cast<char*>(g_static_scratch_addr[g->device]);
  g->ctl_mem = base; g->ctl_cap = ctl_need;
  g->bulk_mem = base + ctl_need; g->bulk_cap = (size_t)AMPNET_STATIC_SCRATCH_BYTES - ctl_need;
  g->arenas_lent = true;
  st = execute(g, 0, cfg->max_active_keys, cfg->deterministic ? 1 : 0, 0, cfg, out, per_instance_loss, nullptr);
  g->arenas_lent = false;
  g->ctl_mem = own_ctl; g->ctl_cap = own_ctl_cap; g->bulk_mem = own_bulk; g->bulk_cap = own_bulk_cap;
  g->leftover_regions.clear();      // they described the lent memory
  return st;
}
