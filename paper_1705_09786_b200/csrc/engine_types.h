// Device-side data structures of the AMPNet engine (shared by the host library and the kernel).
#pragma once
#include <stdint.h>

namespace amp {

constexpr int MAX_PORTS = 8;
constexpr int THREADS = 256;          // threads per CTA
constexpr int WARPS = THREADS / 32;
constexpr int MAX_BATCH_MSGS = 64;    // messages per micro-batch (one warp schedules them, two messages per lane)
constexpr int MAX_BATCH_ROWS = 64;    // payload rows per micro-batch
constexpr int BATCH_BLOCKS = 16;     // batch context blocks in flight between a node's scheduler and its tiles / emitters
constexpr int MAX_SMEM_NODES = 40;    // IR nodes / PPT nodes whose tables are kept in shared memory
constexpr int MAX_SMEM_PPTS = 16;
constexpr int MAX_TILES = 32;        // row tiles per PPT node
constexpr int WALK_STACK = 12;        // continuation frames per walking warp
constexpr int JOIN_UNIT = 4096;       // direct-delivery engine: one whole message in a join counter; a row tile arrives with its share

enum NodeType { SOURCE, LINEAR, LOOKUP, GRUCELL, LOSS_CE, LOSS_MSE, NPT_SUMROWS, COND, PHI, ISU, CONCAT, SPLIT,
                BCAST, GROUP, UNGROUP, FLATMAP, SINK, NPT_LSTM, N_NODE_TYPES };
enum { FWD = 0, BWD = 1 };
enum { HDR_EVAL = 1 };
enum { BATCH_UPDATE = 1, BATCH_END_ROUND = 2, BATCH_TERMINATE = 4 };
enum { ST_OK = 0, ST_TIMEOUT = 4, ST_OVERFLOW = 5 };

// Message header: the state of Sec. 4 (instance id, position, iteration, ...) plus the payload row count.
struct __align__(16) Hdr { int inst, seq, slot, it, u, port, rows, flags; };

struct Ring {            // multi-producer ring of headers; payloads live in the keyed caches
  Hdr* e;
  unsigned* seq;         // per slot: ticket + 1 once published
  unsigned* tail;        // next ticket
  unsigned mask;
};

struct __align__(16) BatchDesc { unsigned sched_start; int count, dir, flags, n_upd, nrows, upd_t, pad1; };   // upd_t: index (from 1) of this update within the run

// Everything a tile or an emitter needs to know about one micro-batch.  With scheduler CTAs the scheduler assembles it
// once and the consumers copy the block; otherwise every consumer derives it from the descriptor and the headers.
struct __align__(16) BatchCtx {
  BatchDesc desc;                       // desc.pad1 != 0: the batch is malformed (the run is being aborted)
  Hdr hdr[MAX_BATCH_MSGS];
  long long key[MAX_BATCH_MSGS];
  int rowoff[MAX_BATCH_MSGS + 4];       // first batch row of every message; [count] = rows of the batch
  int rowmsg[MAX_BATCH_ROWS];                       // message of every batch row
  const float* rowptr[MAX_BATCH_ROWS];              // cached input row (LOOKUP: incoming gradient row) of every batch row
  int rowid[MAX_BATCH_ROWS], rownext[MAX_BATCH_ROWS];           // LOOKUP: table row of every batch row; next batch row with the same table row (-1: none)
  int rowfirst[MAX_BATCH_ROWS];                     // LOOKUP: no earlier batch row has the same table row
};
static_assert(sizeof(BatchCtx) % 16 == 0, "batch context blocks are copied in 16-byte pieces");

struct PPTStats {
  unsigned long long n_updates, n_grads_applied, msgs, batches, batch_rows;
  unsigned long long stale_hist[64];
  int max_staleness, log_n;
  unsigned long long phase_cycles[16];  // leader tile: idle, fetch, headers, compute, update, barrier, emit, loop; [8..] emission detail
  unsigned max_pending[2];              // direct-delivery engine: most messages waiting in the forward / backward ring when a batch was taken
  unsigned long long tc_batches;        // micro-batches (of those counted in `batches`) whose product ran on the tensor cores
};

struct DevNode {
  int type, in_dim, out_dim, act, fn, fn_arg, flags, ppt;
  int n_succ, n_pred;
  int succ_node[MAX_PORTS], succ_port[MAX_PORTS];
  int pred_node[MAX_PORTS], pred_port[MAX_PORTS];
  int U_in, U_out, rows_in, rows_out;   // bounds of the position u and of the payload rows, before / after
  // keyed storage; its meaning depends on the node type
  float* jbuf;            // join / result buffer, jstride floats per key
  long long jstride;
  int* jcnt;              // arrival counter per key
  unsigned char* origin;  // PHI: recorded predecessor per key
  int* rowcnt;            // NPT_SUMROWS: cached row count per key
  float* lossval;         // LOSS: loss per key
  int* predok;            // LOSS_CE: 1 if the arg-max equals the label
  int jalias;             // CONCAT: jbuf is the input cache of the succeeding PPT node; GROUP: jbuf lies inside the
                          // buffer of the succeeding CONCAT
  int jld;                // GROUP: row stride of the assembled rows
};

struct DevPPT {
  int node, kind, in_dim, out_dim, act, flags, muf_override;
  int tc;                             // direct-delivery engine: the forward row tiles (64 rows each) run their products on the tensor cores
  int T, cta0, R, BM;                 // row tiles, first CTA, rows per tile, batch row capacity
  int U, rows_max, J, xld;            // key space, max rows per message, ceil(in_dim / 32) bucket, row stride of xcache (in_dim
                                      // rounded up to 4 floats, padding kept at zero: rows start on 16 bytes for bulk copies)
  float *om, *ov;                     // optimiser state (first / second moment), laid out like W followed by b
  long long opt_t0;                   // updates of this node before the run (Adam's bias correction)
  float *W, *b;                       // LINEAR: W[out][in], b[out]; LOOKUP: W = E[V][d]; GRUCELL: W[3][H][2H], b[3][H]
  float* A;                           // LOOKUP: accumulator [V][d] in device memory; a node whose tiles keep their accumulators in
                                      // device memory (a_global): [tile][nmat][R][ldw]
  int a_global, xwt_rb;               // xwt_rb: output rows per pass of X.W^T (8 or 16; sizes the k-slice scratch)
  int *touched_flag, *touched_list, *touched_n;
  float *xcache, *ycache, *gbuf;      // [key][rows_max][in | out | out]
  float *zc, *rc, *cc;                // GRUCELL caches [key][rows_max][H]
  int* vcache;                        // version at forward time, per key
  Ring ring[2];
  unsigned* sched; unsigned sched_mask;
  BatchDesc* batches; unsigned batch_mask; unsigned* batch_pub;
  Hdr* bhdr;                          // [BATCH_BLOCKS][MAX_BATCH_MSGS] headers of the most recent batches
  BatchCtx* ctxblk;                   // [BATCH_BLOCKS] assembled batch contexts (scheduler CTAs only)
  unsigned long long* sortbuf;
  float* dxpart;                      // [2][T][BM][in_dim] partial input gradients of the row tiles
  float* stage;                       // [2][BM][max(in_dim, out_dim)] reduced input gradients / gathered rows, by batch parity
  long long stage_floats;
  unsigned *emit_pub, *emit_fin;      // per tile: batches handed to its emitter CTAs; set once the last one is out
  unsigned* emit_done;                // [emitter]: last batch (index + 1) the emitter has finished
  int NE, G;                          // emitter CTAs of the node; groups that take batches in turn (emitter q: group q % G,
                                      // member q / G, which emits its share of the messages of every batch of its group)
  unsigned* fetched;                  // batches tile 0 has fetched (paces the scheduler CTA)
  float* part2;                       // GRUCELL scratch
  unsigned* nbar;                     // barrier counter of the node's tiles
  PPTStats* stats;
  int* update_log; int update_log_cap;
  int smem_floats;
  int* injoin[2];                     // direct-delivery engine: arrival counter per key and direction (in units of JOIN_UNIT per message)
  int TB, CB, NS, bwd_smem_floats;    // direct-delivery engine: backward column tiles and input columns per tile; gradient slots per key
                                      // in gbuf ([key][NS][out]: one per successor of the Bcast whose backward sum forms there)
  unsigned* wver;                     // backward tiles that have published their columns, summed over the updates (TB per update)
  // direct-delivery engine, node that feeds a Loss: LT tiles share its messages (tile t takes the tickets t, t + LT, ... of
  // the forward ring) and exchange their partial gradient sums at every update: lh_part[2][LT][out * in + out] by update
  // parity, lh_count = arrivals at the exchanges so far (LT per update), lh_mom = private optimiser moments of tiles 1..LT-1
  int LT, pad1;
  int* lh_count;
  float *lh_part, *lh_mom;
};

struct DevInst {                      // instances + routing tables produced by the structure encoder
  int kind, dense_dim, NT, labels_per_node;
  long long n;
  const long long* offsets;
  const int* tokens;
  const int *left, *right, *parent, *child_slot;
  const int* root;                    // per instance
  const long long* leaf_off; const int* leaf_ids;
  const long long* edge_off;
  const int *esrc, *edst, *etype, *rank_out, *rank_in, *rank_type;
  const long long *out_off, *in_off, *type_off;   // per global node (+1) / per (instance, type) (+1)
  const int *out_list, *in_list, *type_list;      // local edge ids
  const float* dense;
  const int* labels_i;
  const float* labels_f;
};

struct KeyLog { long long inst; int slot; int pad; long long admit, release; };

struct Globals {                      // mutable run state in device memory (zeroed before every run)
  unsigned grid_bar;
  unsigned abort_flag;
  int status;
  unsigned done;
  unsigned long long node_messages, route_hash;
  unsigned long long rounds;
  long long max_active;
  unsigned long long correct, n_pred;
  double total_loss;
  double inf_loss; unsigned long long inf_instances, inf_correct, inf_pred;   // instances that were only evaluated (concurrent inference)
  long long n_keylog;
  unsigned retire_tail;
  int err_node, err_detail;
  unsigned long long walk_cycles[N_NODE_TYPES * 2], walk_steps[N_NODE_TYPES * 2];   // profiling (tune bit 8)
  // cycles by role: [0..7] controller (retire, admit, clear, pump, idle, admissions), then per PPT node p at 8 + 8 p:
  // scheduler (waiting for tile 0, no message pending, forming) and emitters (waiting, loading, emitting, batches)
  unsigned long long role_cycles[8 + 8 * MAX_SMEM_PPTS];
  unsigned long long step_cycles[MAX_SMEM_PPTS][16];   // tile 0 of every node: cycles between the marks inside the arithmetic phase
};

struct Role { int ppt, tile, kind, pad; };   // kind 0: row tile, 1: one of the node's emitter CTAs (pad = which one), 2: the node's scheduler CTA,
                                             // 3: backward column tile (direct-delivery engine)

struct Ctx {
  DevNode* nodes; int n_nodes;
  DevPPT* ppts; int n_ppts;
  Role* roles; int n_ctas;
  DevInst inst;
  Globals* g;
  unsigned long long* node_msgs;       // [n_nodes][2]
  // controller
  int n_sources; int src_nodes[4];
  int n_loss; int loss_nodes[4];
  int ends_per_instance, ends_per_position;   // forward-only instances: Loss / Sink arrivals that finish one = a + b x positions
  int* slot_inst; int* outstanding; int* slot_log;
  KeyLog* keylog;
  unsigned* retire_e; unsigned* retire_seq; unsigned retire_mask;
  const long long* order; long long n_order;
  const unsigned char* inference_only;  // per instance: only evaluated while the others train (may be null)
  float* loss_out;
  // configuration
  int mak, muf, det, eval, IT;
  int wide;                           // the graph has row-wise forks (Ungroup / Group)
  int bf16;                           // payloads rounded to bfloat16 at emission
  int emit_ctas;                      // the nodes have emitter CTAs (0: tiles emit themselves)
  int sched_ctas;                     // every PPT node has a scheduler CTA (its leader) of its own
  int depth;                          // per-batch buffers (partials, staging rows) are reused every `depth` batches
  int tune;                           // experiment switches (environment AMPNET_TUNE): 2 no look-ahead, 4 no per-node counters
  float lr;
  int opt;                            // update rule: 0 SGD, 1 momentum-SGD, 2 Adam
  float mu, beta1, beta2, eps;
  unsigned long long timeout_ns;
  char* ctl_base;                     // start of the control arena (counters are addressed by 32-bit offsets from here)
};

}  // namespace amp
