/* ampnet.h -- C ABI of the B200-native AMPNet training engine.
 *
 * The engine executes the hot path of asynchronous model-parallel (AMP) training of dynamic networks
 * (AMPNet, arXiv 1705.09786): the message-driven execution of a static IR graph.  Forward and backward
 * messages keyed by instance flow through parameterised nodes (Linear, GRU cell, embedding lookup) and
 * control-flow nodes (Cond, Phi, Isu, Concat, Bcast, Group, Ungroup, Flatmap); every parameterised node
 * accumulates gradients locally and applies an SGD update once min_update_frequency gradients have
 * arrived (Sec. 3); max_active_keys bounds the instances in flight (Sec. 3).  On the device this is one
 * persistent kernel whose CTAs own row tiles of the parameterised nodes (weights and fp32 accumulators in
 * shared memory) and exchange messages through lock-free ring queues in device memory.
 *
 * Conventions.  Every call returns a status; nothing aborts the process or traps the GPU; every device-side
 * wait is bounded and reports AMPNET_ETIMEOUT.  Input arrays are caller-owned HOST memory and are copied.
 * Output arrays are caller-allocated HOST memory.  The handle owns all device memory, obtained through the
 * allocator given at creation (cudaMalloc when none is given).  Matrices are row-major [out x in], fp32.
 * Calls on one handle are not thread-safe.  All work is issued on the stream given at creation.
 */
#ifndef AMPNET_H
#define AMPNET_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ampnet_graph ampnet_graph_t; /* opaque, owned by the library */

typedef enum {
  AMPNET_OK = 0,
  AMPNET_EINVAL = 1,    /* malformed argument or IR description (see ampnet_last_error)            */
  AMPNET_ENOMEM = 2,    /* device allocation failed                                                */
  AMPNET_ECUDA = 3,     /* a CUDA runtime call failed                                              */
  AMPNET_ETIMEOUT = 4,  /* a bounded device-side wait gave up; the GPU context stays usable        */
  AMPNET_EOVERFLOW = 5, /* a queue / cache / key-space bound was exceeded; nothing blocked         */
  AMPNET_ESTATE = 6     /* call order wrong (for example run before load)                          */
} ampnet_status_t;

/* ---- IR description (Sec. 4: a static graph of nodes and edges) ---------------------------------------- */

/* node types */
enum {
  AMPNET_SOURCE = 0,      /* controller output: pumps one admitted instance (fn = AMPNET_SRC_*)          */
  AMPNET_LINEAR = 1,      /* PPT: y = act(W x + b), row-wise for matrix payloads                         */
  AMPNET_LOOKUP = 2,      /* PPT: embedding table, in_dim = vocabulary, out_dim = width                  */
  AMPNET_GRUCELL = 3,     /* PPT: x = [a; h] (in_dim = 2H): z = s(Wz x + bz), r = s(Wr x + br),
                             c = tanh(Wc [a; r*h] + bc), h' = (1 - z) * h + z * c                        */
  AMPNET_LOSS_CE = 4,     /* softmax cross-entropy against an integer label; starts the backward pass    */
  AMPNET_LOSS_MSE = 5,    /* (y - t)^2 against a float target                                            */
  AMPNET_NPT_SUMROWS = 6, /* non-parameterised transform: sum of the rows of the payload                 */
  AMPNET_COND = 7,        /* routes on the state (fn = AMPNET_COND_*)                                    */
  AMPNET_PHI = 8,         /* join: records the origin keyed on the state, backpropagates to it           */
  AMPNET_ISU = 9,         /* invertible state update (fn = AMPNET_ISU_*)                                 */
  AMPNET_CONCAT = 10,     /* fn_arg ports of width in_dim -> one payload of width out_dim                */
  AMPNET_SPLIT = 11,      /* inverse of CONCAT: fn_arg successors, successor k gets columns [k w, (k+1) w) */
  AMPNET_BCAST = 12,      /* same payload to fn_arg successors; backward = sum in successor order        */
  AMPNET_GROUP = 13,      /* collect messages by state into one matrix payload (fn = AMPNET_GROUP_*)     */
  AMPNET_UNGROUP = 14,    /* one message per row (fn = AMPNET_UNGROUP_*)                                 */
  AMPNET_FLATMAP = 15,    /* one message per generated state, payload replicated (fn = AMPNET_FLATMAP_*) */
  AMPNET_SINK = 16,       /* answers a forward message with a zero gradient                              */
  AMPNET_NPT_LSTM = 17    /* non-parameterised LSTM gate combination (fn = AMPNET_LSTM_*): gate pre-activations from a
                             LINEAR node on port 0 (and the children's cells [cL; cR] on port 1) -> [h; c]          */
};
enum { AMPNET_ACT_NONE = 0, AMPNET_ACT_RELU = 1, AMPNET_ACT_TANH = 2, AMPNET_ACT_SIGMOID = 3 };
/* state functions; the message state is (inst, seq, slot, it, u, port)                                     */
enum { AMPNET_SRC_DENSE_ROW = 1, AMPNET_SRC_TOKENS = 2, AMPNET_SRC_ZERO_STATE = 3, AMPNET_SRC_TREE_LEAVES = 4,
       AMPNET_SRC_GRAPH_NODES = 5,
       AMPNET_SRC_TREE_LEAVES_GROUPED = 6 }; /* one message with L rows: the tokens of the tree's leaves in leaf order (Sec. 6) */
enum { AMPNET_LSTM_LEAF = 1,   /* [pi, po, pu] (3H): c = s(pi) tanh(pu), h = s(po) tanh(c)                                   */
       AMPNET_LSTM_BRANCH = 2 }; /* [pi, pfL, pfR, po, pu] (5H), [cL; cR]: c = s(pi) tanh(pu) + s(pfL) cL + s(pfR) cR, h = s(po) tanh(c) */
enum { AMPNET_COND_SEQ_END = 1,   /* u < #tokens ? 0 : 1        */
       AMPNET_COND_TREE_ROOT = 2, /* u is the root ? 0 : 1      */
       AMPNET_COND_BY_U = 3,      /* successor = u              */
       AMPNET_COND_IT_LT = 4,     /* it < fn_arg ? 0 : 1        */
       AMPNET_COND_ROUND_ROBIN = 5 }; /* successor = (instance + u) mod successors: replicas of a node (Sec. 5) */
enum { AMPNET_ISU_U_INC = 1, AMPNET_ISU_TREE_PARENT = 2, AMPNET_ISU_IT_INC = 3 };
enum { AMPNET_CONCAT_BY_EDGE = 1, AMPNET_CONCAT_BY_STATE_PORT = 2 };
enum { AMPNET_GROUP_EDGES_BY_TYPE = 1, AMPNET_GROUP_EDGES_BY_DST = 2, AMPNET_GROUP_ALL_NODES = 3 };
enum { AMPNET_UNGROUP_NODES = 1, AMPNET_UNGROUP_TYPE_EDGES = 2,
       AMPNET_UNGROUP_LEAVES = 3 };  /* row i -> u = position of the tree's i-th leaf */
enum { AMPNET_FLATMAP_OUT_EDGES = 1 };
enum { AMPNET_LABEL_PER_INSTANCE = 1, AMPNET_LABEL_PER_TREE_NODE = 2 };
enum { AMPNET_FLAG_SOURCE_ADJACENT = 1 }; /* PPT fed directly by a SOURCE: no input gradient, retire instead */

typedef struct {
  int32_t type, in_dim, out_dim, act;
  int32_t fn, fn_arg;
  int32_t muf_override; /* 0 = use the run configuration's min_update_frequency (per-node threshold)   */
  int32_t flags;
} ampnet_node_desc_t;
typedef struct { int32_t src_node, src_port, dst_node, dst_port; } ampnet_edge_desc_t;
typedef struct {
  int32_t n_nodes, n_edges;
  const ampnet_node_desc_t* nodes; /* host */
  const ampnet_edge_desc_t* edges; /* host */
  int32_t payload_dtype;           /* 0 = fp32 messages; 1 = bf16 messages: every emitted payload is rounded to bfloat16
                                      (round to nearest even), weights, accumulators and cached-activation arithmetic
                                      stay fp32                                                              */
} ampnet_ir_desc_t;

/* IR builders for the model families of Sec. 2 / Sec. 4: multi-layer perceptron (ReLU hidden layers, softmax-CE),
 * variable-length RNN (Fig. 2: Lookup, Concat with the hidden state from Phi, Linear, Isu(t+1), Cond(end?), loop or
 * Linear + Loss), binary tree RNN (leaf / branch cells joined by Phi, classifier at every node, children concatenated
 * on the way up), gated graph neural network (Fig. 3a: per-edge-type Linear messages, GRU update, `steps` iterations,
 * sum-pool read-out with MSE).  Host only; no device is touched.  The arrays are caller-allocated HOST memory of the
 * given capacities; *n_nodes / *n_edges always return the sizes needed, AMPNET_EOVERFLOW says the capacity was too
 * small (call with NULL arrays to size them).                                                                   */
ampnet_status_t ampnet_ir_mlp(const int32_t* dims, int32_t n_dims, ampnet_node_desc_t* nodes, int32_t cap_nodes,
                              int32_t* n_nodes, ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges);
ampnet_status_t ampnet_ir_rnn(int32_t vocab, int32_t emb, int32_t hidden, int32_t classes, int32_t act,
                              ampnet_node_desc_t* nodes, int32_t cap_nodes, int32_t* n_nodes,
                              ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges);
/* binary Tree-LSTM (Sec. 6): leaf and branch cells built from a LINEAR node (gate pre-activations) and an NPT_LSTM node */
ampnet_status_t ampnet_ir_tree_lstm(int32_t vocab, int32_t emb, int32_t hidden, int32_t classes,
                                    ampnet_node_desc_t* nodes, int32_t cap_nodes, int32_t* n_nodes,
                                    ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges);
ampnet_status_t ampnet_ir_tree(int32_t vocab, int32_t emb, int32_t hidden, int32_t classes,
                               ampnet_node_desc_t* nodes, int32_t cap_nodes, int32_t* n_nodes,
                               ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges);
/* the tree model with the leaf operations of a tree grouped into one call (Sec. 6): the controller pumps one message whose
 * rows are the leaves' tokens, LOOKUP and the leaf cell work on that matrix (at most 64 leaves per tree), an UNGROUP in
 * front of the PHI hands every leaf its row and, backward, collects the leaves' gradients into one matrix message.   */
ampnet_status_t ampnet_ir_tree_grouped(int32_t vocab, int32_t emb, int32_t hidden, int32_t classes,
                                       ampnet_node_desc_t* nodes, int32_t cap_nodes, int32_t* n_nodes,
                                       ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges);
ampnet_status_t ampnet_ir_ggnn(int32_t n_node_types, int32_t hidden, int32_t steps, int32_t n_edge_types, int32_t readout,
                               ampnet_node_desc_t* nodes, int32_t cap_nodes, int32_t* n_nodes,
                               ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges);

/* Device-memory allocator supplied by the caller (for example a PyTorch caching allocator).  `alloc` returns a
 * device pointer aligned to 256 bytes or NULL; `free` releases it.  Both are called from the calling thread. */
typedef void* (*ampnet_alloc_fn)(void* ctx, size_t bytes);
typedef void (*ampnet_free_fn)(void* ctx, void* ptr);
typedef struct { ampnet_alloc_fn alloc; ampnet_free_fn free; void* ctx; } ampnet_allocator_t;

/* Sec. 4 "a model = an IR graph + a controller loop".  Validates the IR, places the parameterised nodes on
 * CTAs, allocates and initialises the parameters (seeded).  `cuda_stream` is a cudaStream_t (NULL = default
 * stream); `allocator` may be NULL.  On failure *out is NULL and the status says why.                         */
ampnet_status_t ampnet_graph_create(const ampnet_ir_desc_t* ir, uint64_t init_seed, void* cuda_stream,
                                    const ampnet_allocator_t* allocator, ampnet_graph_t** out);
void ampnet_graph_destroy(ampnet_graph_t*);

/* ---- instances (what the controller pumps, Sec. 4) ----------------------------------------------------- */
enum { AMPNET_KIND_DENSE_ROWS = 0, AMPNET_KIND_SEQUENCES = 1, AMPNET_KIND_BINARY_TREES = 2,
       AMPNET_KIND_TYPED_GRAPHS = 3 };
typedef struct {
  int32_t kind;
  int64_t n_instances;
  const int64_t* offsets;      /* n+1: tokens / tree nodes / graph nodes per instance (NULL for dense rows)   */
  const int32_t* tokens;       /* token id / leaf token id (-1 at inner tree nodes) / graph node type id      */
  const int32_t *left, *right; /* trees: local child ids, -1 at leaves; children precede parents             */
  const int64_t* edge_offsets; /* graphs: n+1                                                                */
  const int32_t *edge_src, *edge_dst, *edge_type; /* graphs: directed edges, local node ids                  */
  const float* dense;          /* dense rows: n x dense_dim                                                  */
  int32_t dense_dim;
  const int32_t* labels_i;     /* class per instance, or per tree node (AMPNET_LABEL_PER_TREE_NODE)          */
  const float* labels_f;       /* regression target per instance                                             */
} ampnet_instances_t;

/* Copies the instances to the device and encodes their structure into routing tables (parents and child
 * slots of trees; out-edge, in-edge and per-type edge lists and ranks of graphs).  split: 0 train, 1 valid.  */
ampnet_status_t ampnet_load_instances(ampnet_graph_t*, int32_t split, const ampnet_instances_t*);

/* ---- training (Sec. 3) ---------------------------------------------------------------------------------- */
typedef struct {
  int32_t max_active_keys;      /* instances in flight                                                       */
  int32_t min_update_frequency; /* gradients accumulated by a node before it updates                         */
  float lr;                     /* SGD: theta -= lr * (accumulated gradient / number of gradients)           */
  int32_t deterministic;        /* 1: canonical round schedule (reproducible; for checking), 0: asynchronous */
  const int64_t* order;         /* host, instance order of the epoch; NULL = dataset order                   */
  int64_t n_order;              /* number of instances to train on (ignored when order == NULL: all)         */
  double timeout_s;             /* bound on the whole device run; 0 = default (120 s)                        */
  int32_t max_batch_rows;       /* cap on payload rows a node processes as one micro-batch; 0 = automatic    */
  int32_t n_ctas;               /* CTAs to use; 0 = one per SM                                               */
} ampnet_run_cfg_t;

typedef struct {
  int64_t instances, node_messages, ppt_messages, rounds;
  double seconds;   /* device time of the run (CUDA events)                                                  */
  double mean_loss; /* mean per-instance loss of the epoch                                                   */
  int32_t max_staleness;
  int64_t max_active_observed;
  uint64_t route_hash; /* order-independent fingerprint of all routed (node, direction, state) messages     */
  int64_t micro_batches, micro_batch_rows; /* batches executed by all nodes and the payload rows in them    */
} ampnet_epoch_stats_t;

/* One pass over the training split: admission under max_active_keys, message-driven forward and backward
 * execution, local updates, retirement; accumulators are flushed at the end.  per_instance_loss: host,
 * n_instances floats (indexed by instance), may be NULL.                                                    */
ampnet_status_t ampnet_run_epoch(ampnet_graph_t*, const ampnet_run_cfg_t*, ampnet_epoch_stats_t* out,
                                 float* per_instance_loss);

/* Forward-only messages over a split; nothing cached, no parameter touched.  accuracy: fraction of correct
 * arg-max predictions over all loss evaluations (0 for MSE).                                                */
ampnet_status_t ampnet_eval(ampnet_graph_t*, int32_t split, int32_t max_active_keys, double* mean_loss,
                            double* accuracy, float* per_instance_loss);

/* ---- parameters and statistics --------------------------------------------------------------------------- */
/* which: LINEAR 0 = W, 1 = b; LOOKUP 0 = E; GRUCELL 0..2 = Wz, Wr, Wc, 3..5 = bz, br, bc.                    */
ampnet_status_t ampnet_param_count(ampnet_graph_t*, int32_t node, int32_t which, int64_t* n);
ampnet_status_t ampnet_get_params(ampnet_graph_t*, int32_t node, int32_t which, float* dst_host, int64_t n);
ampnet_status_t ampnet_set_params(ampnet_graph_t*, int32_t node, int32_t which, const float* src_host, int64_t n);
/* Device address of the same array (*n floats), owned by the handle and valid until it is destroyed.  Between two
 * epochs the caller may read or write it on the handle's stream or after synchronising with it: this is how replicas of
 * the whole model on several GPUs are averaged in place at the end of an epoch (Sec. 5) by a collective library.     */
ampnet_status_t ampnet_param_device_ptr(ampnet_graph_t*, int32_t node, int32_t which, float** dev, int64_t* n);

/* Statistics of the last run.  staleness_hist: 64 bins (updates between a gradient's forward and backward).
 * fwd_msgs / bwd_msgs (messages consumed by the node) and the route fingerprint are collected in the
 * deterministic schedule only; the asynchronous schedule counts the total of node messages.                   */
ampnet_status_t ampnet_get_node_stats(ampnet_graph_t*, int32_t node, int64_t* n_updates, int64_t* n_grads_applied,
                                      int64_t* staleness_hist, int64_t* fwd_msgs, int64_t* bwd_msgs);
/* Gradient count of each update of a node, in order; returns the number of updates through *n.               */
ampnet_status_t ampnet_get_update_log(ampnet_graph_t*, int32_t node, int32_t* n_per_update, int64_t cap, int64_t* n);
/* Key bookkeeping of the last deterministic run: instance, slot, admission round, release round.             */
ampnet_status_t ampnet_get_key_log(ampnet_graph_t*, int64_t* inst, int32_t* slot, int64_t* admit_round,
                                   int64_t* release_round, int64_t cap, int64_t* n);
/* Number of keyed cache entries (join counters, recorded origins) still set after the last run; the
 * forward/backward state invariant of Sec. 4 makes this 0.                                                   */
ampnet_status_t ampnet_leftover_cache_entries(ampnet_graph_t*, int64_t* n);
/* Placement chosen for a parameterised node: number of row tiles (CTAs) and micro-batch row capacity.  Asynchronous
 * runs of graphs that the direct-delivery engine takes (single-row messages; Cond, Phi, Isu, Bcast, Concat, Sink and a
 * Loss fed by a Linear node) report the forward row tiles; a Linear node has backward column tiles besides (none for a
 * node that feeds a Loss: each of its tiles holds all rows, does both directions and takes its share of the messages). */
ampnet_status_t ampnet_get_placement(ampnet_graph_t*, int32_t node, int32_t* n_tiles, int32_t* batch_rows);

/* Where the leader tile of a node spent its SM cycles in the last run: [0] waiting for messages, [1] fetching a
 * batch descriptor, [2] loading headers, [3] staging + arithmetic, [4] local updates, [5] barrier among the node's
 * tiles, [6] emission (walking the parameter-free nodes), [7] loop overhead; [8..15] detail of the emission phase
 * ([8] look-ahead scheduling, [9] reduction of partial gradients, [10]/[12] own walks of warps 0/1, [11]/[13] helping
 * other warps, [14] closing barrier).  After a run of the direct-delivery engine the 16 values are diagnostic marks of
 * the node's first forward tile ([0] waiting for and taking messages, [1] keys, routes and staging of the input rows,
 * [2] rest of the arithmetic phase, [3] update / reload of the weights, [4] arrivals and closing barrier, [5] products,
 * [6] activation and stores / Loss and gradients of a loss head, [7] delivery of those gradients) and, for a Linear node with column tiles, [8..14] of its first backward
 * tile in the same order of work (wait, routes and staging, incoming gradient, input gradient and delivery,
 * accumulation, update and publication, arrivals).  cycles16: 16 values.  batches: micro-batches executed.        */
ampnet_status_t ampnet_get_phase_cycles(ampnet_graph_t*, int32_t node, uint64_t* cycles16, int64_t* batches);
/* Queue occupancy of a node in the last asynchronous run (the benchmark set's stress configuration asks for it; App. A:
 * every worker owns a queue): the largest number of messages that were waiting in the node's forward and in its
 * backward ring at the moment a micro-batch was taken, as seen by the node's first tile.  The deterministic schedule
 * and graphs that run on the interpreter engine report 0.                                                        */
ampnet_status_t ampnet_get_queue_occupancy(ampnet_graph_t*, int32_t node, int64_t* max_pending_fwd, int64_t* max_pending_bwd);
/* Micro-batches of a node in the last run by the unit that ran their product (the stress configuration of the benchmark
 * set asks for this split): tensor_core_batches = forward micro-batches whose product Y^T = W X^T ran as tcgen05
 * instructions (bf16 runs on the direct-delivery engine: nodes with out_dim a multiple of 64 and in_dim a multiple of
 * 16; W and the batch as bfloat16 operands in shared memory, fp32 accumulator in tensor memory; the master weights,
 * the input gradient and the accumulation stay fp32), fma_batches = all others (counted like micro_batches of the epoch
 * statistics: by the node's first forward and first backward tile).  Either pointer may be NULL.                 */
ampnet_status_t ampnet_get_micro_batch_split(ampnet_graph_t*, int32_t node, int64_t* fma_batches, int64_t* tensor_core_batches);

/* ---- concurrent inference (Sec. 1: inference can run while the model trains; Sec. 6 reports inference throughput) --------
 * A training epoch in which the instances i with inference_only[i] != 0 (host array, one byte per loaded instance of
 * the training split) are only evaluated: their messages carry the evaluation flag, travel through the same queues and
 * micro-batch formation as the training messages (a micro-batch holds one kind only), cache nothing, produce no
 * gradients and count towards no update; they occupy a key like any instance.  out->mean_loss is the mean over the
 * training instances, *inference (may be NULL) receives count, mean loss and accuracy of the others;
 * per_instance_loss is indexed by instance for both kinds.                                                        */
typedef struct ampnet_inference_stats { int64_t instances; double mean_loss; double accuracy; } ampnet_inference_stats_t;
ampnet_status_t ampnet_run_epoch_mixed(ampnet_graph_t*, const ampnet_run_cfg_t*, const uint8_t* inference_only,
                                       ampnet_epoch_stats_t* out, float* per_instance_loss, ampnet_inference_stats_t* inference);

/* ---- replicas (Sec. 5) -------------------------------------------------------------------------------------
 * A heavy node is replicated in full between a Cond (AMPNET_COND_ROUND_ROBIN) and a Phi; the copies train
 * independently and are synchronised infrequently, at the end of an epoch, by averaging.  This call replaces the
 * parameters of the n listed nodes (same type and shape, n >= 1) by their element-wise mean, on the device, between
 * two epochs.  Optimiser state is left as it is.  nodes: host array of node indices.
 * Errors: AMPNET_EINVAL (not a parameterised node, shapes differ), AMPNET_ECUDA.                                  */
ampnet_status_t ampnet_average_params(ampnet_graph_t*, const int32_t* nodes, int32_t n);

/* canonical RNN with Linear-1 replicated `replicas` times (replicas = 1: identical to ampnet_ir_rnn) */
ampnet_status_t ampnet_ir_rnn_replicated(int32_t vocab, int32_t emb, int32_t hidden, int32_t classes, int32_t act, int32_t replicas,
                                         ampnet_node_desc_t* nodes, int32_t cap_nodes, int32_t* n_nodes,
                                         ampnet_edge_desc_t* edges, int32_t cap_edges, int32_t* n_edges);

/* ---- update rule of the local updates (Sec. 3; App. A lists the optimiser among the run-time options) -------
 * Every parameterised node applies the chosen rule to the MEAN of its accumulated gradients, g = A / n, whenever
 * it updates (min_update_frequency reached, or the epoch-end flush):
 *   AMPNET_OPT_SGD       theta <- theta - lr g                                   (the default)
 *   AMPNET_OPT_MOMENTUM  v <- momentum v + g;  theta <- theta - lr v
 *   AMPNET_OPT_ADAM      m <- beta1 m + (1-beta1) g;  v <- beta2 v + (1-beta2) g^2;
 *                        theta <- theta - lr (m / (1-beta1^t)) / (sqrt(v / (1-beta2^t)) + eps),  t = updates of this node
 * The moments are per node, owned by the handle (allocated here through the handle's allocator, one or two float
 * arrays of the node's parameter count, in device memory), kept across epochs and touched only at updates; an
 * embedding table moves only the rows (and their moments) that received gradients since its last update.
 * reset_state != 0 zeroes the moments and t.  Arguments that the chosen rule does not use are ignored.
 * Errors: AMPNET_EINVAL (unknown kind, momentum/beta outside [0,1), eps <= 0), AMPNET_ENOMEM, AMPNET_ECUDA.          */
enum { AMPNET_OPT_SGD = 0, AMPNET_OPT_MOMENTUM = 1, AMPNET_OPT_ADAM = 2 };
ampnet_status_t ampnet_set_optimizer(ampnet_graph_t*, int32_t kind, float momentum, float beta1, float beta2, float eps,
                                     int32_t reset_state);

/* FP32 multiply-add rate of the device, measured with a register-only FMA kernel (16 independent chains per thread, 8
 * blocks of 256 threads per SM, best of three timed launches on the default stream): the denominator of the roofline
 * fraction of this path, which is bound by plain FP32 arithmetic.  Needs no handle.  Errors: AMPNET_ECUDA, AMPNET_ENOMEM. */
ampnet_status_t ampnet_measure_fma_peak(int32_t device, double* tflops);

const char* ampnet_last_error(const ampnet_graph_t*); /* library-owned string */

/* ---- a training epoch that allocates nothing (no counterpart in the paper) ------------------------------
 * For callers that must not allocate device memory once they are running: a training loop that has handed all
 * free device memory to another pool, a latency-critical loop that cannot afford the device-wide
 * synchronisation of cudaMalloc/cudaFree, or a host that forbids allocation after start-up.  The handle is
 * created and its instances loaded beforehand (those calls allocate); this call then runs one epoch exactly
 * like ampnet_run_epoch, but its queues, counters and keyed caches live in a fixed array of
 * AMPNET_STATIC_SCRATCH_BYTES inside the library image instead of allocator memory.  It calls no cudaMalloc,
 * cudaFree or other allocating routine.
 *   - A run whose scratch does not fit (large max_active_keys, big structures or vocabularies) is refused with
 *     AMPNET_EINVAL; ampnet_last_error states the bytes needed and the bytes available.  Nothing has run then.
 *   - Every GPU that loads the library holds the array until the process exits.
 *   - The first call on a device looks up the array's device address; make that first call outside any stream
 *     capture.
 *   - All handles and all calls share the one array: what must start at zero is cleared at the start of each
 *     call, the rest keeps the previous call's contents.  Two such calls that overlap on the GPU (different
 *     streams or threads) race; serialise them.
 *   - ampnet_get_node_stats / ampnet_get_update_log / ampnet_get_key_log describe this run until the next call
 *     that uses the array; ampnet_leftover_cache_entries reports 0 after it.
 * Arguments, outputs and statuses are those of ampnet_run_epoch.                                             */
#define AMPNET_STATIC_SCRATCH_BYTES (64u << 20)
ampnet_status_t ampnet_run_epoch_static(ampnet_graph_t*, const ampnet_run_cfg_t*, ampnet_epoch_stats_t* out,
                                        float* per_instance_loss);

#ifdef __cplusplus
}
#endif
#endif /* AMPNET_H */
