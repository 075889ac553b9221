"""ctypes binding of libampnet.so (argument marshalling only)."""
import ctypes as C
import os

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_LIB = None

STATUS = {0: "OK", 1: "EINVAL", 2: "ENOMEM", 3: "ECUDA", 4: "ETIMEOUT", 5: "EOVERFLOW", 6: "ESTATE"}

EXPORTS = ["ampnet_graph_create", "ampnet_graph_destroy", "ampnet_load_instances", "ampnet_run_epoch", "ampnet_eval",
           "ampnet_param_count", "ampnet_get_params", "ampnet_set_params", "ampnet_get_node_stats",
           "ampnet_get_update_log", "ampnet_get_key_log", "ampnet_leftover_cache_entries", "ampnet_get_placement",
           "ampnet_last_error", "ampnet_set_optimizer", "ampnet_average_params", "ampnet_ir_rnn_replicated", "ampnet_run_epoch_mixed", "ampnet_param_device_ptr", "ampnet_run_epoch_static", "ampnet_get_phase_cycles", "ampnet_get_queue_occupancy", "ampnet_get_micro_batch_split", "ampnet_ir_mlp", "ampnet_ir_rnn",
           "ampnet_ir_tree", "ampnet_ir_tree_grouped", "ampnet_ir_ggnn", "ampnet_ir_tree_lstm", "ampnet_measure_fma_peak"]


class InferenceStats(C.Structure):
    _fields_ = [("instances", C.c_int64), ("mean_loss", C.c_double), ("accuracy", C.c_double)]


class AmpnetError(RuntimeError):
    def __init__(self, status, msg):
        super().__init__(f"ampnet status {STATUS.get(status, status)}: {msg}")
        self.status = status


class NodeDesc(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("type", "in_dim", "out_dim", "act", "fn", "fn_arg", "muf_override", "flags")]


class EdgeDesc(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("src_node", "src_port", "dst_node", "dst_port")]


class IRDesc(C.Structure):
    _fields_ = [("n_nodes", C.c_int32), ("n_edges", C.c_int32), ("nodes", C.c_void_p), ("edges", C.c_void_p),
                ("payload_dtype", C.c_int32)]


ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_void_p, C.c_size_t)
FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)


class Allocator(C.Structure):
    _fields_ = [("alloc", ALLOC_FN), ("free", FREE_FN), ("ctx", C.c_void_p)]


class Instances(C.Structure):
    _fields_ = [("kind", C.c_int32), ("n_instances", C.c_int64), ("offsets", C.c_void_p), ("tokens", C.c_void_p),
                ("left", C.c_void_p), ("right", C.c_void_p), ("edge_offsets", C.c_void_p), ("edge_src", C.c_void_p),
                ("edge_dst", C.c_void_p), ("edge_type", C.c_void_p), ("dense", C.c_void_p), ("dense_dim", C.c_int32),
                ("labels_i", C.c_void_p), ("labels_f", C.c_void_p)]


class RunCfg(C.Structure):
    _fields_ = [("max_active_keys", C.c_int32), ("min_update_frequency", C.c_int32), ("lr", C.c_float),
                ("deterministic", C.c_int32), ("order", C.c_void_p), ("n_order", C.c_int64), ("timeout_s", C.c_double),
                ("max_batch_rows", C.c_int32), ("n_ctas", C.c_int32)]


class EpochStats(C.Structure):
    _fields_ = [("instances", C.c_int64), ("node_messages", C.c_int64), ("ppt_messages", C.c_int64),
                ("rounds", C.c_int64), ("seconds", C.c_double), ("mean_loss", C.c_double),
                ("max_staleness", C.c_int32), ("max_active_observed", C.c_int64), ("route_hash", C.c_uint64),
                ("micro_batches", C.c_int64), ("micro_batch_rows", C.c_int64)]


def library_path():
    return os.path.join(_DIR, "libampnet.so")


def load_library():
    """Load libampnet.so; raises if it has not been built (there is no fallback path)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_1705_09786_b200.build` "
                          "(the engine has no CPU or eager fallback)")
    lib = C.CDLL(path)
    P = C.c_void_p
    lib.ampnet_graph_create.argtypes = [C.POINTER(IRDesc), C.c_uint64, P, C.POINTER(Allocator), C.POINTER(P)]
    lib.ampnet_graph_destroy.argtypes = [P]
    lib.ampnet_graph_destroy.restype = None
    lib.ampnet_load_instances.argtypes = [P, C.c_int32, C.POINTER(Instances)]
    lib.ampnet_run_epoch.argtypes = [P, C.POINTER(RunCfg), C.POINTER(EpochStats), P]
    lib.ampnet_run_epoch_static.argtypes = [P, C.POINTER(RunCfg), C.POINTER(EpochStats), P]
    lib.ampnet_eval.argtypes = [P, C.c_int32, C.c_int32, C.POINTER(C.c_double), C.POINTER(C.c_double), P]
    lib.ampnet_param_count.argtypes = [P, C.c_int32, C.c_int32, C.POINTER(C.c_int64)]
    lib.ampnet_get_params.argtypes = [P, C.c_int32, C.c_int32, P, C.c_int64]
    lib.ampnet_set_params.argtypes = [P, C.c_int32, C.c_int32, P, C.c_int64]
    lib.ampnet_get_node_stats.argtypes = [P, C.c_int32, P, P, P, P, P]
    lib.ampnet_get_update_log.argtypes = [P, C.c_int32, P, C.c_int64, C.POINTER(C.c_int64)]
    lib.ampnet_get_key_log.argtypes = [P, P, P, P, P, C.c_int64, C.POINTER(C.c_int64)]
    lib.ampnet_leftover_cache_entries.argtypes = [P, C.POINTER(C.c_int64)]
    lib.ampnet_get_placement.argtypes = [P, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.ampnet_get_phase_cycles.argtypes = [P, C.c_int32, P, C.POINTER(C.c_int64)]
    lib.ampnet_get_queue_occupancy.argtypes = [P, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    lib.ampnet_get_micro_batch_split.argtypes = [P, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    lib.ampnet_set_optimizer.argtypes = [P, C.c_int32, C.c_float, C.c_float, C.c_float, C.c_float, C.c_int32]
    I32, PI = C.c_int32, C.POINTER(C.c_int32)
    tail = [P, I32, PI, P, I32, PI]
    lib.ampnet_ir_mlp.argtypes = [P, I32] + tail
    lib.ampnet_ir_rnn.argtypes = [I32] * 5 + tail
    lib.ampnet_ir_rnn_replicated.argtypes = [I32] * 6 + tail
    lib.ampnet_average_params.argtypes = [P, P, C.c_int32]
    lib.ampnet_run_epoch_mixed.argtypes = [P, P, P, P, P, P]
    lib.ampnet_param_device_ptr.argtypes = [P, C.c_int32, C.c_int32, C.POINTER(C.c_void_p), C.POINTER(C.c_int64)]
    lib.ampnet_ir_tree.argtypes = [I32] * 4 + tail
    lib.ampnet_ir_tree_grouped.argtypes = [I32] * 4 + tail
    lib.ampnet_ir_tree_lstm.argtypes = [I32] * 4 + tail
    lib.ampnet_measure_fma_peak.argtypes = [C.c_int32, C.POINTER(C.c_double)]
    lib.ampnet_ir_ggnn.argtypes = [I32] * 5 + tail
    lib.ampnet_last_error.argtypes = [P]
    lib.ampnet_last_error.restype = C.c_char_p
    _LIB = lib
    return lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def measure_fma_peak(device=0):
    """Measured FP32 FMA rate of the device in TFLOP/s (register-only kernel of the library)."""
    v = C.c_double()
    rc = load_library().ampnet_measure_fma_peak(device, C.byref(v))
    if rc != 0:
        raise AmpnetError(rc, "ampnet_measure_fma_peak failed")
    return v.value


def ir_tables(family, *args):
    """Node and edge tables (int32 [n,8] / [m,4]) of a canonical model family from the library's IR builders.
    family: "mlp" (dims list), "rnn" (vocab, emb, hidden, classes, act), "tree" (vocab, emb, hidden, classes),
    "ggnn" (n_node_types, hidden, steps, n_edge_types, readout)."""
    lib = load_library()
    nn, ne = C.c_int32(), C.c_int32()

    def call(nodes, cn, edges, ce):
        tail = (_p(nodes), cn, C.byref(nn), _p(edges), ce, C.byref(ne))
        if family == "mlp":
            dims = np.ascontiguousarray(args[0], dtype=np.int32)
            return lib.ampnet_ir_mlp(_p(dims), len(dims), *tail)
        return getattr(lib, "ampnet_ir_" + family)(*[int(a) for a in args], *tail)

    rc = call(None, 0, None, 0)
    if rc not in (0, 5):
        raise AmpnetError(rc, f"ampnet_ir_{family} rejected its arguments")
    nodes, edges = np.zeros((nn.value, 8), np.int32), np.zeros((ne.value, 4), np.int32)
    rc = call(nodes, nn.value, edges, ne.value)
    if rc != 0:
        raise AmpnetError(rc, f"ampnet_ir_{family} failed")
    return nodes, edges


class Engine:
    """One IR graph on one GPU.  graph: an object with int32 tables `.nodes` [n,8] and `.edges` [m,4]."""

    def __init__(self, graph, seed=1, device=0, use_torch_allocator=True, payload_bf16=False):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("the AMPNet engine needs a CUDA device (no CPU fallback)")
        self.lib = load_library()
        self.graph = graph
        self.torch = torch
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self._blocks = {}
        self.alloc_calls = self.free_calls = 0      # how often the library called back into the allocator
        self._alloc_struct = None
        if use_torch_allocator:
            def _alloc(ctx, nbytes):
                self.alloc_calls += 1
                try:
                    t = torch.empty(int(nbytes) + 256, dtype=torch.uint8, device=self.device)
                except Exception:
                    return None
                ptr = (t.data_ptr() + 255) & ~255
                self._blocks[ptr] = t
                return ptr

            def _free(ctx, ptr):
                self.free_calls += 1
                self._blocks.pop(ptr, None)

            self._alloc_cb, self._free_cb = ALLOC_FN(_alloc), FREE_FN(_free)
            self._alloc_struct = Allocator(self._alloc_cb, self._free_cb, None)
        nodes = np.ascontiguousarray(graph.nodes, dtype=np.int32)
        edges = np.ascontiguousarray(graph.edges, dtype=np.int32)
        ir = IRDesc(len(nodes), len(edges), _p(nodes), _p(edges), 1 if payload_bf16 else 0)
        self.stream = torch.cuda.current_stream(self.device)
        h = C.c_void_p()
        rc = self.lib.ampnet_graph_create(C.byref(ir), seed, C.c_void_p(self.stream.cuda_stream),
                                          C.byref(self._alloc_struct) if self._alloc_struct else None, C.byref(h))
        if rc != 0:
            raise AmpnetError(rc, "ampnet_graph_create rejected the IR description")
        self.h = h
        self.n = [0, 0]

    def close(self):
        if getattr(self, "h", None):
            self.lib.ampnet_graph_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc):
        if rc != 0:
            raise AmpnetError(rc, self.lib.ampnet_last_error(self.h).decode())

    def load_instances(self, inst, split=0):
        s = Instances(inst.kind, inst.n, _p(inst.offsets), _p(inst.tokens), _p(inst.left), _p(inst.right),
                      _p(inst.edge_offsets), _p(inst.edge_src), _p(inst.edge_dst), _p(inst.edge_type), _p(inst.dense),
                      0 if inst.dense is None else inst.dense.shape[1], _p(inst.labels_i), _p(inst.labels_f))
        self._check(self.lib.ampnet_load_instances(self.h, split, C.byref(s)))
        self.n[split] = inst.n

    def set_params(self, params):
        for (node, which), v in params.items():
            a = np.ascontiguousarray(v, dtype=np.float32).ravel()
            self._check(self.lib.ampnet_set_params(self.h, node, which, _p(a), a.size))

    def get_params(self, node=None, which=None):
        if node is None:
            return {(i, w): self.get_params(i, w) for i in self.graph.ppt_nodes() for w, _ in self.graph.param_shapes(i)}
        n = C.c_int64()
        self._check(self.lib.ampnet_param_count(self.h, node, which, C.byref(n)))
        a = np.empty(n.value, np.float32)
        self._check(self.lib.ampnet_get_params(self.h, node, which, _p(a), n.value))
        return a.reshape(dict(self.graph.param_shapes(node))[which])

    def param_tensors(self):
        """{(node, which): torch tensor} aliasing the parameter arrays in device memory (no copies).  The arrays belong to
        the engine: the tensors must not be used after close(), and not while an epoch is running."""
        import torch

        class _View:                          # what torch.as_tensor needs to wrap a raw device pointer
            def __init__(self, ptr, n):
                self.__cuda_array_interface__ = {"shape": (n,), "typestr": "<f4", "data": (ptr, False), "version": 2}

        out = {}
        for i in self.graph.ppt_nodes():
            for w, shape in self.graph.param_shapes(i):
                ptr, n = C.c_void_p(), C.c_int64()
                self._check(self.lib.ampnet_param_device_ptr(self.h, i, w, C.byref(ptr), C.byref(n)))
                out[(i, w)] = torch.as_tensor(_View(ptr.value, n.value), device=self.device).view(*shape)
        return out

    def run_epoch(self, mak, muf, lr, deterministic=False, order=None, timeout_s=0.0, max_batch_rows=0, n_ctas=0,
                  want_loss=True, static_scratch=False):
        """One training epoch.  static_scratch=True calls ampnet_run_epoch_static: the same epoch with its run
        state in the library's fixed scratch array, for callers that must not allocate device memory (it is
        refused with EINVAL when the run state does not fit; calls sharing the array must not overlap)."""
        order = None if order is None else np.ascontiguousarray(order, dtype=np.int64)
        cfg = RunCfg(mak, muf, lr, int(deterministic), _p(order), 0 if order is None else len(order), timeout_s,
                     max_batch_rows, n_ctas)
        st = EpochStats()
        loss = np.zeros(self.n[0], np.float32) if want_loss else None
        fn = self.lib.ampnet_run_epoch_static if static_scratch else self.lib.ampnet_run_epoch
        self._check(fn(self.h, C.byref(cfg), C.byref(st), _p(loss)))
        return st, loss

    def run_epoch_mixed(self, mak, muf, lr, inference_only, deterministic=False, order=None, timeout_s=0.0):
        """A training epoch in which the instances marked in inference_only (uint8 per instance) are only evaluated.
        Returns (stats, per-instance loss, dict(instances, mean_loss, accuracy) of the inference instances)."""
        order = None if order is None else np.ascontiguousarray(order, dtype=np.int64)
        mask = np.ascontiguousarray(inference_only, dtype=np.uint8)
        if mask.shape != (self.n[0],):
            raise ValueError("inference_only needs one entry per loaded training instance")
        cfg = RunCfg(mak, muf, lr, int(deterministic), _p(order), 0 if order is None else len(order), timeout_s, 0, 0)
        st, inf = EpochStats(), InferenceStats()
        loss = np.zeros(self.n[0], np.float32)
        self._check(self.lib.ampnet_run_epoch_mixed(self.h, C.byref(cfg), _p(mask), C.byref(st), _p(loss), C.byref(inf)))
        return st, loss, dict(instances=inf.instances, mean_loss=inf.mean_loss, accuracy=inf.accuracy)

    def set_optimizer(self, kind="sgd", momentum=0.9, beta1=0.9, beta2=0.999, eps=1e-8, reset=True):
        k = {"sgd": 0, "momentum": 1, "adam": 2}[kind]
        self._check(self.lib.ampnet_set_optimizer(self.h, k, momentum, beta1, beta2, eps, int(reset)))

    def average_params(self, nodes):
        """End-of-epoch replica synchronisation (Sec. 5): the listed nodes get the mean of their parameters."""
        a = np.ascontiguousarray(nodes, dtype=np.int32)
        self._check(self.lib.ampnet_average_params(self.h, _p(a), len(a)))

    def eval(self, split=0, mak=64):
        ml, acc = C.c_double(), C.c_double()
        loss = np.zeros(self.n[split], np.float32)
        self._check(self.lib.ampnet_eval(self.h, split, mak, C.byref(ml), C.byref(acc), _p(loss)))
        return ml.value, acc.value, loss

    def node_stats(self, node):
        nu, ng, fw, bw = C.c_int64(), C.c_int64(), C.c_int64(), C.c_int64()
        hist = np.zeros(64, np.int64)
        self._check(self.lib.ampnet_get_node_stats(self.h, node, C.byref(nu), C.byref(ng), _p(hist), C.byref(fw),
                                                   C.byref(bw)))
        return dict(n_updates=nu.value, n_grads_applied=ng.value, staleness_hist=hist, fwd_msgs=fw.value,
                    bwd_msgs=bw.value)

    def update_log(self, node):
        n = C.c_int64()
        self._check(self.lib.ampnet_get_update_log(self.h, node, None, 0, C.byref(n)))
        a = np.zeros(max(n.value, 1), np.int32)
        self._check(self.lib.ampnet_get_update_log(self.h, node, _p(a), n.value, C.byref(n)))
        return a[:n.value]

    def key_log(self):
        n = C.c_int64()
        self._check(self.lib.ampnet_get_key_log(self.h, None, None, None, None, 0, C.byref(n)))
        m = max(n.value, 1)
        inst, slot = np.zeros(m, np.int64), np.zeros(m, np.int32)
        adm, rel = np.zeros(m, np.int64), np.zeros(m, np.int64)
        self._check(self.lib.ampnet_get_key_log(self.h, _p(inst), _p(slot), _p(adm), _p(rel), n.value, C.byref(n)))
        return inst[:n.value], slot[:n.value], adm[:n.value], rel[:n.value]

    def leftover_cache_entries(self):
        n = C.c_int64()
        self._check(self.lib.ampnet_leftover_cache_entries(self.h, C.byref(n)))
        return n.value

    def phase_cycles(self, node):
        a = np.zeros(16, np.uint64)
        b = C.c_int64()
        self._check(self.lib.ampnet_get_phase_cycles(self.h, node, _p(a), C.byref(b)))
        return a, b.value

    def queue_occupancy(self, node):
        """(forward, backward) high-water marks of the node's rings in the last asynchronous run."""
        f, b = C.c_int64(), C.c_int64()
        self._check(self.lib.ampnet_get_queue_occupancy(self.h, node, C.byref(f), C.byref(b)))
        return f.value, b.value

    def micro_batch_split(self, node):
        """(FMA, tensor-core) micro-batches of the node in the last run."""
        f, t = C.c_int64(), C.c_int64()
        self._check(self.lib.ampnet_get_micro_batch_split(self.h, node, C.byref(f), C.byref(t)))
        return f.value, t.value

    def placement(self, node):
        t, b = C.c_int32(), C.c_int32()
        self._check(self.lib.ampnet_get_placement(self.h, node, C.byref(t), C.byref(b)))
        return t.value, b.value
