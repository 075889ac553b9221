"""ctypes wrapper of the CPU oracle (test infrastructure; never imported by the product package)."""
import ctypes as C
import os
import subprocess
import time

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "ampnet_oracle.cpp")
_LIBS = {}


def _lib_path(real):
    return os.path.join(_DIR, f"liboracle_{real}.so")


def build(real="f64", force=False):
    """Compile the oracle (plain g++ -O2, no BLAS, no intrinsics).  real in {"f64", "f32"}."""
    out = _lib_path(real)
    if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(_SRC):
        return out
    ctype = {"f64": "double", "f32": "float"}[real]
    tmp = out + f".tmp{os.getpid()}"
    subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", f"-DORACLE_REAL={ctype}", "-o", tmp, _SRC])
    os.replace(tmp, out)
    return out


class OracleStats(C.Structure):
    _fields_ = [("instances", C.c_int64), ("node_messages", C.c_int64), ("ppt_messages", C.c_int64),
                ("rounds", C.c_int64), ("seconds", C.c_double), ("mean_loss", C.c_double),
                ("max_staleness", C.c_int32), ("max_active_observed", C.c_int64), ("route_hash", C.c_uint64),
                ("leftover_cache_entries", C.c_int64)]


def _load(real):
    if real in _LIBS:
        return _LIBS[real]
    lib = C.CDLL(build(real))
    P = C.c_void_p
    lib.oracle_create.restype = P
    lib.oracle_create.argtypes = [P, C.c_int, P, C.c_int, C.c_int]
    lib.oracle_destroy.argtypes = [P]
    lib.oracle_last_error.restype = C.c_char_p
    lib.oracle_last_error.argtypes = [P]
    lib.oracle_load_instances.argtypes = [P, C.c_int, C.c_int, C.c_int64] + [P] * 9 + [C.c_int, P, P]
    lib.oracle_param_count.restype = C.c_int64
    lib.oracle_param_count.argtypes = [P, C.c_int, C.c_int]
    for f in (lib.oracle_set_params, lib.oracle_get_params, lib.oracle_get_accum):
        f.argtypes = [P, C.c_int, C.c_int, P, C.c_int64]
    lib.oracle_run_epoch.argtypes = [P, C.c_int, C.c_int, C.c_int, C.c_double, P, C.c_int64, C.c_int,
                                     C.POINTER(OracleStats), P]
    lib.oracle_eval.argtypes = [P, C.c_int, P, P, P]
    lib.oracle_run_epoch_mixed.argtypes = [P, C.c_int, C.c_int, C.c_int, C.c_double, P, C.c_int64, C.c_int, P,
                                           C.POINTER(OracleStats), P, P]
    lib.oracle_set_optimizer.argtypes = [P, C.c_int, C.c_double, C.c_double, C.c_double, C.c_double, C.c_int]
    lib.oracle_get_node_stats.argtypes = [P, C.c_int, P, P, P, P, P]
    lib.oracle_round_bf16.argtypes = [P, P, C.c_int64]
    lib.oracle_get_update_log.restype = C.c_int64
    lib.oracle_get_update_log.argtypes = [P, C.c_int, P, C.c_int64]
    lib.oracle_get_key_log.restype = C.c_int64
    lib.oracle_get_key_log.argtypes = [P, P, P, P, P, C.c_int64]
    _LIBS[real] = lib
    return lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def round_bf16(values, real="f64"):
    """The oracle's payload rounding (to bfloat16, nearest even) applied to an array of float32-representable values."""
    a = np.ascontiguousarray(values, dtype=np.float64)
    out = np.empty_like(a)
    _load(real).oracle_round_bf16(_p(a), _p(out), a.size)
    return out


class Oracle:
    def __init__(self, graph, real="f64", payload_bf16=False):
        self.lib = _load(real)
        self.graph = graph
        nodes, edges = graph.nodes, graph.edges
        self.h = self.lib.oracle_create(_p(nodes), len(nodes), _p(edges), len(edges), int(payload_bf16))
        if not self.h:
            raise ValueError("oracle_create failed: malformed IR description")
        self.n = [0, 0]

    def __del__(self):
        if getattr(self, "h", None):
            self.lib.oracle_destroy(self.h)
            self.h = None

    def _check(self, rc):
        if rc != 0:
            raise RuntimeError("oracle: " + self.lib.oracle_last_error(self.h).decode())

    def load_instances(self, inst, split=0):
        self._keep = getattr(self, "_keep", {})
        self._keep[split] = inst
        dd = 0 if inst.dense is None else inst.dense.shape[1]
        self._check(self.lib.oracle_load_instances(
            self.h, split, inst.kind, inst.n, _p(inst.offsets), _p(inst.tokens), _p(inst.left), _p(inst.right),
            _p(inst.edge_offsets), _p(inst.edge_src), _p(inst.edge_dst), _p(inst.edge_type), _p(inst.dense), dd,
            _p(inst.labels_i), _p(inst.labels_f)))
        self.n[split] = inst.n

    def set_params(self, params):
        for (node, which), v in params.items():
            a = np.ascontiguousarray(v, dtype=np.float64).ravel()
            if self.lib.oracle_set_params(self.h, node, which, _p(a), a.size) != 0:
                raise ValueError(f"set_params({node},{which}): size mismatch")

    def _get(self, fn, node, which):
        n = self.lib.oracle_param_count(self.h, node, which)
        if n < 0:
            raise KeyError((node, which))
        a = np.empty(n, np.float64)
        if fn(self.h, node, which, _p(a), n) != 0:
            raise RuntimeError("oracle get failed")
        shape = dict(self.graph.param_shapes(node))[which]
        return a.reshape(shape)

    def get_params(self, node=None, which=None):
        if node is not None:
            return self._get(self.lib.oracle_get_params, node, which)
        return {(i, w): self._get(self.lib.oracle_get_params, i, w)
                for i in self.graph.ppt_nodes() for w, _ in self.graph.param_shapes(i)}

    def get_accum(self, node, which):
        return self._get(self.lib.oracle_get_accum, node, which)

    def run_epoch(self, mak, muf, lr, order=None, flush=True, split=0):
        n = self.n[split]
        order = np.arange(n, dtype=np.int64) if order is None else np.ascontiguousarray(order, dtype=np.int64)
        st = OracleStats()
        loss = np.zeros(n, np.float64)
        lr = float(np.float32(lr))
        t0 = time.perf_counter()
        self._check(self.lib.oracle_run_epoch(self.h, split, mak, muf, lr, _p(order), len(order), int(flush),
                                              C.byref(st), _p(loss)))
        st.seconds = time.perf_counter() - t0
        return st, loss

    def run_epoch_mixed(self, mak, muf, lr, inference_only, order=None, flush=True, split=0):
        """Training epoch in which the instances marked in inference_only (uint8 per instance) are only evaluated.
        Returns (stats, per-instance loss, dict(instances, mean_loss, accuracy) of the inference instances)."""
        n = self.n[split]
        order = np.arange(n, dtype=np.int64) if order is None else np.ascontiguousarray(order, dtype=np.int64)
        mask = np.ascontiguousarray(inference_only, dtype=np.uint8)
        assert mask.shape == (n,)
        st, loss, inf = OracleStats(), np.zeros(n, np.float64), np.zeros(3, np.float64)
        self._check(self.lib.oracle_run_epoch_mixed(self.h, split, mak, muf, float(np.float32(lr)), _p(order), len(order),
                                                    int(flush), _p(mask), C.byref(st), _p(loss), _p(inf)))
        return st, loss, dict(instances=int(inf[0]), mean_loss=inf[1], accuracy=inf[2])

    def set_optimizer(self, kind="sgd", momentum=0.9, beta1=0.9, beta2=0.999, eps=1e-8, reset=True):
        k = {"sgd": 0, "momentum": 1, "adam": 2}[kind]
        # the hyper-parameters are rounded to fp32 so that a float32 implementation uses the same numbers
        f = lambda v: float(np.float32(v))
        if self.lib.oracle_set_optimizer(self.h, k, f(momentum), f(beta1), f(beta2), f(eps), int(reset)) != 0:
            raise ValueError(kind)

    def average_params(self, nodes):
        """End-of-epoch replica synchronisation (Sec. 5): every listed node gets the mean of their parameters."""
        for which in (0, 1):
            mean = sum(self._get(self.lib.oracle_get_params, n, which) for n in nodes) / len(nodes)
            for n in nodes:
                self.set_params({(n, which): mean})

    def eval(self, split=0):
        ml, acc = C.c_double(), C.c_double()
        loss = np.zeros(self.n[split], np.float64)
        self._check(self.lib.oracle_eval(self.h, split, C.byref(ml), C.byref(acc), _p(loss)))
        return ml.value, acc.value, loss

    def node_stats(self, node):
        nu, ng, fw, bw = C.c_int64(), C.c_int64(), C.c_int64(), C.c_int64()
        hist = np.zeros(64, np.int64)
        self.lib.oracle_get_node_stats(self.h, node, C.byref(nu), C.byref(ng), _p(hist), C.byref(fw), C.byref(bw))
        return dict(n_updates=nu.value, n_grads_applied=ng.value, staleness_hist=hist, fwd_msgs=fw.value,
                    bwd_msgs=bw.value)

    def update_log(self, node):
        n = self.lib.oracle_get_update_log(self.h, node, None, 0)
        a = np.zeros(max(n, 1), np.int32)
        self.lib.oracle_get_update_log(self.h, node, _p(a), n)
        return a[:n]

    def key_log(self):
        n = self.lib.oracle_get_key_log(self.h, None, None, None, None, 0)
        inst, slot = np.zeros(max(n, 1), np.int64), np.zeros(max(n, 1), np.int32)
        adm, rel = np.zeros(max(n, 1), np.int64), np.zeros(max(n, 1), np.int64)
        self.lib.oracle_get_key_log(self.h, _p(inst), _p(slot), _p(adm), _p(rel), n)
        return inst[:n], slot[:n], adm[:n], rel[:n]
