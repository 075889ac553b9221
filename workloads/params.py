"""Seeded parameter initialisers (host generated; loaded into both implementations through set_params)."""
import numpy as np

from . import ir
from .data import MASTER_SEED


def init_params(graph, seed=1, emb_std=0.1):
    """{(node, which): float64 array}.  Linear / GRU matrices ~ U(+-sqrt(6/(in+out))), biases 0,
    embedding tables ~ N(0, emb_std)."""
    rng = np.random.default_rng([MASTER_SEED, 11, int(seed)])
    out = {}
    nodes = graph.nodes
    for i in graph.ppt_nodes():
        t, din, dout = (int(v) for v in nodes[i][:3])
        for which, shape in graph.param_shapes(i):
            if t == ir.LOOKUP:
                out[(i, which)] = rng.standard_normal(shape) * emb_std
            elif len(shape) == 2:
                lim = np.sqrt(6.0 / (din + dout))
                out[(i, which)] = rng.uniform(-lim, lim, size=shape)
            else:
                out[(i, which)] = np.zeros(shape)
    # round to fp32 so that a float32 and a float64 implementation start from the same numbers
    return {k: v.astype(np.float32).astype(np.float64) for k, v in out.items()}
