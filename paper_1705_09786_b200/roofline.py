"""Algorithmic work model of AMP training and the roofline it is measured against (host arithmetic only).

Flop convention (paper, appendix "Throughput calculation for the GGSNN model"): a forward mat-vec costs
2*in*out per payload row; the backward pass is counted as transpose-multiply plus gradient accumulation,
i.e. twice the forward cost when the input gradient is needed and once when it is not (a node fed directly
by the controller); a local update costs 2 flops per parameter.  Elementwise work is ignored.
"""
import numpy as np

from workloads import ir   # integer codes of the IR format only

SM_COUNT = 148             # B200: 2 dies x 74 SMs
# dram__bytes_read.sum + dram__bytes_write.sum of the persistent kernel per instance, from the ncu captures summarised
# under profiles/ (captured on a small case; traffic grows in proportion to the instances processed): the tree workload
# on ampnet_engine_direct (600 trees: 14.31 + 16.74 MB), the graph workload on ampnet_engine (1,000 graphs), the stress
# configuration on ampnet_engine_direct (60 trees: 328.2 + 391.2 MB)
MEASURED_DRAM_BYTES_PER_INSTANCE = {"tree": 51753.0, "ggnn": 858646.0, "stress": 11989589.0}
FP32_LANES_PER_SM = 128


def fma_peak_tflops(sm_mhz, sm_count=SM_COUNT):
    """FP32 FMA peak = SMs x 128 lanes x 2 flop x clock."""
    return sm_count * FP32_LANES_PER_SM * 2 * sm_mhz * 1e6 / 1e12


def appendix_c_estimate(H=200, N=30, E=30, C=4, steps=4, device_flops=1e12, factor=0.5, bytes_per_float=4):
    """The paper's own closed-form estimate for a network of 1-TFLOPS devices; used to pin the convention."""
    fwdop = 2 * max(2 * N * H * H, E * H * H / C)
    bwdop = 6 * max(2 * N * H * H, E * H * H / C)
    throughput = factor * device_flops / ((fwdop + bwdop) * steps)
    bandwidth_bits = 8 * bytes_per_float * throughput * max(N, E) * H
    memory_bytes = 4 * (2 * H * H) * bytes_per_float
    return dict(fwdop=fwdop, bwdop=bwdop, throughput=throughput, bandwidth_bits=bandwidth_bits,
                memory_bytes=memory_bytes)


def gradient_rows(graph, inst):
    """{ppt node: payload rows it receives per epoch (forward = backward)} from the instance structure."""
    name = graph.name
    if name == "mlp":
        return {n: inst.n for n in graph.ppt_nodes()}
    if name == "rnn":
        T = int(np.diff(inst.offsets).sum())
        return {graph.index("lookup"): T, graph.index("linear1"): T, graph.index("linear2"): inst.n}
    if name in ("tree", "tree_grouped"):                   # (grouping changes the messages, not the payload rows)
        L = (np.diff(inst.offsets) + 1) // 2
        return {graph.index("lookup"): int(L.sum()), graph.index("leaf_cell"): int(L.sum()),
                graph.index("branch_cell"): int((L - 1).sum()), graph.index("classifier"): int((2 * L - 1).sum())}
    if name == "tree_lstm":
        L = (np.diff(inst.offsets) + 1) // 2
        return {graph.index("lookup"): int(L.sum()), graph.index("leaf_gates"): int(L.sum()),
                graph.index("branch_gates"): int((L - 1).sum()), graph.index("classifier"): int((2 * L - 1).sum())}
    if name == "ggnn":
        steps = int(graph.nodes[graph.index("cond_it")][5])
        N = int(np.diff(inst.offsets).sum())
        rows = {graph.index("lookup"): N, graph.index("gru"): steps * N, graph.index("readout1"): inst.n,
                graph.index("readout2"): inst.n}
        cnt = np.bincount(inst.edge_type, minlength=ir.N_EDGE_TYPES)
        for c in range(ir.N_EDGE_TYPES):
            rows[graph.index(f"edge_linear{c}")] = steps * int(cnt[c])
        return rows
    raise ValueError(name)


def node_messages(graph, inst):
    """Logical node-messages per epoch of the canonical IR graphs (closed forms of the routing)."""
    name = graph.name
    if name == "mlp":
        return (2 * len(graph.ppt_nodes()) + 1) * inst.n
    if name == "rnn":
        T = np.diff(inst.offsets)
        return int((13 * T + 3).sum())
    if name == "tree":
        L = (np.diff(inst.offsets) + 1) // 2
        return int((33 * L - 18).sum())
    if name == "tree_lstm":
        L = (np.diff(inst.offsets) + 1) // 2
        return int((55 * L - 32).sum())
    if name == "ggnn":
        steps = int(graph.nodes[graph.index("cond_it")][5])
        N, D = np.diff(inst.offsets), np.diff(inst.edge_offsets)
        gid = np.repeat(np.arange(inst.n), D)
        Dc = np.zeros((inst.n, ir.N_EDGE_TYPES), np.int64)
        np.add.at(Dc, (gid, inst.edge_type), 1)
        Cp = (Dc > 0).sum(1)
        return int((steps * (6 * N + 4 * D + 8 * Cp + 16) + 9).sum())
    raise ValueError(name)


def algorithmic_flops(graph, inst, updates=None):
    """Flops of one epoch.  updates: {node: number of local updates} (None = ignore the update term)."""
    rows = gradient_rows(graph, inst)
    nodes = graph.nodes
    total = 0.0
    for n, r in rows.items():
        t, din, dout, flags = int(nodes[n][0]), int(nodes[n][1]), int(nodes[n][2]), int(nodes[n][7])
        if t == ir.LOOKUP:
            continue
        nmat = 3 if t == ir.GRUCELL else 1
        fwd = 2.0 * din * dout * nmat
        bwd = fwd if (flags & ir.FLAG_SOURCE_ADJACENT) else 2 * fwd
        total += r * (fwd + bwd)
        if updates:
            total += updates.get(n, 0) * 2.0 * (din * dout + dout) * nmat
    return total


def payload_bytes(graph, inst):
    """Bytes of PPT-to-PPT payloads written and read once each (fp32): the HBM term of the roofline."""
    rows = gradient_rows(graph, inst)
    nodes = graph.nodes
    total = 0.0
    for n, r in rows.items():
        din, dout = int(nodes[n][1]), int(nodes[n][2])
        t = int(nodes[n][0])
        width_in = 1 if t == ir.LOOKUP else din
        total += r * 4.0 * 2 * 2 * (width_in + dout)     # x and y, forward and backward, write + read
    return total


def reload_bytes(graph, inst):
    """Device-memory bytes of a design that reloads the weights for every message (the per-message mat-vec the paper
    argues existing frameworks are bound by): W read forward, W read backward, accumulator read and written, per
    payload row and matrix."""
    rows = gradient_rows(graph, inst)
    nodes = graph.nodes
    total = 0.0
    for n, r in rows.items():
        t, din, dout = int(nodes[n][0]), int(nodes[n][1]), int(nodes[n][2])
        if t == ir.LOOKUP:
            continue
        total += r * 4.0 * 4 * din * dout * (3 if t == ir.GRUCELL else 1)
    return total


def roofline_instances_per_s(graph, inst, sm_mhz, hbm_gbs):
    """On-chip-resident-weight roofline: weights never reloaded; bound by FP32 FMA or by payload traffic."""
    F = algorithmic_flops(graph, inst) / inst.n
    B = payload_bytes(graph, inst) / inst.n
    t = max(F / (fma_peak_tflops(sm_mhz) * 1e12), B / (hbm_gbs * 1e9))
    return 1.0 / t, F, B
