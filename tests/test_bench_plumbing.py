"""Host logic of the benchmark: the flop model against the paper's appendix numbers, and the N > 1 rank plumbing
(independent replicas, max-over-ranks time) with world_size 2 on the gloo backend."""
import os
import socket
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_flop_convention_reproduces_the_papers_appendix_estimate():
    """fwd = 2*in*out per row, bwd = 3x fwd: the paper's closed form gives 6.5e3 samples/s, 1.2e9 bit/s, 1.2 MB."""
    from paper_1705_09786_b200 import roofline as rf
    import helpers
    gold = {k: float(v) for k, v in helpers.read_golden(os.path.join(GOLD, "appendix_c.txt"))}
    est = rf.appendix_c_estimate()
    assert abs(est["throughput"] - gold["throughput_samples_per_s"]) / gold["throughput_samples_per_s"] < 0.01
    assert abs(est["bandwidth_bits"] - gold["bandwidth_bits_per_s"]) / gold["bandwidth_bits_per_s"] < 0.05
    assert abs(est["memory_bytes"] - gold["memory_bytes"]) / gold["memory_bytes"] < 0.08
    # the same convention applied to our GRU step: fwd + bwd of the 3 gate matrices = 3 * 3 * 2*(2H*H) per node row
    assert est["fwdop"] + est["bwdop"] == 8 * 2 * 30 * 200 * 200


def test_work_model_counts(oracle_mod):
    """Gradient rows and node-message closed forms used by the benchmark equal what the oracle counts."""
    from paper_1705_09786_b200 import roofline as rf
    from workloads import ir, data, params as wp
    cases = [(ir.mlp((8, 6, 6, 3)), data.mlp_instances(n=9, dim=8, classes=3)),
             (ir.rnn(emb=6, hidden=6), data.list_instances(n=7, max_len=5)),
             (ir.tree(vocab=30, emb=6, hidden=5, classes=3), data.tree_instances(n=5, max_leaves=7, vocab=30, classes=3)),
             (ir.ggnn(hidden=4, readout=3), data.graph_instances(n=4, min_nodes=3, max_nodes=6))]
    for g, inst in cases:
        o = oracle_mod.Oracle(g)
        o.load_instances(inst)
        o.set_params(wp.init_params(g))
        st, _ = o.run_epoch(mak=3, muf=5, lr=0.01)
        assert rf.node_messages(g, inst) == st.node_messages
        for n, rows in rf.gradient_rows(g, inst).items():
            assert o.node_stats(n)["n_grads_applied"] == rows
    g, inst = cases[0]
    # 3 layers: (8*6 + 6*6 + 6*3) * 2 forward; backward 1x for the first layer, 2x for the others
    want = inst.n * (2 * 48 * 2 + 2 * 36 * 3 + 2 * 18 * 3)
    assert rf.algorithmic_flops(g, inst) == want
    assert rf.fma_peak_tflops(1965.0) == pytest.approx(74.45, rel=1e-3)
    # weight-reload bytes: every message pair reads W twice and reads + writes the accumulator (4 x 4 bytes x in x out)
    assert rf.reload_bytes(g, inst) == inst.n * 16 * (48 + 36 + 18)
    gt, it = cases[2]
    L = (np.diff(it.offsets) + 1) // 2
    assert rf.reload_bytes(gt, it) == 16 * (L.sum() * 6 * 5 + (L - 1).sum() * 10 * 5 + (2 * L - 1).sum() * 5 * 3)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import bench
    r, w = bench.dist_init("gloo")
    assert (r, w) == (rank, world)
    _, inst, _ = bench.make_workload("rnn", rank, n=50)          # every rank draws its own shard
    bench.barrier()
    value, tmax = bench.aggregate(units_this_rank=100 * (rank + 1), seconds_this_rank=1.0 + rank)
    # end-of-epoch averaging of the replicas' parameters (Sec. 5): rank r holds r + 1 and 10 (r + 1)
    import torch
    from paper_1705_09786_b200.replicas import average_across_ranks
    params = [torch.full((3, 2), float(rank + 1)), torch.full((5,), 10.0 * (rank + 1))]
    n = average_across_ranks(params)
    assert n == world and torch.all(params[0] == 1.5) and torch.all(params[1] == 15.0)
    q.put((rank, value, tmax, int(inst.tokens[:64].sum())))
    import torch.distributed as dist
    dist.destroy_process_group()


def test_replica_aggregation_world_size_2_gloo():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, v0, t0, s0), (r1, v1, t1, s1) = out
    assert v0 == v1 == pytest.approx(300 / 2.0)       # units of all ranks / the slowest rank's time
    assert t0 == t1 == 2.0
    assert s0 != s1                                   # independent shards


def test_replica_sync_note_when_the_collective_raises():
    """bench.py with N > 1 averages the replicas at the end of every epoch; if the collective raises, the ranks go on as
    independent replicas and the JSON line's config.replica_sync says so (and averaging is not tried again)."""
    import bench
    calls = []

    def ok(views):
        calls.append("ok")

    def broken(views):
        calls.append("broken")
        raise RuntimeError("NCCL error")

    avg = {"on": True, "note": "end-of-epoch parameter averaging over NCCL"}
    bench.average_replicas([], avg, ok)
    assert avg["on"] and calls == ["ok"]
    bench.average_replicas([], avg, broken)
    assert not avg["on"] and "RuntimeError" in avg["note"] and "independent replicas" in avg["note"]
    bench.average_replicas([], avg, broken)                      # switched off: the collective is not called again
    assert calls == ["ok", "broken"]
    single = {"on": False, "note": "single replica"}
    bench.average_replicas([], single, broken)
    assert single == {"on": False, "note": "single replica"}
