#!/usr/bin/env python
"""Benchmark of the AMPNet training hot path on B200.

A step is one epoch of asynchronous model-parallel training (admission, message-driven forward and backward
execution, local updates, retirement) over one seeded synthetic workload.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload tree|ggnn|rnn|mlp] [--impl ours|reference]

`--impl reference` times the CPU oracle (test infrastructure) on a bounded sample of the same workload.
With N > 1 (torchrun) every rank trains an independent replica on its own shard; there is no collective on
the data path.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import ir, data, params as wp  # noqa: E402

WORKLOADS = {
    # name: (graph builder, instance generator, full size, mak, muf, lr)
    "mlp": (ir.mlp, data.mlp_instances, 2048, 4, 32, 0.01),
    "rnn": (ir.rnn, data.list_instances, 20000, 16, 50, 0.05),
    "tree": (ir.tree, data.tree_instances, 8544, 64, 100, 0.05),
    "ggnn": (ir.ggnn, data.graph_instances, 130000, 128, 200, 0.01),
    # the tree model with the leaf operations of a tree grouped into one matrix message (Sec. 6); runs on the interpreter engine
    "tree_grouped": (lambda: ir.tree(grouped_leaves=True), data.tree_instances, 8544, 64, 100, 0.05),
    # the paper's sentiment model proper: binary Tree-LSTM (leaf and branch cells) on the same trees as "tree"
    "tree_lstm": (ir.tree_lstm, data.tree_instances, 8544, 64, 100, 0.05),
    # throughput stress: binary tree RNN, hidden 512, 64..512 leaves, bf16 messages with fp32 accumulators
    "stress": (lambda: ir.tree(vocab=20000, emb=512, hidden=512, classes=5),
               lambda n, split=0: data.tree_instances(n=n, min_leaves=64, max_leaves=512, split=split, config_index=5),
               50000, 64, 64, 0.01),
}
STRESS_BENCH_INSTANCES = 1000     # the stress workload is timed on a prefix of this many trees per step
BASELINE_CONFIGS = ("mlp", "rnn", "tree", "ggnn", "stress")      # the five configurations of the benchmark set
SWEEP_MAK = (1, 8, 64, 256, 1024)
SWEEP_MUF = (1, 64, 1024)
GGNN_BENCH_INSTANCES = 20000      # the graph workload is timed on a prefix of this many graphs per step


def make_workload(name, rank=0, n=None):
    build_graph, gen, full, mak, muf, lr = WORKLOADS[name]
    if n is None:
        n = GGNN_BENCH_INSTANCES if name == "ggnn" else STRESS_BENCH_INSTANCES if name == "stress" else full
    inst = gen(n=n, split=0 if rank == 0 else 100 + rank)
    return build_graph(), inst, dict(mak=mak, muf=muf, lr=lr, full=full, bf16=(name == "stress"))


# ---------------------------------------------------------------------------------------------------
# process-group plumbing (kept in functions so that the N > 1 path is testable with gloo on CPU)
# ---------------------------------------------------------------------------------------------------
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1)), int(os.environ.get("LOCAL_RANK", 0))


def dist_init(backend):
    import torch.distributed as dist
    rank, world, _ = dist_env()
    if world > 1 and not dist.is_initialized():
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def all_max(x, device="cpu"):
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def all_sum(x, device="cpu"):
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def aggregate(units_this_rank, seconds_this_rank, device="cpu"):
    """Whole-job throughput: units of all ranks / the slowest rank's time."""
    total = all_sum(units_this_rank, device)
    t = all_max(seconds_this_rank, device)
    return total / t if t > 0 else 0.0, t


# ---------------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.stop_flag, self.proc = index, [], threading.Event(), None

    def run(self):
        # one nvidia-smi process that prints a line every 100 ms (starting a process per sample takes longer than that)
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-i", str(self.index),
                                          "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            for line in self.proc.stdout:
                if self.stop_flag.is_set():
                    break
                if line.strip():
                    self.samples.append([v.strip() for v in line.strip().split(",")])
            return
        except Exception:
            self.proc = None
        while not self.stop_flag.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-i",
                                      str(self.index)], capture_output=True, text=True, timeout=5).stdout.strip()
                if out:
                    self.samples.append([v.strip() for v in out.split(",")])
            except Exception:
                pass
            self.stop_flag.wait(0.2)

    def summary(self):
        self.stop_flag.set()
        proc = getattr(self, "proc", None)
        if proc is not None and proc.poll() is None:
            proc.terminate()                                   # (the process this sampler started, nothing else)
        self.join(timeout=6)
        sm = [float(s[0]) for s in self.samples if s and s[0].replace(".", "").isdigit()]
        mx = [float(s[1]) for s in self.samples if len(s) > 1 and s[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for s in self.samples for i in range(4) if len(s) > 2 + i and s[2 + i] == "Active"})
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f), "measured"
    except Exception:
        return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0}, "fallback"


def host_description():
    model = "unknown"
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return {"nproc": os.cpu_count(), "cpu_model": model}


def time_oracle(graph, inst, cfg, target_s=12.0, probe=48):
    """The oracle as it stands, single-threaded, on a bounded prefix of the workload."""
    import oracle as oracle_mod
    o = oracle_mod.Oracle(graph, payload_bf16=cfg.get("bf16", False))
    p = wp.init_params(graph)
    probe = min(probe, inst.n)
    o.load_instances(inst.head(probe))
    o.set_params(p)
    st, _ = o.run_epoch(mak=cfg["mak"], muf=cfg["muf"], lr=cfg["lr"])
    per = st.seconds / probe
    n = int(max(probe, min(inst.n, target_s / max(per, 1e-9))))
    sample = inst.head(n)
    o.load_instances(sample)
    o.set_params(p)
    st, _ = o.run_epoch(mak=cfg["mak"], muf=cfg["muf"], lr=cfg["lr"])
    return dict(instances=n, seconds=st.seconds, inst_per_s=n / st.seconds, msgs_per_s=st.node_messages / st.seconds)


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    graph, inst, cfg = make_workload(args.workload, n=args.instances)
    times, units, msgs = [], 0, 0
    res = None
    for k in range(args.warmup + args.steps):
        res = time_oracle(graph, inst, cfg, target_s=8.0 if args.steps > 1 else 12.0)
        if k >= args.warmup:
            times.append(res["seconds"]); units += res["instances"]; msgs += res["msgs_per_s"] * res["seconds"]
    tot = sum(times)
    value = units / tot
    sample = f"first {res['instances']} of {inst.n} instances per step, one epoch each"
    line = {"impl": "reference", "metric": "training_instances_per_s", "value": value, "unit": "instances/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "node_messages_per_s": msgs / tot,
            "config": workload_config(args.workload, inst, cfg, "canonical round schedule on the host"),
            "cpu_baseline": dict({"value": value, "unit": "instances/s", "cores": 1, "kind": "oracle", "sample": sample,
                                  "arithmetic": "f64 build of the oracle, single thread"}, **host_description()),
            "e2e": {"value": value, "unit": "instances/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def workload_config(name, inst, cfg, mode):
    return {"workload": name, "messages": "bf16 payloads, fp32 accumulators" if cfg.get("bf16") else "fp32", "instances_per_step": int(inst.n), "full_dataset_instances": cfg["full"],
            "max_active_keys": cfg["mak"], "min_update_frequency": cfg["muf"], "lr": cfg["lr"], "mode": mode,
            "l2": "flushed between steps (256 MiB write)", "parallelism": "replicas, no collective"}


def input_bytes(inst):
    return int(sum(a.nbytes for a in (inst.offsets, inst.tokens, inst.left, inst.right, inst.edge_offsets, inst.edge_src,
                                      inst.edge_dst, inst.edge_type, inst.dense, inst.labels_i, inst.labels_f)
                   if a is not None))


def split_counts(eng, graph):
    """Micro-batches of the last run by the unit that ran their product, counted on the device (first forward and first
    backward tile of every node)."""
    fma = tensor = 0
    for n in graph.ppt_nodes():
        f, t = eng.micro_batch_split(n)
        fma += f
        tensor += t
    return {"micro_batches_fma": int(fma), "micro_batches_tensor_core": int(tensor)}


def micro_batch_split(eng, graph):
    c = split_counts(eng, graph)
    total = max(1, c["micro_batches_fma"] + c["micro_batches_tensor_core"])
    return {"fma": c["micro_batches_fma"] / total, "tensor_core": c["micro_batches_tensor_core"] / total, **c,
            "note": "tensor cores (tcgen05, bf16 operands, fp32 accumulation) run the forward products of nodes with out_dim % 64 == 0 "
                    "and in_dim % 16 == 0 in bf16 runs (the stress configuration's cells); everything else runs on FP32 FMA"}


def average_replicas(views, averaging, average_fn=None):
    """End-of-epoch replica synchronisation (Sec. 5) inside the timed region.  If the collective cannot run the ranks
    continue as independent replicas and `averaging` (reported as config.replica_sync) says so."""
    if not averaging["on"]:
        return
    try:
        if average_fn is None:
            from paper_1705_09786_b200.replicas import average_across_ranks as average_fn
        average_fn(views)
    except Exception as exc:                                   # keep measuring independent replicas
        averaging.update(on=False, note=f"averaging unavailable ({type(exc).__name__}); independent replicas")


def roofline_object(rf, graph, inst, workload, flops, kernel_s, peak_tf, peaks, peak_kind, mak, rate_one_key, n1):
    """The roofline record of one workload: algorithmic flops of a launch / its device time against the FP32 FMA peak
    measured in this run, with the resident-weight roofline and the concurrency ceiling beside it."""
    sm_mhz = float(peaks.get("sm_max_mhz", 1965.0))
    achieved = flops / kernel_s / 1e12
    roof_inst, F, B = rf.roofline_instances_per_s(graph, inst, sm_mhz, float(peaks.get("hbm_gbs", 6650.0)))
    per_inst = rf.MEASURED_DRAM_BYTES_PER_INSTANCE.get(workload)
    return {"bound": "alu", "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s", "frac": achieved / peak_tf,
            "traffic": per_inst * inst.n if per_inst else None,
            "traffic_note": ("ncu capture on a small case, scaled by instances processed (see profiles/)" if per_inst
                             else "no ncu capture for this workload"),
            "peak_kind": "measured in this run: register-only FP32 FMA kernel (ampnet_measure_fma_peak)",
            "peak_derived": rf.fma_peak_tflops(sm_mhz),
            "peak_derived_kind": f"148 SMs x 128 FP32 lanes x 2 x {sm_mhz:.0f} MHz ({peak_kind} max SM clock)",
            "concurrency_ceiling_instances_per_s": mak * rate_one_key,
            "concurrency_ceiling_kind": f"max_active_keys x the rate at one key in flight ({rate_one_key:.0f}/s on {n1} instances)",
            "kernel": "one persistent launch per step (ampnet_engine_direct; ampnet_engine for graphs with row-wise groups)",
            "kernel_ms": kernel_s * 1e3, "algorithmic_flop_per_launch": flops, "flop_per_instance": F,
            "payload_bytes_per_instance": B, "resident_weight_roofline_instances_per_s": roof_inst,
            "weight_reload_roofline_instances_per_s": float(peaks.get("hbm_gbs", 6650.0)) * 1e9 / (rf.reload_bytes(graph, inst) / inst.n),
            "weight_reload_roofline_kind": "a per-message mat-vec that reads W forward and backward and updates the accumulator in device memory (context)",
            "frac_of_resident_weight_roofline": (inst.n / kernel_s) / roof_inst}


def one_key_rate(eng, inst, cfg, timeout):
    n1 = max(8, min(inst.n, 64))
    eng.load_instances(inst.head(n1))
    st1, _ = eng.run_epoch(mak=1, muf=cfg["muf"], lr=0.0, deterministic=False, timeout_s=timeout, want_loss=False)
    eng.load_instances(inst)
    return n1 / st1.seconds, n1


def run_ours(args):
    import torch
    import paper_1705_09786_b200 as amp
    from paper_1705_09786_b200 import roofline as rf
    rank, world, local = dist_env()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist_init("nccl")
    graph, inst, cfg = make_workload(args.workload, rank, n=args.instances)
    eng = amp.Engine(graph, device=local, payload_bf16=cfg["bf16"])
    eng.load_instances(inst)
    p0 = wp.init_params(graph)
    eng.set_params(p0)
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)

    # With more than one rank the replicas are averaged in place at the end of every epoch (Sec. 5), inside the timed
    # region; if the collective cannot run, the ranks stay independent replicas and the line says so.
    averaging = {"on": world > 1, "note": "end-of-epoch parameter averaging over NCCL" if world > 1 else "single replica"}
    views = list(eng.param_tensors().values()) if world > 1 else []

    def step():
        eng.set_params(p0)                                     # every step starts from the same parameters (untimed)
        flush_buf.fill_(1)                                     # evict L2 between steps (outside the timed events)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        st, _ = eng.run_epoch(mak=cfg["mak"], muf=cfg["muf"], lr=cfg["lr"], deterministic=False, timeout_s=args.timeout,
                              want_loss=False)
        average_replicas(views, averaging)
        e1.record(stream)
        e1.synchronize()
        return st, e0.elapsed_time(e1) * 1e-3

    for _ in range(args.warmup):
        step()
    sampler = ClockSampler(local)
    sampler.start()
    torch.cuda.synchronize()
    barrier()
    step_s, kern_s, msgs, last = [], [], 0, None
    for _ in range(args.steps):
        st, s = step()
        step_s.append(s); kern_s.append(st.seconds); msgs += st.node_messages; last = st
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.summary()
    updates = {n: eng.node_stats(n)["n_updates"] for n in graph.ppt_nodes()}     # of the last timed step
    placement = {graph.names[n]: eng.placement(n) for n in graph.ppt_nodes()}
    queue_occ = {graph.names[n]: list(eng.queue_occupancy(n)) for n in graph.ppt_nodes()}
    split = micro_batch_split(eng, graph)
    secs = sum(step_s)
    value, tmax = aggregate(inst.n * args.steps, secs, dev)
    msg_rate, _ = aggregate(msgs, secs, dev)

    # ---- end to end: host buffers in, per-instance losses out, every step --------------------------------
    pinned = {}
    for k in ("offsets", "tokens", "left", "right", "edge_offsets", "edge_src", "edge_dst", "edge_type", "dense",
              "labels_i", "labels_f"):
        a = getattr(inst, k)
        if a is not None:
            pinned[k] = torch.from_numpy(a).pin_memory()
            setattr(inst, k, pinned[k].numpy())
    e2e_steps = max(1, min(args.steps, 3))
    torch.cuda.synchronize()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        eng.load_instances(inst)
        st, loss = eng.run_epoch(mak=cfg["mak"], muf=cfg["muf"], lr=cfg["lr"], deterministic=False, timeout_s=args.timeout)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_value, _ = aggregate(inst.n * e2e_steps, e2e_s, dev)

    # ---- forward-only throughput (the paper's inference column): the same instances, evaluation messages only -----
    eng.eval(0, mak=cfg["mak"])
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    eng.eval(0, mak=cfg["mak"])
    torch.cuda.synchronize()
    inference_rate = inst.n / (time.perf_counter() - t0)

    # ---- diagnostics: the FP32 FMA rate of this GPU, measured; the concurrency ceiling mak x (rate at one key) ------
    fma_measured = amp.measure_fma_peak(local)
    rate_one_key, n1 = one_key_rate(eng, inst, cfg, args.timeout)
    # ---- the other configurations of the benchmark set, briefly (single GPU only): same timing rules, fewer steps ----
    others = None
    if world == 1 and not args.no_other_configs and args.instances is None:
        eng.close()
        eng = None
        others = {}
        for name in BASELINE_CONFIGS:
            if name == args.workload:
                continue
            g2, inst2, cfg2 = make_workload(name, rank)
            e2 = amp.Engine(g2, device=local, payload_bf16=cfg2["bf16"])
            e2.load_instances(inst2)
            e2.set_params(wp.init_params(g2))
            ks, ms = [], 0
            for k in range(3 + 2):                               # three warm-up epochs, two timed
                flush_buf.fill_(1)
                st2, _ = e2.run_epoch(mak=cfg2["mak"], muf=cfg2["muf"], lr=cfg2["lr"], deterministic=False,
                                      timeout_s=args.timeout, want_loss=False)
                if k >= 3:
                    ks.append(st2.seconds); ms += st2.node_messages
                if k < 4:
                    e2.set_params(wp.init_params(g2))
            fl = rf.algorithmic_flops(g2, inst2, {n: e2.node_stats(n)["n_updates"] for n in g2.ppt_nodes()})
            occ2 = {g2.names[n]: list(e2.queue_occupancy(n)) for n in g2.ppt_nodes()}
            split2 = micro_batch_split(e2, g2)
            split2.pop("note")
            r1, m1 = one_key_rate(e2, inst2, cfg2, args.timeout)
            peaks2, kind2 = measured_peaks()
            others[name] = {"instances_per_s": 2 * inst2.n / sum(ks), "node_messages_per_s": ms / sum(ks),
                            "tflops": fl / (sum(ks) / 2) / 1e12, "instances_per_step": int(inst2.n),
                            "full_dataset_instances": cfg2["full"], "max_active_keys": cfg2["mak"],
                            "min_update_frequency": cfg2["muf"], "steps": 2, "warmup": 3,
                            "timing": "device time of the persistent kernel (CUDA events around the launch), parameters reset before every epoch",
                            "roofline": roofline_object(rf, g2, inst2, name, fl, sum(ks) / 2, fma_measured, peaks2, kind2,
                                                        cfg2["mak"], r1, m1),
                            "queue_occupancy_max_pending_fwd_bwd": occ2, "micro_batch_split": split2}
            if not args.no_cpu_baseline:
                r = time_oracle(g2, inst2, cfg2, target_s=4.0, probe=16)
                others[name]["cpu_baseline"] = dict({"value": r["inst_per_s"], "unit": "instances/s", "cores": 1, "kind": "oracle",
                                                     "sample": f"first {r['instances']} of {inst2.n} instances, one epoch, {r['seconds']:.1f} s",
                                                     "arithmetic": "f64 build of the oracle, single thread"}, **host_description())
            e2.close()

    sweep = None
    if args.sweep and rank == 0:
        # max_active_keys x min_update_frequency grid on a prefix (one epoch each, parameters reset)
        sweep = []
        for mak in SWEEP_MAK:
            sub = inst.head(max(20, min(inst.n, 30 * mak if mak < 64 else 400)))
            eng.load_instances(sub)
            for muf in SWEEP_MUF:
                eng.set_params(p0)
                st, _ = eng.run_epoch(mak=mak, muf=muf, lr=cfg["lr"], deterministic=False, timeout_s=args.timeout,
                                      want_loss=False)
                sweep.append({"max_active_keys": mak, "min_update_frequency": muf, "instances": int(sub.n),
                              "instances_per_s": sub.n / st.seconds, "node_messages_per_s": st.node_messages / st.seconds,
                              "rows_per_micro_batch": st.micro_batch_rows / max(1, st.micro_batches),
                              "max_active_observed": int(st.max_active_observed), "max_staleness": int(st.max_staleness),
                              "queue_occupancy_max_pending_fwd_bwd": {graph.names[n]: list(eng.queue_occupancy(n)) for n in graph.ppt_nodes()},
                              **split_counts(eng, graph)})
        eng.load_instances(inst)
    if rank == 0:
        peaks, peak_kind = measured_peaks()
        flops = rf.algorithmic_flops(graph, inst, updates)
        peak_tf = fma_measured                       # measured in this run; the derived figure is reported beside it
        kavg = float(np.mean(kern_s))
        roofline = roofline_object(rf, graph, inst, args.workload, flops, kavg, peak_tf, peaks, peak_kind, cfg["mak"],
                                   rate_one_key, n1)
        cpu = None
        if not args.no_cpu_baseline:
            r = time_oracle(graph, inst, cfg)
            cpu = dict({"value": r["inst_per_s"], "unit": "instances/s", "cores": 1, "kind": "oracle",
                        "sample": f"first {r['instances']} of {inst.n} instances, one epoch, {r['seconds']:.1f} s",
                        "node_messages_per_s": r["msgs_per_s"], "arithmetic": "f64 build of the oracle, single thread"},
                       **host_description())
        line = {"metric": "training_instances_per_s", "value": value, "unit": "instances/s", "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tmax / args.steps,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "node_messages_per_s": msg_rate,
                "config": dict(workload_config(args.workload, inst, cfg, "asynchronous (free-running persistent kernel)"),
                               parallelism="replicas, no collective" if world == 1 or not averaging["on"] else
                               "replicas, parameters averaged at the end of every epoch (NCCL all-reduce)",
                               replica_sync=averaging["note"]),
                "roofline": roofline, "cpu_baseline": cpu,
                "e2e": {"value": e2e_value, "unit": "instances/s", "h2d_bytes_per_step": input_bytes(inst),
                        "d2h_bytes_per_step": int(inst.n * 4 + 512), "steps": e2e_steps},
                "clocks": clocks, "gpu_launches": args.steps,
                "step_ms": {"all": [round(1e3 * v, 3) for v in step_s], "best": 1e3 * min(step_s), "median": 1e3 * float(np.median(step_s)),
                            "note": "this rank's steps (CUDA events around launch + averaging)"},
                "stats": {"mean_loss_last_step": last.mean_loss, "max_staleness": int(last.max_staleness),
                          "rows_per_micro_batch": last.micro_batch_rows / max(1, last.micro_batches),
                          "placement": placement, "inference_instances_per_s": inference_rate,
                          "queue_occupancy_max_pending_fwd_bwd": queue_occ,
                          "micro_batch_split": split}}
        if sweep is not None:
            line["sweep"] = sweep
        if others is not None:
            for o in others.values():
                o["frac_of_fma_peak"] = o["tflops"] / fma_measured
            line["other_configs"] = others
        print(json.dumps(line), flush=True)
    if eng is not None:
        eng.close()
    import torch.distributed as dist
    if dist.is_initialized():
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="tree", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--instances", type=int, default=None, help="instances per step (default: the workload's size)")
    ap.add_argument("--timeout", type=float, default=300.0, help="bound on one device run, seconds")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true", help="skip the brief runs of the other configurations")
    ap.add_argument("--sweep", action="store_true", help="also run the max_active_keys x min_update_frequency grid")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
