"""Where the time of one instance goes when a single key is in flight: `python -m paper_1705_09786_b200.hop_latency`.

With max_active_keys = 1 nothing overlaps, so the latency of an instance is the sum of its hops and the kernel's own cycle
counters (ampnet_get_phase_cycles: the first forward and the first backward tile of every parameterised node) split it
into the time those tiles worked and the time they waited for the next message.  What is left after the work of all
nodes is the hand-over between tiles: arrival counters, ticket, entry store, the consumer's poll.  The asynchronous mode
of the MLP, list and tree workloads (the direct-delivery engine) is measured; sizes are kept small (seconds).
"""
import argparse

import numpy as np

from workloads import data, ir, params as wp

from . import Engine

CASES = {"mlp": (lambda: ir.mlp((784, 256, 256, 10)), lambda n: data.mlp_instances(n=n), 2048, 32),
         "rnn": (ir.rnn, lambda n: data.list_instances(n=n), 3000, 50),
         "tree": (ir.tree, lambda n: data.tree_instances(n=n), 600, 100)}
F_PHASES = ("front", "rest", "update", "arrive", "product", "epilogue/loss", "loss-head dx")       # phase marks 1..7 of a forward tile
B_PHASES = ("front", "dpre", "dx", "accumulate", "update", "arrive")                                # marks 9..14 of a backward tile


def measure(family, sm_mhz):
    build, make, n, muf = CASES[family]
    g, inst = build(), make(n)
    e = Engine(g)
    e.load_instances(inst)
    e.set_params(wp.init_params(g))
    for _ in range(3):
        st, _ = e.run_epoch(mak=1, muf=muf, lr=0.01, deterministic=False, timeout_s=60)
    per_inst = st.seconds * 1e6 / inst.n
    lines = [f"{family}: {per_inst:.1f} us per instance with one key in flight ({inst.n / st.seconds:.0f} instances/s), "
             f"{st.node_messages / inst.n:.1f} node messages per instance"]
    busy_total = 0.0
    for node in g.ppt_nodes():
        a, _ = e.phase_cycles(node)
        us = a.astype(np.float64) / sm_mhz / inst.n                    # microseconds per instance
        f_busy, b_busy = us[1:8].sum() + us[15], us[9:15].sum()
        busy_total += f_busy + b_busy
        f = ", ".join(f"{k} {v:.2f}" for k, v in zip(F_PHASES, us[1:8]) if v >= 0.005)
        b = ", ".join(f"{k} {v:.2f}" for k, v in zip(B_PHASES, us[9:15]) if v >= 0.005)
        lines.append(f"  {g.names[node]:<12} forward tile works {f_busy:6.2f} us per instance ({f})" +
                     (f"; backward tile {b_busy:6.2f} us ({b})" if b_busy > 0 else ""))
    lines.append(f"  tiles at work {busy_total:.1f} us, hand-overs and the controller {per_inst - busy_total:.1f} us per instance")
    e.close()
    return lines


def main():
    ap = argparse.ArgumentParser(description=__doc__)
    ap.add_argument("--families", default="mlp,rnn,tree")
    ap.add_argument("--sm-mhz", type=float, default=None, help="SM clock the cycle counters ran at (default: the device's maximum)")
    args = ap.parse_args()
    import torch
    mhz = args.sm_mhz or getattr(torch.cuda.get_device_properties(0), "clock_rate", 1965000) / 1e3
    for fam in args.families.split(","):
        print("\n".join(measure(fam, mhz)))


if __name__ == "__main__":
    main()
