"""Time the rank-driven partitioners and the batched list-scheduling simulation on one configuration.

    python -m paper_1711_01912_b200.sim_case --config 6 [--P 4096] [--reps 3]

Prints the device time (CUDA events) of tfps_ranks, tfps_critical_path + tfps_cp_partition, tfps_batch_split and of
tfps_simulate under both policies (candidates simulated per second), and the makespans of the two generated
partitions under the PCT policy next to the mean over the configuration's random candidates.
"""
from __future__ import annotations

import argparse

import numpy as np


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=6, choices=[1, 2, 3, 4, 6])
    ap.add_argument("--P", type=int, default=0)
    ap.add_argument("--reps", type=int, default=3)
    args = ap.parse_args()

    import torch
    from . import inputs, tfps

    w = inputs.paper_shaped(2, P=args.P or 4096) if args.config == 6 else inputs.make_config(args.config)
    if args.P:
        w.P = args.P
    n, P = w.graph.n, w.P
    ldp = tfps.round_up_ldp(P)
    G = tfps.graph_from_workload(w)
    host = np.zeros((n, ldp), np.uint8)
    for r0, blk in w.part_blocks():
        host[r0:r0 + blk.shape[0], :P] = blk[:, :P]
    part = torch.from_numpy(host).cuda()

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.reps):
            out = fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.reps, out

    ms_rank, (up, down, total) = timed(G.ranks)
    ms_cp, (cp_part, cp_bad) = timed(lambda: G.cp_partition(G.critical_path(down)))
    ms_bs, (bs_part, bs_bad) = timed(lambda: G.batch_split(total))
    print(f"{w.name} n={n} m={w.graph.m} k={w.devices.k} P={P}: ranks {ms_rank:.3f} ms, critical path + CP partition "
          f"{ms_cp:.3f} ms ({cp_bad} unplaced), Batch Split {ms_bs:.3f} ms ({bs_bad} unplaced)", flush=True)
    out = G.eval_batch(part, P)
    for name, policy in (("FIFO", tfps.SCHED_FIFO), ("PCT", tfps.SCHED_PCT), ("MSR", tfps.SCHED_MSR)):
        prio = out["blevel"] if policy == tfps.SCHED_PCT else None
        ms, (_, mk) = timed(lambda: G.simulate(part, P, policy, prio, want_start=False))
        G.status()
        print(f"  simulate {name}: {ms:.2f} ms for {P} candidates = {P / ms * 1e3:,.0f} candidates/s; makespan of the random "
              f"candidates: mean {mk.double().mean().item():,.0f}, best {mk.min().item():,} (critical path mean "
              f"{out['cp'][:P].double().mean().item():,.0f})", flush=True)
    # the two generated partitions, evaluated and simulated like any candidate
    two = torch.zeros((n, 16), dtype=torch.uint8, device="cuda")
    two[:, 0] = cp_part
    two[:, 1] = bs_part
    o2 = G.eval_batch(two, 2)
    for name, policy in (("FIFO", tfps.SCHED_FIFO), ("PCT", tfps.SCHED_PCT), ("MSR", tfps.SCHED_MSR)):
        _, mk = G.simulate(two, 2, policy, o2["blevel"] if policy == tfps.SCHED_PCT else None, want_start=False)
        G.status()
        print(f"  {name}: makespan of the Critical Path partition {int(mk[0]):,} (CP {int(o2['cp'][0]):,}), of the Batch Split "
              f"partition {int(mk[1]):,} (CP {int(o2['cp'][1]):,})", flush=True)
    G.close()


if __name__ == "__main__":
    main()
