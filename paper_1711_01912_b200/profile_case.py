"""Time one configuration of the evaluation with chosen kernel shape (also the driver used for ncu captures).

    python -m paper_1711_01912_b200.profile_case --config 3 [--P 2368] [--variant auto|sliced|level]
                                                 [--cpt 0|1|2|4|8] [--warps 0..32] [--reps 5]

Builds the seeded workload (optionally with fewer candidates), evaluates all outputs and prints the device time
of the phases (loads/validation, forward pass, backward pass) from the library's own CUDA events, the kernel
family that ran and the forward pass' byte rates.  --cpt / --warps set the tuning overrides
TFPS_SLICED_CPT / TFPS_SLICED_WARPS (0 = the library's choice).
"""
from __future__ import annotations

import argparse
import os

import numpy as np


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=3, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--P", type=int, default=0, help="number of candidates (default: the config's)")
    ap.add_argument("--variant", default="auto", choices=["auto", "sliced", "level"])
    ap.add_argument("--cpt", type=int, default=0)
    ap.add_argument("--warps", type=int, default=0)
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--layers", type=int, default=0, help="config 5 only: fewer layers of the same width (smaller capture)")
    args = ap.parse_args()

    import torch
    from . import inputs, tfps

    os.environ["TFPS_SLICED_CPT"] = str(args.cpt)
    os.environ["TFPS_SLICED_WARPS"] = str(args.warps)
    w = inputs.config5(layers=args.layers) if (args.config == 5 and args.layers) else inputs.make_config(args.config)
    if args.P:
        w.P = args.P
    n, m, P = w.graph.n, w.graph.m, w.P
    ldp = tfps.round_up_ldp(P)
    g = tfps.graph_from_workload(w)
    host = np.zeros((n, ldp), np.uint8)
    for r0, blk in w.part_blocks():
        host[r0:r0 + blk.shape[0], :P] = blk
    part = torch.from_numpy(host).cuda()
    out = {}
    flags = {"auto": tfps.EVAL_AUTO, "sliced": tfps.EVAL_SLICED, "level": tfps.EVAL_LEVEL_SYNC}[args.variant]
    for _ in range(2):
        g.eval_batch(part, P, flags=flags, out=out, check=False)
    g.status()
    ph = np.zeros(3)
    for _ in range(args.reps):
        g.eval_batch(part, P, flags=flags | tfps.EVAL_PROFILE, out=out, check=False)
        ph += np.array(tfps.tfps_phase_times(g.handle))
    ph /= args.reps
    print(f"{w.name} n={n} m={m} P={P} variant={args.variant} cpt={args.cpt} warps={args.warps} "
          f"kernel={tfps.tfps_last_pass_kernel(g.handle)}: loads {ph[0]:.3f} ms, forward {ph[1]:.3f} ms, "
          f"backward {ph[2]:.3f} ms | forward compulsory {9 * n * P / ph[1] / 1e6:.0f} GB/s, "
          f"logical {9 * (n + m) * P / ph[1] / 1e6:.0f} GB/s", flush=True)
    g.close()


if __name__ == "__main__":
    main()
