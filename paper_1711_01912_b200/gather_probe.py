"""Prints the rate at which the current GPU gathers 1 KiB row segments, for several working-set sizes.

    python -m paper_1711_01912_b200.gather_probe [--mb 8 32 64 128 512]

This is the access pattern of the step-synchronous record passes (a neighbour's levels and ids for one tile of
candidates) without their arithmetic: the ceiling of those passes in bytes gathered per second.
"""
from __future__ import annotations

import argparse


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--mb", type=int, nargs="+", default=[8, 32, 64, 128, 512], help="working-set sizes in MiB")
    ap.add_argument("--rows-per-warp", type=int, default=4096)
    ap.add_argument("--window-mb", type=int, nargs="+", default=[16, 84], help="wavefront probe: window sizes in MiB")
    args = ap.parse_args()
    import torch
    from . import tfps
    torch.cuda.set_device(0)
    for mb in args.mb:
        gbs = tfps.tfps_probe_gather_bandwidth(mb << 20, args.rows_per_warp)
        print(f"working set {mb:5d} MiB: {gbs:8.0f} GB/s gathered", flush=True)
    # the wavefront of a pass: 4 GiB written once, every row after reading rows among the last `window` MiB
    for layout in (0, 1):
        for window in args.window_mb:
            for reads in (0, 1, 2, 3):
                gbs = tfps.tfps_probe_wavefront_bandwidth(4 << 30, window << 20, reads, layout)
                print(f"wavefront, layout {layout}, window {window:4d} MiB, {reads} rows read per row written: {gbs:8.0f} GB/s "
                      f"(read + written)", flush=True)


if __name__ == "__main__":
    main()
