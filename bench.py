#!/usr/bin/env python
"""Benchmark of the batched critical-path evaluation path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 5] [--impl reference]

One step = one full evaluation (per-device loads and violation flags, forward
pass, backward pass, critical-path lengths) of ALL candidate partitions of the
synthetic workload.  The default workload is the largest configuration (config
5: 1,048,576 vertices, 8,192 candidates); its level matrices are int64
[n][P], so a step evaluates the candidates in chunks of 4,096 columns and reuses
one pair of level matrices.  Configs 3 and 4 are timed in the same run and
reported as sub-records under "per_config".  Prints one JSON line (rank 0).

With --gpus N > 1 and no torchrun environment the script starts N ranks itself.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "candidate_partitions_evaluated_per_s"
UNIT = "candidates/s"
CHUNK = 4096   # candidates whose level matrices are resident at a time (config 5)


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def captured_traffic(kernel: str, workload: str):
    """DRAM bytes per vertex-candidate of a pass kernel from the ncu capture summarised under profiles/ (None when
    there is no capture of this kernel on this workload: the figure is a property of that kernel and graph)."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.json")) as f:
            for rec in json.load(f)["captures"]:
                if rec["kernel"] == kernel and rec["workload"] == workload:
                    return rec
    except Exception:
        pass
    return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        inside = [l for (t, l) in self.lines if t0 <= t <= t1 + 0.1] or [l for (_, l) in self.lines[-3:]]
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in inside:
            p = [x.strip() for x in l.split(",")]
            try:
                sm.append(float(p[0])); mx.append(float(p[1])); pw.append(float(p[2]))
                for nm, v in zip(names, p[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            except Exception:
                pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": float(np.median(pw)) if pw else None, "reasons": sorted(reasons), "samples": len(sm)}


def base_workload(cfg: int):
    """Configurations 1-5; 6 = the paper's own set-up (Section 5.1: 50 devices, speeds U[10,100], link rates U[10,60],
    costs U[1,100]) on the largest of its Table 1 graph shapes, with 4,096 random candidates."""
    from paper_1711_01912_b200 import inputs
    return inputs.paper_shaped(2, P=4096) if cfg == 6 else inputs.make_config(cfg)


def make_workload(cfg: int, rank: int):
    """The seeded workload of a configuration; other ranks draw other candidate partitions of the same graph (weak
    scaling: rank r owns slice r of a global batch of world x P candidates)."""
    w = base_workload(cfg)
    if rank:
        w.seed = w.seed + 1000 * rank
    return w


# ---------------------------------------------------------------------------------------------------------------
# CPU oracle legs (cpu_baseline and --impl reference): the oracle as it stands, fanned out over host processes
# ---------------------------------------------------------------------------------------------------------------
_ORACLE = {}


def _oracle_init(cfg: int):
    import oracle
    from paper_1711_01912_b200 import inputs
    w = base_workload(cfg)
    c = inputs.to_csr(w.graph)
    _ORACLE["w"] = w
    _ORACLE["og"] = oracle.OracleGraph(w.graph.n, c.in_ptr, c.in_src, c.in_t, c.out_ptr, c.out_dst, c.out_t, w.graph.c, w.graph.mem)


def _oracle_eval(part_cols: np.ndarray) -> float:
    import oracle
    w, og = _ORACLE["w"], _ORACLE["og"]
    d = w.devices
    t0 = time.perf_counter()
    oracle.eval_batch(og, d.k, d.s, d.C, d.B, d.scale, np.ascontiguousarray(part_cols), want_levels=True)
    return time.perf_counter() - t0


class OraclePool:
    """One spawned process per host core, each holding the oracle's copy of the graph."""

    def __init__(self, cfg: int, cores: int):
        import multiprocessing as mp
        self.cores = cores
        self.pool = mp.get_context("spawn").Pool(cores, initializer=_oracle_init, initargs=(cfg,))
        self.pool.map(_noop, range(cores))   # wait until every worker has built its graph

    def time_columns(self, part_cols: np.ndarray) -> float:
        """Wall seconds for the given candidate columns, one slice per process."""
        pieces = [p for p in np.array_split(part_cols, self.cores, axis=1) if p.shape[1] > 0]
        t0 = time.perf_counter()
        self.pool.map(_oracle_eval, pieces)
        return time.perf_counter() - t0

    def close(self):
        self.pool.close()
        self.pool.join()


def _noop(_):
    return 0


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def oracle_baseline(cfg: int, part_host: np.ndarray, P: int, budget_s: float):
    """cpu_baseline record: single-thread rate on a few columns, then the all-cores rate on a sample sized for about
    `budget_s` seconds of wall time."""
    cores = host_cores()
    _oracle_init(cfg)
    probe = np.ascontiguousarray(part_host[:, :4])
    per = _oracle_eval(probe) / 4
    pool = OraclePool(cfg, cores)
    try:
        # the processes share the memory system: size the sample from the rate of a short parallel run
        trial = np.ascontiguousarray(part_host[:, :2 * cores])
        rate = trial.shape[1] / pool.time_columns(trial)
        count = int(max(cores, min(P, budget_s * rate)))
        cols = (np.arange(count, dtype=np.int64) * max(1, P // count)) % P
        sample = np.ascontiguousarray(part_host[:, cols])
        dt = pool.time_columns(sample)
    finally:
        pool.close()
    name = _ORACLE["w"].name
    return {"value": count / dt, "unit": UNIT, "cores": cores, "host_cores": cores, "kind": "oracle",
            "single_thread_value": 1.0 / per,
            "sample": f"{count} of {P} candidates of {name}, all outputs, one process per core ({cores}), {dt:.1f} s; "
                      f"single thread: {per:.3f} s per candidate"}, cols


def run_reference(args):
    """The CPU oracle as the reference arm: each step evaluates a bounded sample of the workload's candidates."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = make_workload(args.config, 0)
    cores = host_cores()
    _oracle_init(args.config)
    probe = w.part_columns(np.arange(4))
    per = _oracle_eval(probe) / 4
    budget = 60.0 / max(1, args.steps + args.warmup)   # wall seconds per step
    pool = OraclePool(args.config, cores)
    try:
        trial = w.part_columns(np.arange(2 * cores))
        rate = trial.shape[1] / pool.time_columns(trial)
        count = int(max(cores, min(w.P, budget * rate)))
        cols = (np.arange(count, dtype=np.int64) * max(1, w.P // count)) % w.P
        sample = w.part_columns(cols)
        for _ in range(args.warmup):
            pool.time_columns(sample)
        t0 = time.perf_counter()
        for _ in range(args.steps):
            pool.time_columns(sample)
        dt = (time.perf_counter() - t0) / args.steps
    finally:
        pool.close()
    value = count / dt
    desc = f"{count} of {w.P} candidates per step, all outputs, one process per core ({cores})"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": w.name, "n": w.graph.n, "m": w.graph.m, "k": w.devices.k, "P": w.P, "sample": desc},
        "edge_relaxations_per_s": value * 2 * w.graph.m,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "host_cores": cores, "kind": "oracle",
                         "single_thread_value": 1.0 / per, "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------------------------------
def inputs_sha256(w, host_np: np.ndarray) -> str:
    h = hashlib.sha256()
    g, d = w.graph, w.devices
    for arr in (g.src, g.dst, g.t, g.c, g.mem, d.s, d.C, d.B):
        if arr is not None:
            h.update(np.ascontiguousarray(arr).tobytes())
    h.update(memoryview(host_np).cast("B"))
    return h.hexdigest()


def measure_config(cfg: int, args, rank: int, world: int, local: int, steps: int, min_seconds: float, headline: bool):
    """Times one configuration: device-resident steps, per-phase times, the end-to-end (host buffers) path and, on
    request, the CPU oracle.  Returns the record for the JSON line."""
    import torch
    import torch.distributed as dist
    from paper_1711_01912_b200 import tfps

    w = make_workload(cfg, rank)
    n, m, k, P = w.graph.n, w.graph.m, w.devices.k, w.P
    chunk = min(P, CHUNK) if cfg == 5 else P
    nchunks = (P + chunk - 1) // chunk
    ldp = tfps.round_up_ldp(P)          # host matrix [n][ldp]
    ldc = tfps.round_up_ldp(chunk)      # resident chunk matrices [n][ldc]
    t_setup = time.perf_counter()
    g = tfps.graph_from_workload(w)
    level, order, lp, L = g.topo_levels()
    setup_s = time.perf_counter() - t_setup
    del level, order

    host_part = torch.empty((n, ldp), dtype=torch.uint8).pin_memory()
    host_np = host_part.numpy()
    host_np[:, P:] = 0
    for r0, blk in w.part_blocks():
        host_np[r0:r0 + blk.shape[0], :P] = blk
    sha = inputs_sha256(w, host_np) if rank == 0 else None
    parts, widths = [], []
    for c in range(nchunks):
        wd = min(chunk, P - c * chunk)
        t = torch.zeros((n, ldc), dtype=torch.uint8, device="cuda")
        t[:, :wd] = host_part[:, c * chunk:c * chunk + wd].cuda(non_blocking=True)
        parts.append(t)
        widths.append(wd)
    flags = {"auto": tfps.EVAL_AUTO, "sliced": tfps.EVAL_SLICED, "level_sync": tfps.EVAL_LEVEL_SYNC}[args.variant]
    want = ("tlevel", "blevel", "cp", "load", "memload", "viol")
    # one pair of level matrices for all chunks, summaries per chunk
    tl = torch.empty((n, ldc), dtype=torch.int64, device="cuda")
    bl = torch.empty((n, ldc), dtype=torch.int64, device="cuda")
    outs = []
    for c in range(nchunks):
        outs.append({"tlevel": tl, "blevel": bl,
                     "cp": torch.empty(max(widths[c], 1), dtype=torch.int64, device="cuda"),
                     "load": torch.empty((k, ldc), dtype=torch.int64, device="cuda"),
                     "memload": torch.empty((k, ldc), dtype=torch.int64, device="cuda"),
                     "viol": torch.empty(max(widths[c], 1), dtype=torch.int64, device="cuda")})

    def step(profile=False):
        ph = np.zeros(3)
        for c in range(nchunks):
            g.eval_batch(parts[c], widths[c], want=want, flags=flags | (tfps.EVAL_PROFILE if profile else 0), out=outs[c], check=False)
            if profile:
                ph += np.array(tfps.tfps_phase_times(g.handle))
        return ph

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        if world > 1:
            t = torch.tensor([x], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            return float(t.item())
        return x

    warmup = max(3, args.warmup)
    for _ in range(warmup):
        step()
    g.status()
    barrier()
    if not headline:
        # sub-records choose their own step count: a timed region of at least `min_seconds`
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); step(); e1.record(); torch.cuda.synchronize()
        steps = int(min(5000, max(steps, math.ceil(min_seconds * 1e3 / max(e0.elapsed_time(e1), 1e-3)))))
    sampler = ClockSampler(local).start()
    time.sleep(0.25)
    launches0 = tfps.tfps_kernel_launches()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    wall0 = time.time()
    ev0.record()
    for _ in range(steps):
        step()
    ev1.record()
    barrier()
    wall1 = time.time()
    launches = tfps.tfps_kernel_launches() - launches0
    clocks = sampler.stop(wall0, wall1)
    g.status()
    ms = max_over_ranks(ev0.elapsed_time(ev1) / steps)

    # per-phase device time (forward pass = dominant kernel): CUDA events recorded by the library on the launching stream
    phase = np.zeros(3)
    reps = max(3, min(steps, 10))
    for _ in range(reps):
        phase += step(profile=True)
    phase /= reps   # per step, summed over the step's chunks
    loads_ms, fwd_ms, bwd_ms = float(phase[0]), float(phase[1]), float(phase[2])
    kernel_name = tfps.tfps_last_pass_kernel(g.handle)
    cp_dev = torch.cat([outs[c]["cp"][:widths[c]] for c in range(nchunks)]).cpu()

    rec = {}
    spot = None
    if args.cpu_baseline and world == 1 and (headline or args.cpu_baseline_all):
        cpu, cols = oracle_baseline(cfg, host_np, P, 15.0 if headline else 6.0)
        rec["cpu_baseline"] = cpu
        # the first sampled columns double as a parity check of the timed configuration (levels of the last chunk
        # are still resident; cp of every chunk is)
        import oracle
        d = w.devices
        sel = cols[:4]
        ref = oracle.eval_batch(_ORACLE["og"], d.k, d.s, d.C, d.B, d.scale, np.ascontiguousarray(host_np[:, sel]), want_levels=True)
        assert np.array_equal(cp_dev.numpy()[sel], ref.cp), "cp differs from the oracle"
        last0 = (nchunks - 1) * chunk
        lastsel = np.array([last0, P - 1])
        ref2 = oracle.eval_batch(_ORACLE["og"], d.k, d.s, d.C, d.B, d.scale, np.ascontiguousarray(host_np[:, lastsel]), want_levels=True)
        tsel = torch.from_numpy(lastsel - last0).cuda()
        assert np.array_equal(tl[:, tsel].cpu().numpy(), ref2.tlevel)
        assert np.array_equal(bl[:, tsel].cpu().numpy(), ref2.blevel)
        spot = "cp of 4 sampled candidates and tlevel, blevel of 2 candidates of the last chunk bit-exact against the oracle"

    # end to end through the host-buffer entry point: ids H2D from pinned memory, summaries D2H.  The resident
    # matrices go first: the entry point keeps its own staging buffers and level scratch.
    del tl, bl, outs, parts
    torch.cuda.empty_cache()
    res_cp = torch.empty(P, dtype=torch.int64).pin_memory()
    res_ld = torch.empty((k, ldp), dtype=torch.int64).pin_memory()
    res_ml = torch.empty((k, ldp), dtype=torch.int64).pin_memory()
    res_vi = torch.empty(P, dtype=torch.int64).pin_memory()
    stream = torch.cuda.current_stream().cuda_stream

    def e2e_step():
        tfps.tfps_eval_batch_host(g.handle, P, ldp, host_part.data_ptr(), None, None, res_cp.data_ptr(),
                                  res_ld.data_ptr(), res_ml.data_ptr(), res_vi.data_ptr(), flags, stream)

    e2e_steps = max(2, min(steps, 5))
    for _ in range(2):
        e2e_step()
    barrier()
    ev0.record()
    for _ in range(e2e_steps):
        e2e_step()
    ev1.record()
    barrier()
    e2e_ms = max_over_ranks(ev0.elapsed_time(ev1) / e2e_steps)
    assert torch.equal(res_cp, cp_dev), "end-to-end and device-resident runs disagree"
    g.close()
    del g
    torch.cuda.empty_cache()

    peak, peak_kind = measured_peak_gbs()
    # dominant kernel = the forward pass; one step launches it once per chunk.  Compulsory bytes per launch: one id
    # read and one level write per vertex-candidate; logical bytes add one neighbour level and one neighbour id per
    # relaxation (served by shared memory or L2 when resident)
    launches_fwd = nchunks
    fwd_launch_ms = fwd_ms / launches_fwd
    compulsory = 9.0 * n * (P / nchunks)
    logical = 9.0 * (n + m) * (P / nchunks)
    achieved = compulsory / (fwd_launch_ms * 1e-3) / 1e9
    cap = captured_traffic(kernel_name, w.name)
    step_bytes = (2 * 9.0 + 1.0) * n * P   # both passes and the id re-read of the loads kernel
    mhz = clocks.get("sm_mhz") or 0.0
    rec.update({
        "workload": w.name, "ms_per_step": ms, "steps": steps, "value": world * P / (ms * 1e-3),
        "edge_relaxations_per_s": world * 2.0 * m * P / (ms * 1e-3),
        "ms_x_sm_mhz": ms * mhz,
        "phase_ms": {"loads_validate_viol": loads_ms, "forward": fwd_ms, "backward": bwd_ms,
                     "note": "per step (all chunks), CUDA events on the pass stream" +
                             ("; the loads kernel runs beside the lean passes on its own stream and the backward figure "
                              "includes the wait for it" if kernel_name.startswith("pass_lean") else "")},
        "roofline": {"bound": "hbm", "kernel": kernel_name + "<forward>",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}", "bytes_per_launch": compulsory, "launches_per_step": launches_fwd,
                     "launch_ms": fwd_launch_ms,
                     "traffic": (cap["bytes_per_vertex_candidate"] * n * (P / nchunks)) if cap else None,
                     "traffic_source": (cap["source"] if cap else None),
                     "achieved_logical": logical / (fwd_launch_ms * 1e-3) / 1e9,
                     "frac_whole_step": step_bytes / (ms * 1e-3) / 1e9 / peak,
                     "note": "achieved = compulsory bytes 9*n*P_launch (1 B id read + 8 B level write per vertex-candidate) / "
                             "forward launch time; achieved_logical adds 9 B per relaxation for neighbour reads (shared "
                             "memory or L2, not DRAM); frac_whole_step = 19*n*P bytes of both passes and the loads kernel / "
                             "step time / peak"},
        "e2e": {"value": world * P / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": n * ldp, "d2h_bytes_per_step": 8 * (2 * P + 2 * k * ldp),
                "api": "tfps_eval_batch_host (pinned host ids in; cp, load, memload, viol out; level matrices stay on the device)"},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "config": {"workload": w.name, "n": n, "m": m, "levels": L, "k": k, "P": P, "chunk": chunk, "chunks_per_step": nchunks,
                   "ldp": ldp, "scale": w.devices.scale, "variant": args.variant, "outputs": list(want),
                   "l2": f"inputs+outputs per step {(n * ldp * 17) / 1e9:.1f} GB >> 126 MB L2, no explicit flush",
                   "setup_ms_graph_levels_tables": setup_s * 1e3, "inputs_sha256": sha,
                   "candidates": "rank r owns slice r of a global batch of n_gpus x P candidates (no data-path collective)"},
    })
    if spot:
        rec["parity_spot_check"] = spot
    return rec


def run_gpu(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    head = measure_config(args.config, args, rank, world, local, args.steps, 0.0, True)
    subs = {}
    if args.config == 5 and not args.no_sub_configs:
        for cfg in (3, 4):
            r = measure_config(cfg, args, rank, world, local, 3, 2.0, False)
            subs[f"cfg{cfg}"] = {key: r[key] for key in ("workload", "ms_per_step", "steps", "value", "edge_relaxations_per_s",
                                                         "ms_x_sm_mhz", "phase_ms", "roofline", "e2e", "clocks", "config")
                                 if key in r}
            if "cpu_baseline" in r:
                subs[f"cfg{cfg}"]["cpu_baseline"] = r["cpu_baseline"]
    if rank == 0:
        line = {
            "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int64", "data": "synthetic", "config": head["config"],
            "edge_relaxations_per_s": head["edge_relaxations_per_s"], "ms_x_sm_mhz": head["ms_x_sm_mhz"],
            "phase_ms": head["phase_ms"], "roofline": head["roofline"], "e2e": head["e2e"],
            "gpu_launches": head["gpu_launches"], "clocks": head["clocks"], "host_cores": host_cores(),
        }
        for key in ("cpu_baseline", "parity_spot_check"):
            if key in head:
                line[key] = head[key]
        if subs:
            line["per_config"] = subs
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def spawn_ranks(args) -> int:
    """--gpus N without a torchrun environment: start N ranks of this script (one process per GPU)."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=5, choices=[1, 2, 3, 4, 5, 6], help="1-5: the configurations; 6: the paper's own set-up (50 devices) on its largest graph shape")
    ap.add_argument("--impl", default="tfps", choices=["tfps", "reference"])
    ap.add_argument("--variant", default="auto", choices=["auto", "sliced", "level_sync"])
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--cpu-baseline-all", action="store_true", help="time the oracle on the sub-record configurations too")
    ap.add_argument("--no-sub-configs", action="store_true", help="config 5 only: skip the sub-records of configs 3 and 4")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
