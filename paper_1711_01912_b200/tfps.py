"""ctypes binding of libtfps.so (argument marshalling only).

Module-level ``tfps_*`` functions mirror the C ABI of ``include/tfps.h`` one to
one and take raw addresses/ints.  ``Graph`` wraps them for callers that hold
numpy arrays (host) and torch CUDA tensors (device memory and streams only --
every step of the evaluation runs in the library's kernels).

There is no CPU fallback: if the shared library is missing or cannot be loaded
an ImportError is raised at first use.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtfps.so")

OK = 0
ERR_INVALID_ARG, ERR_BAD_CSR, ERR_CYCLE, ERR_BAD_DEVICES, ERR_BAD_PARTITION = -1, -2, -3, -4, -5
ERR_OVERFLOW, ERR_WORKSPACE, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT, ERR_STATE = -6, -7, -8, -9, -10, -11
K_MAX = 64
I32, I64 = 0, 1
HOST, DEVICE = 0, 1
EVAL_AUTO, EVAL_LEVEL_SYNC, EVAL_SLICED, EVAL_NO_VALIDATE, EVAL_SCRATCH_LEVELS, EVAL_PROFILE = 0, 1, 2, 16, 32, 64

EXPORTS = [
    "tfps_strerror", "tfps_last_error", "tfps_graph_create", "tfps_graph_destroy", "tfps_graph_info",
    "tfps_devices_set", "tfps_topo_levels", "tfps_eval_workspace_bytes", "tfps_eval_batch",
    "tfps_eval_batch_host", "tfps_get_status", "tfps_transpose_u8", "tfps_phase_times", "tfps_kernel_launches",
    "tfps_eval_cp_noalloc", "tfps_last_pass_kernel", "tfps_probe_gather_bandwidth", "tfps_constraints_set", "tfps_eval_constraints", "tfps_critical_mask",
    "tfps_ranks", "tfps_critical_path", "tfps_batch_split", "tfps_cp_partition", "tfps_simulate", "tfps_msr_weights_set", "tfps_probe_wavefront_bandwidth",
]


class TfpsError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"tfps error {code}: {message}")
        self.code = code


_lib = None


def lib() -> ctypes.CDLL:
    """Load libtfps.so (built by ``paper_1711_01912_b200.build``); never falls back to anything else."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_1711_01912_b200.build` "
                          "(or __graft_entry__.build()); there is no CPU fallback")
    L = ctypes.CDLL(LIB_PATH)
    vp, i64, i32, ci, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int, ctypes.c_size_t
    L.tfps_strerror.restype = ctypes.c_char_p
    L.tfps_strerror.argtypes = [ci]
    L.tfps_last_error.restype = ctypes.c_char_p
    L.tfps_last_error.argtypes = []
    L.tfps_graph_create.restype = ci
    L.tfps_graph_create.argtypes = [ctypes.POINTER(vp), i64, i64, vp, vp, vp, vp, vp, vp, ci, vp, vp, ci, ci, vp]
    L.tfps_graph_destroy.restype = ci
    L.tfps_graph_destroy.argtypes = [vp]
    L.tfps_graph_info.restype = ci
    L.tfps_graph_info.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64), ctypes.POINTER(i32), ctypes.POINTER(i32)]
    L.tfps_devices_set.restype = ci
    L.tfps_devices_set.argtypes = [vp, ci, vp, vp, vp, i64]
    L.tfps_topo_levels.restype = ci
    L.tfps_topo_levels.argtypes = [vp, vp, vp, vp, i64, ctypes.POINTER(i32), vp]
    L.tfps_eval_workspace_bytes.restype = sz
    L.tfps_eval_workspace_bytes.argtypes = [vp, i64, i64, ci]
    L.tfps_eval_batch.restype = ci
    L.tfps_eval_batch.argtypes = [vp, i64, i64, vp, vp, vp, vp, vp, vp, vp, vp, sz, ci, vp]
    L.tfps_eval_batch_host.restype = ci
    L.tfps_eval_batch_host.argtypes = [vp, i64, i64, vp, vp, vp, vp, vp, vp, vp, ci, vp]
    L.tfps_phase_times.restype = ci
    L.tfps_phase_times.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    L.tfps_kernel_launches.restype = i64
    L.tfps_kernel_launches.argtypes = []
    L.tfps_constraints_set.restype = ci
    L.tfps_constraints_set.argtypes = [vp, i64, vp, vp, i64, vp, vp]
    L.tfps_eval_constraints.restype = ci
    L.tfps_eval_constraints.argtypes = [vp, i64, i64, vp, vp, vp, vp]
    L.tfps_critical_mask.restype = ci
    L.tfps_critical_mask.argtypes = [i64, i64, i64, vp, vp, vp, vp, vp]
    L.tfps_ranks.restype = ci
    L.tfps_ranks.argtypes = [vp, vp, vp, vp, vp]
    L.tfps_critical_path.restype = ci
    L.tfps_critical_path.argtypes = [vp, vp, vp, ctypes.POINTER(ctypes.c_int64), vp]
    L.tfps_batch_split.restype = ci
    L.tfps_batch_split.argtypes = [vp, vp, vp, ctypes.POINTER(ctypes.c_int64), vp]
    L.tfps_cp_partition.restype = ci
    L.tfps_cp_partition.argtypes = [vp, vp, i64, vp, ctypes.POINTER(ctypes.c_int64), vp]
    L.tfps_msr_weights_set.restype = ci
    L.tfps_msr_weights_set.argtypes = [vp, i64, i64, i64, i64]
    L.tfps_simulate.restype = ci
    L.tfps_simulate.argtypes = [vp, i64, i64, vp, ci, vp, vp, vp, vp]
    L.tfps_probe_wavefront_bandwidth.restype = ci
    L.tfps_probe_wavefront_bandwidth.argtypes = [sz, sz, ci, ci, ctypes.POINTER(ctypes.c_double)]
    L.tfps_probe_gather_bandwidth.restype = ci
    L.tfps_probe_gather_bandwidth.argtypes = [sz, ci, ctypes.POINTER(ctypes.c_double)]
    L.tfps_last_pass_kernel.restype = ctypes.c_char_p
    L.tfps_last_pass_kernel.argtypes = [vp]
    L.tfps_eval_cp_noalloc.restype = ci
    L.tfps_eval_cp_noalloc.argtypes = [vp, i64, i64, vp, vp, ci, vp]
    L.tfps_get_status.restype = ci
    L.tfps_get_status.argtypes = [vp, vp]
    L.tfps_transpose_u8.restype = ci
    L.tfps_transpose_u8.argtypes = [vp, vp, i64, i64, i64, vp]
    _lib = L
    return L


def _check(rc: int) -> None:
    if rc != OK:
        raise TfpsError(rc, lib().tfps_last_error().decode() or lib().tfps_strerror(rc).decode())


# ---- one-to-one wrappers (raw addresses in, status checked) ---------------------------------
def tfps_strerror(status: int) -> str:
    return lib().tfps_strerror(status).decode()


def tfps_last_error() -> str:
    return lib().tfps_last_error().decode()


def tfps_graph_create(n, m, in_ptr, in_src, in_t, out_ptr, out_dst, out_t, t_dtype, c, mem, mem_dtype, ptr_space,
                      stream=0) -> int:
    h = ctypes.c_void_p()
    _check(lib().tfps_graph_create(ctypes.byref(h), n, m, in_ptr, in_src, in_t, out_ptr, out_dst, out_t, t_dtype, c,
                                   mem, mem_dtype, ptr_space, stream))
    return h.value


def tfps_graph_destroy(g) -> None:
    _check(lib().tfps_graph_destroy(g))


def tfps_graph_info(g):
    n, m, L, k = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int32(), ctypes.c_int32()
    _check(lib().tfps_graph_info(g, ctypes.byref(n), ctypes.byref(m), ctypes.byref(L), ctypes.byref(k)))
    return n.value, m.value, L.value, k.value


def tfps_devices_set(g, k, s, C, B, scale) -> None:
    _check(lib().tfps_devices_set(g, k, s, C, B, scale))


def tfps_topo_levels(g, level, order, level_ptr, cap, stream=0) -> int:
    L = ctypes.c_int32()
    _check(lib().tfps_topo_levels(g, level, order, level_ptr, cap, ctypes.byref(L), stream))
    return L.value


def tfps_eval_workspace_bytes(g, P, ldp, flags) -> int:
    return int(lib().tfps_eval_workspace_bytes(g, P, ldp, flags))


def tfps_eval_batch(g, P, ldp, part, tlevel, blevel, cp, load, memload, viol, workspace, workspace_bytes, flags,
                    stream=0) -> None:
    _check(lib().tfps_eval_batch(g, P, ldp, part, tlevel, blevel, cp, load, memload, viol, workspace, workspace_bytes,
                                 flags, stream))


def tfps_eval_batch_host(g, P, ldp, part, tlevel, blevel, cp, load, memload, viol, flags, stream=0) -> None:
    _check(lib().tfps_eval_batch_host(g, P, ldp, part, tlevel, blevel, cp, load, memload, viol, flags, stream))


def tfps_phase_times(g):
    ms = (ctypes.c_float * 3)()
    _check(lib().tfps_phase_times(g, ms))
    return [float(x) for x in ms]


def tfps_last_pass_kernel(g) -> str:
    return lib().tfps_last_pass_kernel(g).decode()


def tfps_kernel_launches() -> int:
    return int(lib().tfps_kernel_launches())


def tfps_constraints_set(g, npairs, pair_a, pair_b, ndev, dc_vertex, dc_device) -> None:
    _check(lib().tfps_constraints_set(g, npairs, pair_a, pair_b, ndev, dc_vertex, dc_device))


def tfps_eval_constraints(g, P, ldp, part, coll_viol, dev_viol, stream) -> None:
    _check(lib().tfps_eval_constraints(g, P, ldp, part, coll_viol, dev_viol, stream))


def tfps_critical_mask(n, P, ldp, tlevel, blevel, cp, mask, stream) -> None:
    _check(lib().tfps_critical_mask(n, P, ldp, tlevel, blevel, cp, mask, stream))


def tfps_ranks(handle, up, down, total, stream) -> None:
    _check(lib().tfps_ranks(handle, up, down, total, stream))


def tfps_critical_path(handle, down, path, stream) -> int:
    ln = ctypes.c_int64(0)
    _check(lib().tfps_critical_path(handle, down, path, ctypes.byref(ln), stream))
    return int(ln.value)


def tfps_batch_split(handle, total, part, stream) -> int:
    bad = ctypes.c_int64(0)
    _check(lib().tfps_batch_split(handle, total, part, ctypes.byref(bad), stream))
    return int(bad.value)


def tfps_cp_partition(handle, path, length, part, stream) -> int:
    bad = ctypes.c_int64(0)
    _check(lib().tfps_cp_partition(handle, path, length, part, ctypes.byref(bad), stream))
    return int(bad.value)


SCHED_FIFO, SCHED_PCT, SCHED_MSR = 0, 1, 2


def tfps_msr_weights_set(handle, alpha, beta, gamma, delta) -> None:
    _check(lib().tfps_msr_weights_set(handle, alpha, beta, gamma, delta))


def tfps_simulate(handle, P, ldp, part, policy, prio, start, makespan, stream) -> None:
    _check(lib().tfps_simulate(handle, P, ldp, part, policy, prio, start, makespan, stream))


def tfps_probe_wavefront_bandwidth(total_bytes: int, window_bytes: int, reads: int, layout: int = 0) -> float:
    out = ctypes.c_double(0.0)
    _check(lib().tfps_probe_wavefront_bandwidth(total_bytes, window_bytes, reads, layout, ctypes.byref(out)))
    return out.value


def tfps_probe_gather_bandwidth(working_set_bytes: int, rows_per_warp: int = 4096) -> float:
    """GB/s at which the current device gathers pseudo-random 1 KiB row segments of a buffer of that size."""
    out = ctypes.c_double(0.0)
    _check(lib().tfps_probe_gather_bandwidth(int(working_set_bytes), int(rows_per_warp), ctypes.byref(out)))
    return float(out.value)


NOALLOC_SCRATCH_BYTES = 32 << 20


def tfps_eval_cp_noalloc(g, P, ldp, part, cp, flags=0, stream=0) -> None:
    """Critical-path lengths with the level scratch inside the library: no device allocation happens in this call."""
    _check(lib().tfps_eval_cp_noalloc(g, P, ldp, part, cp, flags, stream))


def tfps_get_status(g, stream=0) -> None:
    _check(lib().tfps_get_status(g, stream))


def tfps_transpose_u8(src, dst, P, n, ldp, stream=0) -> None:
    _check(lib().tfps_transpose_u8(src, dst, P, n, ldp, stream))


# ---- convenience layer ------------------------------------------------------------------------
def _np(a, dtype):
    return np.ascontiguousarray(np.asarray(a), dtype=dtype)


def _addr(a) -> Optional[int]:
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        return a.ctypes.data
    return a.data_ptr()  # torch tensor


def _stream() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


def round_up_ldp(P: int) -> int:
    return max(16, (P + 15) // 16 * 16)


class Graph:
    """Owns a tfps_graph handle built from host numpy CSR arrays (or, with ``device_arrays``, from copies of them
    placed in device memory first: the library then fetches them itself, ptr_space = TFPS_DEVICE)."""

    def __init__(self, n, in_ptr, in_src, in_t, c, out_ptr=None, out_dst=None, out_t=None, mem=None, device_arrays=False):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("tfps needs a CUDA device; there is no CPU fallback")
        in_t = np.asarray(in_t)
        t_np = np.int32 if in_t.dtype == np.int32 else np.int64
        self._keep = [_np(in_ptr, np.int64), _np(in_src, np.int32), _np(in_t, t_np), _np(c, np.int32)]
        outs = [None, None, None]
        if out_ptr is not None:
            outs = [_np(out_ptr, np.int64), _np(out_dst, np.int32), _np(out_t, t_np)]
        mem_a, mem_dt = None, I64
        if mem is not None:
            mem = np.asarray(mem)
            mem_dt = I32 if mem.dtype == np.int32 else I64
            mem_a = _np(mem, np.int32 if mem_dt == I32 else np.int64)
        self.n = int(n)
        self.m = int(self._keep[1].shape[0])
        space = HOST
        if device_arrays:
            def dev(a):
                return None if a is None else torch.from_numpy(a).cuda() if a.size else torch.zeros(1, dtype=torch.from_numpy(a).dtype, device="cuda")
            self._keep = [dev(a) for a in self._keep]
            outs = [dev(a) for a in outs]
            mem_a = dev(mem_a)
            torch.cuda.synchronize()
            space = DEVICE
        self.handle = tfps_graph_create(self.n, self.m, _addr(self._keep[0]), _addr(self._keep[1]),
                                        _addr(self._keep[2]), _addr(outs[0]), _addr(outs[1]), _addr(outs[2]),
                                        I32 if t_np == np.int32 else I64, _addr(self._keep[3]), _addr(mem_a), mem_dt,
                                        space, _stream())
        self._keep = None
        self.k = 0

    def close(self):
        if getattr(self, "handle", None):
            tfps_graph_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def devices_set(self, k, s, C, B, scale):
        s = _np(s, np.int32); C = _np(C, np.int64); B = _np(B, np.int64)
        tfps_devices_set(self.handle, int(k), _addr(s), _addr(C), _addr(B), int(scale))
        self.k = int(k)

    def topo_levels(self):
        import torch
        level = torch.empty(max(self.n, 1), dtype=torch.int32, device="cuda")
        order = torch.empty(max(self.n, 1), dtype=torch.int32, device="cuda")
        lp = np.zeros(self.n + 2, np.int64)
        L = tfps_topo_levels(self.handle, _addr(level), _addr(order), _addr(lp), lp.shape[0], _stream())
        return level[: self.n], order[: self.n], lp[: L + 1].copy(), L

    def eval_batch(self, part, P=None, want=("tlevel", "blevel", "cp", "load", "memload", "viol"), flags=EVAL_AUTO,
                   out: Optional[Dict] = None, check=True) -> Dict:
        """part: torch uint8 CUDA tensor [n][ldp].  Returns a dict of torch CUDA tensors."""
        import torch
        assert part.is_cuda and part.dtype == torch.uint8 and part.dim() == 2 and part.is_contiguous()
        n, ldp = part.shape
        assert n == self.n
        P = ldp if P is None else int(P)
        out = {} if out is None else out
        dev = part.device

        def buf(name, shape, dtype):
            if name not in want:
                return None
            if name not in out:
                out[name] = torch.empty(shape, dtype=dtype, device=dev)
            return out[name]

        tl = buf("tlevel", (n, ldp), torch.int64)
        bl = buf("blevel", (n, ldp), torch.int64)
        cp = buf("cp", (max(P, 1),), torch.int64)
        ld = buf("load", (self.k, ldp), torch.int64)
        ml = buf("memload", (self.k, ldp), torch.int64)
        vi = buf("viol", (max(P, 1),), torch.int64)  # bit pattern of uint64
        ws, ws_bytes = None, 0
        if cp is not None and tl is None and bl is None:
            ws_bytes = tfps_eval_workspace_bytes(self.handle, P, ldp, flags | EVAL_SCRATCH_LEVELS)
            if "workspace" not in out or out["workspace"].numel() < ws_bytes:
                out["workspace"] = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device=dev)
            ws = out["workspace"]
        tfps_eval_batch(self.handle, P, ldp, _addr(part), _addr(tl), _addr(bl), _addr(cp), _addr(ld), _addr(ml),
                        _addr(vi), _addr(ws), ws_bytes, flags, _stream())
        if check:
            self.status()
        return out

    def eval_batch_host(self, part: np.ndarray, P=None, want=("cp", "load", "memload", "viol"), flags=EVAL_AUTO) -> Dict:
        """part: host uint8 [n][ldp] (numpy, or a pinned torch CPU tensor).  Returns numpy arrays."""
        n, ldp = part.shape
        P = ldp if P is None else int(P)
        res = {}
        tl = np.zeros((n, ldp), np.int64) if "tlevel" in want else None
        bl = np.zeros((n, ldp), np.int64) if "blevel" in want else None
        cp = np.zeros(max(P, 1), np.int64) if "cp" in want else None
        ld = np.zeros((self.k, ldp), np.int64) if "load" in want else None
        ml = np.zeros((self.k, ldp), np.int64) if "memload" in want else None
        vi = np.zeros(max(P, 1), np.uint64) if "viol" in want else None
        tfps_eval_batch_host(self.handle, P, ldp, _addr(part), _addr(tl), _addr(bl), _addr(cp), _addr(ld), _addr(ml),
                             _addr(vi), flags, _stream())
        for name, a in (("tlevel", tl), ("blevel", bl), ("cp", cp), ("load", ld), ("memload", ml), ("viol", vi)):
            if a is not None:
                res[name] = a
        return res

    def constraints_set(self, pairs, devcons):
        """pairs: [npairs][2] vertices that must share a device (Eq. 3); devcons: [ndev][2] (vertex, device) (Eq. 4)."""
        pairs = _np(pairs, np.int32).reshape(-1, 2)
        devcons = _np(devcons, np.int32).reshape(-1, 2)
        pa, pb = np.ascontiguousarray(pairs[:, 0]), np.ascontiguousarray(pairs[:, 1])
        dv, dd = np.ascontiguousarray(devcons[:, 0]), np.ascontiguousarray(devcons[:, 1])
        tfps_constraints_set(self.handle, pairs.shape[0], _addr(pa), _addr(pb), devcons.shape[0], _addr(dv), _addr(dd))

    def eval_constraints(self, part, P=None):
        """Violated collocation pairs and device constraints per candidate: two int32 CUDA tensors [P]."""
        import torch
        n, ldp = part.shape
        P = ldp if P is None else int(P)
        coll = torch.empty(max(P, 1), dtype=torch.int32, device=part.device)
        dev = torch.empty(max(P, 1), dtype=torch.int32, device=part.device)
        tfps_eval_constraints(self.handle, P, ldp, _addr(part), _addr(coll), _addr(dev), _stream())
        return coll[:P], dev[:P]

    def ranks(self):
        """(upRank, downRank, totalRank): three int64 CUDA tensors [n] (Eq. 5, Eq. 6, Section 3.2.1)."""
        import torch
        up, down, total = (torch.zeros(max(self.n, 1), dtype=torch.int64, device="cuda") for _ in range(3))
        tfps_ranks(self.handle, _addr(up), _addr(down), _addr(total), _stream())
        return up[:self.n], down[:self.n], total[:self.n]

    def critical_path(self, down):
        """int32 CUDA tensor: the vertices of the critical path from its source to its sink (Section 3.2.2)."""
        import torch
        path = torch.zeros(max(self.n, 1), dtype=torch.int32, device="cuda")
        ln = tfps_critical_path(self.handle, _addr(down), _addr(path), _stream())
        return path[:ln]

    def batch_split(self, total):
        """(uint8 CUDA tensor [n] of devices, number of vertices no device could take): Batch Split (Section 3.2.1)."""
        import torch
        part = torch.zeros(max(self.n, 1), dtype=torch.uint8, device="cuda")
        bad = tfps_batch_split(self.handle, _addr(total), _addr(part), _stream())
        return part[:self.n], bad

    def cp_partition(self, path):
        """(uint8 CUDA tensor [n] of devices, unplaced count): Critical Path partitioning (Section 3.2.2, Eq. 7)."""
        import torch
        part = torch.zeros(max(self.n, 1), dtype=torch.uint8, device="cuda")
        bad = tfps_cp_partition(self.handle, _addr(path) if path.numel() else None, int(path.numel()), _addr(part), _stream())
        return part[:self.n], bad

    def simulate(self, part, P, policy=SCHED_FIFO, prio=None, want_start=True):
        """List-scheduling simulation of every candidate (Section 4): (start int64 [n][ldp] or None, makespan int64 [P])."""
        import torch
        n, ldp = part.shape
        start = torch.zeros((n, ldp), dtype=torch.int64, device=part.device) if want_start else None
        mk = torch.zeros(max(int(P), 1), dtype=torch.int64, device=part.device)
        tfps_simulate(self.handle, int(P), ldp, _addr(part), policy, _addr(prio), _addr(start), _addr(mk), _stream())
        return start, mk[:int(P)]

    def status(self):
        tfps_get_status(self.handle, _stream())


def critical_mask(out: Dict, P: int):
    """uint8 CUDA tensor [n][ldp]: 1 where a vertex lies on a longest path of the candidate (from eval_batch outputs)."""
    import torch
    tl, bl, cp = out["tlevel"], out["blevel"], out["cp"]
    n, ldp = tl.shape
    mask = torch.zeros((n, ldp), dtype=torch.uint8, device=tl.device)
    tfps_critical_mask(n, int(P), ldp, _addr(tl), _addr(bl), _addr(cp), _addr(mask), _stream())
    return mask


def transpose_u8(src, ldp: Optional[int] = None):
    """src: torch uint8 CUDA tensor [P][n] -> [n][ldp] (padding columns zero-initialised by torch)."""
    import torch
    P, n = src.shape
    ldp = round_up_ldp(P) if ldp is None else ldp
    dst = torch.zeros((n, ldp), dtype=torch.uint8, device=src.device)
    tfps_transpose_u8(_addr(src), _addr(dst), P, n, ldp, _stream())
    return dst


def graph_from_workload(w) -> "Graph":
    """Build a Graph (and set its device tables) from an ``inputs.Workload``."""
    from . import inputs
    c = inputs.to_csr(w.graph)
    g = Graph(w.graph.n, c.in_ptr, c.in_src, c.in_t, w.graph.c, c.out_ptr, c.out_dst, c.out_t, w.graph.mem)
    d = w.devices
    g.devices_set(d.k, d.s, d.C, d.B, d.scale)
    return g
