"""TEST INFRASTRUCTURE -- not part of the product path.

ctypes front end of the plain C oracle (``tfps_oracle.c``): topological levels
and, per candidate partition, tlevel / blevel (the PCT of Eq. 12) / critical
path length / per-device load, memory load and capacity-violation bits.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may
import this package.  It imports nothing from the CUDA package and shares no
code with it.  The shared object is compiled with gcc on first use.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tfps_oracle.c")
_LIB = os.path.join(_HERE, "libtfps_oracle.so")

OK, BAD_ARG, CYCLE, OVERFLOW, BAD_PARTITION = 0, -1, -2, -3, -4


class OracleError(RuntimeError):
    def __init__(self, code: int):
        names = {BAD_ARG: "BAD_ARG", CYCLE: "CYCLE", OVERFLOW: "OVERFLOW", BAD_PARTITION: "BAD_PARTITION"}
        super().__init__(f"oracle error {names.get(code, code)}")
        self.code = code


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc, -O2, no vectorisation tricks of our own)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _get():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P = ctypes.c_void_p
        lib.oracle_topo_levels.restype = ctypes.c_int
        lib.oracle_topo_levels.argtypes = [ctypes.c_int64, P, P, P, P, P, P, P, P, P]
        lib.oracle_default_mem.restype = ctypes.c_int
        lib.oracle_default_mem.argtypes = [ctypes.c_int64, P, P, P]
        lib.oracle_eval_partition.restype = ctypes.c_int
        lib.oracle_eval_partition.argtypes = (
            [ctypes.c_int64] + [P] * 8 + [ctypes.c_int32, P, P, P, ctypes.c_int64, P, P, ctypes.c_int64] + [P] * 6
        )
        lib.oracle_eval_constraints.restype = ctypes.c_int
        lib.oracle_eval_constraints.argtypes = [ctypes.c_int64, P, ctypes.c_int64, ctypes.c_int64, P, P, ctypes.c_int64, P, P, P, P]
        lib.oracle_critical_mask.restype = ctypes.c_int
        lib.oracle_critical_mask.argtypes = [ctypes.c_int64, P, ctypes.c_int64, P, ctypes.c_int64, ctypes.c_int64, P, ctypes.c_int64]
        lib.oracle_ranks.restype = ctypes.c_int
        lib.oracle_ranks.argtypes = [ctypes.c_int64] + [P] * 9
        lib.oracle_batch_split.restype = ctypes.c_int
        lib.oracle_batch_split.argtypes = [ctypes.c_int64, P, P, ctypes.c_int32, P, P, P, P]
        lib.oracle_critical_path.restype = ctypes.c_int
        lib.oracle_critical_path.argtypes = [ctypes.c_int64, P, P, P, P, P, P]
        lib.oracle_cp_partition.restype = ctypes.c_int
        lib.oracle_cp_partition.argtypes = [ctypes.c_int64, P, ctypes.c_int64, P, P, ctypes.c_int32, P, P, ctypes.c_int64, P, P]
        lib.oracle_simulate.restype = ctypes.c_int
        lib.oracle_simulate.argtypes = ([ctypes.c_int64] + [P] * 5 + [ctypes.c_int32, P, P, ctypes.c_int64, P, ctypes.c_int64,
                                        ctypes.c_int32, P, ctypes.c_int64, P, P, P])
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _arr(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=dtype)


class OracleGraph:
    """Graph + topological structure held by the oracle (numpy arrays only)."""

    def __init__(self, n, in_ptr, in_src, in_t, out_ptr, out_dst, out_t, c, mem=None):
        self.n = int(n)
        self.in_ptr = _arr(in_ptr, np.int64)
        self.in_src = _arr(in_src, np.int32)
        self.in_t = _arr(in_t, np.int64)
        self.out_ptr = _arr(out_ptr, np.int64)
        self.out_dst = _arr(out_dst, np.int32)
        self.out_t = _arr(out_t, np.int64)
        self.c = _arr(c, np.int32)
        self.m = int(self.in_src.shape[0])
        assert self.in_ptr.shape[0] == self.n + 1 and self.out_ptr.shape[0] == self.n + 1
        assert self.out_dst.shape[0] == self.m
        lib = _get()
        self.level = np.zeros(self.n, np.int32)
        self.order = np.zeros(self.n, np.int32)
        self.topo = np.zeros(self.n, np.int32)
        lp = np.zeros(self.n + 2, np.int64)
        L = ctypes.c_int32(0)
        rc = lib.oracle_topo_levels(self.n, _p(self.in_ptr), _p(self.in_src), _p(self.out_ptr), _p(self.out_dst),
                                    _p(self.level), _p(self.order), _p(lp), ctypes.byref(L), _p(self.topo))
        if rc:
            raise OracleError(rc)
        self.num_levels = int(L.value)
        self.level_ptr = lp[: self.num_levels + 1].copy()
        if mem is None:
            self.mem = np.zeros(self.n, np.int64)
            rc = lib.oracle_default_mem(self.n, _p(self.out_ptr), _p(self.out_t), _p(self.mem))
            if rc:
                raise OracleError(rc)
        else:
            self.mem = _arr(mem, np.int64)


class OracleResult:
    __slots__ = ("tlevel", "blevel", "cp", "load", "memload", "viol")


def eval_partition(g: OracleGraph, k: int, s, C, B, S: int, p: np.ndarray, want_levels: bool = True) -> OracleResult:
    """Evaluate one candidate partition p (uint8[n], any stride)."""
    lib = _get()
    s = _arr(s, np.int32)
    C = _arr(C, np.int64)
    B = _arr(B, np.int64).reshape(k, k)
    assert p.dtype == np.uint8 and p.ndim == 1 and p.shape[0] == g.n
    stride = p.strides[0] if g.n > 1 else 1
    res = OracleResult()
    res.tlevel = np.zeros(g.n, np.int64) if want_levels else None
    res.blevel = np.zeros(g.n, np.int64) if want_levels else None
    res.load = np.zeros(k, np.int64)
    res.memload = np.zeros(k, np.int64)
    cp = ctypes.c_int64(0)
    viol = ctypes.c_uint64(0)
    rc = lib.oracle_eval_partition(
        g.n, _p(g.in_ptr), _p(g.in_src), _p(g.in_t), _p(g.out_ptr), _p(g.out_dst), _p(g.out_t),
        _p(g.c), _p(g.mem), k, _p(s), _p(C), _p(B), int(S), _p(g.topo),
        ctypes.c_void_p(p.ctypes.data), stride,
        _p(res.tlevel), _p(res.blevel), ctypes.byref(cp), _p(res.load), _p(res.memload), ctypes.byref(viol))
    if rc:
        raise OracleError(rc)
    res.cp = int(cp.value)
    res.viol = int(viol.value)
    return res


class OracleBatch:
    __slots__ = ("tlevel", "blevel", "cp", "load", "memload", "viol")


def eval_batch(g: OracleGraph, k: int, s, C, B, S: int, part: np.ndarray,
               cols: Optional[Sequence[int]] = None, want_levels: bool = True) -> OracleBatch:
    """Evaluate the listed candidate columns of the id matrix part[n][P], one
    candidate after the other.  Outputs are laid out [n][len(cols)] and
    [k][len(cols)] like the library's."""
    assert part.dtype == np.uint8 and part.ndim == 2 and part.shape[0] == g.n
    cols = list(range(part.shape[1])) if cols is None else list(cols)
    out = OracleBatch()
    q = len(cols)
    out.tlevel = np.zeros((g.n, q), np.int64) if want_levels else None
    out.blevel = np.zeros((g.n, q), np.int64) if want_levels else None
    out.cp = np.zeros(q, np.int64)
    out.load = np.zeros((k, q), np.int64)
    out.memload = np.zeros((k, q), np.int64)
    out.viol = np.zeros(q, np.uint64)
    for i, j in enumerate(cols):
        r = eval_partition(g, k, s, C, B, S, part[:, j], want_levels)
        if want_levels:
            out.tlevel[:, i] = r.tlevel
            out.blevel[:, i] = r.blevel
        out.cp[i] = r.cp
        out.load[:, i] = r.load
        out.memload[:, i] = r.memload
        out.viol[i] = r.viol
    return out


def eval_constraints(part: np.ndarray, pairs, devcons, cols: Optional[Sequence[int]] = None):
    """Collocation constraints (Eq. 3: pairs of vertices that must share a device) and device constraints (Eq. 4:
    (vertex, device) pairs that must hold) of the listed candidate columns of part[n][P].  Returns two int64 arrays:
    the number of violated collocation pairs and of violated device constraints per candidate."""
    lib = _get()
    assert part.dtype == np.uint8 and part.ndim == 2
    n = part.shape[0]
    pairs = _arr(pairs, np.int32).reshape(-1, 2)
    devcons = _arr(devcons, np.int32).reshape(-1, 2)
    pa, pb = np.ascontiguousarray(pairs[:, 0]), np.ascontiguousarray(pairs[:, 1])
    dv, dd = np.ascontiguousarray(devcons[:, 0]), np.ascontiguousarray(devcons[:, 1])
    cols = list(range(part.shape[1])) if cols is None else list(cols)
    coll = np.zeros(len(cols), np.int64)
    dev = np.zeros(len(cols), np.int64)
    for i, j in enumerate(cols):
        col = part[:, j]
        a, b = ctypes.c_int64(0), ctypes.c_int64(0)
        rc = lib.oracle_eval_constraints(n, ctypes.c_void_p(col.ctypes.data), col.strides[0] if n > 1 else 1,
                                         pairs.shape[0], _p(pa), _p(pb), devcons.shape[0], _p(dv), _p(dd),
                                         ctypes.byref(a), ctypes.byref(b))
        if rc:
            raise OracleError(rc)
        coll[i], dev[i] = a.value, b.value
    return coll, dev


def critical_mask(tlevel: np.ndarray, blevel: np.ndarray, cp: np.ndarray) -> np.ndarray:
    """mask[v][j] = 1 where vertex v lies on a longest path of candidate j (tlevel + blevel == cp), from the
    [n][q] level matrices and the [q] critical-path lengths of an OracleBatch."""
    lib = _get()
    tl = _arr(tlevel, np.int64)
    bl = _arr(blevel, np.int64)
    n, q = tl.shape
    mask = np.zeros((n, q), np.uint8)
    for j in range(q):
        rc = lib.oracle_critical_mask(n, ctypes.c_void_p(tl[:, j].ctypes.data), q, ctypes.c_void_p(bl[:, j].ctypes.data), q,
                                      int(cp[j]), ctypes.c_void_p(mask[:, j].ctypes.data), q)
        if rc:
            raise OracleError(rc)
    return mask


def ranks(g: OracleGraph):
    """(upRank, downRank, totalRank) of every vertex, int64 [n] each (Eq. 5, Eq. 6, Section 3.2.1)."""
    lib = _get()
    up = np.zeros(g.n, np.int64)
    down = np.zeros(g.n, np.int64)
    total = np.zeros(g.n, np.int64)
    rc = lib.oracle_ranks(g.n, _p(g.in_ptr), _p(g.in_src), _p(g.out_ptr), _p(g.out_dst), _p(g.c), _p(g.topo),
                          _p(up), _p(down), _p(total))
    if rc:
        raise OracleError(rc)
    return up, down, total


def batch_split(total, mem, k: int, s, C):
    """Batch Split partition (Section 3.2.1): (part uint8 [n], number of vertices no device could take)."""
    lib = _get()
    total = _arr(total, np.int64)
    mem = _arr(mem, np.int64)
    s = _arr(s, np.int32)
    C = _arr(C, np.int64)
    n = total.shape[0]
    part = np.zeros(n, np.uint8)
    bad = ctypes.c_int64(0)
    rc = lib.oracle_batch_split(n, _p(total), _p(mem), k, _p(s), _p(C), _p(part), ctypes.byref(bad))
    if rc:
        raise OracleError(rc)
    return part, int(bad.value)


def critical_path(g: OracleGraph, down) -> np.ndarray:
    """Vertices of the critical path of the Critical Path strategy, source to sink (Section 3.2.2, steps 1-4)."""
    lib = _get()
    down = _arr(down, np.int64)
    path = np.zeros(max(1, g.n), np.int32)
    ln = ctypes.c_int64(0)
    rc = lib.oracle_critical_path(g.n, _p(g.in_ptr), _p(g.in_src), _p(g.out_ptr), _p(down), _p(path), ctypes.byref(ln))
    if rc:
        raise OracleError(rc)
    return path[: int(ln.value)].copy()


def cp_partition(g: OracleGraph, path, k: int, s, C, S: int):
    """Critical Path partition (Section 3.2.2, Eq. 7): (part uint8 [n], number of vertices no device could take)."""
    lib = _get()
    path = _arr(path, np.int32)
    s = _arr(s, np.int32)
    C = _arr(C, np.int64)
    part = np.zeros(g.n, np.uint8)
    bad = ctypes.c_int64(0)
    rc = lib.oracle_cp_partition(g.n, _p(path), path.shape[0], _p(g.c), _p(g.mem), k, _p(s), _p(C), S, _p(part),
                                 ctypes.byref(bad))
    if rc:
        raise OracleError(rc)
    return part, int(bad.value)


def simulate(g: OracleGraph, k: int, s, B, S: int, p, policy: int, prio=None, msr_weights=(1, 1, 1, 5)):
    """List-scheduling simulation of one candidate (Section 4): (start times int64 [n], makespan).
    policy 0 = FIFO, 1 = PCT with prio = the candidate's path computation times (blevel, Eq. 12), 2 = MSR (Eq. 13)
    with the weights (alpha, beta, gamma, delta)."""
    lib = _get()
    s = _arr(s, np.int32)
    B = _arr(B, np.int64)
    p = _arr(p, np.uint8)
    pr = None if prio is None else _arr(prio, np.int64)
    start = np.zeros(g.n, np.int64)
    mk = ctypes.c_int64(0)
    w = _arr(msr_weights, np.int64)
    rc = lib.oracle_simulate(g.n, _p(g.in_ptr), _p(g.out_ptr), _p(g.out_dst), _p(g.out_t), _p(g.c), k, _p(s), _p(B), S,
                             _p(p), 1, policy, _p(pr), 1, _p(w), _p(start), ctypes.byref(mk))
    if rc:
        raise OracleError(rc)
    return start, int(mk.value)
