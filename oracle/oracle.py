"""ctypes front end of the CPU oracle (test infrastructure, never used by the product path).

Builds ``ftc_oracle.c`` with gcc on first use and exposes one scenario (`run`) or a batch
(`batch`) with numpy arrays. Nothing here touches CUDA.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ftc_oracle.c")
_LIB = os.path.join(_HERE, "libftc_oracle.so")

DTYPES = {np.dtype(np.int32): 0, np.dtype(np.int64): 1, np.dtype(np.uint64): 2, np.dtype(np.float32): 3}
OPS = {"sum": 0, "max": 1, "xor": 2}
STATUS_NAMES = {0: "OK", 1: "ROOT_FAILED", 2: "NO_CLEAN_SUBTREE", 3: "NO_LIVE_ROOT_CANDIDATE",
                4: "PRECONDITION_INOP_ROOT"}
UNUSED = 0xFFFFFFFF


class Cfg(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("P", "f", "k", "dtype", "op", "max_inop", "sweep", "track_sets", "partners_descending", "arity")]


class Out(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("result", "status", "cand", "cand_flag", "holders", "expanded", "msgs",
                                          "contrib", "sends", "events", "uc_values", "tree_values", "tree_sent",
                                          "tree_sets", "cand_nfail", "nfail", "failed")]


def build(force: bool = False) -> str:
    """Compile the oracle into a shared library next to its source (gcc, -O2, no fp contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-ffp-contract=off", "-fPIC", "-shared",
                               "-o", _LIB, _SRC])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ftc_oracle_run.restype = C.c_int
        _lib.ftc_oracle_run.argtypes = [C.POINTER(Cfg), C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32,
                                        C.POINTER(Out)]
        _lib.ftc_oracle_batch.restype = C.c_int
        _lib.ftc_oracle_batch.argtypes = [C.POINTER(Cfg), C.c_int, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p]
        _lib.ftc_oracle_schedule.restype = C.c_int
        _lib.ftc_oracle_schedule.argtypes = [C.c_uint32, C.c_uint32, C.c_uint32, C.POINTER(C.c_uint32)]
    return _lib


def schedule(P: int, f: int, arity: int = 2) -> dict:
    """q, r, H and the round counts of one reduce / one allreduce attempt (subtrees: `arity`-ary heaps)."""
    buf = (C.c_uint32 * 5)()
    if lib().ftc_oracle_schedule(P, f, arity, buf) != 0:
        raise ValueError("P must be at least f+2")
    return dict(q=buf[0], r=buf[1], H=buf[2], rounds_reduce=buf[3], rounds_attempt=buf[4])


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _prep_inop(inop, max_inop):
    if inop is None or max_inop == 0:
        return None
    a = np.ascontiguousarray(inop, dtype=np.uint32)
    return a


def run(x: np.ndarray, f: int, op: str, prefail, inop=None, root: int = 0, allreduce: bool = False,
        sweep: int = 0, track_sets: bool = False, detail: bool = False, arity: int = 2,
        partners_descending: bool = False) -> dict:
    """Simulate one scenario. x: [P][k]; prefail: uint32 words or an iterable of failed ids;
    inop: [(victim, round), ...]. Returns result, status fields and (detail=True) instrumentation."""
    x = np.ascontiguousarray(x)
    P, k = x.shape
    W = (P + 31) // 32
    if not (isinstance(prefail, np.ndarray) and prefail.dtype == np.uint32):
        words = np.zeros(W, dtype=np.uint32)
        for p in prefail:
            words[p >> 5] |= np.uint32(1 << (p & 31))
        prefail = words
    prefail = np.ascontiguousarray(prefail)
    inop_a = None
    max_inop = 0
    if inop is not None and len(inop):
        inop_a = np.ascontiguousarray(np.asarray(inop, dtype=np.uint32).reshape(-1, 2))
        max_inop = inop_a.shape[0]
    cfg = Cfg(P, f, k, DTYPES[x.dtype], OPS[op], max_inop, sweep, 1 if track_sets else 0, int(partners_descending), arity)
    res = np.zeros(k, dtype=x.dtype)
    status = np.zeros(4, dtype=np.uint32)
    out = Out()
    out.result, out.status = _ptr(res), _ptr(status)
    extra = {}
    if detail:
        extra = dict(cand=np.zeros((f + 1, k), x.dtype), cand_flag=np.zeros(f + 1, np.uint32),
                     holders=np.zeros(W, np.uint32), expanded=np.zeros((P, k), x.dtype),
                     msgs=np.zeros(8, np.uint64), sends=np.zeros(P, np.uint32), events=np.zeros(P, np.uint32),
                     uc_values=np.zeros((P, k), x.dtype), tree_values=np.zeros((P, k), x.dtype),
                     tree_sent=np.zeros(P, np.uint32), cand_nfail=np.zeros(f + 1, np.uint32), nfail=np.zeros(1, np.uint32))
        if track_sets:
            extra["contrib"] = np.zeros(W, np.uint32)
            extra["tree_sets"] = np.zeros((P, W), np.uint32)
            extra["failed"] = np.zeros(W, np.uint32)
        for name, arr in extra.items():
            setattr(out, name, _ptr(arr))
    rc = lib().ftc_oracle_run(C.byref(cfg), 1 if allreduce else 0, _ptr(x), _ptr(prefail), _ptr(inop_a), root,
                              C.byref(out))
    if rc != 0:
        raise RuntimeError(f"oracle returned {rc}")
    d = dict(result=res, status=status, code=int(status[0] & 0xFF), subtree=int((status[0] >> 8) & 0xFF),
             attempts=int((status[0] >> 16) & 0xFF), count=int(status[1]), inop_included=int(status[2]),
             n_holders=int(status[3]))
    d.update(extra)
    return d


def batch(x: np.ndarray, f: int, op: str, prefail: np.ndarray, inop=None, roots=None, root: int = 0,
          allreduce: bool = False, arity: int = 2, partners_descending: bool = False):
    """Simulate S scenarios one after the other. x: [S][P][k]; prefail: [S][W] uint32;
    inop: [S][max_inop][2] uint32 or None; roots: [S] uint32 or None. Returns (result [S][k], status [S][4])."""
    x = np.ascontiguousarray(x)
    S, P, k = x.shape
    prefail = np.ascontiguousarray(prefail, dtype=np.uint32)
    max_inop = 0
    if inop is not None:
        inop = np.ascontiguousarray(inop, dtype=np.uint32)
        max_inop = inop.shape[1]
    if roots is not None:
        roots = np.ascontiguousarray(roots, dtype=np.uint32)
    cfg = Cfg(P, f, k, DTYPES[x.dtype], OPS[op], max_inop, 0, 0, int(partners_descending), arity)
    res = np.zeros((S, k), dtype=x.dtype)
    status = np.zeros((S, 4), dtype=np.uint32)
    rc = lib().ftc_oracle_batch(C.byref(cfg), 1 if allreduce else 0, S, _ptr(x), _ptr(prefail), _ptr(inop),
                                _ptr(roots), max(root, 0), _ptr(res), _ptr(status))
    if rc != 0:
        raise RuntimeError(f"oracle returned {rc}")
    return res, status
