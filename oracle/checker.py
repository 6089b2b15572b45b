"""Direct-definition checker (test infrastructure).

Independent of the simulator's mechanics: given the inputs of a scenario and a set C of process ids,
the reduction over exactly C is evaluated from its plain definition. Semantics items 3 and 4 of the
reduce (and 4, 5 of the allreduce) then read: Live <= C <= Live + InOp, C and PreFailed disjoint, and
the delivered value equals the reduction over C.
"""
from __future__ import annotations

import math

import numpy as np


def reduce_over(x: np.ndarray, members, op: str):
    """Reduction of rows `members` of x [P][k] by its textbook definition. Integer sums wrap (two's
    complement); float32 inputs are summed in float64 and returned with the sum of magnitudes."""
    members = list(members)
    sel = x[members] if members else x[:0]
    if x.dtype == np.float32:
        s64 = sel.astype(np.float64)
        return s64.sum(axis=0), np.abs(s64).sum(axis=0)
    if op == "sum":
        with np.errstate(over="ignore"):
            return sel.view(np.uint32 if x.dtype.itemsize == 4 else np.uint64).sum(
                axis=0, dtype=np.uint32 if x.dtype.itemsize == 4 else np.uint64).view(x.dtype)
    if op == "max":
        return sel.max(axis=0)
    if op == "xor":
        return np.bitwise_xor.reduce(sel, axis=0)
    raise ValueError(op)


def value_matches(x: np.ndarray, members, op: str, y: np.ndarray) -> bool:
    """Does y equal the reduction over `members`? Exact for integers; for float32 within
    1e-6 * ceil(log2 P) relative to the sum of magnitudes."""
    if x.dtype == np.float32:
        s, mag = reduce_over(x, members, op)
        tol = 1e-6 * math.ceil(math.log2(x.shape[0])) * mag
        return bool(np.all(np.abs(y.astype(np.float64) - s) <= tol))
    return bool(np.array_equal(reduce_over(x, members, op), y))


def bits(words: np.ndarray, P: int):
    return [p for p in range(P) if (int(words[p >> 5]) >> (p & 31)) & 1]


def contribution_allowed(P: int, C, prefailed, inop_victims) -> bool:
    """Live <= C <= Live + InOp and C disjoint from PreFailed."""
    C, pre, vic = set(C), set(prefailed), set(inop_victims) - set(prefailed)
    live = set(range(P)) - pre - vic
    return live <= C and C <= (live | vic) and not (C & pre)
