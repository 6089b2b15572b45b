"""Checks of a finished batch that hold at any size, computed with torch (on the device the batch lives on) from the
plain definition.

For workloads whose failures stay within the tolerated number f (the configurations of the benchmark), section
"Semantics" fixes what a correct batch looks like without replaying the schedule:
  - the outcome of every scenario follows from the failure masks alone (a reduce toward a root that failed before
    the operation is a no-op; an allreduce uses one attempt per leading root candidate that had failed);
  - the result is the reduction over exactly the processes the status record claims as included: everybody who
    had not failed before the operation, minus the in-operation victims the record does not list as included.
Nothing here shares code with the kernels (torch reductions over the raw inputs) or with the CPU oracle.
Used by the full-size tests and by ``bench.py --full-config`` on every batch.
"""
from __future__ import annotations

import numpy as np

UNUSED = 0xFFFFFFFF


def _bit(prefail: np.ndarray, proc: np.ndarray) -> np.ndarray:
    rows = np.arange(prefail.shape[0])
    return ((prefail[rows, proc >> 5] >> (proc & 31).astype(np.uint32)) & 1).astype(bool)


def check_status_fields(w, st: np.ndarray) -> dict:
    """Status records against what the masks imply. Returns counts for the report; raises AssertionError."""
    P, f, S = w.P, w.f, w.S
    npre = np.unpackbits(w.prefail.view(np.uint8), axis=1).sum(axis=1).astype(np.int64)
    nvic = np.zeros(S, dtype=np.int64) if w.inop is None else (w.inop[:, :, 0] != UNUSED).sum(axis=1)
    assert (npre + nvic <= f).all(), "workload exceeds the tolerated number of failures: outcomes are not implied by the masks"
    first = np.full(S, max(w.root, 0), dtype=np.int64) if w.roots is None else w.roots.astype(np.int64)
    code = st[:, 0] & 0xFF
    if w.collective == "allreduce":
        lead = np.zeros(S, dtype=np.int64)
        alive = np.ones(S, dtype=bool)
        for a in range(f + 1):
            dead = _bit(w.prefail, (first + a) % P)
            lead += (alive & dead)
            alive &= dead
        assert (code == 0).all(), "an allreduce with at most f failures always finds a live root candidate"
        assert np.array_equal((st[:, 0] >> 16) & 0xFF, lead + 1), "one attempt per leading dead candidate"
        assert np.array_equal(st[:, 3], P - npre - nvic), "everybody alive at the end holds the value"
        ok = np.ones(S, dtype=bool)
    else:
        root_dead = _bit(w.prefail, first)
        assert np.array_equal(code, root_dead.astype(np.uint32)), "reduce: no-op exactly when the root had failed"
        ok = ~root_dead
        assert not st[~ok, 1:].any()
    incl_vic = np.array([bin(int(v)).count("1") for v in st[:, 2]], dtype=np.int64)
    assert np.array_equal(st[ok, 1], (P - npre - nvic + incl_vic)[ok]), "included count"
    assert (((st[ok, 0] >> 8) & 0xFF) <= f).all(), "selected child"
    return {"ok_scenarios": int(ok.sum()), "noop_scenarios": int((~ok).sum()), "retried": int((((st[:, 0] >> 16) & 0xFF) > 1).sum())}


def excluded_lists(w, st: np.ndarray):
    """(scenario, process) pairs excluded from the result according to the masks and status word 2."""
    pre_s, pre_p = np.nonzero(np.unpackbits(w.prefail.view(np.uint8), axis=1, bitorder="little")[:, :w.P])
    if w.inop is None:
        return pre_s, pre_p
    vs, vslot = np.nonzero(w.inop[:, :, 0] != UNUSED)
    out = ((st[vs, 2] >> vslot.astype(np.uint32)) & 1) == 0
    return np.concatenate([pre_s, vs[out]]), np.concatenate([pre_p, w.inop[vs[out], vslot[out], 0].astype(np.int64)])


def _xor_over_processes(x):
    """xor-reduction over dim 1 of an int64 tensor [S][P][k] by halving (torch has no xor reduction)."""
    import torch
    cur = x
    while cur.shape[1] > 1:
        n = cur.shape[1]
        h = n // 2
        nxt = torch.bitwise_xor(cur[:, :h], cur[:, h:2 * h])
        if n & 1:
            nxt[:, 0] ^= cur[:, n - 1]
        cur = nxt
    return cur[:, 0]


def check_results_by_definition(w, d_x, d_out, st: np.ndarray, chunk: int = 0) -> dict:
    """d_out against the reduction torch computes over exactly the included processes (raises AssertionError).
    Works through the batch in chunks of about 1 GiB of inputs (temporaries stay a few GiB)."""
    import torch
    chunk = chunk or max(1, (1 << 30) // (w.P * w.k * np.dtype(w.dtype).itemsize))
    es, ep = excluded_lists(w, st)
    ok = (st[:, 0] & 0xFF) == 0
    keep = ok[es]
    es, ep = es[keep], ep[keep]                        # excluded processes of scenarios that produced a result
    dev = d_x.device
    es_t, ep_t = torch.from_numpy(es).to(dev), torch.from_numpy(ep).to(dev)
    ok_t = torch.from_numpy(ok).to(dev)
    name = np.dtype(w.dtype).name
    report = {"excluded_pairs": int(len(es))}
    if name == "float32":
        import math
        tol = 1e-6 * math.ceil(math.log2(w.P))           # relative to the sum of magnitudes
        worst = 0.0
        for s0 in range(0, w.S, chunk):
            s1 = min(s0 + chunk, w.S)
            xd = d_x[s0:s1].double()
            ref, mag = xd.sum(dim=1), xd.abs().sum(dim=1)
            sel = (es_t >= s0) & (es_t < s1)
            ref.index_add_(0, es_t[sel] - s0, -d_x[es_t[sel], ep_t[sel]].double())
            err = ((d_out[s0:s1].double() - ref).abs() / mag)[ok_t[s0:s1]]
            if err.numel():
                worst = max(worst, err.max().item())
        assert worst <= tol, f"float32 sum off by {worst} of the sum of magnitudes (bound {tol})"
        report["worst_relative_error"] = worst
    elif w.op == "max":
        lowest = torch.iinfo(d_x.dtype).min
        for s0 in range(0, w.S, chunk):
            s1 = min(s0 + chunk, w.S)
            x2 = d_x[s0:s1].clone()
            sel = (es_t >= s0) & (es_t < s1)
            x2[es_t[sel] - s0, ep_t[sel]] = lowest
            ref = x2.amax(dim=1)
            ref[~ok_t[s0:s1]] = 0
            assert torch.equal(ref, d_out[s0:s1]), "max over the included processes"
    else:
        xi = d_x.view(torch.int64) if d_x.dtype == torch.uint64 else d_x
        oi = d_out.view(torch.int64) if d_out.dtype == torch.uint64 else d_out
        order = np.argsort(es, kind="stable")
        es_o, ep_o = es[order], ep[order]
        nth = np.arange(len(es_o)) - np.searchsorted(es_o, es_o, side="left")      # position within its scenario
        for s0 in range(0, w.S, chunk):
            s1 = min(s0 + chunk, w.S)
            if w.op == "sum":
                ref = xi[s0:s1].sum(dim=1)                                           # wraps like the method's sum
            else:
                ref = _xor_over_processes(xi[s0:s1])
            inb = (es_o >= s0) & (es_o < s1)
            for j in range(int(nth[inb].max()) + 1 if inb.any() else 0):
                pick = inb & (nth == j)                                              # one excluded process per scenario
                a, b = torch.from_numpy(es_o[pick]).to(dev), torch.from_numpy(ep_o[pick]).to(dev)
                if w.op == "sum":
                    ref[a - s0] -= xi[a, b]
                else:
                    ref[a - s0] ^= xi[a, b]
            ref[~ok_t[s0:s1]] = 0
            assert torch.equal(ref, oi[s0:s1]), f"{w.op} over the included processes"
    return report
