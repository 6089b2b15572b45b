"""Helpers for the GPU parity tests: run a batch through the C ABI and through the CPU oracle."""
from __future__ import annotations

import numpy as np

from oracle import oracle as O
from paper_2602_22445_b200 import binding as B

NP2TORCH = {"int32": "int32", "int64": "int64", "uint64": "uint64", "float32": "float32"}


def to_dev(a):
    import torch
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint64:
        return torch.from_numpy(a.view(np.int64)).cuda().view(torch.uint64)
    if a.dtype == np.uint32:
        return torch.from_numpy(a.view(np.int32)).cuda().view(torch.uint32)
    return torch.from_numpy(a).cuda()


def to_host(t, dtype):
    import torch
    if t.dtype == torch.uint64:
        return t.view(torch.int64).cpu().numpy().view(np.uint64)
    if t.dtype == torch.uint32:
        return t.view(torch.int32).cpu().numpy().view(np.uint32)
    return t.cpu().numpy()


def run_gpu(x, f, op, prefail, inop=None, roots=None, root=0, allreduce=False, flags=0, d_x=None):
    """x: [S][P][k] numpy (or None with d_x a device tensor). Returns (out [S][k], status [S][4]) as numpy."""
    import torch
    if d_x is None:
        d_x = to_dev(x)
    S, P, k = d_x.shape
    np_dtype = np.dtype(str(d_x.dtype).replace("torch.", ""))
    max_inop = 0 if inop is None else inop.shape[1]
    desc = B.make_desc(P, f, k, B.dtype_code(d_x.dtype), op, root=-1 if roots is not None else root,
                       max_inop=max_inop, flags=flags)
    d_pf = to_dev(np.ascontiguousarray(prefail, dtype=np.uint32))
    d_inop = to_dev(np.ascontiguousarray(inop, dtype=np.uint32)) if max_inop else None
    d_roots = to_dev(np.ascontiguousarray(roots, dtype=np.uint32)) if roots is not None else None
    d_out = torch.empty((S, k), dtype=d_x.dtype, device="cuda")
    d_out.view(torch.uint8).fill_(0x5A)                     # stale bytes must not survive
    d_status = torch.full((max(S, 1), 4), 0x7FFFFFFF, dtype=torch.int32, device="cuda")[:S].contiguous()
    wsb = B.ftc_workspace_bytes(desc, S, allreduce)
    d_ws = torch.empty(max(wsb, 16), dtype=torch.uint8, device="cuda")
    fn = B.ftc_allreduce_batch if allreduce else B.ftc_reduce_batch
    fn(desc, S, d_x, d_pf, d_inop, d_roots, d_out, d_status.view(torch.uint32) if S else d_status, d_ws)
    torch.cuda.synchronize()
    return to_host(d_out, np_dtype), d_status.cpu().numpy().view(np.uint32), desc


def run_oracle(x, f, op, prefail, inop=None, roots=None, root=0, allreduce=False, arity=2, partners_descending=False):
    return O.batch(x, f, op, prefail, inop=inop, roots=roots, root=root, allreduce=allreduce, arity=arity,
                   partners_descending=partners_descending)


def run_oracle_mt(x, f, op, prefail, inop=None, roots=None, root=0, allreduce=False, chunk=None, partners_descending=False, arity=2):
    """run_oracle over chunks of scenarios on all host cores (threads: the C call releases the interpreter lock)."""
    import os
    from concurrent.futures import ThreadPoolExecutor
    S = x.shape[0]
    cores = os.cpu_count() or 1
    chunk = chunk or max(1, (S + 4 * cores - 1) // (4 * cores))
    O.lib()
    cuts = [(a, min(a + chunk, S)) for a in range(0, S, chunk)]

    def work(ab):
        a, b = ab
        return O.batch(x[a:b], f, op, prefail[a:b], inop=None if inop is None else inop[a:b],
                       roots=None if roots is None else roots[a:b], root=root, allreduce=allreduce,
                       arity=arity, partners_descending=partners_descending)

    with ThreadPoolExecutor(max_workers=cores) as ex:
        parts = list(ex.map(work, cuts))
    return np.concatenate([q[0] for q in parts]), np.concatenate([q[1] for q in parts])


def assert_same(got, want, what=""):
    g_out, g_st = got[0], got[1]
    w_out, w_st = want
    bad_st = np.nonzero((g_st != w_st).any(axis=1))[0]
    assert bad_st.size == 0, f"{what}: status differs at scenarios {bad_st[:8]}: gpu {g_st[bad_st[:4]]} oracle {w_st[bad_st[:4]]}"
    gb, wb = g_out.view(np.uint8).reshape(g_out.shape[0], -1), w_out.view(np.uint8).reshape(w_out.shape[0], -1)
    bad = np.nonzero((gb != wb).any(axis=1))[0]
    assert bad.size == 0, f"{what}: result differs at scenarios {bad[:8]}: gpu {g_out[bad[:2]]} oracle {w_out[bad[:2]]} status {w_st[bad[:2]]}"
