"""What every root child delivers, on the staged tiles (ftc_candidates_batch, kernel "staged"): value, delivered /
failed bit and size of the failed-process list of all f+1 children, compared with the CPU oracle scenario by scenario,
at batch sizes of more than two scenarios per launched block, with up to f+1 pre-operation failures, in-operation
victims (the root of a reduce among them) and per-scenario roots; and the same inputs through the general kernel."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest

from oracle import oracle as O
from paper_2602_22445_b200 import binding as B
from tests.gpu_util import to_dev, to_host
from tests.test_gpu_variants import DT, make_batch

pytestmark = pytest.mark.gpu


def gpu_candidates(d_x, f, op, pf, inop, roots, allreduce, flags=0):
    import torch
    S, P, k = d_x.shape
    desc = B.make_desc(P, f, k, B.dtype_code(d_x.dtype), op, root=-1, max_inop=inop.shape[1], flags=flags)
    d_cand = torch.empty((S, f + 1, k), dtype=d_x.dtype, device="cuda")
    d_cand.view(torch.uint8).fill_(0x5A)
    d_info = torch.full((S, f + 1, 2), 0x7FFFFFFF, dtype=torch.int32, device="cuda")
    d_ws = torch.empty(max(256, B.ftc_candidates_workspace_bytes(desc, S)), dtype=torch.uint8, device="cuda")
    B.ftc_candidates_batch(desc, S, allreduce, d_x, to_dev(pf), to_dev(inop), to_dev(roots), d_cand, d_info, d_ws)
    torch.cuda.synchronize()
    return to_host(d_cand, None), d_info.cpu().numpy(), desc


def oracle_candidates(x, f, op, pf, inop, roots, allreduce, descending=False):
    S, P, k = x.shape
    cand = np.zeros((S, f + 1, k), dtype=x.dtype)
    info = np.zeros((S, f + 1, 2), dtype=np.int32)
    O.lib()

    def work(i):
        d = O.run(x[i], f, op, pf[i], inop=[tuple(e) for e in inop[i]], root=int(roots[i]), allreduce=allreduce, detail=True,
                  partners_descending=descending)
        if d["attempts"] == 0:
            info[i, :, 0] = 2
            return
        cand[i] = d["cand"]
        info[i, :, 0] = d["cand_flag"]
        info[i, :, 1] = d["cand_nfail"]

    with ThreadPoolExecutor(max_workers=os.cpu_count() or 1) as ex:
        list(ex.map(work, range(S)))
    return cand, info


def assert_candidates(got, want, what):
    bad = np.nonzero((got[1] != want[1]).any(axis=(1, 2)))[0]
    assert bad.size == 0, f"{what}: info differs at scenarios {bad[:6]}: gpu {got[1][bad[:2]].tolist()} oracle {want[1][bad[:2]].tolist()}"
    S = got[0].shape[0]
    gb, wb = got[0].view(np.uint8).reshape(S, -1), want[0].view(np.uint8).reshape(S, -1)
    bad = np.nonzero((gb != wb).any(axis=1))[0]
    assert bad.size == 0, f"{what}: values differ at scenarios {bad[:6]} info {want[1][bad[:2]].tolist()}"


CASES = [
    # P, f, k, dtype, op, allreduce, scenarios (0 = a little more than two per block), flags
    (4096, 4, 32, "i32", "max", True, 0, 0),                 # the P=4096 configuration's shape
    (4096, 4, 32, "i32", "max", False, 300, 0),              # reduce: the root may die during the operation
    (65536, 8, 4, "u64", "sum", True, 0, 0),                 # the P=65536 configuration's shape
    (65536, 8, 4, "u64", "xor", False, 160, 0),
    (16384, 1, 8, "i32", "sum", True, 400, 0),               # groups of two
    (2000, 2, 8, "i64", "max", False, 900, 0),               # small blocks, no short group (1999 = 666*3 + 1: one member)
    (20011, 7, 2, "u64", "xor", True, 300, 0),               # ragged heap, wide groups
    (5000, 0, 8, "i32", "sum", False, 500, 0),               # no tolerance: one child, groups of one
    (3000, 3, 16, "i32", "sum", True, 500, B.FTC_PARTNERS_DESCENDING),
    (1024, 3, 16, "i32", "sum", True, 3000, 0),              # the float32 configuration's shape with integers
    (1024, 3, 16, "f32", "sum", True, 3000, 0),              # the float32 configuration: every member folds in its own order
    (1024, 3, 16, "f32", "sum", False, 700, B.FTC_PARTNERS_DESCENDING),
    (4099, 1, 16, "f32", "sum", True, 300, 0),               # groups of two, a short group of one member plus the root
    (20000, 7, 8, "f32", "sum", False, 120, 0),              # several warps per block, groups of eight
    (300, 2, 64, "f32", "sum", True, 900, 0),                # 256-byte vectors: two lane rows
]


@pytest.mark.parametrize("P,f,k,dname,op,allreduce,S,flags", CASES)
def test_all_children_on_the_staged_tiles(P, f, k, dname, op, allreduce, S, flags):
    desc = B.make_desc(P, f, k, B.dtype_code(np.dtype(DT[dname])), op, root=-1, max_inop=2, flags=flags)
    assert B.ftc_candidates_kernel_name(desc) == "staged"
    if S == 0:
        S = 2 * 2 * 148 + 5
    d_x, x, pf, inop, roots = make_batch(P, f, k, dname, allreduce, S, seed=17 * P + f)
    if not allreduce:                                         # some reduce roots die at some round of the operation
        R = O.schedule(P, f)["rounds_reduce"]
        for i in range(3, S, 9):
            inop[i, 1] = (roots[i], (i // 9) % (R + 2))
    got = gpu_candidates(d_x, f, op, pf, inop, roots, allreduce, flags)
    want = oracle_candidates(x, f, op, pf, inop, roots, allreduce, descending=bool(flags & B.FTC_PARTNERS_DESCENDING))
    assert_candidates(got, want, f"P={P} f={f} k={k} {dname} {op} allreduce={allreduce}")
    flags_seen = set(np.unique(want[1][:, :, 0]).tolist())
    assert {0, 1} <= flags_seen or f == 0
    if dname == "f32" and f >= 2:                             # each member folds in its own order: children 0 and 2 differ by
        clean = np.nonzero((want[1][:, :, 0] == 0).all(axis=1) & (want[1][:, :, 1] == 0).all(axis=1))[0]     # rounding (0 and 1 never do:
        assert clean.size and any(not np.array_equal(want[0][i, 0], want[0][i, 2]) for i in clean[:50])       # x1 + x0 = x0 + x1)
    general = gpu_candidates(d_x, f, op, pf, inop, roots, allreduce, flags | B.FTC_KERNEL_GENERIC)
    assert B.ftc_candidates_kernel_name(general[2]) == "generic"
    assert_candidates(general, want, "general kernel")


def test_kernel_choice():
    assert B.ftc_candidates_kernel_name(B.make_desc(4096, 4, 32, B.FTC_I32, "max")) == "staged"
    assert B.ftc_candidates_kernel_name(B.make_desc(1024, 3, 16, B.FTC_F32, "sum")) == "staged"           # one heap array per child
    assert B.ftc_candidates_kernel_name(B.make_desc(64, 2, 8, B.FTC_I64, "sum")) == "generic"             # a few KB per scenario
    assert B.ftc_candidates_kernel_name(B.make_desc(4096, 4, 5, B.FTC_I32, "max")) == "generic"           # odd vector length
    assert B.ftc_candidates_kernel_name(B.make_desc(4096, 4, 32, B.FTC_I32, "max", flags=B.FTC_TREE_ARITY(4))) == "generic"


@pytest.mark.parametrize("P,f,k,dname,op", [(4096, 4, 32, "i32", "max"), (1024, 3, 16, "f32", "sum")])
def test_a_wait_that_gives_up_is_reported_per_scenario(P, f, k, dname, op):
    """With FTC_DEBUG_ONE_POLL the kernel's waits for its copies look once and give up: a scenario then either matches the
    oracle or reports 3 ("a bounded wait ran out") for every child with zero values; the call returns by itself, and a
    normal call afterwards on the same buffers matches the oracle again."""
    S = 2 * 4 * 148 + 3
    d_x, x, pf, inop, roots = make_batch(P, f, k, dname, True, S, seed=5 * P + f)
    want = oracle_candidates(x, f, op, pf, inop, roots, True)
    cand, info, _ = gpu_candidates(d_x, f, op, pf, inop, roots, True, B.FTC_DEBUG_ONE_POLL)
    gave_up = (info[:, :, 0] == 3).all(axis=1)
    assert ((info[:, :, 0] == 3).any(axis=1) == gave_up).all()          # all children of a scenario or none
    assert not cand[gave_up].any() and not info[gave_up][:, :, 1].any()
    assert np.array_equal(info[~gave_up], want[1][~gave_up])
    assert np.array_equal(cand[~gave_up].view(np.uint8), want[0][~gave_up].view(np.uint8))
    assert gave_up.any()                                                # tile copies are waited for right after their issue
    assert_candidates(gpu_candidates(d_x, f, op, pf, inop, roots, True), want, "normal call after the give-up run")
