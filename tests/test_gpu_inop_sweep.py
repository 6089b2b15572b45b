"""Exhaustive in-operation sweep at a size the CPU oracle does not reach in full: every pre-operation failure set of
size <= 1, every victim, every failure round, P = 64, f = 2 (37 000 and 63 000 scenarios). Item 4 of the
reduce semantics (a failed process' value is included whole or not at all) and items 4, 5 of the allreduce
semantics are checked on every scenario with torch arithmetic; a random sample goes through the oracle as well."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2602_22445_b200 import binding as B
from paper_2602_22445_b200 import scenarios as sc
from tests.gpu_util import run_gpu, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("collective", ["reduce", "allreduce"])
def test_every_victim_and_round(collective):
    import torch
    P, f, k = 64, 2, 2
    sched = O.schedule(P, f)
    R = sched["rounds_attempt"] if collective == "allreduce" else sched["rounds_reduce"]
    pre_sets = [()] + [(p,) for p in range(P)]
    victims = range(f + 1, P) if collective == "allreduce" else range(P)       # allreduce: not a root candidate
    w = sc.inop_sweep(P, f, k, sc.KIND_U64_FULL, "sum", pre_sets, range(0, R + 2), collective, victims)
    assert w.S > 30000
    x = w.host_inputs()
    out, st, _ = run_gpu(x, f, "sum", w.prefail, w.inop, None, 0, collective == "allreduce")
    code = st[:, 0] & 0xFF
    vic, rnd = w.inop[:, 0, 0].astype(np.int64), w.inop[:, 0, 1].astype(np.int64)
    pre0 = (w.prefail[:, 0] & 1).astype(bool)                                  # process 0 failed before the operation
    if collective == "reduce":
        root_dead = pre0 | ((vic == 0) & (rnd < R))
        assert np.array_equal(code == B.FTC_ST_ROOT_FAILED, root_dead) and (code[~root_dead] == 0).all()
    else:
        assert (code == 0).all()
        assert np.array_equal((st[:, 0] >> 16) & 0xFF, 1 + pre0.astype(np.int64))   # second attempt iff candidate 0 was dead
    ok = code == 0
    # the contribution set the status claims: everybody but the pre-failed, and the victim iff its bit is set
    npre = np.unpackbits(w.prefail.view(np.uint8), axis=1).sum(axis=1)
    incl = (st[:, 2] & 1).astype(bool)
    assert np.array_equal(st[ok, 1], (P - npre - 1 + incl)[ok])
    X = torch.from_numpy(x.view(np.int64)).cuda()
    total = X.sum(dim=1)
    rows = torch.arange(w.S, device="cuda")
    pre_s, pre_p = np.nonzero(np.unpackbits(w.prefail.view(np.uint8), axis=1, bitorder="little")[:, :P])
    total.index_add_(0, torch.from_numpy(pre_s).cuda(), -X[torch.from_numpy(pre_s).cuda(), torch.from_numpy(pre_p).cuda()])
    excl = torch.from_numpy(~incl).cuda()
    total[excl] -= X[rows[excl], torch.from_numpy(vic).cuda()[excl]]
    got = torch.from_numpy(out.view(np.int64)).cuda()
    okt = torch.from_numpy(ok).cuda()
    assert torch.equal(got[okt], total[okt])                                   # whole or not at all, nobody twice
    assert not got[~okt].any()
    # a victim that performs every send of the reduce is included; one that fails before sending anything is not
    base = np.where((collective == "allreduce") & pre0, R, 0)
    assert incl[ok & (rnd - base >= sched["rounds_reduce"])].all() and not incl[ok & (rnd <= base)].any()
    assert 0 < incl[ok].mean() < 1
    if collective == "allreduce":                                              # everybody alive at the end holds the value
        dead_end = rnd < base + R
        assert np.array_equal(st[:, 3], P - npre - dead_end)
    idx = np.random.Generator(np.random.PCG64(1)).choice(w.S, 600, replace=False)
    want_out, want_st = O.batch(x[idx], f, "sum", w.prefail[idx], w.inop[idx], None, 0, collective == "allreduce")
    assert np.array_equal(st[idx], want_st) and np.array_equal(out[idx], want_out)
