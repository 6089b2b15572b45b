"""Parity at the full sizes and in the launch configuration bench.py times (same entry point, same batch size,
device-generated inputs): sampled scenarios against the CPU oracle bit for bit, and every scenario of the batch
against properties that hold at any size (status fields derived from the masks; the result equals a reduction that
torch computes over exactly the processes the status record claims to be included)."""
import numpy as np
import pytest

import bench
from oracle import oracle as O
from paper_2602_22445_b200 import binding as B
from paper_2602_22445_b200 import scenarios as sc

pytestmark = pytest.mark.gpu


def run_full(name):
    import torch
    S = bench.DEFAULT_BATCH[name]
    sched = O.schedule(*{"c3": (1024, 3), "c4": (4096, 4), "c5": (65536, 8), "c5r": (65536, 8)}[name])
    w = bench.make_workload(name, S, 0, sched["rounds_attempt"])
    tdt = getattr(torch, np.dtype(w.dtype).name)
    allred = w.collective == "allreduce"
    desc = B.make_desc(w.P, w.f, w.k, B.dtype_code(tdt), w.op, root=-1 if w.roots is not None else 0,
                       max_inop=0 if w.inop is None else w.inop.shape[1])
    d_x = torch.empty((S, w.P, w.k), dtype=tdt, device="cuda")
    B.ftc_fill_inputs(w.kind, w.seed, 0, S, w.P, w.k, d_x)
    d_pf, d_inop, d_roots = bench.upload(w, torch)
    d_out = torch.empty((S, w.k), dtype=tdt, device="cuda")
    d_st = torch.empty((S, 4), dtype=torch.int32, device="cuda")
    fn = B.ftc_allreduce_batch if allred else B.ftc_reduce_batch
    fn(desc, S, d_x, d_pf, d_inop, d_roots, d_out, d_st, None)
    torch.cuda.synchronize()
    st = d_st.cpu().numpy().view(np.uint32)
    return w, sched, d_x, d_out, st


def want_dtype(w):
    return np.dtype(w.dtype)


def sample_against_oracle(w, d_out, st, n, seed):
    import torch
    rng = np.random.Generator(np.random.PCG64(seed))
    npre = np.unpackbits(w.prefail.view(np.uint8), axis=1).sum(axis=1)
    interesting = np.nonzero(npre > 0)[0]
    idx = np.unique(np.concatenate([rng.choice(w.S, n // 2, replace=False), rng.choice(interesting, n // 2, replace=False)]))
    x = w.host_inputs(idx)
    want_out, want_st = O.batch(x, w.f, w.op, w.prefail[idx], None if w.inop is None else w.inop[idx],
                                None if w.roots is None else w.roots[idx], max(w.root, 0), w.collective == "allreduce")
    d_sel = d_out.view(torch.int64) if d_out.dtype == torch.uint64 else d_out      # torch cannot index uint64
    got = d_sel[torch.from_numpy(idx).cuda()].cpu().numpy().view(want_dtype(w))
    assert np.array_equal(st[idx], want_st), "status differs from the oracle on sampled scenarios"
    assert np.array_equal(got.view(np.uint8), want_out.view(np.uint8)), "result differs from the oracle on sampled scenarios"


def excluded_lists(w, st):
    """(scenario, process) pairs excluded from the result according to masks and status word 2."""
    pre_s, pre_p = np.nonzero(np.unpackbits(w.prefail.view(np.uint8), axis=1, bitorder="little")[:, :w.P])
    if w.inop is None:
        return pre_s, pre_p
    vs, vslot = np.nonzero(w.inop[:, :, 0] != sc.UNUSED)
    out = ((st[vs, 2] >> vslot) & 1) == 0
    return np.concatenate([pre_s, vs[out]]), np.concatenate([pre_p, w.inop[vs[out], vslot[out], 0].astype(np.int64)])


def check_status_fields(w, sched, st):
    P, f = w.P, w.f
    npre = np.unpackbits(w.prefail.view(np.uint8), axis=1).sum(axis=1)
    nvic = np.zeros(w.S, dtype=np.int64) if w.inop is None else (w.inop[:, :, 0] != sc.UNUSED).sum(axis=1)
    assert ((st[:, 0] & 0xFF) == 0).all()                       # at most f failures: never an error outcome
    first = np.zeros(w.S, dtype=np.int64) if w.roots is None else w.roots.astype(np.int64)
    lead = np.zeros(w.S, dtype=np.int64)
    if w.collective == "allreduce":
        alive = np.ones(w.S, dtype=bool)
        for a in range(f + 1):
            c = (first + a) % P
            dead = ((w.prefail[np.arange(w.S), c >> 5] >> (c & 31).astype(np.uint32)) & 1).astype(bool)
            lead += (alive & dead)
            alive &= dead
        assert np.array_equal((st[:, 0] >> 16) & 0xFF, lead + 1)             # one attempt per dead leading candidate
        assert np.array_equal(st[:, 3], P - npre - nvic)                     # everybody alive at the end holds the value
    incl_vic = np.array([bin(v).count("1") for v in st[:, 2]])
    assert np.array_equal(st[:, 1], P - npre - nvic + incl_vic)
    assert (((st[:, 0] >> 8) & 0xFF) <= f).all()


def test_config4_full_batch():
    import torch
    w, sched, d_x, d_out, st = run_full("c4")
    sample_against_oracle(w, d_out, st, 24, 4)
    check_status_fields(w, sched, st)
    es, ep = excluded_lists(w, st)
    x2 = d_x.clone()
    x2[torch.from_numpy(es).cuda(), torch.from_numpy(ep).cuda()] = torch.iinfo(torch.int32).min
    assert torch.equal(x2.amax(dim=1), d_out)                               # max over exactly the included processes
    assert len(es) > 1000


def test_config5_full_batch():
    import torch
    w, sched, d_x, d_out, st = run_full("c5")
    sample_against_oracle(w, d_out, st, 4, 5)
    check_status_fields(w, sched, st)
    es, ep = excluded_lists(w, st)
    total = d_x.view(torch.int64).sum(dim=1)                                # wraps mod 2^64 like the method's sum
    es_t, ep_t = torch.from_numpy(es).cuda(), torch.from_numpy(ep).cuda()
    total.index_add_(0, es_t, -d_x.view(torch.int64)[es_t, ep_t])
    assert torch.equal(total, d_out.view(torch.int64))


def test_config3_full_batch_float32():
    import torch
    w, sched, d_x, d_out, st = run_full("c3")
    sample_against_oracle(w, d_out, st, 48, 3)
    check_status_fields(w, sched, st)
    es, ep = excluded_lists(w, st)
    es_t, ep_t = torch.from_numpy(es).cuda(), torch.from_numpy(ep).cuda()
    tol = 1e-6 * 10                                                         # 1e-6 * ceil(log2 1024), relative to sum |x|
    worst = 0.0
    for s0 in range(0, w.S, 32768):
        sl = slice(s0, s0 + 32768)
        xd = d_x[sl].double()
        ref, mag = xd.sum(dim=1), xd.abs().sum(dim=1)
        sel = (es_t >= s0) & (es_t < s0 + 32768)
        ref.index_add_(0, es_t[sel] - s0, -d_x[es_t[sel], ep_t[sel]].double())
        err = ((d_out[sl].double() - ref).abs() / mag).max().item()
        worst = max(worst, err)
    assert worst <= tol, worst
