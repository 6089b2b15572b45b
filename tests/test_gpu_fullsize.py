"""Parity at the full sizes and in the launch configuration bench.py times (same entry point, same batch size,
device-generated inputs): sampled scenarios against the CPU oracle bit for bit, and every scenario of the batch
against properties that hold at any size (paper_2602_22445_b200.verify: status fields derived from the masks; the
result equals a reduction that torch computes over exactly the processes the status record claims to be included)."""
import numpy as np
import pytest

import bench
from oracle import oracle as O
from paper_2602_22445_b200 import binding as B
from paper_2602_22445_b200 import scenarios as sc

pytestmark = pytest.mark.gpu


def run_full(name, flags=0, arity=2):
    import torch
    S = bench.DEFAULT_BATCH[name]
    sched = O.schedule(*{"c3": (1024, 3), "c4": (4096, 4), "c5": (65536, 8), "c5r": (65536, 8)}[name], arity)     # in-operation rounds are drawn within an attempt of this shape
    w = bench.make_workload(name, S, 0, sched["rounds_attempt"])
    tdt = getattr(torch, np.dtype(w.dtype).name)
    allred = w.collective == "allreduce"
    desc = B.make_desc(w.P, w.f, w.k, B.dtype_code(tdt), w.op, root=-1 if w.roots is not None else 0,
                       max_inop=0 if w.inop is None else w.inop.shape[1], flags=flags)
    d_x = torch.empty((S, w.P, w.k), dtype=tdt, device="cuda")
    B.ftc_fill_inputs(w.kind, w.seed, 0, S, w.P, w.k, d_x)
    d_pf, d_inop, d_roots = bench.upload(w, torch)
    d_out = torch.empty((S, w.k), dtype=tdt, device="cuda")
    d_st = torch.empty((S, 4), dtype=torch.int32, device="cuda")
    fn = B.ftc_allreduce_batch if allred else B.ftc_reduce_batch
    fn(desc, S, d_x, d_pf, d_inop, d_roots, d_out, d_st, None)
    torch.cuda.synchronize()
    st = d_st.cpu().numpy().view(np.uint32)
    return w, sched, d_x, d_out, st, B.ftc_kernel_name(desc, allred)


def want_dtype(w):
    return np.dtype(w.dtype)


def sample_against_oracle(w, d_out, st, n, seed, arity=2):
    import torch
    rng = np.random.Generator(np.random.PCG64(seed))
    npre = np.unpackbits(w.prefail.view(np.uint8), axis=1).sum(axis=1)
    interesting = np.nonzero(npre > 0)[0]
    idx = np.unique(np.concatenate([rng.choice(w.S, n // 2, replace=False), rng.choice(interesting, n // 2, replace=False)]))
    x = w.host_inputs(idx)
    want_out, want_st = O.batch(x, w.f, w.op, w.prefail[idx], None if w.inop is None else w.inop[idx],
                                None if w.roots is None else w.roots[idx], max(w.root, 0), w.collective == "allreduce", arity)
    d_sel = d_out.view(torch.int64) if d_out.dtype == torch.uint64 else d_out      # torch cannot index uint64
    got = d_sel[torch.from_numpy(idx).cuda()].cpu().numpy().view(want_dtype(w))
    assert np.array_equal(st[idx], want_st), "status differs from the oracle on sampled scenarios"
    assert np.array_equal(got.view(np.uint8), want_out.view(np.uint8)), "result differs from the oracle on sampled scenarios"


@pytest.mark.parametrize("name,n_sample", [("c4", 24), ("c5", 4), ("c5r", 4), ("c3", 48)])
def test_full_batch(name, n_sample):
    from paper_2602_22445_b200 import verify
    w, sched, d_x, d_out, st, _ = run_full(name)
    sample_against_oracle(w, d_out, st, n_sample, len(name) + n_sample)
    counts = verify.check_status_fields(w, st)
    rep = verify.check_results_by_definition(w, d_x, d_out, st)
    assert rep["excluded_pairs"] > 1000 and counts["ok_scenarios"] > w.S * 0.99
    if name == "c5r":
        assert counts["noop_scenarios"] >= 0 and counts["ok_scenarios"] + counts["noop_scenarios"] == w.S


@pytest.mark.parametrize("name,arity,n_sample", [("c4", 4, 16), ("c4", 1, 16), ("c3", 3, 32), ("c5", 1, 4)])
def test_full_batch_other_subtree_shapes(name, arity, n_sample):
    """The same batches with a-ary heaps or binomial trees (arity 1, the oracle's code for them) below the root's children:
    the level kernel in the launch configuration the bench's legs time."""
    from paper_2602_22445_b200 import verify
    w, sched, d_x, d_out, st, kernel = run_full(name, B.FTC_TREE_BINOMIAL if arity == 1 else B.FTC_TREE_ARITY(arity), arity)
    assert kernel == "levels"
    sample_against_oracle(w, d_out, st, n_sample, 7 * arity + n_sample, arity)
    counts = verify.check_status_fields(w, st)
    rep = verify.check_results_by_definition(w, d_x, d_out, st)
    assert rep["excluded_pairs"] > 1000 and counts["ok_scenarios"] > w.S * 0.99
