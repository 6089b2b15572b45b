"""GPU parity of the message accounting (ftc_message_counts_batch) against the CPU oracle's counters, which
count every send the simulated processes perform; plus the closed forms of the theorem on the number of messages
and the (f+1)-fold bound of the allreduce theorem at full batch size."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2602_22445_b200 import binding as B
from paper_2602_22445_b200 import scenarios as sc
from tests.gpu_util import to_dev, to_host

pytestmark = pytest.mark.gpu


def gpu_counts(P, f, allreduce, prefail, inop=None, roots=None, root=0):
    import torch
    S = prefail.shape[0]
    max_inop = 0 if inop is None else inop.shape[1]
    desc = B.make_desc(P, f, 1, B.FTC_I32, "sum", root=-1 if roots is not None else root, max_inop=max_inop)
    d_msgs = torch.full((S, B.FTC_MSG_WORDS), -1, dtype=torch.int64, device="cuda")
    B.ftc_message_counts_batch(desc, S, allreduce, to_dev(np.ascontiguousarray(prefail, dtype=np.uint32)),
                               to_dev(np.ascontiguousarray(inop, dtype=np.uint32)) if max_inop else None,
                               to_dev(np.ascontiguousarray(roots, dtype=np.uint32)) if roots is not None else None,
                               d_msgs.view(torch.uint64))
    torch.cuda.synchronize()
    return to_host(d_msgs.view(torch.uint64), np.uint64)


def oracle_counts(P, f, allreduce, prefail, inop=None, roots=None, root=0):
    S = prefail.shape[0]
    x = np.zeros((P, 1), dtype=np.int32)
    out = np.zeros((S, 8), dtype=np.uint64)
    for i in range(S):
        d = O.run(x, f, "sum", prefail[i], inop=None if inop is None else inop[i],
                  root=int(roots[i]) if roots is not None else root, allreduce=allreduce, detail=True)
        out[i] = d["msgs"]
    return out


def assert_counts(got, want, what):
    bad = np.nonzero((got != want).any(axis=1))[0]
    assert bad.size == 0, f"{what}: scenarios {bad[:6]}: gpu {got[bad[:3]]} oracle {want[bad[:3]]}"


def closed_forms(P, f):
    m, q, r = f + 1, (P - 1) // (f + 1), (P - 1) % (f + 1)
    return f * m * q + (r + 1) * r, P - 1


@pytest.mark.parametrize("allreduce", [False, True])
def test_random_patterns_small_P(allreduce):
    """Random pre- and in-operation failures (more than f of them as well), random roots, in-operation victims
    that may be root candidates (nothing is played then)."""
    rng = np.random.Generator(np.random.PCG64(77 + allreduce))
    for f in range(0, 5):
        for P in (f + 2, f + 3, 9, 17, 33, 64, 100):
            if P < f + 2:
                continue
            S = 160
            ratt = O.schedule(P, f)["rounds_attempt"]
            sets = [tuple(rng.choice(P, size=min(int(rng.integers(0, f + 3)), P), replace=False)) for _ in range(S)]
            pf = sc.sets_to_masks(sets, P)
            roots = rng.integers(0, P, size=S).astype(np.uint32)
            inop = np.full((S, 3, 2), sc.UNUSED, dtype=np.uint32)
            for i in range(S):
                for j in range(int(rng.integers(0, 4))):
                    v = int(rng.integers(0, P))
                    if allreduce and rng.random() < 0.85 and P > 2 * (f + 1):
                        while (v - int(roots[i])) % P <= f:
                            v = int(rng.integers(0, P))
                    inop[i, j] = (v, int(rng.integers(0, (f + 1) * ratt + 3)))
            got = gpu_counts(P, f, allreduce, pf, inop, roots)
            want = oracle_counts(P, f, allreduce, pf, inop, roots)
            assert_counts(got, want, f"P={P} f={f} allreduce={allreduce}")


def test_exhaustive_victim_and_round():
    """Every (victim, round) of one in-operation failure, alone and beside one pre-operation failure."""
    for P, f in ((7, 1), (11, 2), (14, 3), (22, 2)):
        for allreduce in (False, True):
            R = O.schedule(P, f)["rounds_attempt" if allreduce else "rounds_reduce"]
            cases = [(pre, v, t) for v in range(P) for t in range(0, 2 * R + 2) for pre in ((), ((v + 3) % P,), (0,))]
            pf = sc.sets_to_masks([c[0] for c in cases], P)
            inop = np.full((len(cases), 1, 2), sc.UNUSED, dtype=np.uint32)
            inop[:, 0, 0] = [c[1] for c in cases]
            inop[:, 0, 1] = [c[2] for c in cases]
            got = gpu_counts(P, f, allreduce, pf, inop)
            want = oracle_counts(P, f, allreduce, pf, inop)
            assert_counts(got, want, f"P={P} f={f} allreduce={allreduce}")


def test_configurations_against_oracle():
    w = sc.config1()
    assert_counts(gpu_counts(w.P, w.f, False, w.prefail), oracle_counts(w.P, w.f, False, w.prefail), "C1")
    w = sc.config2()
    ids = np.arange(0, w.S, 16 * 7)
    assert_counts(gpu_counts(w.P, w.f, False, w.prefail[ids]), oracle_counts(w.P, w.f, False, w.prefail[ids]), "C2")
    w = sc.config3(S=96)
    assert_counts(gpu_counts(w.P, w.f, True, w.prefail), oracle_counts(w.P, w.f, True, w.prefail), "C3")
    w = sc.config4(O.schedule(4096, 4)["rounds_attempt"], S=48)
    assert_counts(gpu_counts(w.P, w.f, True, w.prefail, w.inop), oracle_counts(w.P, w.f, True, w.prefail, w.inop), "C4")
    for coll in ("reduce", "allreduce"):
        w = sc.config5(coll, "sum", S=6)
        allred = coll == "allreduce"
        assert_counts(gpu_counts(w.P, w.f, allred, w.prefail, None, w.roots),
                      oracle_counts(w.P, w.f, allred, w.prefail, None, w.roots), f"C5 {coll}")


@pytest.mark.parametrize("name", ["c3", "c4", "c5"])
def test_full_batches_closed_forms_and_bound(name):
    """At the batch sizes the benchmark runs: failure-free scenarios send exactly the closed-form numbers, reduce
    and broadcast alike; no scenario sends more per attempt; all attempts together stay within (f+1) times one
    failure-free allreduce; the attempt count of the status record and of the message counts agree."""
    if name == "c3":
        w = sc.config3(S=1 << 16)
    elif name == "c4":
        w = sc.config4(O.schedule(4096, 4)["rounds_attempt"], S=1 << 14)
    else:
        w = sc.config5("allreduce", "sum", S=1 << 12)
    got = gpu_counts(w.P, w.f, True, w.prefail, w.inop, w.roots, max(w.root, 0)).astype(np.int64)
    uc0, tree0 = closed_forms(w.P, w.f)
    one = np.array([uc0, tree0, tree0, uc0], dtype=np.int64)
    nfail = np.unpackbits(w.prefail.view(np.uint8), axis=1).sum(axis=1)
    if w.inop is not None:
        nfail = nfail + (w.inop[:, :, 0] != sc.UNUSED).sum(axis=1)
    free = nfail == 0
    assert free.sum() > 0
    assert (got[free, 4:] == one).all() and (got[free, :4] == one).all()
    assert (got[:, 4:] <= one).all()
    assert (got[:, :4] <= (w.f + 1) * one).all()
    # every attempt before the last one is a reduce toward a dead candidate: between one and f of them
    extra = got[:, 0] - got[:, 4]
    assert ((extra == 0) | (got[:, 1] - got[:, 5] > 0)).all()
    assert (got[~free, 4:].sum(axis=1) < one.sum()).all()        # a failed process always costs at least one message
