"""GPU parity of the failed-process list (ftc_failed_list_batch; first and second scheme of section "Failure
information") against the CPU oracle, whose processes append ids to their lists one by one and hand them up the
tree: the bitmask over process ids and its size, for random failure patterns (more than f failures too), every
(victim, round) of one in-operation failure, the other partner order and subtree shapes, and samples of the
configurations. On the full batches: the size equals P minus the included count of the status record."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2602_22445_b200 import binding as B
from paper_2602_22445_b200 import scenarios as sc
from tests.gpu_util import run_gpu, to_dev

pytestmark = pytest.mark.gpu


def gpu_lists(P, f, allreduce, prefail, inop=None, roots=None, root=0, flags=0):
    import torch
    S, W = prefail.shape[0], (P + 31) // 32
    max_inop = 0 if inop is None else inop.shape[1]
    desc = B.make_desc(P, f, 1, B.FTC_I32, "sum", root=-1 if roots is not None else root, max_inop=max_inop, flags=flags)
    d_failed = torch.full((S, W), -1, dtype=torch.int32, device="cuda")
    d_nfail = torch.full((S,), -1, dtype=torch.int32, device="cuda")
    B.ftc_failed_list_batch(desc, S, allreduce, to_dev(np.ascontiguousarray(prefail, dtype=np.uint32)),
                            to_dev(np.ascontiguousarray(inop, dtype=np.uint32)) if max_inop else None,
                            to_dev(np.ascontiguousarray(roots, dtype=np.uint32)) if roots is not None else None,
                            d_failed, d_nfail)
    torch.cuda.synchronize()
    return d_failed.cpu().numpy().view(np.uint32), d_nfail.cpu().numpy().view(np.uint32)


def oracle_lists(P, f, allreduce, prefail, inop=None, roots=None, root=0, track=True, **kw):
    S, W = prefail.shape[0], (P + 31) // 32
    x = np.zeros((P, 1), dtype=np.int32)
    failed, nfail = np.zeros((S, W), dtype=np.uint32), np.zeros(S, dtype=np.uint32)
    for i in range(S):
        d = O.run(x, f, "sum", prefail[i], inop=None if inop is None else inop[i],
                  root=int(roots[i]) if roots is not None else root, allreduce=allreduce, detail=True, track_sets=track, **kw)
        nfail[i] = d["nfail"][0]
        if track:
            failed[i] = d["failed"]
    return failed, nfail


def assert_lists(got, want, what):
    bad = np.nonzero((got[0] != want[0]).any(axis=1) | (got[1] != want[1]))[0]
    assert bad.size == 0, f"{what}: scenarios {bad[:6]}: gpu {got[0][bad[:2]]} {got[1][bad[:3]]} oracle {want[0][bad[:2]]} {want[1][bad[:3]]}"


def random_patterns(rng, P, f, S, allreduce):
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
    return pf, inop, roots


@pytest.mark.parametrize("allreduce", [False, True])
def test_random_patterns(allreduce):
    rng = np.random.Generator(np.random.PCG64(311 + allreduce))
    seen_sizes = set()
    for f in range(0, 5):
        for P in (f + 2, f + 3, 9, 17, 33, 64, 100, 333):
            if P < f + 2:
                continue
            pf, inop, roots = random_patterns(rng, P, f, 120, allreduce)
            got = gpu_lists(P, f, allreduce, pf, inop, roots)
            want = oracle_lists(P, f, allreduce, pf, inop, roots)
            assert_lists(got, want, f"P={P} f={f} allreduce={allreduce}")
            assert np.array_equal(got[1], np.unpackbits(got[0].view(np.uint8), axis=1).sum(axis=1))   # duplicate-free
            seen_sizes |= set(got[1].tolist())
    assert {0, 1, 2, 3} <= seen_sizes


def test_exhaustive_victim_and_round():
    for P, f in ((7, 1), (11, 2), (14, 3), (22, 2)):
        for allreduce in (False, True):
            R = O.schedule(P, f)["rounds_attempt" if allreduce else "rounds_reduce"]
            cases = [(pre, v, t) for v in range(P) for t in range(0, 2 * R + 2) for pre in ((), ((v + 3) % P,), (0,))]
            pf = sc.sets_to_masks([c[0] for c in cases], P)
            inop = np.full((len(cases), 1, 2), sc.UNUSED, dtype=np.uint32)
            inop[:, 0, 0] = [c[1] for c in cases]
            inop[:, 0, 1] = [c[2] for c in cases]
            assert_lists(gpu_lists(P, f, allreduce, pf, inop), oracle_lists(P, f, allreduce, pf, inop), f"P={P} f={f} allreduce={allreduce}")


@pytest.mark.parametrize("flags,kw", [(B.FTC_PARTNERS_DESCENDING, dict(partners_descending=True)),
                                      (B.FTC_TREE_ARITY(3), dict(arity=3)), (B.FTC_TREE_BINOMIAL, dict(arity=1))])
def test_other_partner_order_and_subtree_shapes(flags, kw):
    rng = np.random.Generator(np.random.PCG64(5))
    for P, f in ((23, 2), (64, 3), (130, 4)):
        pf, inop, roots = random_patterns(rng, P, f, 100, False)
        assert_lists(gpu_lists(P, f, False, pf, inop, roots, flags=flags), oracle_lists(P, f, False, pf, inop, roots, **kw), f"P={P} f={f} {kw}")


def test_configurations():
    w = sc.config2()
    ids = np.arange(0, w.S, 16 * 11)
    assert_lists(gpu_lists(w.P, w.f, False, w.prefail[ids]), oracle_lists(w.P, w.f, False, w.prefail[ids]), "C2")
    w = sc.config3(S=64)
    assert_lists(gpu_lists(w.P, w.f, True, w.prefail), oracle_lists(w.P, w.f, True, w.prefail), "C3")
    w = sc.config4(O.schedule(4096, 4)["rounds_attempt"], S=40)
    assert_lists(gpu_lists(w.P, w.f, True, w.prefail, w.inop), oracle_lists(w.P, w.f, True, w.prefail, w.inop), "C4")
    w = sc.config5("allreduce", "sum", S=6)                     # sizes only: the oracle's id sets would take P*P bits
    got = gpu_lists(w.P, w.f, True, w.prefail, None, w.roots)
    want = oracle_lists(w.P, w.f, True, w.prefail, None, w.roots, track=False)
    assert np.array_equal(got[1], want[1])
    assert np.array_equal(got[0], w.prefail)                    # pre-operation failures only: the list is the failure set


def test_full_batch_sizes_agree_with_the_status_records():
    """P=4096 configuration, 16384 scenarios: the list's size is P minus the included count of the batch call's status
    record, the list holds every pre-failed process, and beyond those only in-operation victims."""
    w = sc.config4(O.schedule(4096, 4)["rounds_attempt"], S=1 << 14)
    got_failed, got_n = gpu_lists(w.P, w.f, True, w.prefail, w.inop)
    import torch
    d_x = torch.zeros((w.S, w.P, 4), dtype=torch.int32, device="cuda")
    _, st, _ = run_gpu(None, w.f, "max", w.prefail, w.inop, None, 0, True, 0, d_x=d_x)
    assert ((st[:, 0] & 0xFF) == 0).all()
    assert np.array_equal(got_n, w.P - st[:, 1])
    assert not (w.prefail & ~got_failed).any()
    extra = got_failed & ~w.prefail
    vic = np.zeros_like(extra)
    for slot in range(w.inop.shape[1]):
        v = w.inop[:, slot, 0]
        use = v != sc.UNUSED
        vic[np.nonzero(use)[0], v[use] >> 5] |= (np.uint32(1) << (v[use] & 31).astype(np.uint32))
    assert not (extra & ~vic).any() and extra.any()
