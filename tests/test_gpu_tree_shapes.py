"""GPU parity for subtree shapes other than the binary heap: a-ary heaps (FTC_TREE_ARITY) and binomial trees
(FTC_TREE_BINOMIAL) below the root's children, through every entry point, against the CPU oracle playing the same shape."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2602_22445_b200 import binding as B
from paper_2602_22445_b200 import scenarios as sc
from tests.gpu_util import assert_same, run_gpu, run_oracle, to_dev, to_host

pytestmark = pytest.mark.gpu

ARITIES = [3, 4, 7, 1]            # 1 stands for the binomial tree (the oracle's code for it)


def shape_flags(arity):
    return B.FTC_TREE_BINOMIAL if arity == 1 else B.FTC_TREE_ARITY(arity)


def random_case(rng, S, P, f, k, dtype, allreduce, arity):
    x = rng.standard_normal((S, P, k)).astype(np.float32) if dtype == np.float32 else \
        rng.integers(0, 2**63 - 1, size=(S, P, k)).astype(dtype)
    pf = sc.picks_to_masks(sc.random_subsets(rng, S, P, rng.integers(0, f + 3, size=S)), P)
    R = O.schedule(P, f, arity)["rounds_attempt"]
    inop = np.zeros((S, 2, 2), dtype=np.uint32)
    inop[:, :, 0] = rng.integers((f + 1) if allreduce else 0, P, size=(S, 2))
    inop[:, :, 1] = rng.integers(0, R + 3, size=(S, 2))
    inop[rng.random((S, 2)) < 0.3, 0] = sc.UNUSED
    roots = (np.zeros(S) if allreduce else rng.integers(0, P, size=S)).astype(np.uint32)
    return x, pf, inop, roots


@pytest.mark.parametrize("arity", ARITIES)
@pytest.mark.parametrize("allreduce", [False, True])
def test_exhaustive_failure_sets_small_P(arity, allreduce):
    rng = np.random.Generator(np.random.PCG64(50 + arity))
    for f in (0, 1, 2, 3):
        for P in (f + 2, 9, 14, 23):
            if P < f + 2:
                continue
            sets = sc.all_failure_sets(P, min(f + 1, 2))
            roots = rng.integers(0, P, size=len(sets)).astype(np.uint32)
            x = rng.integers(0, 2**64, size=(len(sets), P, 2), dtype=np.uint64)
            pf = sc.sets_to_masks(sets, P)
            got = run_gpu(x, f, "sum", pf, None, roots, 0, allreduce, shape_flags(arity))
            assert B.ftc_kernel_name(got[2], allreduce) == "levels"
            want = run_oracle(x, f, "sum", pf, None, roots, 0, allreduce, arity)
            assert_same(got, want, f"P={P} f={f} arity={arity}")


@pytest.mark.parametrize("arity", ARITIES)
@pytest.mark.parametrize("allreduce", [False, True])
def test_exhaustive_inop_victim_and_round(arity, allreduce):
    for P, f in ((11, 2), (20, 1), (29, 3)):
        R = O.schedule(P, f, arity)["rounds_attempt" if allreduce else "rounds_reduce"]
        cases = [(pre, v, t) for v in range(P) for t in range(0, R + 2) for pre in ((), ((v + 3) % P,))]
        S = len(cases)
        x = np.random.Generator(np.random.PCG64(P)).integers(0, 2**64, size=(S, P, 2), dtype=np.uint64)
        pf = sc.sets_to_masks([c[0] for c in cases], P)
        inop = np.zeros((S, 1, 2), dtype=np.uint32)
        inop[:, 0, 0] = [c[1] for c in cases]
        inop[:, 0, 1] = [c[2] for c in cases]
        got = run_gpu(x, f, "sum", pf, inop, None, 0, allreduce, shape_flags(arity))
        want = run_oracle(x, f, "sum", pf, inop, None, 0, allreduce, arity)
        assert_same(got, want, f"P={P} f={f} arity={arity}")


@pytest.mark.parametrize("arity", [3, 5, 1])
def test_configuration_shapes(arity):
    """Samples of the large configurations on the other shapes: float32 bit for bit, in-operation failures,
    per-scenario roots at P = 65536."""
    w = sc.config3(S=64)
    x = w.host_inputs()
    got = run_gpu(x, w.f, w.op, w.prefail, None, None, 0, True, shape_flags(arity))
    assert_same(got, run_oracle(x, w.f, w.op, w.prefail, None, None, 0, True, arity), f"C3 arity={arity}")
    w = sc.config4(O.schedule(4096, 4, arity)["rounds_attempt"], S=24)
    x = w.host_inputs()
    got = run_gpu(x, w.f, w.op, w.prefail, w.inop, None, 0, True, shape_flags(arity))
    assert_same(got, run_oracle(x, w.f, w.op, w.prefail, w.inop, None, 0, True, arity), f"C4 arity={arity}")
    for coll in ("reduce", "allreduce"):
        w = sc.config5(coll, "sum", S=3)
        x = w.host_inputs()
        got = run_gpu(x, w.f, w.op, w.prefail, None, w.roots, 0, coll == "allreduce", shape_flags(arity))
        assert_same(got, run_oracle(x, w.f, w.op, w.prefail, None, w.roots, 0, coll == "allreduce", arity), f"C5 {coll}")


@pytest.mark.parametrize("arity", ARITIES)
def test_expanded_candidates_messages_and_noalloc(arity):
    import torch
    rng = np.random.Generator(np.random.PCG64(300 + arity))
    flags = shape_flags(arity)
    for P, f, k, dtype in ((10, 2, 4, np.uint64), (41, 1, 3, np.float32), (130, 3, 2, np.int32)):
        S = 50
        for allreduce in (False, True):
            x, pf, inop, roots = random_case(rng, S, P, f, k, dtype, allreduce, arity)
            d_x = to_dev(x)
            ref = [O.run(x[i], f, "sum", pf[i], inop=[tuple(e) for e in inop[i]], root=int(roots[i]), allreduce=allreduce,
                         detail=True, arity=arity) for i in range(S)]
            # every root child's delivery
            desc = B.make_desc(P, f, k, B.dtype_code(d_x.dtype), "sum", root=-1, max_inop=2, flags=flags)
            d_cand = torch.zeros((S, f + 1, k), dtype=d_x.dtype, device="cuda")
            d_info = torch.zeros((S, f + 1, 2), dtype=torch.int32, device="cuda")
            d_ws = torch.empty(B.ftc_candidates_workspace_bytes(desc, S), dtype=torch.uint8, device="cuda")
            B.ftc_candidates_batch(desc, S, allreduce, d_x, to_dev(pf), to_dev(inop), to_dev(roots), d_cand, d_info, d_ws)
            # message counts
            d_msgs = torch.zeros((S, B.FTC_MSG_WORDS), dtype=torch.int64, device="cuda")
            B.ftc_message_counts_batch(desc, S, allreduce, to_dev(pf), to_dev(inop), to_dev(roots), d_msgs.view(torch.uint64))
            torch.cuda.synchronize()
            cand, info, msgs = to_host(d_cand, x.dtype), d_info.cpu().numpy(), d_msgs.cpu().numpy().view(np.uint64)
            for i, d in enumerate(ref):
                assert np.array_equal(msgs[i], d["msgs"]), (P, f, i, msgs[i], d["msgs"])
                if d["attempts"] == 0:
                    continue
                assert np.array_equal(info[i, :, 0], d["cand_flag"]) and np.array_equal(info[i, :, 1], d["cand_nfail"]), (P, f, i)
                assert np.array_equal(cand[i].view(np.uint8), d["cand"].view(np.uint8)), (P, f, i)
            if allreduce:
                # expanded output: the value in every holder's slot
                desc_e = B.make_desc(P, f, k, B.dtype_code(d_x.dtype), "sum", root=-1, max_inop=2, flags=flags | B.FTC_OUT_EXPANDED)
                d_out = torch.zeros((S, P, k), dtype=d_x.dtype, device="cuda")
                d_st = torch.zeros((S, 4), dtype=torch.int32, device="cuda")
                d_ws = torch.empty(B.ftc_workspace_bytes(desc_e, S, True), dtype=torch.uint8, device="cuda")
                B.ftc_allreduce_batch(desc_e, S, d_x, to_dev(pf), to_dev(inop), to_dev(roots), d_out, d_st, d_ws)
                torch.cuda.synchronize()
                out, st = to_host(d_out, x.dtype), d_st.cpu().numpy().view(np.uint32)
                for i, d in enumerate(ref):
                    assert np.array_equal(st[i], d["status"]), (P, i)
                    assert np.array_equal(out[i].view(np.uint8), d["expanded"].view(np.uint8)), (P, f, i)
            else:
                # the entry point that brings its own scratch
                d_out = torch.zeros((S, k), dtype=d_x.dtype, device="cuda")
                d_st = torch.zeros((S, 4), dtype=torch.int32, device="cuda")
                B.ftc_reduce_batch_noalloc(desc, S, d_x, to_dev(pf), to_dev(inop), to_dev(roots), d_out, d_st)
                torch.cuda.synchronize()
                out, st = to_host(d_out, x.dtype), d_st.cpu().numpy().view(np.uint32)
                for i, d in enumerate(ref):
                    assert np.array_equal(st[i], d["status"]) and np.array_equal(out[i].view(np.uint8), d["result"].view(np.uint8)), (P, i)


def test_arity_in_the_descriptor():
    import torch
    z = torch.zeros(4096, dtype=torch.int32, device="cuda")
    for bad in (1, 33, 255):
        d = B.make_desc(8, 1, 4, B.FTC_I32, "sum", flags=B.FTC_TREE_ARITY(bad))
        assert B.ftc_reduce_batch(d, 1, z, z, None, None, z, z, z, check=False) == B.FTC_EINVAL
    both = B.make_desc(8, 1, 4, B.FTC_I32, "sum", flags=B.FTC_TREE_ARITY(3) | B.FTC_TREE_BINOMIAL)
    assert B.ftc_reduce_batch(both, 1, z, z, None, None, z, z, z, check=False) == B.FTC_EINVAL
    assert B.ftc_schedule_info(B.make_desc(65536, 8, 4, B.FTC_U64, "sum", flags=B.FTC_TREE_BINOMIAL))["H"] == O.schedule(65536, 8, 1)["H"]
    d2 = B.make_desc(4096, 4, 32, B.FTC_I32, "max", flags=B.FTC_TREE_ARITY(2))
    assert B.ftc_kernel_name(d2, True) == "staged"                       # 2 is the default shape
    assert B.ftc_schedule_info(B.make_desc(65536, 8, 4, B.FTC_U64, "sum", flags=B.FTC_TREE_ARITY(3)))["H"] == O.schedule(65536, 8, 3)["H"]


# ---------------------------------------------------------------------------------------------
# the other partner order (FTC_PARTNERS_DESCENDING), alone and together with another subtree shape
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("arity", [2, 3, 1])
@pytest.mark.parametrize("allreduce", [False, True])
def test_descending_partners(arity, allreduce):
    flags = B.FTC_PARTNERS_DESCENDING | (0 if arity == 2 else shape_flags(arity))
    rng = np.random.Generator(np.random.PCG64(900 + arity))
    # every (victim, round), alone and beside one pre-operation failure: the order decides whom a dying process reached
    for P, f in ((6, 2), (11, 2), (20, 1), (29, 3)):
        R = O.schedule(P, f, arity)["rounds_attempt" if allreduce else "rounds_reduce"]
        cases = [(pre, v, t) for v in range(P) for t in range(0, R + 2) for pre in ((), ((v + 3) % P,))]
        S = len(cases)
        x = rng.integers(0, 2**64, size=(S, P, 2), dtype=np.uint64)
        pf = sc.sets_to_masks([c[0] for c in cases], P)
        inop = np.zeros((S, 1, 2), dtype=np.uint32)
        inop[:, 0, 0] = [c[1] for c in cases]
        inop[:, 0, 1] = [c[2] for c in cases]
        got = run_gpu(x, f, "sum", pf, inop, None, 0, allreduce, flags)
        assert B.ftc_kernel_name(got[2], allreduce) == {2: "staged", 3: "levels", 1: "levels"}[arity]    # the order is known to the shared-memory kernels
        assert_same(got, run_oracle(x, f, "sum", pf, inop, None, 0, allreduce, arity, True), f"P={P} f={f} arity={arity}")
    # float32 bit for bit, random failures and roots, expanded output and message counts
    import torch
    for P, f, k in ((41, 3, 4), (130, 2, 16), (1024, 3, 16)):
        S = 40
        x, pf, inop, roots = random_case(rng, S, P, f, k, np.float32, allreduce, arity)
        got = run_gpu(x, f, "sum", pf, inop, roots, 0, allreduce, flags)
        assert_same(got, run_oracle(x, f, "sum", pf, inop, roots, 0, allreduce, arity, True), f"f32 P={P} f={f} arity={arity}")
        desc = B.make_desc(P, f, k, B.FTC_F32, "sum", root=-1, max_inop=2, flags=flags)
        d_msgs = torch.zeros((S, B.FTC_MSG_WORDS), dtype=torch.int64, device="cuda")
        B.ftc_message_counts_batch(desc, S, allreduce, to_dev(pf), to_dev(inop), to_dev(roots), d_msgs.view(torch.uint64))
        torch.cuda.synchronize()
        msgs = d_msgs.cpu().numpy().view(np.uint64)
        ref = [O.run(x[i], f, "sum", pf[i], inop=[tuple(e) for e in inop[i]], root=int(roots[i]), allreduce=allreduce, detail=True,
                     arity=arity, partners_descending=True) for i in range(S)]
        d_cand = torch.zeros((S, f + 1, k), dtype=torch.float32, device="cuda")
        d_info = torch.zeros((S, f + 1, 2), dtype=torch.int32, device="cuda")
        d_cws = torch.empty(B.ftc_candidates_workspace_bytes(desc, S), dtype=torch.uint8, device="cuda")
        B.ftc_candidates_batch(desc, S, allreduce, to_dev(x), to_dev(pf), to_dev(inop), to_dev(roots), d_cand, d_info, d_cws)
        torch.cuda.synchronize()
        cand, info = d_cand.cpu().numpy(), d_info.cpu().numpy()
        for i, d in enumerate(ref):
            assert np.array_equal(msgs[i], d["msgs"]), (P, f, i)
            if d["attempts"]:
                assert np.array_equal(info[i, :, 0], d["cand_flag"]) and np.array_equal(info[i, :, 1], d["cand_nfail"]), (P, f, i)
                assert np.array_equal(cand[i].view(np.uint8), d["cand"].view(np.uint8)), (P, f, i)
        if allreduce:
            desc_e = B.make_desc(P, f, k, B.FTC_F32, "sum", root=-1, max_inop=2, flags=flags | B.FTC_OUT_EXPANDED)
            d_out = torch.zeros((S, P, k), dtype=torch.float32, device="cuda")
            d_st = torch.zeros((S, 4), dtype=torch.int32, device="cuda")
            d_ws = torch.empty(B.ftc_workspace_bytes(desc_e, S, True), dtype=torch.uint8, device="cuda")
            B.ftc_allreduce_batch(desc_e, S, to_dev(x), to_dev(pf), to_dev(inop), to_dev(roots), d_out, d_st, d_ws)
            torch.cuda.synchronize()
            out, st = d_out.cpu().numpy(), d_st.cpu().numpy().view(np.uint32)
            for i, d in enumerate(ref):
                assert np.array_equal(st[i], d["status"]) and np.array_equal(out[i].view(np.uint8), d["expanded"].view(np.uint8)), (P, i)
