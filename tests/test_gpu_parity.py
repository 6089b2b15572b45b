"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, element by element.

Integer and bitwise results, status records and float32 results are all compared bit for bit (the
schedule fixes the float32 combine order, so no tolerance is needed; the documented fallback tolerance
1e-6*ceil(log2 P) relative to the sum of magnitudes is checked against a float64 sum as well).
"""
import itertools

import numpy as np
import pytest

from oracle import checker as K
from oracle import oracle as O
from paper_2602_22445_b200 import binding as B
from paper_2602_22445_b200 import scenarios as sc
from tests.gpu_util import assert_same, run_gpu, run_oracle, to_dev, to_host

pytestmark = pytest.mark.gpu

KERNELS = [0, B.FTC_KERNEL_DIRECT, B.FTC_KERNEL_GENERIC]


def check_workload(w, idx=None, flags=0, collective=None):
    ids = np.arange(w.S) if idx is None else np.asarray(idx)
    x = w.host_inputs(ids)
    pf = w.prefail[ids]
    inop = None if w.inop is None else w.inop[ids]
    roots = None if w.roots is None else w.roots[ids]
    allred = (collective or w.collective) == "allreduce"
    got = run_gpu(x, w.f, w.op, pf, inop, roots, max(w.root, 0), allred, flags)
    want = run_oracle(x, w.f, w.op, pf, inop, roots, max(w.root, 0), allred)
    assert_same(got, want, f"{w.name} flags={flags:#x}")
    return x, got


@pytest.mark.parametrize("flags", KERNELS)
def test_config1_all_scenarios(flags):
    w = sc.config1()
    x, (out, st, _) = check_workload(w, flags=flags)
    assert (st[:, 0] & 0xFF).tolist() == [0, 1] + [0] * 7       # the set {0} kills the root: no-op


@pytest.mark.parametrize("flags", KERNELS)
def test_config2_all_scenarios(flags):
    w = sc.config2()
    assert w.S == 33296
    x, (out, st, desc) = check_workload(w, flags=flags)
    assert B.ftc_kernel_name(desc) == {0: "staged", B.FTC_KERNEL_DIRECT: "tiled", B.FTC_KERNEL_GENERIC: "generic"}[flags]
    live_ok = (st[:, 0] & 0xFF) == 0
    assert live_ok.sum() == 16 * (2081 - 1 - 63)                 # every set without process 0 succeeds


@pytest.mark.parametrize("flags", KERNELS)
def test_config3_sample_float32_bit_exact(flags):
    w = sc.config3(S=384)
    x, (out, st, _) = check_workload(w, flags=flags)
    for i in range(0, 384, 37):                                   # and within the documented tolerance of float64
        live = [p for p in range(w.P) if not (w.prefail[i, p >> 5] >> (p & 31)) & 1]
        assert K.value_matches(x[i], live, "sum", out[i])
    assert set((st[:, 0] >> 16) & 0xFF) >= {1, 2}                 # some first candidates were dead


@pytest.mark.parametrize("flags", KERNELS)
def test_config4_sample_with_inop_failures(flags):
    ratt = O.schedule(4096, 4)["rounds_attempt"]
    w = sc.config4(ratt, S=96)
    check_workload(w, flags=flags)


@pytest.mark.parametrize("collective,op", [("reduce", "sum"), ("reduce", "xor"), ("allreduce", "sum"), ("allreduce", "xor")])
def test_config5_sample(collective, op):
    w = sc.config5(collective, op, S=12)
    check_workload(w)


@pytest.mark.parametrize("flags", KERNELS[1:])
def test_config5_sample_other_kernels(flags):
    w = sc.config5("allreduce", "sum", S=4)
    check_workload(w, flags=flags)


# ---------------------------------------------------------------------------------------------
# exhaustive small cases and edge cases
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("flags", KERNELS)
@pytest.mark.parametrize("allreduce", [False, True])
def test_exhaustive_failure_sets_small_P(flags, allreduce):
    rng = np.random.Generator(np.random.PCG64(5))
    for f in (0, 1, 2, 3):
        for P in (f + 2, f + 3, 7, 9, 13, 16):
            if P < f + 2:
                continue
            sets = sc.all_failure_sets(P, min(f + 1, 3))          # one more failure than tolerated as well
            roots = rng.integers(0, P, size=len(sets)).astype(np.uint32)
            x = rng.integers(0, 2**64, size=(len(sets), P, 2), dtype=np.uint64)
            pf = sc.sets_to_masks(sets, P)
            got = run_gpu(x, f, "sum", pf, None, roots, 0, allreduce, flags)
            want = run_oracle(x, f, "sum", pf, None, roots, 0, allreduce)
            assert_same(got, want, f"P={P} f={f}")


@pytest.mark.parametrize("flags", KERNELS)
@pytest.mark.parametrize("allreduce", [False, True])
def test_exhaustive_inop_victim_and_round(flags, allreduce):
    """Every (victim, round) with zero or one pre-operation failure."""
    for P, f in ((7, 1), (11, 2), (14, 3)):
        R = O.schedule(P, f)["rounds_attempt" if allreduce else "rounds_reduce"]
        cases = []
        for victim in range(P):
            for t in range(0, 2 * R + 2):
                cases.append(((), victim, t))
                cases.append((((victim + 3) % P,), victim, t))
                cases.append(((0,), victim, t))
        S = len(cases)
        x = np.random.Generator(np.random.PCG64(P)).integers(0, 2**64, size=(S, P, 2), dtype=np.uint64)
        pf = sc.sets_to_masks([c[0] for c in cases], P)
        inop = np.zeros((S, 2, 2), dtype=np.uint32)
        inop[:, 0, 0] = [c[1] for c in cases]
        inop[:, 0, 1] = [c[2] for c in cases]
        inop[:, 1, 0] = sc.UNUSED
        got = run_gpu(x, f, "sum", pf, inop, None, 0, allreduce, flags)
        want = run_oracle(x, f, "sum", pf, inop, None, 0, allreduce)
        assert_same(got, want, f"P={P} f={f}")


DT = {"i32": np.int32, "i64": np.int64, "u64": np.uint64, "f32": np.float32}


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes_ops_and_failure_patterns(seed):
    """Random (P, f, k, dtype, op), up to f+2 pre-operation failures, up to 3 in-operation failures (victims may
    repeat, may be pre-failed, may be the reduce root), per-scenario roots, both collectives, both kernels."""
    rng = np.random.Generator(np.random.PCG64(1000 + seed))
    for _ in range(10):
        f = int(rng.integers(0, 6))
        P = int(rng.integers(f + 2, 400))
        dname = ["i32", "i64", "u64", "f32"][int(rng.integers(0, 4))]
        op = "sum" if dname == "f32" else ["sum", "max", "xor"][int(rng.integers(0, 3))]
        k = int(rng.choice([1, 2, 3, 4, 8, 12, 16, 32, 64, 128] if DT[dname]().itemsize == 4 else [1, 2, 3, 4, 6, 8, 16, 64]))
        S = 40
        allred = bool(rng.integers(0, 2))
        if dname == "f32":
            x = rng.standard_normal((S, P, k)).astype(np.float32)
        else:
            info = np.iinfo(DT[dname])
            x = rng.integers(info.min, info.max, size=(S, P, k), dtype=DT[dname], endpoint=True)
        sizes = rng.integers(0, f + 3, size=S)
        pf = sc.picks_to_masks(sc.random_subsets(rng, S, P, np.minimum(sizes, P - 1)), P)
        R = O.schedule(P, f)["rounds_attempt"]
        inop = np.zeros((S, 3, 2), dtype=np.uint32)
        lo = f + 1 if allred and P > f + 2 else 0
        inop[:, :, 0] = rng.integers(lo, P, size=(S, 3))
        inop[:, :, 1] = rng.integers(0, 2 * R + 2, size=(S, 3))
        inop[rng.random((S, 3)) < 0.4, 0] = sc.UNUSED
        roots = rng.integers(0, P, size=S).astype(np.uint32)
        if allred and lo:
            roots = rng.integers(0, 1, size=S).astype(np.uint32)      # candidates 0..f stay clear of the victims
        for flags in KERNELS:
            got = run_gpu(x, f, op, pf, inop, roots, 0, allred, flags)
            want = run_oracle(x, f, op, pf, inop, roots, 0, allred)
            assert_same(got, want, f"P={P} f={f} k={k} {dname} {op} allreduce={allred} flags={flags:#x}")


def test_chunk_counts_up_to_32_and_beyond():
    """k*elem = 16 B .. 512 B in a power-of-two number of 16-byte chunks run on the staged tiles, other multiples of 16 bytes
    (80 B here) on the level kernel, larger vectors and sizes that are no multiple of 16 bytes on the general one."""
    rng = np.random.Generator(np.random.PCG64(3))
    P, f, S = 300, 2, 16
    pf = sc.picks_to_masks(sc.random_subsets(rng, S, P, rng.integers(0, 3, size=S)), P)
    for k, kernel in ((4, "staged"), (8, "staged"), (16, "staged"), (32, "staged"), (64, "staged"), (128, "staged"),
                      (256, "generic"), (20, "levels"), (5, "generic")):
        x = rng.integers(-2**31, 2**31 - 1, size=(S, P, k), dtype=np.int32)
        got = run_gpu(x, f, "max", pf)
        assert B.ftc_kernel_name(got[2]) == kernel
        assert_same(got, run_oracle(x, f, "max", pf), f"k={k}")


def test_wide_groups_f_up_to_31():
    rng = np.random.Generator(np.random.PCG64(8))
    for f in (9, 12, 31):
        P, S, k = 40 * (f + 1) + 5, 12, 4
        x = rng.integers(0, 2**64, size=(S, P, k), dtype=np.uint64)
        pf = sc.picks_to_masks(sc.random_subsets(rng, S, P, rng.integers(0, f + 1, size=S)), P)
        for allred in (False, True):
            for flags in KERNELS:
                assert_same(run_gpu(x, f, "sum", pf, allreduce=allred, flags=flags),
                            run_oracle(x, f, "sum", pf, allreduce=allred), f"f={f}")


def test_empty_batch_and_argument_errors():
    import torch
    d = B.make_desc(8, 1, 4, B.FTC_I32, "sum")
    z = torch.zeros(16, dtype=torch.int32, device="cuda")
    assert B.ftc_reduce_batch(d, 0, None, None, None, None, None, None) == B.FTC_OK
    bad = [B.make_desc(2, 1, 4, B.FTC_I32, "sum"), B.make_desc(8, 1, 0, B.FTC_I32, "sum"),
           B.make_desc(8, 1, 4, B.FTC_I32, "sum", root=8), B.make_desc(8, 32, 4, B.FTC_I32, "sum"),
           B.make_desc(64, 1, 4, B.FTC_I32, "sum", max_inop=33)]
    for desc in bad:
        assert B.ftc_reduce_batch(desc, 1, z, z, z, z, z, z, check=False) == B.FTC_EINVAL
    assert B.ftc_reduce_batch(B.make_desc(8, 1, 4, B.FTC_F32, "xor"), 1, z, z, z, z, z, z, check=False) == B.FTC_EUNSUPPORTED
    assert B.ftc_reduce_batch(B.make_desc(8, 1, 4, 9, "sum"), 1, z, z, z, z, z, z, check=False) == B.FTC_EUNSUPPORTED
    assert B.ftc_reduce_batch(d, 1, None, z, None, None, z, z, check=False) == B.FTC_EINVAL
    assert B.ftc_reduce_batch(B.make_desc(8, 1, 4, B.FTC_I32, "sum", root=-1), 1, z, z, None, None, z, z, check=False) == B.FTC_EINVAL
    assert B.ftc_reduce_batch(d, 1, z[1:], z, None, None, z, z, check=False) == B.FTC_EINVAL          # misaligned
    g = B.make_desc(8, 1, 1, B.FTC_I32, "sum")                                                          # needs workspace
    assert B.ftc_workspace_bytes(g, 4) > 0
    assert B.ftc_reduce_batch(g, 4, z, z, None, None, z, z, None, check=False) == B.FTC_EWORKSPACE
    with pytest.raises(B.FtcError):
        B.ftc_reduce_batch(g, 4, z, z, None, None, z, z, None)
    torch.cuda.synchronize()


def test_bad_per_scenario_root_is_a_status_not_an_error():
    rng = np.random.Generator(np.random.PCG64(2))
    x = rng.integers(0, 100, size=(3, 10, 4), dtype=np.int32)
    pf = np.zeros((3, 1), dtype=np.uint32)
    out, st, _ = run_gpu(x, 1, "sum", pf, roots=np.array([2, 10, 9], dtype=np.uint32))
    assert (st[:, 0] & 0xFF).tolist() == [0, B.FTC_ST_BAD_ROOT, 0] and not out[1].any()
    assert np.array_equal(out[0], x[0].sum(axis=0)) and np.array_equal(out[2], x[2].sum(axis=0))


def test_mask_bits_beyond_P_are_ignored():
    P, f = 40, 2
    x = np.random.Generator(np.random.PCG64(2)).integers(0, 2**64, size=(2, P, 2), dtype=np.uint64)
    pf = np.zeros((2, 2), dtype=np.uint32)
    pf[1, 1] = 0xFFFFFF00                    # bits 40..63
    out, st, _ = run_gpu(x, f, "sum", pf)
    want = run_oracle(x, f, "sum", np.zeros((2, 2), dtype=np.uint32))
    assert_same((out, st), want)


def test_device_input_generator_matches_host_generator():
    import torch
    for kind, tdt in ((sc.KIND_I32_PM20, torch.int32), (sc.KIND_I64_PM40, torch.int64), (sc.KIND_F32_NORMAL, torch.float32),
                      (sc.KIND_I32_FULL, torch.int32), (sc.KIND_U64_FULL, torch.uint64)):
        S, P, k, first = 5, 70, 6, 123456
        d = torch.empty((S, P, k), dtype=tdt, device="cuda")
        B.ftc_fill_inputs(kind, 0xABCDEF12345, first, S, P, k, d)
        torch.cuda.synchronize()
        host = sc.gen_inputs(kind, 0xABCDEF12345, np.arange(S) + first, P, k)
        got = to_host(d, host.dtype)
        assert np.array_equal(got.view(np.uint8), host.view(np.uint8)), kind


def test_host_buffer_entry_points_match_device_ones():
    import torch
    ratt = O.schedule(4096, 4)["rounds_attempt"]
    w = sc.config4(ratt, S=40)
    x = w.host_inputs()
    desc = B.make_desc(w.P, w.f, w.k, B.FTC_I32, "max", max_inop=2)
    out = np.full((w.S, w.k), 7, dtype=np.int32)
    st = np.full((w.S, 4), 7, dtype=np.uint32)
    nbytes = B.ftc_host_staging_bytes(desc, 16)                 # forces three chunks
    staging = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    B.ftc_allreduce_batch_host(desc, w.S, x, w.prefail, np.ascontiguousarray(w.inop), None, out, st, staging)
    assert_same((out, st), run_oracle(x, w.f, "max", w.prefail, w.inop, None, 0, True), "host variant")
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    assert B.ftc_allreduce_batch_host(desc, w.S, x, w.prefail, np.ascontiguousarray(w.inop), None, out, st, small,
                                      check=False) == B.FTC_EWORKSPACE


# ---------------------------------------------------------------------------------------------
# expanded allreduce output: the value in the slot of every holder, zeros elsewhere
# ---------------------------------------------------------------------------------------------
def run_gpu_expanded(x, f, op, pf, inop, roots, flags):
    import torch
    d_x = to_dev(x)
    S, P, k = d_x.shape
    max_inop = 0 if inop is None else inop.shape[1]
    desc = B.make_desc(P, f, k, B.dtype_code(d_x.dtype), op, root=-1, max_inop=max_inop, flags=flags | B.FTC_OUT_EXPANDED)
    d_out = torch.empty((S, P, k), dtype=d_x.dtype, device="cuda")
    d_out.view(torch.uint8).fill_(0x5A)
    d_st = torch.full((S, 4), 0x7FFFFFFF, dtype=torch.int32, device="cuda")
    wsb = B.ftc_workspace_bytes(desc, S, True)
    assert wsb >= S * k * x.dtype.itemsize
    d_ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    B.ftc_allreduce_batch(desc, S, d_x, to_dev(pf), to_dev(inop) if max_inop else None, to_dev(roots), d_out, d_st, d_ws)
    torch.cuda.synchronize()
    return to_host(d_out, x.dtype), d_st.cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("flags", KERNELS)
def test_expanded_output_matches_oracle_holders(flags):
    rng = np.random.Generator(np.random.PCG64(77))
    for P, f, k, dtype in ((10, 2, 4, np.uint64), (37, 1, 3, np.int32), (64, 3, 8, np.float32), (200, 0, 4, np.int32)):
        S = 60
        x = rng.standard_normal((S, P, k)).astype(np.float32) if dtype == np.float32 else \
            rng.integers(0, 2**31 - 1, size=(S, P, k)).astype(dtype)
        pf = sc.picks_to_masks(sc.random_subsets(rng, S, P, rng.integers(0, f + 3, size=S), lo=0), P)
        R = O.schedule(P, f)["rounds_attempt"]
        inop = np.zeros((S, 2, 2), dtype=np.uint32)
        inop[:, :, 0] = rng.integers(f + 1, P, size=(S, 2))
        inop[:, :, 1] = rng.integers(0, R + 3, size=(S, 2))
        inop[rng.random((S, 2)) < 0.3, 0] = sc.UNUSED
        roots = np.zeros(S, dtype=np.uint32)
        got, st = run_gpu_expanded(x, f, "sum", pf, inop, roots, flags)
        for i in range(S):
            d = O.run(x[i], f, "sum", pf[i], inop=[tuple(e) for e in inop[i]], root=0, allreduce=True, detail=True)
            assert np.array_equal(st[i], d["status"]), (P, i)
            assert np.array_equal(got[i].view(np.uint8), d["expanded"].view(np.uint8)), (P, f, i, d["code"])


def test_expanded_needs_allreduce_and_workspace():
    import torch
    z = torch.zeros(4096, dtype=torch.int32, device="cuda")
    d = B.make_desc(8, 1, 4, B.FTC_I32, "sum", flags=B.FTC_OUT_EXPANDED)
    assert B.ftc_reduce_batch(d, 1, z, z, None, None, z, z, z, check=False) == B.FTC_EUNSUPPORTED
    assert B.ftc_allreduce_batch(d, 1, z, z, None, None, z, z, None, check=False) == B.FTC_EWORKSPACE


# ---------------------------------------------------------------------------------------------
# what every root child delivers: value, delivered / failed bit, size of the failed-process list
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("allreduce", [False, True])
def test_candidates_of_every_root_child_match_oracle(allreduce):
    import torch
    rng = np.random.Generator(np.random.PCG64(91))
    for P, f, k, dtype in ((7, 1, 1, np.int64), (14, 2, 4, np.uint64), (41, 3, 3, np.float32), (130, 4, 2, np.int32), (9, 0, 2, np.int32)):
        S = 80
        x = rng.standard_normal((S, P, k)).astype(np.float32) if dtype == np.float32 else \
            rng.integers(0, 2**31 - 1, size=(S, P, k)).astype(dtype)
        pf = sc.picks_to_masks(sc.random_subsets(rng, S, P, rng.integers(0, f + 3, size=S)), P)
        R = O.schedule(P, f)["rounds_attempt"]
        inop = np.zeros((S, 2, 2), dtype=np.uint32)
        inop[:, :, 0] = rng.integers((f + 1) if allreduce else 0, P, size=(S, 2))
        inop[:, :, 1] = rng.integers(0, R + 3, size=(S, 2))
        inop[rng.random((S, 2)) < 0.3, 0] = sc.UNUSED
        roots = (np.zeros(S) if allreduce else rng.integers(0, P, size=S)).astype(np.uint32)
        d_x = to_dev(x)
        desc = B.make_desc(P, f, k, B.dtype_code(d_x.dtype), "sum", root=-1, max_inop=2)
        d_cand = torch.empty((S, f + 1, k), dtype=d_x.dtype, device="cuda")
        d_cand.view(torch.uint8).fill_(0x5A)
        d_info = torch.full((S, f + 1, 2), 0x7FFFFFFF, dtype=torch.int32, device="cuda")
        d_ws = torch.empty(B.ftc_candidates_workspace_bytes(desc, S), dtype=torch.uint8, device="cuda")
        B.ftc_candidates_batch(desc, S, allreduce, d_x, to_dev(pf), to_dev(inop), to_dev(roots), d_cand, d_info, d_ws)
        torch.cuda.synchronize()
        cand, info = to_host(d_cand, x.dtype), d_info.cpu().numpy()
        for i in range(S):
            d = O.run(x[i], f, "sum", pf[i], inop=[tuple(e) for e in inop[i]], root=int(roots[i]), allreduce=allreduce, detail=True)
            if d["attempts"] == 0:
                assert (info[i, :, 0] == 2).all() and not cand[i].any()
                continue
            assert np.array_equal(info[i, :, 0], d["cand_flag"]), (P, f, i, d["code"])
            assert np.array_equal(info[i, :, 1], d["cand_nfail"]), (P, f, i)
            assert np.array_equal(cand[i].view(np.uint8), d["cand"].view(np.uint8)), (P, f, i)


# ---------------------------------------------------------------------------------------------
# a sparsely filled last heap level: its rows stay out of the warp tiles and are folded one by one
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("P,f,k,dname", [(1024, 3, 16, "f32"),     # 256 rows: one row (the short group) on the last level
                                         (533, 1, 4, "i32"),       # 266 rows, 10 on the last level; staged whole
                                         (1598, 2, 8, "i64"),      # 533 rows, 21 on the last level, short group among them
                                         (2056, 7, 4, "f32")])     # 257 rows: one row on the last level, wide groups
@pytest.mark.parametrize("allreduce", [False, True])
def test_sparse_last_level_failures_roots_and_victims_there(P, f, k, dname, allreduce):
    rng = np.random.Generator(np.random.PCG64(P + f))
    S, m = 96, f + 1
    Gmax = (P - 1 + m - 1) // m
    first_last = (1 << (Gmax.bit_length() - 1)) - 1                 # first row of the last heap level
    tail = list(range(first_last * m + 1, P))                        # processes of the last level's rows
    assert 0 < len(tail) <= (m * (first_last + 1)) // 8 + m
    x = rng.standard_normal((S, P, k)).astype(np.float32) if dname == "f32" else \
        rng.integers(np.iinfo(DT[dname]).min, np.iinfo(DT[dname]).max, size=(S, P, k), dtype=DT[dname])
    R = O.schedule(P, f)
    sets, inop, roots = [], np.full((S, 2, 2), sc.UNUSED, dtype=np.uint32), np.zeros(S, dtype=np.uint32)
    for i in range(S):
        n_tail = int(rng.integers(0, min(f, len(tail)) + 1))
        dead = set(int(v) for v in rng.choice(tail, size=n_tail, replace=False))
        dead |= set(int(v) for v in rng.integers(0, P, size=int(rng.integers(0, f + 1 - n_tail + 1))))
        roots[i] = int(rng.choice(tail)) if rng.random() < 0.5 else int(rng.integers(0, P))
        if allreduce and rng.random() < 0.5:
            roots[i] = P - 1 - int(rng.integers(0, 2))               # candidates wrap around to process 0
        for j in range(2):
            if rng.random() < 0.6:
                v = int(rng.choice(tail)) if rng.random() < 0.7 else int(rng.integers(0, P))
                if allreduce and (v - int(roots[i])) % P <= f:
                    continue
                inop[i, j] = (v, int(rng.integers(0, R["rounds_attempt"] + 2)))
        sets.append(sorted(dead))
    pf = sc.sets_to_masks(sets, P)
    op = "sum" if dname == "f32" else "max"
    for flags in KERNELS:
        got = run_gpu(x, f, op, pf, inop, roots, 0, allreduce, flags)
        want = run_oracle(x, f, op, pf, inop, roots, 0, allreduce)
        assert_same(got, want, f"P={P} f={f} k={k} {dname} allreduce={allreduce} flags={flags:#x}")
        assert ((want[1][:, 0] & 0xFF) == 0).sum() > S // 3


# ---------------------------------------------------------------------------------------------
# many processes with wide vectors: the staged kernel's array of tile results moves into the workspace
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("P,f,k,dname,S", [(16384, 5, 16, "u64", 6), (65536, 4, 32, "i32", 2), (1024, 3, 128, "f32", 24),
                                           (65536, 8, 16, "f32", 2)])
def test_large_heap_array_in_the_workspace_and_without(P, f, k, dname, S):
    import torch
    rng = np.random.Generator(np.random.PCG64(P + k))
    x = rng.standard_normal((S, P, k)).astype(np.float32) if dname == "f32" else \
        rng.integers(np.iinfo(DT[dname]).min, np.iinfo(DT[dname]).max, size=(S, P, k), dtype=DT[dname])
    pf = sc.picks_to_masks(sc.random_subsets(rng, S, P, rng.integers(0, f + 1, size=S)), P)
    roots = rng.integers(0, P, size=S).astype(np.uint32)
    op = "sum" if dname in ("f32", "u64") else "max"
    want = run_oracle(x, f, op, pf, None, roots, 0, True)
    desc = B.make_desc(P, f, k, B.dtype_code(np.dtype(DT[dname])), op, root=-1)
    assert B.ftc_kernel_name(desc, True) == "staged" and B.ftc_workspace_bytes(desc, S, True) > 0
    got = run_gpu(x, f, op, pf, None, roots, 0, True)                   # with the workspace the library asks for
    assert_same(got, want, f"P={P} k={k} {dname} with workspace")
    # without a workspace the shape still runs (array in shared memory, or another kernel) unless only the general
    # kernel is left, which reports the missing workspace
    d_x, d_out = to_dev(x), torch.zeros((S, k), dtype=to_dev(x).dtype, device="cuda")
    d_st = torch.zeros((S, 4), dtype=torch.int32, device="cuda")
    rc = B.ftc_allreduce_batch(desc, S, d_x, to_dev(pf), None, to_dev(roots), d_out, d_st.view(torch.uint32), None, check=False)
    torch.cuda.synchronize()
    if rc == B.FTC_OK:
        assert_same((to_host(d_out, x.dtype), d_st.cpu().numpy().view(np.uint32)), want, f"P={P} k={k} {dname} without workspace")
    else:
        assert rc == B.FTC_EWORKSPACE


# ---------------------------------------------------------------------------------------------
# float32 vectors of 16 and 32 bytes in groups of a multiple of 128 bytes: tiles arrive by swizzled tensor copies
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("P,f,k,S", [(16384, 3, 8, 6), (8200, 7, 4, 10), (1030, 3, 8, 40), (20000, 15, 4, 4), (4099, 1, 16, 12),
                                     (5000, 3, 4, 12), (20001, 1, 8, 5), (40000, 3, 4, 3), (1500, 3, 4, 30)])   # the last four: 64-byte groups
@pytest.mark.parametrize("allreduce", [False, True])
def test_float32_small_vectors_swizzled_tiles(P, f, k, S, allreduce):
    rng = np.random.Generator(np.random.PCG64(3 * P + k))
    x = rng.standard_normal((S, P, k)).astype(np.float32)
    pf = sc.picks_to_masks(sc.random_subsets(rng, S, P, rng.integers(0, f + 2, size=S)), P)
    pf[0] = 0                                                        # one failure-free scenario
    R = O.schedule(P, f)["rounds_attempt"]
    inop = np.full((S, 2, 2), sc.UNUSED, dtype=np.uint32)
    roots = rng.integers(0, P, size=S).astype(np.uint32)
    roots[1 % S] = P - 1                                             # root in the last (short or full) group
    for i in range(S):
        for j in range(2):
            if rng.random() < 0.5:
                v = int(rng.integers(0, P))
                if allreduce and (v - int(roots[i])) % P <= f:
                    continue
                inop[i, j] = (v, int(rng.integers(0, R + 2)))
    got = run_gpu(x, f, "sum", pf, inop, roots, 0, allreduce)
    assert B.ftc_kernel_name(got[2], allreduce) == "staged"
    assert_same(got, run_oracle(x, f, "sum", pf, inop, roots, 0, allreduce), f"P={P} f={f} k={k} allreduce={allreduce}")


@pytest.mark.parametrize("P,f,k,dname,S", [(8200, 7, 4, "f32", 10), (16384, 5, 16, "u64", 5), (5000, 3, 4, "f32", 9)])
def test_host_buffer_entry_point_on_swizzled_and_workspace_shapes(P, f, k, dname, S):
    """The host-buffer call goes chunk by chunk through device staging: tensor maps are built per chunk, and the
    staging holds the workspace for the tile results."""
    import torch
    rng = np.random.Generator(np.random.PCG64(P))
    x = rng.standard_normal((S, P, k)).astype(np.float32) if dname == "f32" else rng.integers(0, 2**63, size=(S, P, k), dtype=np.uint64)
    pf = sc.picks_to_masks(sc.random_subsets(rng, S, P, rng.integers(0, f + 1, size=S)), P)
    roots = rng.integers(0, P, size=S).astype(np.uint32)
    desc = B.make_desc(P, f, k, B.dtype_code(np.dtype(DT[dname])), "sum", root=-1)
    out = np.zeros((S, k), dtype=DT[dname])
    st = np.zeros((S, 4), dtype=np.uint32)
    staging = torch.empty(B.ftc_host_staging_bytes(desc, 4), dtype=torch.uint8, device="cuda")     # several chunks
    B.ftc_reduce_batch_host(desc, S, x, pf, None, roots, out, st, staging)
    assert_same((out, st), run_oracle(x, f, "sum", pf, None, roots, 0, False), f"host variant P={P} k={k} {dname}")
