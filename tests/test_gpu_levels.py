"""GPU parity for the level kernel (shared-memory tiles evaluated level by level), which plays subtrees that are a-ary heaps
of arity 3 and more, binomial trees (arity 1 here, the oracle's code for them), and binary heaps on request: against the CPU
oracle playing the same shape, bit for bit."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2602_22445_b200 import scenarios as sc

from paper_2602_22445_b200 import binding as B
from tests.gpu_util import assert_same, run_gpu, run_oracle_mt
from tests.test_gpu_variants import DT, make_batch

pytestmark = pytest.mark.gpu


def flags_for(arity):
    return B.FTC_KERNEL_LEVELS if arity == 2 else B.FTC_TREE_BINOMIAL if arity == 1 else B.FTC_TREE_ARITY(arity)


SHAPES = [
    # P, f, k, dtype, op: one tile, several tiles, several levels above the tiles, ragged last levels, a short last group
    (7, 1, 4, "i32", "sum"), (40, 3, 2, "u64", "xor"), (150, 3, 16, "f32", "sum"), (1024, 3, 16, "f32", "sum"),
    (1000, 0, 4, "f32", "sum"), (2003, 2, 8, "i64", "max"), (4096, 4, 32, "i32", "max"), (5000, 15, 4, "i32", "xor"),
    (16384, 1, 8, "i32", "sum"), (65536, 8, 4, "u64", "sum"), (30011, 7, 64, "f32", "sum"), (9000, 31, 2, "i64", "sum"),
]


# The shape with P = 30011 and 256-byte vectors has a heap array (the rows of all levels down to the tiles' roots) beyond the
# kernel's shared-memory budget at every arity: the general kernel plays it. (4096 processes at arity 5 or 32 and 65536 at
# arity 8 fit only because the kernel may take a larger buffer to make its forests one level deeper.)
TOO_WIDE = set()


@pytest.mark.parametrize("arity", [1, 2, 3, 4, 5, 8, 32])
@pytest.mark.parametrize("P,f,k,dname,op", SHAPES)
def test_level_kernel_matches_the_oracle(arity, P, f, k, dname, op):
    S = max(3, min(40, int(4e6 // (P * k))))
    for allreduce in (False, True):
        d_x, x, pf, inop, roots = make_batch(P, f, k, dname, allreduce, S, seed=arity * 1000 + P + k)
        got = run_gpu(None, f, op, pf, inop, roots, 0, allreduce, flags_for(arity), d_x=d_x)
        fits = (P, k) != (30011, 64) and (arity, P) not in TOO_WIDE
        assert B.ftc_kernel_name(got[2], allreduce) == ("levels" if fits else "staged" if arity == 2 else "generic")
        assert_same(got, run_oracle_mt(x, f, op, pf, inop, roots, 0, allreduce, arity=arity), f"P={P} f={f} k={k} {dname} {op} arity={arity} allreduce={allreduce}")


@pytest.mark.parametrize("arity", [1, 3, 4])
def test_level_kernel_with_descending_partners(arity):
    for P, f, k in ((150, 3, 16), (4099, 4, 8)):
        d_x, x, pf, inop, roots = make_batch(P, f, k, "f32", True, 30, seed=P)
        got = run_gpu(None, f, "sum", pf, inop, roots, 0, True, flags_for(arity) | B.FTC_PARTNERS_DESCENDING, d_x=d_x)
        assert B.ftc_kernel_name(got[2], True) == "levels"
        assert_same(got, run_oracle_mt(x, f, "sum", pf, inop, roots, 0, True, arity=arity, partners_descending=True), f"P={P} arity={arity}")


WIDE_SHAPES = [
    # vectors of 3, 5, 6 and 12 chunks of 16 bytes (not a power of two: the register tiles cannot hold them)
    (300, 2, 12, "f32", "sum"), (4099, 4, 20, "i32", "max"), (1024, 3, 12, "u64", "xor"), (20011, 7, 6, "i64", "sum"), (700, 1, 48, "f32", "sum"),
]


@pytest.mark.parametrize("arity", [1, 2, 4])
@pytest.mark.parametrize("P,f,k,dname,op", WIDE_SHAPES)
def test_vectors_of_any_number_of_chunks(arity, P, f, k, dname, op):
    """Vectors that are a multiple of 16 bytes but not a power-of-two number of chunks: binary heaps take the level kernel by
    themselves here (no flag), the other shapes as always."""
    S = max(3, min(40, int(4e6 // (P * k))))
    flags = 0 if arity == 2 else flags_for(arity)
    for allreduce in (False, True):
        d_x, x, pf, inop, roots = make_batch(P, f, k, dname, allreduce, S, seed=arity * 77 + P + k)
        got = run_gpu(None, f, op, pf, inop, roots, 0, allreduce, flags, d_x=d_x)
        assert B.ftc_kernel_name(got[2], allreduce) == "levels"
        assert_same(got, run_oracle_mt(x, f, op, pf, inop, roots, 0, allreduce, arity=arity), f"P={P} f={f} k={k} {dname} {op} arity={arity} allreduce={allreduce}")


EDGE_SHAPES = [
    # the smallest process counts (P = f + 2: one group, one row), a single full group plus the root, one row more than a tile,
    # the widest group (f = 31), the widest vectors (31 and 32 chunks), two processes
    (3, 1, 4, "i32", "sum"), (2, 0, 4, "f32", "sum"), (33, 31, 4, "i32", "xor"), (34, 31, 2, "u64", "sum"), (65, 31, 4, "f32", "sum"),
    (5, 3, 8, "f32", "sum"), (6, 3, 8, "i64", "max"), (1000, 0, 124, "f32", "sum"), (300, 2, 128, "i32", "max"), (130, 1, 64, "u64", "xor"),
]


@pytest.mark.parametrize("arity", [1, 2, 3, 32])
@pytest.mark.parametrize("P,f,k,dname,op", EDGE_SHAPES)
def test_level_kernel_edge_shapes(arity, P, f, k, dname, op):
    """Degenerate shapes, and batches of one and two scenarios: whichever kernel the shape gets, the oracle decides."""
    for allreduce in (False, True):
        for S in (1, 2, 37):
            d_x, x, pf, inop, roots = make_batch(P, f, k, dname, allreduce, S, seed=arity + 13 * P + k + S)
            got = run_gpu(None, f, op, pf, inop, roots, 0, allreduce, flags_for(arity), d_x=d_x)
            assert B.ftc_kernel_name(got[2], allreduce) in ("levels", "generic", "staged")
            assert_same(got, run_oracle_mt(x, f, op, pf, inop, roots, 0, allreduce, arity=arity), f"P={P} f={f} k={k} {dname} {op} arity={arity} allreduce={allreduce} S={S}")


def test_shapes_the_level_kernel_leaves_to_the_general_one():
    for k, dt in ((3, B.FTC_F32), (6, B.FTC_I32), (1, B.FTC_U64)):            # not a multiple of 16 bytes
        assert B.ftc_kernel_name(B.make_desc(100, 2, k, dt, "sum", flags=B.FTC_TREE_ARITY(4)), True) == "generic"
    assert B.ftc_kernel_name(B.make_desc(100, 2, 4, B.FTC_I32, "sum", flags=B.FTC_TREE_ARITY(4) | B.FTC_KERNEL_GENERIC), True) == "generic"
    assert B.ftc_kernel_name(B.make_desc(100, 2, 6, B.FTC_I32, "sum", flags=B.FTC_TREE_BINOMIAL), True) == "generic"
    assert B.ftc_kernel_name(B.make_desc(100, 2, 4, B.FTC_I32, "sum", flags=B.FTC_TREE_BINOMIAL), True) == "levels"
    assert B.ftc_kernel_name(B.make_desc(100, 2, 4, B.FTC_I32, "sum"), True) == "staged"


@pytest.mark.parametrize("arity,P,f,k,dname,op,allreduce", [(4, 4096, 4, 32, "i32", "max", True), (3, 1024, 3, 16, "f32", "sum", True),
                                                            (8, 16384, 1, 8, "i32", "sum", False), (2, 150, 3, 16, "f32", "sum", True),
                                                            (1, 5000, 2, 8, "i64", "max", True)])
def test_level_kernel_gives_up_cleanly(arity, P, f, k, dname, op, allreduce):
    """With FTC_DEBUG_ONE_POLL the waits for the asynchronous copies look once and give up: a scenario is then either
    played correctly or reports FTC_ST_INTERNAL_TIMEOUT with zero bytes, a block that reported it does so for all its
    later scenarios, the call returns by itself, and the next normal call on the same buffers matches the oracle."""
    flags = flags_for(arity)
    desc = B.make_desc(P, f, k, B.dtype_code(np.dtype(DT[dname])), op, root=-1, max_inop=2, flags=flags)
    assert B.ftc_kernel_name(desc, allreduce) == "levels"
    blocks = B.ftc_launch_blocks(desc, 1 << 30, allreduce)
    S = 2 * blocks + 3
    d_x, x, pf, inop, roots = make_batch(P, f, k, dname, allreduce, S, seed=5 + P)
    want = run_oracle_mt(x, f, op, pf, inop, roots, 0, allreduce, arity=arity)
    out, st, _ = run_gpu(None, f, op, pf, inop, roots, 0, allreduce, flags | B.FTC_DEBUG_ONE_POLL, d_x=d_x)
    timed_out = (st[:, 0] & 0xFF) == B.FTC_ST_INTERNAL_TIMEOUT
    ob, wb = out.view(np.uint8).reshape(S, -1), want[0].view(np.uint8).reshape(S, -1)
    assert not ob[timed_out].any() and not st[timed_out, 1:].any()
    assert np.array_equal(st[~timed_out], want[1][~timed_out]) and np.array_equal(ob[~timed_out], wb[~timed_out])
    for b in range(blocks):
        seq = timed_out[b::blocks]
        assert np.array_equal(seq, np.sort(seq)), (b, seq)
    assert timed_out.any()
    assert_same(run_gpu(None, f, op, pf, inop, roots, 0, allreduce, flags, d_x=d_x), want, "normal call after the give-up run")


def seeded_shapes():
    rng = np.random.Generator(np.random.PCG64(20260223))
    out = []
    for _ in range(40):
        f = int(rng.choice([0, 1, 1, 2, 3, 3, 4, 7, 15]))
        P = int(rng.choice([rng.integers(f + 2, 300), rng.integers(300, 3000), rng.integers(3000, 30000)]))
        dname = ["i32", "i64", "u64", "f32", "f32"][int(rng.integers(0, 5))]
        op = "sum" if dname == "f32" else ["sum", "max", "xor"][int(rng.integers(0, 3))]
        k = int(rng.choice([4, 8, 12, 16, 20, 24, 32, 44, 64, 128] if np.dtype(DT[dname]).itemsize == 4 else [2, 4, 6, 8, 10, 16, 22, 64]))
        out.append((P, f, k, dname, op, bool(rng.integers(0, 2)), int(rng.choice([1, 2, 3, 4, 5, 7, 8, 16, 32])), bool(rng.integers(0, 3) == 0)))
    return out


@pytest.mark.parametrize("P,f,k,dname,op,allreduce,arity,descending", seeded_shapes())
def test_seeded_random_shapes_and_patterns(P, f, k, dname, op, allreduce, arity, descending):
    """Random shapes, subtree shapes and partner orders with failure patterns beyond what the schedule tolerates (up to f + 2
    processes failed beforehand, two in-operation victims at any round up to twice an attempt, any root): whatever kernel the
    shape gets, results and status records equal the oracle's."""
    rng = np.random.Generator(np.random.PCG64(P * 31 + k + arity))
    S = max(2, min(24, int(3e6 // (P * k))))
    dt = DT[dname]
    x = rng.standard_normal((S, P, k)).astype(np.float32) if dname == "f32" else \
        rng.integers(np.iinfo(dt).min, np.iinfo(dt).max, size=(S, P, k), dtype=dt, endpoint=True)
    pf = sc.picks_to_masks(sc.random_subsets(rng, S, P, np.minimum(rng.integers(0, f + 3, size=S), P - 1)), P)
    R = O.schedule(P, f, arity)["rounds_attempt"]
    inop = np.zeros((S, 2, 2), dtype=np.uint32)
    lo = f + 1 if allreduce and P > 2 * f + 4 else 0                 # keeps the victims clear of the root candidates 0..f
    inop[:, :, 0] = rng.integers(lo, P, size=(S, 2))
    inop[:, :, 1] = rng.integers(0, 2 * R + 2, size=(S, 2))
    inop[rng.random((S, 2)) < 0.4, 0] = sc.UNUSED
    roots = rng.integers(0, P, size=S).astype(np.uint32)
    if allreduce and lo:
        roots[:] = 0
    flags = flags_for(arity) | (B.FTC_PARTNERS_DESCENDING if descending else 0)
    got = run_gpu(x, f, op, pf, inop, roots, 0, allreduce, flags)
    assert B.ftc_kernel_name(got[2], allreduce) in ("levels", "generic", "staged")
    assert_same(got, run_oracle_mt(x, f, op, pf, inop, roots, 0, allreduce, arity=arity, partners_descending=descending),
                f"P={P} f={f} k={k} {dname} {op} allreduce={allreduce} arity={arity} descending={descending}")
