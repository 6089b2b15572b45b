"""Every instantiation of the shared-memory kernel that the dispatcher can pick, with several scenarios per block.

One thread block plays scenarios b, b + blocks, b + 2*blocks, ... and its warps keep their copy pipelines running
across the scenario boundaries (running buffer indices, mbarrier parities, source pointers or tensor coordinates).
So each case here asks the library which instantiation it would run (and asserts the name), sizes the batch to a
little more than three scenarios per launched block, places pre-operation failures (up to f+1), per-scenario roots
(the last group among them) and in-operation victims with rounds over the whole attempt, and compares results and
status records of ALL scenarios with the CPU oracle bit for bit (float32 too: the schedule fixes the order).
"""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2602_22445_b200 import binding as B
from paper_2602_22445_b200 import scenarios as sc
from tests.gpu_util import assert_same, run_gpu, run_oracle_mt, to_host

pytestmark = pytest.mark.gpu

DT = {"i32": np.int32, "i64": np.int64, "u64": np.uint64, "f32": np.float32}
KIND = {"i32": sc.KIND_I32_FULL, "i64": sc.KIND_I64_PM40, "u64": sc.KIND_U64_FULL, "f32": sc.KIND_F32_NORMAL}


def make_batch(P, f, k, dname, allreduce, S, seed):
    """Device-generated inputs (copied back for the oracle) and a seeded failure pattern per scenario."""
    import torch
    rng = np.random.Generator(np.random.PCG64(seed))
    if dname == "f32":
        # normal deviates from numpy: full mantissas, so float32 sums round at every addition and every fold order shows
        x = rng.standard_normal((S, P, k), dtype=np.float32)
        d_x = torch.from_numpy(x).cuda()
    else:
        d_x = torch.empty((S, P, k), dtype=getattr(torch, np.dtype(DT[dname]).name), device="cuda")
        B.ftc_fill_inputs(KIND[dname], seed, 0, S, P, k, d_x)
        torch.cuda.synchronize()
        x = to_host(d_x, DT[dname])
    sizes = rng.integers(0, f + 2, size=S)
    sizes[rng.random(S) < 0.35] = 0                                   # a good third without pre-operation failures
    pf = sc.picks_to_masks(sc.random_subsets(rng, S, P, np.minimum(sizes, P - 1)), P)
    roots = rng.integers(0, P, size=S).astype(np.uint32)
    roots[rng.random(S) < 0.1] = P - 1                                # the root in the last group
    roots[rng.random(S) < 0.1] = 0
    for i in range(7, S, 50):                                         # a failed root: no-op reduce, second allreduce attempt
        pf[i, roots[i] >> 5] |= np.uint32(1 << (roots[i] & 31))
    for i in range(11, S, 100):                                       # every root candidate failed
        for c in range(f + 1):
            v = (int(roots[i]) + c) % P
            pf[i, v >> 5] |= np.uint32(1 << (v & 31))
    R = O.schedule(P, f)["rounds_attempt"]
    inop = np.full((S, 2, 2), sc.UNUSED, dtype=np.uint32)
    vic = rng.integers(0, P, size=(S, 2))
    rnd = rng.integers(0, R + 2, size=(S, 2))
    use = rng.random((S, 2)) < 0.4
    if allreduce:                                                     # victims stay clear of the f+1 root candidates
        use &= ((vic - roots[:, None].astype(np.int64)) % P) > f
    inop[:, :, 0] = np.where(use, vic, sc.UNUSED)
    inop[:, :, 1] = np.where(use, rnd, 0)
    return d_x, x, pf, inop, roots


CASES = [
    # name, P, f, k, dtype, op, allreduce
    ("staged/lean", 1024, 3, 16, "f32", "sum", True),                 # the float32 configuration's shape
    ("staged/lean", 2000, 2, 8, "i64", "max", False),
    ("staged/large", 4096, 4, 32, "i32", "max", True),                # the P=4096 configuration's shape
    ("staged/large", 65536, 8, 4, "u64", "sum", False),               # the P=65536 configuration: reduce, sum
    ("staged/large", 65536, 8, 4, "u64", "xor", False),               #   reduce, xor
    ("staged/large", 65536, 8, 4, "u64", "xor", True),                #   allreduce, xor
    ("staged/large", 65536, 8, 4, "u64", "sum", True),                #   allreduce, sum
    ("staged/batched-lean", 16384, 1, 8, "i32", "sum", True),         # groups of 64 bytes in blocks of 4-8 warps
    ("staged/batched-lean", 40000, 3, 4, "i32", "xor", False),
    ("staged/batched-lean", 20011, 7, 2, "u64", "max", True),         # groups of 128 bytes, ragged
    ("staged/lean-swz", 1030, 3, 8, "f32", "sum", True),              # 128-byte lines
    ("staged/lean-swz", 5000, 3, 4, "f32", "sum", False),             # 64-byte groups
    ("staged/batched-swz", 16384, 3, 8, "f32", "sum", False),
    ("staged/batched-swz", 40000, 3, 4, "f32", "sum", True),          # 64-byte groups in large blocks
    ("staged/whole", 150, 3, 16, "f32", "sum", True),                 # 9.6 KB per scenario
    ("staged/whole", 700, 6, 4, "i32", "xor", False),                 # 11 KB, a heap too deep for one warp tile
    ("staged/warp", 64, 2, 8, "i64", "sum", False),                   # the P=64 configuration's shape
    ("staged/warp", 150, 3, 4, "f32", "sum", True),                   # short last group, 16-byte vectors
    ("staged/warp-pair", 64, 3, 4, "i32", "max", True),               # a heap shallower than the warp tile: two scenarios per warp
    ("staged/warp-pair", 30, 1, 4, "f32", "sum", False),              # eight lanes would do
    ("staged/warp-pair", 120, 7, 4, "u64", "xor", True),              # groups of eight, 32-byte vectors
    ("staged/warp-pair", 17, 0, 4, "i32", "sum", True),               # no tolerance: every failure goes to the general routines
    ("staged/warp", 500, 1, 4, "i32", "xor", False),                  # 8 KB, lane-local sub-heaps of three levels
    ("staged/warp", 40, 4, 32, "i32", "max", True),                   # 128-byte vectors
    ("staged/warp", 12, 0, 64, "f32", "sum", False),                  # no tolerance: groups of one, 256-byte vectors
    ("staged/warp", 9, 1, 128, "i32", "sum", True),                   # 512-byte vectors: one lane row
    ("staged/warp", 100, 5, 4, "u64", "sum", True),
    ("staged/warp", 1024, 7, 2, "i32", "sum", False),                 # kbytes = 8: not this kernel (checked below)
    ("tiled", 4096, 4, 32, "i32", "max", True),
]


@pytest.mark.parametrize("variant,P,f,k,dname,op,allreduce", CASES)
def test_every_variant_with_several_scenarios_per_block(variant, P, f, k, dname, op, allreduce):
    flags = B.FTC_KERNEL_DIRECT if variant == "tiled" else 0
    desc = B.make_desc(P, f, k, B.dtype_code(np.dtype(DT[dname])), op, root=-1, max_inop=2, flags=flags)
    if k * np.dtype(DT[dname]).itemsize % 16:
        assert B.ftc_kernel_variant(desc, allreduce) == "generic"
        return
    assert B.ftc_kernel_variant(desc, allreduce) == variant
    blocks = B.ftc_launch_blocks(desc, 1 << 30, allreduce)
    assert blocks >= 148
    S = 3 * blocks + 5
    if S * P * k * np.dtype(DT[dname]).itemsize > (3 << 30):         # keep the batch under 3 GiB: still > 2 per block
        S = 2 * blocks + 5
    d_x, x, pf, inop, roots = make_batch(P, f, k, dname, allreduce, S, seed=1000 * P + 10 * f + k)
    got = run_gpu(None, f, op, pf, inop, roots, 0, allreduce, flags, d_x=d_x)
    want = run_oracle_mt(x, f, op, pf, inop, roots, 0, allreduce)
    assert_same(got, want, f"{variant} P={P} f={f} k={k} {dname} {op} allreduce={allreduce} S={S} blocks={blocks}")
    codes = want[1][:, 0] & 0xFF
    assert (codes == 0).sum() > S // 2 and (codes != 0).any()         # most scenarios succeed, some do not


DESC_CASES = [c for c in CASES if c[4] == "f32"] + [("staged/warp-pair", 64, 3, 4, "f32", "sum", True), ("staged/large", 4096, 4, 32, "i32", "max", True), ("staged/warp", 64, 2, 8, "i64", "sum", False),
                                                    ("tiled", 1024, 3, 16, "f32", "sum", True), ("tiled", 300, 2, 8, "f32", "sum", False)]


@pytest.mark.parametrize("variant,P,f,k,dname,op,allreduce", DESC_CASES)
def test_descending_partner_order_on_every_variant(variant, P, f, k, dname, op, allreduce):
    """The other partner order (Algorithm "Up-correction" leaves it open): which partners a dying process reached and the
    float32 fold order change with it; the shared-memory kernels play it too."""
    flags = B.FTC_PARTNERS_DESCENDING | (B.FTC_KERNEL_DIRECT if variant == "tiled" else 0)
    desc = B.make_desc(P, f, k, B.dtype_code(np.dtype(DT[dname])), op, root=-1, max_inop=2, flags=flags)
    assert B.ftc_kernel_variant(desc, allreduce) == variant
    blocks = B.ftc_launch_blocks(desc, 1 << 30, allreduce)
    S = min(2 * blocks + 3, max(8, (1 << 30) // (P * k * np.dtype(DT[dname]).itemsize)))
    d_x, x, pf, inop, roots = make_batch(P, f, k, dname, allreduce, S, seed=31 * P + k)
    got = run_gpu(None, f, op, pf, inop, roots, 0, allreduce, flags, d_x=d_x)
    want = run_oracle_mt(x, f, op, pf, inop, roots, 0, allreduce, partners_descending=True)
    assert_same(got, want, f"descending {variant} P={P} f={f} k={k} {dname} {op} allreduce={allreduce}")
    if dname == "f32" and f >= 2:                                     # the order is observable: ascending gives other bits somewhere
        other = run_oracle_mt(x, f, op, pf, inop, roots, 0, allreduce)
        assert not np.array_equal(other[0].view(np.uint8), want[0].view(np.uint8))


# Shapes and failure patterns drawn at random once (seeded), kept as a fixed list: mid-size and large process counts,
# every element type, vector widths of 16 to 512 bytes, group sizes of 1 to 16.
def fuzz_cases():
    rng = np.random.Generator(np.random.PCG64(20260222))
    out = []
    for _ in range(36):
        f = int(rng.choice([0, 1, 1, 2, 3, 3, 4, 7, 15]))
        P = int(rng.choice([rng.integers(f + 2, 300), rng.integers(300, 3000), rng.integers(3000, 30000)]))
        dname = ["i32", "i64", "u64", "f32", "f32"][int(rng.integers(0, 5))]
        op = "sum" if dname == "f32" else ["sum", "max", "xor"][int(rng.integers(0, 3))]
        k = int(rng.choice([4, 8, 16, 32, 64, 128] if np.dtype(DT[dname]).itemsize == 4 else [2, 4, 8, 16, 64]))
        out.append((P, f, k, dname, op, bool(rng.integers(0, 2))))
    return out


@pytest.mark.parametrize("P,f,k,dname,op,allreduce", fuzz_cases())
def test_seeded_random_shapes(P, f, k, dname, op, allreduce):
    S = max(2, min(24, int(3e6 // (P * k))))
    d_x, x, pf, inop, roots = make_batch(P, f, k, dname, allreduce, S, seed=7 * P + k)
    got = run_gpu(None, f, op, pf, inop, roots, 0, allreduce, 0, d_x=d_x)
    assert B.ftc_kernel_variant(got[2], allreduce).split("/")[0] in ("staged", "tiled", "generic")
    assert_same(got, run_oracle_mt(x, f, op, pf, inop, roots, 0, allreduce), f"P={P} f={f} k={k} {dname} {op} allreduce={allreduce}")


# ---------------------------------------------------------------------------------------------
# the give-up path of the kernel's bounded waits
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("P,f,k,dname,op,allreduce", [(1024, 3, 16, "f32", "sum", True), (4096, 4, 32, "i32", "max", True),
                                                      (16384, 3, 8, "f32", "sum", False), (16384, 1, 8, "i32", "sum", True),
                                                      (64, 2, 8, "i64", "sum", False), (150, 3, 16, "f32", "sum", True),
                                                      (64, 3, 4, "i32", "max", True)])
def test_a_wait_that_gives_up_poisons_its_block_and_nothing_else(P, f, k, dname, op, allreduce):
    """With FTC_DEBUG_ONE_POLL the waits for the asynchronous copies look once and give up. Then: a scenario is either
    played correctly (bit-equal to the oracle) or reports FTC_ST_INTERNAL_TIMEOUT with zero bytes; once a block has
    reported it, every later scenario of that block does; the call returns by itself; and a normal call afterwards on
    the same buffers is bit-equal to the oracle again."""
    desc = B.make_desc(P, f, k, B.dtype_code(np.dtype(DT[dname])), op, root=-1, max_inop=2)
    variant = B.ftc_kernel_variant(desc, allreduce)
    assert variant.startswith("staged/")
    blocks = B.ftc_launch_blocks(desc, 1 << 30, allreduce)
    S = 2 * blocks + 3
    d_x, x, pf, inop, roots = make_batch(P, f, k, dname, allreduce, S, seed=99 + P)
    want = run_oracle_mt(x, f, op, pf, inop, roots, 0, allreduce)
    out, st, _ = run_gpu(None, f, op, pf, inop, roots, 0, allreduce, B.FTC_DEBUG_ONE_POLL, d_x=d_x)
    code = st[:, 0] & 0xFF
    timed_out = code == B.FTC_ST_INTERNAL_TIMEOUT
    ob, wb = out.view(np.uint8).reshape(S, -1), want[0].view(np.uint8).reshape(S, -1)
    assert not ob[timed_out].any() and not st[timed_out, 1:].any()
    assert ((st[timed_out, 0] >> 8) & 0xFF == 0xFF).all()
    assert np.array_equal(st[~timed_out], want[1][~timed_out]) and np.array_equal(ob[~timed_out], wb[~timed_out])
    if not variant.startswith("staged/warp"):                         # sticky per block (the warp kernel hands its blocks runs of
        for b in range(blocks):                                       # consecutive scenarios, whose length the test does not know)
            seq = timed_out[b::blocks]
            assert np.array_equal(seq, np.sort(seq)), (b, seq)
    if variant not in ("staged/whole", "staged/warp", "staged/warp-pair"):   # tile copies are waited for right after their issue
        assert timed_out.any()
    assert_same(run_gpu(None, f, op, pf, inop, roots, 0, allreduce, 0, d_x=d_x), want, f"normal call after the give-up run, {variant}")
