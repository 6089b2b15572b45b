"""The reduce entry point that uses the library's built-in scratch array (collected last on purpose).

Some callers may not allocate device memory at the point where they need a reduce: a latency-critical loop
that cannot afford the device-wide stall of an allocation, or a plug-in living inside another framework's
memory budget. For them ftc_reduce_batch_noalloc keeps the general kernel's scratch inside the library.
The test calls it through the C ABI twice in a row -- the second call finds the first call's leftovers in
the array -- and wants bit-identical results and status records to ftc_reduce_batch on the same inputs
(integer and float32 alike: both run the same kernel, so no tolerance is needed), and to the CPU oracle,
which shares no code with either. The second round also checks that the call took no device memory.
"""
import numpy as np
import pytest

from paper_2602_22445_b200 import binding as B
from paper_2602_22445_b200 import scenarios as sc
from tests.gpu_util import run_gpu, run_oracle, to_dev, to_host

pytestmark = pytest.mark.gpu


def run_noalloc(x, f, op, prefail, inop=None, roots=None, root=0, free_unchanged=False):
    import torch
    d_x = to_dev(x)
    S, P, k = d_x.shape
    max_inop = 0 if inop is None else inop.shape[1]
    desc = B.make_desc(P, f, k, B.dtype_code(d_x.dtype), op, root=-1 if roots is not None else root, max_inop=max_inop)
    d_pf = to_dev(np.ascontiguousarray(prefail, dtype=np.uint32))
    d_inop = to_dev(np.ascontiguousarray(inop, dtype=np.uint32)) if max_inop else None
    d_roots = to_dev(np.ascontiguousarray(roots, dtype=np.uint32)) if roots is not None else None
    d_out = torch.empty((S, k), dtype=d_x.dtype, device="cuda")
    d_out.view(torch.uint8).fill_(0xA5)
    d_st = torch.full((S, 4), 0x7FFFFFFF, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    B.ftc_reduce_batch_noalloc(desc, S, d_x, d_pf, d_inop, d_roots, d_out, d_st)
    torch.cuda.synchronize()
    if free_unchanged:                                   # the device's free memory as the driver reports it
        assert torch.cuda.mem_get_info()[0] == free_before
    return to_host(d_out, x.dtype), d_st.cpu().numpy().view(np.uint32)


def make_case(seed, P, f, k, dtype, S):
    rng = np.random.Generator(np.random.PCG64(seed))
    if dtype == np.float32:
        x = rng.standard_normal((S, P, k)).astype(np.float32)
    else:
        info = np.iinfo(dtype)
        x = rng.integers(info.min, info.max, size=(S, P, k), dtype=dtype, endpoint=True)
    pf = sc.picks_to_masks(sc.random_subsets(rng, S, P, rng.integers(0, f + 2, size=S)), P)
    inop = np.zeros((S, 2, 2), dtype=np.uint32)
    inop[:, :, 0] = rng.integers(0, P, size=(S, 2))
    inop[:, :, 1] = rng.integers(0, 12, size=(S, 2))
    roots = rng.integers(0, P, size=S).astype(np.uint32)
    return x, pf, inop, roots


def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    cases = [make_case(1, 333, 2, 5, np.int32, 700),          # odd k: many blocks share the array
             make_case(2, 1024, 3, 16, np.float32, 300),
             make_case(3, 4096, 4, 32, np.int32, 90)]          # 105 KB per block: fewer blocks than usual fit
    for rep in range(2):
        for x, pf, inop, roots in cases:
            f = {333: 2, 1024: 3, 4096: 4}[x.shape[1]]
            op = "sum" if x.dtype == np.float32 else ("max" if x.shape[1] == 4096 else "sum")
            want_out, want_st, _ = run_gpu(x, f, op, pf, inop, roots, flags=B.FTC_KERNEL_GENERIC)
            got_out, got_st = run_noalloc(x, f, op, pf, inop, roots, free_unchanged=rep == 1)
            assert np.array_equal(got_st, want_st), (rep, x.shape)
            assert np.array_equal(got_out.view(np.uint8), want_out.view(np.uint8)), (rep, x.shape)
            orc_out, orc_st = run_oracle(x, f, op, pf, inop, roots)
            assert np.array_equal(got_st, orc_st), (rep, x.shape)
            assert np.array_equal(got_out.view(np.uint8), orc_out.view(np.uint8)), (rep, x.shape)


def test_noalloc_rejects_shapes_beyond_the_built_in_scratch():
    import torch
    z = torch.zeros(64, dtype=torch.int32, device="cuda")
    # one block's slice: ceil((P-1)/(f+1)) * k * 8 bytes = 65536 * 32 * 8 = 16 MiB > 8 MiB
    big = B.make_desc(2 * 65536 + 1, 1, 32, B.FTC_U64, "sum")
    assert B.ftc_reduce_batch_noalloc(big, 1, z, z, None, None, z, z, check=False) == B.FTC_ETOOLARGE
    assert "built-in scratch" in B.ftc_strerror(B.FTC_ETOOLARGE)
    assert B.ftc_reduce_batch_noalloc(B.make_desc(8, 1, 0, B.FTC_I32, "sum"), 1, z, z, None, None, z, z,
                                      check=False) == B.FTC_EINVAL
    assert B.ftc_reduce_batch_noalloc(B.make_desc(8, 1, 4, B.FTC_I32, "sum"), 0, None, None, None, None, None, None) == B.FTC_OK
    torch.cuda.synchronize()
