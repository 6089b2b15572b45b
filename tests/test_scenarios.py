"""Host-side scenario generators: determinism, value ranges, failure-pattern structure."""
import numpy as np

from paper_2602_22445_b200 import scenarios as sc


def popcount_rows(m):
    return np.unpackbits(m.view(np.uint8), axis=1).sum(axis=1)


def test_inputs_are_a_function_of_seed_scenario_process_element():
    a = sc.gen_inputs(sc.KIND_U64_FULL, 5, [3, 9], 16, 4)
    b = sc.gen_inputs(sc.KIND_U64_FULL, 5, [9], 16, 4)
    assert np.array_equal(a[1], b[0]) and not np.array_equal(a[0], a[1])
    assert not np.array_equal(a, sc.gen_inputs(sc.KIND_U64_FULL, 6, [3, 9], 16, 4))


def test_splitmix64_first_outputs_of_seed_zero():
    # first outputs of the published splitmix64 generator started at state 0
    got = sc._hash(0, np.arange(3, dtype=np.uint64))
    assert [int(v) for v in got] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_value_ranges_and_moments():
    x = sc.gen_inputs(sc.KIND_I32_PM20, 1, range(64), 64, 8)
    assert x.dtype == np.int32 and x.min() >= -(1 << 20) and x.max() <= (1 << 20) and x.min() < -(1 << 19)
    y = sc.gen_inputs(sc.KIND_I64_PM40, 1, range(64), 64, 8)
    assert y.dtype == np.int64 and abs(int(y.min())) <= (1 << 40) and int(y.max()) > (1 << 39)
    z = sc.gen_inputs(sc.KIND_F32_NORMAL, 1, range(32), 256, 16)
    assert z.dtype == np.float32 and abs(float(z.mean())) < 0.02 and abs(float(z.std()) - 1.0) < 0.02
    w = sc.gen_inputs(sc.KIND_I32_FULL, 1, range(8), 64, 8)
    assert w.dtype == np.int32 and w.min() < -(1 << 30) and w.max() > (1 << 30)


def test_config1_and_2_enumerate_all_small_failure_sets():
    c1 = sc.config1()
    assert c1.S == 9 and popcount_rows(c1.prefail).tolist() == [0] + [1] * 8
    c2 = sc.config2(draws=2)
    assert c2.S == 2081 * 2 and popcount_rows(c2.prefail).max() == 2
    assert len({m.tobytes() for m in c2.prefail}) == 2081


def test_config3_sizes_uniform_and_distinct():
    w = sc.config3(S=4000)
    n = popcount_rows(w.prefail)
    assert n.max() == 3 and all(abs((n == i).mean() - 0.25) < 0.04 for i in range(4))
    assert np.array_equal(w.prefail, sc.config3(S=4000).prefail)


def test_config4_victims_avoid_candidates_and_prefailed():
    w = sc.config4(28, S=3000)
    assert w.inop.shape == (3000, 2, 2) and popcount_rows(w.prefail).max() == 2
    vic, rnd = w.inop[:, :, 0].astype(np.int64), w.inop[:, :, 1]
    used = vic != sc.UNUSED
    assert (vic[used] >= w.f + 1).all() and (vic[used] < w.P).all()
    assert (rnd[used] >= 1).all() and (rnd[used] < 28).all() and set(np.unique(used.sum(axis=1))) == {0, 1, 2}
    for i in np.nonzero(used.any(axis=1))[0][:500]:
        for v in vic[i][used[i]]:
            assert not (w.prefail[i, v >> 5] >> (v & 31)) & 1
        if used[i].all():
            assert vic[i, 0] != vic[i, 1]


def test_config5_roots_and_sizes():
    w = sc.config5(S=2000)
    n = popcount_rows(w.prefail)
    assert n.max() == 8 and n.min() == 0 and w.roots.shape == (2000,) and w.roots.max() < w.P
    assert w.host_inputs([0, 1]).shape == (2, 65536, 4)
