"""Pins of the CPU oracle against what the paper and plain mathematics fix (no GPU needed).

Each test names the passage of the paper it rests on. A mistake in the simulator (a dropped
message, a wrong group or tree index, a value combined twice, a swapped operand) fails at least
one of them.
"""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import checker as K
from oracle import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
U64 = np.uint64


def rand_u64(P, k, seed):
    return np.random.Generator(np.random.PCG64(seed)).integers(0, 2**64, size=(P, k), dtype=np.uint64)


def uc_messages(n, f):      # Theorem on the number of messages, up-correction phase
    a = ((n - 1) % (f + 1)) + 1
    return f * (f + 1) * ((n - 1) // (f + 1)) + a * (a - 1)


# ---------------------------------------------------------------------------------------------
# worked example (section "Reduce", prose around the second tree figure)
# ---------------------------------------------------------------------------------------------
def parse_golden():
    d = {}
    for line in open(os.path.join(GOLDEN, "worked_example_n7_f1.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *rest = line.split()
        d[key] = rest
    return d


def test_worked_example_every_printed_number():
    g = parse_golden()
    n, f = int(g["n"][0]), int(g["f"][0])
    failed = [int(v) for v in g["failed"]]
    x = np.arange(n, dtype=np.int64).reshape(n, 1)
    d = O.run(x, f, "sum", failed, detail=True, track_sets=True)
    assert d["code"] == 0 and int(d["result"][0]) == int(g["expected_result"][0]) == 20
    for item in g["after_upcorrection"]:
        p, v = map(int, item.split(":"))
        assert int(d["uc_values"][p, 0]) == v, (p, v)
    for item in g["tree_message"]:
        p, v = map(int, item.split(":"))
        assert d["tree_sent"][p] & 1 and int(d["tree_values"][p, 0]) == v
    for p in map(int, g["no_message"]):
        assert d["tree_sent"][p] == 0
    for item in g["label"]:
        p, ids = item.split(":")
        assert K.bits(d["tree_sets"][int(p)], n) == [int(i) for i in ids.split(",")]
    # the root's child that reports "no failures" is process 2 and its flag is clear
    assert d["subtree"] == 1 and d["cand_flag"][1] == 0 and d["cand_flag"][0] == 2
    assert K.bits(d["contrib"], n) == [0, 2, 3, 4, 5, 6]


def test_worked_example_tree_shape_and_groups():
    """The figure's tree and the exchanging pairs, observed through who receives whose value."""
    g = parse_golden()
    n, f = 7, 1
    x = (U64(1) << np.arange(n, dtype=np.uint64)).reshape(n, 1)      # one-hot inputs: sums are set labels
    d = O.run(x, f, "sum", [], detail=True, track_sets=True)
    # up-correction: exactly the printed pairs hold each other's value, the root holds only its own
    groups = [tuple(int(i) for i in grp.split(",")) for grp in g["groups"]]
    for grp in groups:
        want = sum(1 << i for i in grp)
        for p in grp:
            assert int(d["uc_values"][p, 0]) == want
    assert int(d["uc_values"][0, 0]) == 1
    # tree: a process' message carries its group plus everything its children sent
    parent = dict(tuple(map(int, it.split(":"))) for it in g["parent"])
    msg = {p: int(d["tree_values"][p, 0]) for p in range(1, n)}
    for p in range(1, n):
        kids = [c for c, par in parent.items() if par == p]
        expect = int(d["uc_values"][p, 0])
        for c in kids:
            expect += msg[c]          # multiset sum: a label counted twice would show as a carry
        assert msg[p] == expect


# ---------------------------------------------------------------------------------------------
# Theorem (number of messages) and "when processes fail, fewer messages are sent"
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n,f", [(n, f) for f in range(0, 5) for n in range(f + 2, 20)] +
                         [(8, 1), (64, 2), (1024, 3), (4096, 4)])
def test_message_counts_failure_free(n, f):
    x = np.ones((n, 1), dtype=np.int32)
    d = O.run(x, f, "sum", [], detail=True)
    assert int(d["msgs"][0]) == uc_messages(n, f)
    assert int(d["msgs"][1]) == n - 1
    assert int(d["result"][0]) == n


def test_message_counts_config5_and_printed_values():
    # values evaluated from the theorem for the five configurations
    table = {(8, 1): (8, 7), (64, 2): (126, 63), (1024, 3): (3072, 1023), (4096, 4): (16380, 4095),
             (65536, 8): (524274, 65535)}
    for (n, f), (uc, tree) in table.items():
        assert uc_messages(n, f) == uc and tree == n - 1
    n, f = 65536, 8
    d = O.run(np.ones((n, 1), dtype=np.int32), f, "sum", [], detail=True)
    assert (int(d["msgs"][0]), int(d["msgs"][1])) == table[(n, f)]


@pytest.mark.parametrize("n,f", [(7, 1), (11, 2), (14, 3), (9, 2)])
def test_fewer_messages_with_failures_and_nobody_sends_more(n, f):
    x = np.ones((n, 1), dtype=np.int32)
    base = O.run(x, f, "sum", [], detail=True)
    for size in range(1, f + 1):
        for dead in itertools.combinations(range(n), size):
            d = O.run(x, f, "sum", dead, detail=True)
            assert np.all(d["sends"] <= base["sends"])
            for p in dead:
                assert d["sends"][p] == 0
            live = [p for p in range(n) if p not in dead]
            assert np.array_equal(d["sends"][live], base["sends"][live])     # no process sends more, or fewer
            assert int(d["msgs"][0] + d["msgs"][1]) == int(base["sends"][live].sum())


# ---------------------------------------------------------------------------------------------
# Semantics of reduce with pre-operation failures: unique correct result = reduction over the
# non-failed processes (sections "Semantics", "Failure information": "only one correct result")
# ---------------------------------------------------------------------------------------------
def _exhaustive_cases():
    for f in (1, 2, 3):
        for n in range(f + 2, 13):
            yield n, f


@pytest.mark.parametrize("n,f", list(_exhaustive_cases()))
def test_reduce_equals_direct_reduction_over_survivors_exhaustive(n, f):
    x = rand_u64(n, 2, 1000 * n + f)       # random 64-bit weights: a sum matches only if every survivor is in
    roots = range(n) if n <= 9 else (0, 1, f + 1, n - 1)      # exactly once and no failed process is in at all
    for size in range(0, f + 1):
        for dead in itertools.combinations(range(n), size):
            for root in roots:
                d = O.run(x, f, "sum", dead, root=root, track_sets=True, detail=True)
                live = [p for p in range(n) if p not in dead]
                if root in dead:
                    assert d["code"] == 1 and not d["result"].any()          # reduce to a failed root: no-op
                    continue
                assert d["code"] == 0, (n, f, dead, root)                     # a failure-free subtree exists
                assert np.array_equal(d["result"], K.reduce_over(x, live, "sum"))
                assert K.bits(d["contrib"], n) == live and d["count"] == len(live)
                assert d["cand_flag"][d["subtree"]] == 0
                assert all(d["cand_flag"][s] != 0 for s in range(d["subtree"]))


@pytest.mark.parametrize("op,dtype", [("max", np.int32), ("xor", np.uint64), ("sum", np.int64), ("max", np.int64),
                                      ("max", np.uint64), ("xor", np.int32)])
def test_other_ops_and_dtypes_match_definition(op, dtype):
    n, f = 11, 2
    rng = np.random.Generator(np.random.PCG64(7))
    info = np.iinfo(dtype)
    x = rng.integers(info.min, info.max, size=(n, 3), dtype=dtype, endpoint=True)
    for dead in itertools.chain([()], itertools.combinations(range(n), 1), itertools.combinations(range(n), 2)):
        for root in (0, 4):
            if root in dead:
                continue
            d = O.run(x, f, op, dead, root=root)
            live = [p for p in range(n) if p not in dead]
            assert np.array_equal(d["result"], K.reduce_over(x, live, op)), (op, dead, root)


def test_integer_sum_wraps():
    x = np.full((5, 1), 2**31 - 1, dtype=np.int32)
    d = O.run(x, 1, "sum", [])
    assert int(d["result"][0]) == ((5 * (2**31 - 1) + 2**31) % 2**32) - 2**31


def test_more_than_f_failures_never_yield_a_wrong_value():
    """Outside the theorems' hypothesis: the result is right or the root reports no failure-free subtree."""
    n, f = 10, 2
    x = rand_u64(n, 1, 5)
    seen = set()
    for dead in itertools.combinations(range(1, n), f + 1):
        d = O.run(x, f, "sum", dead)
        live = [p for p in range(n) if p not in dead]
        seen.add(d["code"])
        if d["code"] == 0:
            assert np.array_equal(d["result"], K.reduce_over(x, live, "sum"))
        else:
            assert d["code"] == 2 and not d["result"].any()
    assert seen == {0, 2}


# ---------------------------------------------------------------------------------------------
# copies of every value that reach the root in the failure-free case (section "Algorithm":
# "include each value f+1 times", made exact): a process of a full group is in f+1 child
# messages; a member of the last, short group (root included) in r child messages
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n,f", [(7, 1), (8, 1), (12, 2), (13, 3), (16, 3), (30, 4)])
def test_copies_of_each_value_at_the_root(n, f):
    d = O.run(np.ones((n, 1), np.int32), f, "sum", [], detail=True, track_sets=True)
    q, r = (n - 1) // (f + 1), (n - 1) % (f + 1)
    copies = np.zeros(n, dtype=int)
    for s in range(f + 1):
        child = s + 1
        for p in K.bits(d["tree_sets"][child], n):
            copies[p] += 1
    for p in range(1, n):
        full = (p - 1) // (f + 1) < q
        assert copies[p] == (f + 1 if full else r)
    assert copies[0] == r
    # sizes of the root's subtrees differ by at most one (definition of the I(f)-tree)
    sizes = [int(d["tree_values"][s + 1, 0]) for s in range(f + 1)]    # inputs are 1: value = values included
    assert d["cand_flag"].tolist() == [0] * (f + 1)
    incl = [len(K.bits(d["tree_sets"][s + 1], n)) for s in range(f + 1)]
    assert incl == sizes


# ---------------------------------------------------------------------------------------------
# in-operation failures (Theorem on the semantics, item 4): every (victim, round), value equals the
# reduction over Live plus a subset of the victims, never a partial or doubled contribution
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n,f", [(6, 1), (7, 1), (8, 2), (11, 2), (12, 3), (14, 3)])
def test_inop_reduce_allowed_results_exhaustive(n, f):
    x = rand_u64(n, 1, 77 * n + f)
    rounds = O.schedule(n, f)["rounds_reduce"]
    outcomes = set()
    for victim in range(n):
        for t in range(1, rounds + 2):
            for pre in itertools.chain([()], itertools.combinations([p for p in range(1, n) if p != victim], 1)
                                       if f >= 2 else []):
                d = O.run(x, f, "sum", pre, inop=[(victim, t)], track_sets=True, detail=True)
                if victim == 0:
                    if t < rounds:
                        assert d["code"] == 1            # the root failed: no-op
                        continue
                assert d["code"] == 0, (victim, t, pre)
                C = K.bits(d["contrib"], n)
                assert K.contribution_allowed(n, C, pre, [victim])
                assert np.array_equal(d["result"], K.reduce_over(x, C, "sum"))
                assert d["count"] == len(C) and d["inop_included"] == int(victim in C)
                outcomes.add(victim in C)
                if t >= rounds:
                    assert victim in C                   # it completed every send of the reduce
    # with f = 1 a victim's only up-correction send is round 0, so a round >= 1 always includes it
    assert outcomes == ({True, False} if f >= 2 else {True})


def test_inop_value_can_arrive_along_one_path_and_not_another():
    """Section "Failure information": a process that completes up-correction but not its tree send
    reaches the root through its partners only."""
    n, f = 7, 1
    x = (U64(1) << np.arange(n, dtype=np.uint64)).reshape(n, 1)
    sch = O.schedule(n, f)
    # process 3 (depth 2) sends to its partner 4 in round 0, its tree send is round f+H-2 = 1
    d = O.run(x, f, "sum", [], inop=[(3, 1)], detail=True, track_sets=True)
    assert d["cand_flag"].tolist() == [1, 0] and d["subtree"] == 1
    assert K.bits(d["contrib"], n) == list(range(n))
    d = O.run(x, f, "sum", [], inop=[(4, 1)], detail=True, track_sets=True)    # 4 is in subtree 1
    assert d["cand_flag"].tolist() == [0, 1] and d["subtree"] == 0
    assert K.bits(d["contrib"], n) == list(range(n))
    assert sch["rounds_reduce"] == 3


# ---------------------------------------------------------------------------------------------
# allreduce (Algorithm "Allreduce", its semantics and the theorem on its number of messages)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n,f", [(6, 1), (9, 2), (12, 3), (13, 2)])
def test_allreduce_semantics_exhaustive_pre_op(n, f):
    x = rand_u64(n, 2, 31 * n + f)
    free = O.run(x, f, "sum", [], allreduce=True, detail=True)
    per_attempt = int(free["msgs"][:4].sum())
    assert int(free["msgs"][2]) == n - 1                       # the value travels down the same tree
    assert int(free["msgs"][0]) == uc_messages(n, f) and int(free["msgs"][1]) == n - 1
    for size in range(0, f + 1):
        for dead in itertools.combinations(range(n), size):
            for first in (0, 3):
                d = O.run(x, f, "sum", dead, root=first, allreduce=True, detail=True, track_sets=True)
                live = [p for p in range(n) if p not in dead]
                lead = 0
                while (first + lead) % n in dead:
                    lead += 1
                assert d["code"] == 0 and d["attempts"] == lead + 1       # one attempt per failed candidate
                want = K.reduce_over(x, live, "sum")
                assert np.array_equal(d["result"], want)
                assert K.bits(d["holders"], n) == live and d["n_holders"] == len(live)
                for p in range(n):                                       # every live process holds the same bits
                    assert np.array_equal(d["expanded"][p], want if p in live else np.zeros_like(want))
                assert int(d["msgs"][:4].sum()) <= (f + 1) * per_attempt   # at most (f+1)-fold
                ev = d["events"]
                assert all(ev[p] == 3 for p in live) and all(ev[p] == 0 for p in dead)


def test_allreduce_no_live_candidate_and_inop_candidate():
    n, f = 8, 1
    x = rand_u64(n, 1, 3)
    d = O.run(x, f, "sum", [0, 1], allreduce=True)
    assert d["code"] == 3 and d["attempts"] == 2 and not d["result"].any()
    d = O.run(x, f, "sum", [], inop=[(1, 2)], allreduce=True)
    assert d["code"] == 4


@pytest.mark.parametrize("n,f", [(7, 1), (10, 2), (13, 3)])
def test_allreduce_inop_all_or_nothing_and_consistent(n, f):
    """Allreduce semantics items 4 and 5 under one in-operation failure outside the candidates."""
    x = rand_u64(n, 1, 900 + n)
    R = O.schedule(n, f)["rounds_attempt"]
    for victim in range(f + 1, n):
        for t in range(1, R + 1):
            d = O.run(x, f, "sum", [], inop=[(victim, t)], allreduce=True, detail=True, track_sets=True)
            assert d["code"] == 0
            C = K.bits(d["contrib"], n)
            assert K.contribution_allowed(n, C, [], [victim])
            want = K.reduce_over(x, C, "sum")
            holders = K.bits(d["holders"], n)
            alive_end = [p for p in range(n) if p != victim or t >= R]
            assert holders == alive_end
            for p in holders:
                assert np.array_equal(d["expanded"][p], want)


def test_allreduce_dead_first_candidate_then_inop_victim_counts_as_failed_before():
    """A victim that dies during a fruitless first attempt is dead from the start of the second."""
    n, f = 9, 2
    x = rand_u64(n, 1, 11)
    R = O.schedule(n, f)["rounds_attempt"]
    d = O.run(x, f, "sum", [0], inop=[(5, 1)], allreduce=True, detail=True, track_sets=True)
    assert d["attempts"] == 2 and K.bits(d["contrib"], n) == [1, 2, 3, 4, 6, 7, 8]
    # second attempt, root 1: process 5 (group {4,5,6}, subtree of root child 2 -> unclean once 5 is gone) sends
    # to 4 in local round 0 and to 6 in local round 1; subtree of child 1 has the dead process 0 at its top,
    # so the root takes child 3, whose member of that group is 6
    d = O.run(x, f, "sum", [0], inop=[(5, R + 1)], allreduce=True, detail=True, track_sets=True)
    assert d["attempts"] == 2 and d["subtree"] == 2 and K.bits(d["contrib"], n) == [1, 2, 3, 4, 6, 7, 8]
    d = O.run(x, f, "sum", [0], inop=[(5, R + 2)], allreduce=True, detail=True, track_sets=True)
    assert d["attempts"] == 2 and d["subtree"] == 2 and K.bits(d["contrib"], n) == [1, 2, 3, 4, 5, 6, 7, 8]
    assert K.bits(d["holders"], n) == [1, 2, 3, 4, 6, 7, 8]


# ---------------------------------------------------------------------------------------------
# protocol items 1, 2, 5 of the reduce semantics, seen through the event log
# ---------------------------------------------------------------------------------------------
def test_reduce_events_init_and_deliver_once():
    n, f = 12, 2
    x = rand_u64(n, 1, 2)
    for dead in itertools.combinations(range(1, n), 2):
        d = O.run(x, f, "sum", dead, detail=True)
        for p in range(n):
            assert d["events"][p] == (0 if p in dead else 3)        # init once, deliver exactly once


# ---------------------------------------------------------------------------------------------
# the scheduler is irrelevant: any interleaving of the processes gives the same messages
# ---------------------------------------------------------------------------------------------
def test_result_independent_of_scheduler_order():
    n, f = 23, 3
    x = np.random.Generator(np.random.PCG64(4)).standard_normal((n, 3)).astype(np.float32)
    for allred in (False, True):
        for dead, inop in (((), ()), ((2,), ((9, 2),)), ((5, 6), ((7, 1), (22, 4)))):
            ref = O.run(x, f, "sum", dead, inop=list(inop), allreduce=allred, detail=True)
            for sweep in (1, 2, 3, 99):
                d = O.run(x, f, "sum", dead, inop=list(inop), allreduce=allred, sweep=sweep, detail=True)
                for key in ("result", "status", "cand", "cand_flag", "msgs", "sends", "tree_values", "expanded"):
                    assert np.array_equal(ref[key], d[key]), (key, sweep)


# ---------------------------------------------------------------------------------------------
# float32
# ---------------------------------------------------------------------------------------------
def test_f32_within_tolerance_of_float64_sum():
    n, f = 1024, 3
    rng = np.random.Generator(np.random.PCG64(9))
    x = rng.standard_normal((n, 16)).astype(np.float32)
    for dead in ((), (0,), (1, 2, 3), (17, 500, 1023)):
        d = O.run(x, f, "sum", dead, allreduce=True)
        live = [p for p in range(n) if p not in dead]
        assert d["code"] == 0 and K.value_matches(x, live, "sum", d["result"])


def test_f32_small_integers_are_exact():
    n, f = 200, 3
    x = np.random.Generator(np.random.PCG64(1)).integers(-1000, 1000, size=(n, 4)).astype(np.float32)
    d = O.run(x, f, "sum", [3, 50])
    live = [p for p in range(n) if p not in (3, 50)]
    assert np.array_equal(d["result"].astype(np.int64), x[live].astype(np.int64).sum(axis=0))


def test_f32_combine_order_of_the_documented_reading():
    """n=5, f=1: groups {1,2},{3,4}; tree 0->{1,2}, 1->{3}, 2->{4}. The root takes child 1:
    result = x0 + ((x1+x2) + (x3+x4)), each parenthesis one float32 rounding, accumulator left."""
    x = np.array([[1.0], [1e8], [3.0], [-1e8], [5.0]], dtype=np.float32)
    f32 = np.float32
    want = f32(x[0, 0] + f32(f32(x[1, 0] + x[2, 0]) + f32(x[3, 0] + x[4, 0])))
    d = O.run(x, 1, "sum", [])
    assert d["result"][0] == want
    # with process 1 failed the root takes child 2: x0 + ((x2) + (x4 + x3))
    want2 = f32(x[0, 0] + f32(x[2, 0] + f32(x[4, 0] + x[3, 0])))
    d = O.run(x, 1, "sum", [1])
    assert d["result"][0] == want2 and d["subtree"] == 1


def test_schedule_constants_of_the_five_configurations():
    want = {(8, 1): (3, 4, 8), (64, 2): (5, 7, 14), (1024, 3): (9, 12, 24), (4096, 4): (10, 14, 28),
            (65536, 8): (13, 21, 42)}
    for (n, f), (H, rr, ra) in want.items():
        s = O.schedule(n, f)
        assert (s["H"], s["rounds_reduce"], s["rounds_attempt"]) == (H, rr, ra)
        assert s["H"] == 1 + math.floor(math.log2(math.ceil((n - 1) / (f + 1))))


# ---------------------------------------------------------------------------------------------
# hand-evaluated cases of the documented readings (orders and the round clock), so that a change
# of a reading cannot slip through unnoticed
# ---------------------------------------------------------------------------------------------
def test_reading_children_order_and_root_first_in_last_group_f32():
    f32 = np.float32
    # n=7, f=1: 1 -> {3,5}: message of 1 = ((x1+x2) + (x3+x4)) + (x5+x6); root adds its own on the left
    x = np.array([[0.5], [1e8], [1.0], [-1e8], [3.0], [7.0], [-5.0]], dtype=np.float32)
    v1 = f32(f32(f32(x[1, 0] + x[2, 0]) + f32(x[3, 0] + x[4, 0])) + f32(x[5, 0] + x[6, 0]))
    d = O.run(x, 1, "sum", [], detail=True)
    assert d["tree_values"][1, 0] == v1 and d["result"][0] == f32(x[0, 0] + v1)
    swapped = f32(f32(f32(x[1, 0] + x[2, 0]) + f32(x[5, 0] + x[6, 0])) + f32(x[3, 0] + x[4, 0]))
    assert swapped != v1            # the inputs do tell the two orders apart
    # n=6, f=2: groups {1,2,3} and the short one {4,5,root}; the root takes child 1, whose subtree holds 4:
    # message of 4 = (x4 + x0) + x5 (the root is the first partner), message of 1 = ((x1+x2)+x3) + that
    y = np.array([[1e8], [2.0], [3.0], [4.0], [-1e8], [1.0]], dtype=np.float32)
    m4 = f32(f32(y[4, 0] + y[0, 0]) + y[5, 0])
    assert m4 != f32(f32(y[4, 0] + y[5, 0]) + y[0, 0])
    d = O.run(y, 2, "sum", [], detail=True)
    assert d["tree_values"][4, 0] == m4
    assert d["result"][0] == f32(f32(f32(y[1, 0] + y[2, 0]) + y[3, 0]) + m4) and d["subtree"] == 0


def test_reading_round_clock_of_tree_sends():
    """n=7, f=1: H=2; leaves (depth 2) send to their parents in round f+H-2 = 1, root children in round 2."""
    x = (U64(1) << np.arange(7, dtype=np.uint64)).reshape(7, 1)
    flags = lambda vic, t: O.run(x, 1, "sum", [], inop=[(vic, t)], detail=True)["cand_flag"].tolist()
    assert flags(3, 1) == [1, 0] and flags(3, 2) == [0, 0]
    assert flags(1, 2) == [2, 0] and flags(1, 3) == [0, 0]
    assert flags(2, 2) == [0, 2] and flags(2, 3) == [0, 0]


def test_reading_partner_order_decides_whom_a_dying_process_reached():
    """n=6, f=2, short last group {4, 5, root}: process 5 sends to the root in round 0 and to 4 in round 1.
    Subtree of child 1 (holding 4) is chosen; it has 5's value only if the second send happened."""
    x = (U64(1) << np.arange(6, dtype=np.uint64)).reshape(6, 1)
    d = O.run(x, 2, "sum", [], inop=[(5, 1)], detail=True, track_sets=True)
    assert d["subtree"] == 0 and K.bits(d["contrib"], 6) == [0, 1, 2, 3, 4]
    d = O.run(x, 2, "sum", [], inop=[(5, 2)], detail=True, track_sets=True)
    assert d["subtree"] == 0 and K.bits(d["contrib"], 6) == [0, 1, 2, 3, 4, 5]
    # full group {1,2,3}: process 3 sends to 1 in round 0, to 2 in round 1, up the tree in round f+H-1 = 2
    d = O.run(x, 2, "sum", [1], inop=[(3, 1)], detail=True, track_sets=True)
    assert d["subtree"] == 1 and K.bits(d["contrib"], 6) == [0, 2, 4, 5]
    d = O.run(x, 2, "sum", [1], inop=[(3, 2)], detail=True, track_sets=True)
    assert d["subtree"] == 1 and K.bits(d["contrib"], 6) == [0, 2, 3, 4, 5]


def test_reading_broadcast_correction_is_sent_by_tree_holders_only():
    """n=10, f=2, allreduce from root 0 with 2 and 3 failed beforehand and 4 dying after its first
    correction send (three failures: outside the theorems, played anyway). 4 is the only process of
    {4,5,6} the tree reaches; it hands the value to 5 and dies; 5 does not pass it on to 6."""
    x = rand_u64(10, 1, 8)
    sch = O.schedule(10, 2)
    assert (sch["H"], sch["rounds_reduce"], sch["rounds_attempt"]) == (2, 4, 8)
    first_corr = sch["rounds_reduce"] + sch["H"]                # round of correction iteration 0
    d = O.run(x, 2, "sum", [2, 3], inop=[(4, first_corr + 1)], allreduce=True, detail=True, track_sets=True)
    assert d["code"] == 0 and d["subtree"] == 0
    assert K.bits(d["holders"], 10) == [0, 1, 5, 7, 8, 9]
    d = O.run(x, 2, "sum", [2, 3], inop=[(4, first_corr + 2)], allreduce=True, detail=True, track_sets=True)
    # a failure round equal to the attempt's length: every send was made and the process is alive at the end
    assert first_corr + 2 == sch["rounds_attempt"] and K.bits(d["holders"], 10) == [0, 1, 4, 5, 6, 7, 8, 9]
    d = O.run(x, 2, "sum", [2, 3], inop=[(4, first_corr)], allreduce=True, detail=True, track_sets=True)
    assert K.bits(d["holders"], 10) == [0, 1, 7, 8, 9]


def test_leaf_has_no_tree_down_send_to_miss():
    """f = 0: the deepest leaves would send down the tree in the round the attempt ends; they have no
    children, so a failure round equal to the attempt's length leaves them alive and holding the value."""
    n = 12
    x = rand_u64(n, 1, 6)
    sch = O.schedule(n, 0)
    assert sch["rounds_attempt"] == 2 * sch["H"]
    leaf = n - 1
    d = O.run(x, 0, "sum", [], inop=[(leaf, sch["rounds_attempt"])], allreduce=True, detail=True)
    assert d["n_holders"] == n and leaf in K.bits(d["holders"], n)
    d = O.run(x, 0, "sum", [], inop=[(leaf, sch["rounds_attempt"] - 1)], allreduce=True, detail=True)
    assert d["n_holders"] == n - 1 and leaf not in K.bits(d["holders"], n)


# ---------------------------------------------------------------------------------------------
# failure information, first and second scheme (section "Failure information"): a child without a failure
# in its subtree hands the root the complete list of failed processes; concatenated lists are disjoint, so
# the list's size can be tracked instead of the list
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n,f", [(7, 1), (9, 2), (12, 2), (13, 3)])
def test_failed_process_list_is_complete_and_duplicate_free(n, f):
    x = rand_u64(n, 1, 5 * n + f)
    for size in range(0, f + 1):
        for dead in itertools.combinations(range(n), size):
            for root in (0, 2):
                if root in dead:
                    continue
                d = O.run(x, f, "sum", dead, root=root, track_sets=True, detail=True)
                assert K.bits(d["failed"], n) == list(dead)                 # complete list from the clean child
                assert int(d["nfail"][0]) == len(dead)                      # its size: no id listed twice
                assert d["cand_flag"][d["subtree"]] == 0


def test_failed_list_under_inop_failure_is_the_complement_of_the_contributions():
    n, f = 11, 2
    x = rand_u64(n, 1, 3)
    R = O.schedule(n, f)["rounds_reduce"]
    for victim in range(1, n):
        for t in range(1, R + 1):
            for pre in ((), ((victim % (n - 1)) + 1,)):
                if victim in pre:
                    continue
                d = O.run(x, f, "sum", pre, inop=[(victim, t)], track_sets=True, detail=True)
                C = K.bits(d["contrib"], n)
                assert K.bits(d["failed"], n) == [p for p in range(n) if p not in C]
                assert int(d["nfail"][0]) == n - len(C)


# ---------------------------------------------------------------------------------------------
# Other subtree shapes: below each root child an a-ary heap instead of the binary one. The paper fixes only
# the I(f)-tree property (f+1 root children, subtree sizes within one of each other: definition before the
# first theorem of section "Properties"), so every statement pinned above must hold for these shapes too.
# ---------------------------------------------------------------------------------------------
ARITIES = [3, 4, 5, 1]          # 1 = binomial tree


def test_arity_tree_structure_by_hand():
    """n = 14, f = 1, ternary: subtree 0 holds ranks 1,3,..,13 (local index j = (v-1)/2); node j has children
    3j+1..3j+3, so rank 1 receives from 3, 5, 7 and rank 3 from 9, 11, 13. A tree message carries the groups of
    the sender's whole subtree (each group {2j+1, 2j+2}; the short last group {13} also holds the root)."""
    n, f = 14, 1
    x = (U64(1) << np.arange(n, dtype=np.uint64)).reshape(n, 1)
    d = O.run(x, f, "sum", [], detail=True, track_sets=True, arity=3)
    sets = {v: K.bits(d["tree_sets"][v], n) for v in range(1, n)}
    assert sets[3] == sorted([3, 4, 9, 10, 11, 12, 13, 0])
    assert sets[5] == [5, 6] and sets[7] == [7, 8] and sets[9] == [9, 10] and sets[13] == [0, 13]
    assert sets[1] == list(range(n))                       # root child 1 collects every group once
    assert sets[2] == sorted([2, 1] + sets[4] + sets[6] + sets[8])
    assert sets[4] == sorted([4, 3, 10, 9, 12, 11])          # j = 1 of subtree 1: children j = 4, 5 (rank 14 does not exist)
    assert int(d["result"][0]) == (1 << n) - 1
    # depth of the deepest node: rows 0..6 fill ternary levels 1 + 3 + 3, binary levels 1 + 2 + 4: H = 3 either way;
    # n = 20 (rows 0..9): binary 1+2+4+3 -> H = 4, ternary 1+3+6 -> H = 3
    assert O.schedule(14, 1, 3)["H"] == 3 and O.schedule(14, 1, 2)["H"] == 3
    assert O.schedule(20, 1, 2)["H"] == 4 and O.schedule(20, 1, 3)["H"] == 3 and O.schedule(20, 1, 4)["H"] == 3


def test_arity_f32_children_combined_in_ascending_order():
    """Algorithm "reduce_non_root" with three children: data <- ((data + c1) + c2) + c3 in float32."""
    n, f = 5, 0                      # one subtree: ranks 1..4, rank 1 has children 2, 3, 4; no up-correction
    vals = np.array([0.0, 1.0, 2.0**24, 1.0, -(2.0**24)], dtype=np.float32).reshape(n, 1)
    d = O.run(vals, f, "sum", [], arity=3)
    acc = np.float32(1.0)
    for c in (2, 3, 4):
        acc = np.float32(acc + vals[c, 0])
    assert d["result"][0] == np.float32(np.float32(0.0) + acc) and d["result"][0] == np.float32(0.0)
    d2 = O.run(vals, f, "sum", [], arity=2)               # binary: 1 <- (1 + (2 + 4)) + 3: another rounding
    assert d2["result"][0] == np.float32(2.0)


def test_binomial_tree_structure_by_hand():
    """n = 14, f = 1, binomial: in subtree 0 (ranks 1,3,..,13; local index j = (v-1)/2) the parent of j is j without
    its lowest set bit: 0 <- 1, 2, 4;  2 <- 3;  4 <- 5, 6. So rank 1 receives from ranks 3, 5, 9, rank 5 from 7,
    rank 9 from 11 and 13; depth = 1 + number of set bits of j, the deepest being j = 3, 5, 6 at depth 3."""
    n, f = 14, 1
    x = (U64(1) << np.arange(n, dtype=np.uint64)).reshape(n, 1)
    d = O.run(x, f, "sum", [], detail=True, track_sets=True, arity=1)
    sets = {v: K.bits(d["tree_sets"][v], n) for v in range(1, n)}
    assert sets[3] == [3, 4] and sets[7] == [7, 8] and sets[11] == [11, 12] and sets[13] == [0, 13]
    assert sets[5] == [5, 6, 7, 8]                                  # j = 2 with its child j = 3
    assert sets[9] == sorted([9, 10, 11, 12, 13, 0])                # j = 4 with j = 5 and j = 6 (short group: the root too)
    assert sets[1] == list(range(n))
    assert int(d["result"][0]) == (1 << n) - 1
    assert O.schedule(14, 1, 1)["H"] == 3 and O.schedule(17, 0, 1)["H"] == 1 + 4     # 16 rows: j = 15 has four set bits
    # a leaf that dies before its tree send (depth 3: round f+H-3 = 1) taints only its own chain: 7 -> 5 -> 1
    d = O.run(x, f, "sum", [], inop=[(7, 1)], detail=True, track_sets=True, arity=1)
    assert d["cand_flag"].tolist() == [1, 0] and d["subtree"] == 1


def test_binomial_f32_children_in_ascending_order():
    n, f = 5, 0                      # one subtree: ranks 1..4 = j 0..3; 0 <- 1, 2;  2 <- 3
    vals = np.array([0.0, 1.0, 2.0**24, 1.0, -(2.0**24)], dtype=np.float32).reshape(n, 1)
    d = O.run(vals, f, "sum", [], arity=1)
    inner = np.float32(vals[3, 0] + vals[4, 0])                     # rank 3 (j = 2) takes rank 4 (j = 3)
    want = np.float32(np.float32(np.float32(vals[1, 0] + vals[2, 0]) + inner))   # rank 1: its j = 1 child, then j = 2
    assert d["result"][0] == np.float32(np.float32(0.0) + want)


@pytest.mark.parametrize("arity", ARITIES)
def test_arity_message_counts_do_not_depend_on_the_shape(arity):
    for f in range(0, 4):
        for n in list(range(f + 2, 24)) + [64, 257]:
            d = O.run(np.ones((n, 1), dtype=np.int32), f, "sum", [], detail=True, arity=arity)
            assert (int(d["msgs"][0]), int(d["msgs"][1])) == (uc_messages(n, f), n - 1)
            assert int(d["result"][0]) == n
            da = O.run(np.ones((n, 1), dtype=np.int32), f, "sum", [], allreduce=True, detail=True, arity=arity)
            assert [int(v) for v in da["msgs"][:4]] == [uc_messages(n, f), n - 1, n - 1, uc_messages(n, f)]


@pytest.mark.parametrize("arity", ARITIES)
@pytest.mark.parametrize("n,f", [(9, 1), (14, 1), (13, 2), (16, 2), (17, 3)])
def test_arity_reduce_equals_direct_reduction_exhaustive(n, f, arity):
    x = rand_u64(n, 2, 500 * n + f + arity)
    for size in range(0, f + 1):
        for dead in itertools.combinations(range(n), size):
            for root in (0, 2, n - 1):
                d = O.run(x, f, "sum", dead, root=root, track_sets=True, detail=True, arity=arity)
                live = [p for p in range(n) if p not in dead]
                if root in dead:
                    assert d["code"] == 1 and not d["result"].any()
                    continue
                assert d["code"] == 0
                assert np.array_equal(d["result"], K.reduce_over(x, live, "sum"))
                assert K.bits(d["contrib"], n) == live and d["count"] == len(live)


@pytest.mark.parametrize("arity", ARITIES)
@pytest.mark.parametrize("n,f", [(10, 1), (14, 2), (17, 3)])
def test_arity_inop_allowed_results_and_allreduce_consistency(n, f, arity):
    x = rand_u64(n, 1, 91 * n + f + arity)
    sch = O.schedule(n, f, arity)
    for victim in range(f + 1, n):
        for t in range(1, sch["rounds_attempt"] + 2):
            for allred in (False, True):
                if not allred and t > sch["rounds_reduce"] + 1:
                    continue
                d = O.run(x, f, "sum", [1] if f >= 2 and victim != 1 else [], inop=[(victim, t)], allreduce=allred,
                          track_sets=True, detail=True, arity=arity)
                pre = [1] if f >= 2 and victim != 1 else []
                assert d["code"] == 0
                C = K.bits(d["contrib"], n)
                assert K.contribution_allowed(n, C, pre, [victim])
                assert np.array_equal(d["result"], K.reduce_over(x, C, "sum"))
                if allred:
                    holders = K.bits(d["holders"], n)
                    alive_end = [p for p in range(n) if p not in pre and not (p == victim and t < sch["rounds_attempt"])]
                    assert holders == alive_end                  # at most f failures: every survivor holds the value
                    for p in holders:
                        assert np.array_equal(d["expanded"][p], d["result"])


# ---------------------------------------------------------------------------------------------
# The other partner order: Algorithm "Up-correction" leaves the order of "p in group \ {self}" open; besides the
# ascending order (root first) the oracle plays the descending one (root last). Every semantic pin must hold for it.
# ---------------------------------------------------------------------------------------------
def test_descending_partner_order_decides_whom_a_dying_process_reached():
    """The mirror image of the ascending case: n=6, f=2, short last group {4, 5, root}: process 5 now sends to 4 in
    round 0 and to the root in round 1; process 3 of the full group {1,2,3} sends to 2 first, then to 1."""
    x = (U64(1) << np.arange(6, dtype=np.uint64)).reshape(6, 1)
    d = O.run(x, 2, "sum", [], inop=[(5, 1)], detail=True, track_sets=True, partners_descending=True)
    assert d["subtree"] == 0 and K.bits(d["contrib"], 6) == [0, 1, 2, 3, 4, 5]      # 4 (subtree 0) got 5's value
    d = O.run(x, 2, "sum", [1], inop=[(3, 1)], detail=True, track_sets=True, partners_descending=True)
    assert d["subtree"] == 1 and K.bits(d["contrib"], 6) == [0, 2, 3, 4, 5]          # 2 got 3's value in round 0
    d = O.run(x, 2, "sum", [2], inop=[(3, 1)], detail=True, track_sets=True, partners_descending=True)
    assert d["subtree"] == 0 and K.bits(d["contrib"], 6) == [0, 1, 4, 5]             # the send to 2 was wasted, 1 got nothing


def test_descending_partner_order_f32_fold():
    """Group {1,2,3} (f=2, n=4, root 0 in no group): rank 1 folds own + x3 + x2, where ascending gives own + x2 + x3."""
    vals = np.array([0.0, 1.0, 2.0**24, -(2.0**24)], dtype=np.float32).reshape(4, 1)
    asc = O.run(vals, 2, "sum", [])
    desc = O.run(vals, 2, "sum", [], partners_descending=True)
    a = np.float32(np.float32(vals[1, 0] + vals[2, 0]) + vals[3, 0])      # (1 + 2^24) - 2^24 = 0
    b = np.float32(np.float32(vals[1, 0] + vals[3, 0]) + vals[2, 0])      # (1 - 2^24) + 2^24 = 0 as well: use the root add
    assert asc["result"][0] == np.float32(np.float32(0.0) + a)
    assert desc["result"][0] == np.float32(np.float32(0.0) + b)
    vals2 = np.array([0.0, 2.0**24, 1.0, 1.0 - 2.0**-23], dtype=np.float32).reshape(4, 1)   # order of the two small addends shows
    asc, desc = O.run(vals2, 2, "sum", []), O.run(vals2, 2, "sum", [], partners_descending=True)
    assert asc["result"][0] == np.float32(np.float32(vals2[1, 0] + vals2[2, 0]) + vals2[3, 0])
    assert desc["result"][0] == np.float32(np.float32(vals2[1, 0] + vals2[3, 0]) + vals2[2, 0])


@pytest.mark.parametrize("n,f", [(7, 1), (9, 2), (12, 2), (13, 3), (16, 3)])
def test_descending_partner_order_semantics(n, f):
    x = rand_u64(n, 2, 17 * n + f)
    base = O.run(np.ones((n, 1), dtype=np.int32), f, "sum", [], allreduce=True, detail=True, partners_descending=True)
    assert [int(v) for v in base["msgs"][:4]] == [uc_messages(n, f), n - 1, n - 1, uc_messages(n, f)]
    for size in range(0, f + 1):
        for dead in itertools.combinations(range(n), size):
            for root in (0, n - 1):
                d = O.run(x, f, "sum", dead, root=root, track_sets=True, detail=True, partners_descending=True)
                live = [p for p in range(n) if p not in dead]
                if root in dead:
                    assert d["code"] == 1
                    continue
                assert d["code"] == 0 and np.array_equal(d["result"], K.reduce_over(x, live, "sum"))
                assert K.bits(d["contrib"], n) == live
    sch = O.schedule(n, f)
    for victim in range(f + 1, n):
        for t in range(1, sch["rounds_attempt"] + 2):
            d = O.run(x, f, "sum", [], inop=[(victim, t)], allreduce=True, track_sets=True, detail=True, partners_descending=True)
            C = K.bits(d["contrib"], n)
            assert d["code"] == 0 and K.contribution_allowed(n, C, [], [victim])
            assert np.array_equal(d["result"], K.reduce_over(x, C, "sum"))
            alive_end = [p for p in range(n) if not (p == victim and t < sch["rounds_attempt"])]
            assert K.bits(d["holders"], n) == alive_end
