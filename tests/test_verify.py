"""The any-size checks (paper_2602_22445_b200.verify) against the CPU oracle: they accept what the oracle produces for
small samples of the benchmark workloads (torch on the CPU here) and reject planted mistakes."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2602_22445_b200 import scenarios as sc
from paper_2602_22445_b200 import verify


def oracle_batch(w):
    x = w.host_inputs()
    out, st = O.batch(x, w.f, w.op, w.prefail, w.inop, w.roots, max(w.root, 0), w.collective == "allreduce")
    return x, out, st


def as_t(a):
    return torch.from_numpy(a.view(np.int64)).view(torch.uint64) if a.dtype == np.uint64 else torch.from_numpy(a)


def small_workloads():
    ratt = O.schedule(4096, 4)["rounds_attempt"]
    yield sc.config3(S=48)
    yield sc.config4(ratt, S=24)
    yield sc.config5("allreduce", "sum", S=3)
    w = sc.config5("reduce", "xor", S=4)
    w.prefail[1, w.roots[1] >> 5] |= np.uint32(1 << (w.roots[1] & 31))       # one no-op reduce
    yield w


@pytest.mark.parametrize("w", list(small_workloads()), ids=lambda w: f"{w.name}-{w.collective}-{w.op}")
def test_checks_accept_the_oracle_and_reject_planted_mistakes(w):
    x, out, st = oracle_batch(w)
    counts = verify.check_status_fields(w, st)
    assert counts["ok_scenarios"] + counts["noop_scenarios"] == w.S
    verify.check_results_by_definition(w, as_t(x), as_t(out), st, chunk=5)
    bad = out.copy()
    i = int(np.nonzero((st[:, 0] & 0xFF) == 0)[0][-1])
    if w.op == "max":                                   # the value of an excluded process instead of the maximum
        bad[i, 0] = np.iinfo(np.int32).max if bad[i, 0] != np.iinfo(np.int32).max else 0
    elif out.dtype == np.float32:
        bad[i, 0] += np.float32(1.0)
    else:
        bad[i, 0] ^= bad.dtype.type(1)
    with pytest.raises(AssertionError):
        verify.check_results_by_definition(w, as_t(x), as_t(bad), st, chunk=5)
    st2 = st.copy()
    st2[i, 1] -= 1                                      # one process too few included
    with pytest.raises(AssertionError):
        verify.check_status_fields(w, st2)
    if w.collective == "allreduce":
        st3 = st.copy()
        st3[i, 0] += 1 << 16                            # an attempt too many
        with pytest.raises(AssertionError):
            verify.check_status_fields(w, st3)


def test_a_dropped_failed_process_is_noticed():
    """The definition check must see a result that still includes a process that had failed before the operation."""
    w = sc.config5("allreduce", "sum", S=2)
    dead = np.nonzero(np.unpackbits(w.prefail.view(np.uint8), axis=1, bitorder="little").sum(axis=1))[0]
    if dead.size == 0:
        w.prefail[0, 3] |= np.uint32(1 << 7)
    x, out, st = oracle_batch(w)
    i = int(np.nonzero(np.unpackbits(w.prefail.view(np.uint8), axis=1, bitorder="little").sum(axis=1))[0][0])
    victim = int(np.nonzero(np.unpackbits(w.prefail[i].view(np.uint8), bitorder="little"))[0][0])
    wrong = out.copy()
    with np.errstate(over="ignore"):
        wrong[i] += x[i, victim]                        # as if the failed process had been combined after all
    with pytest.raises(AssertionError):
        verify.check_results_by_definition(w, as_t(x), as_t(wrong), st)
