"""Seeded synthetic scenarios: input vectors and failure patterns.

This module holds no arithmetic of the reduce/allreduce method itself. It only
produces the data a scenario consists of:

* input values, from a stateless counter-based generator (the splitmix64 output
  function applied to ``seed + GAMMA * (counter + 1)``), so that any scenario can
  be regenerated alone, on the host (here, numpy) or on the device (the library's
  ``ftc_fill_inputs`` implements the same published function);
* failure patterns (pre-operation failure bitmasks, in-operation (victim, round)
  entries, per-scenario roots), from ``numpy.random.Generator(PCG64(seed))``.

The paper evaluates nothing and names no dataset; the five workloads below are the
synthetic configurations this repository is measured on.
"""
from __future__ import annotations

import itertools
from dataclasses import dataclass, field

import numpy as np

GAMMA = np.uint64(0x9E3779B97F4A7C15)
M1 = np.uint64(0xBF58476D1CE4E5B9)
M2 = np.uint64(0x94D049BB133111EB)
UNUSED = 0xFFFFFFFF

# value kinds (shared numbering with the device generator)
KIND_I32_PM20 = 0   # int32 uniform in [-2^20, 2^20]
KIND_I64_PM40 = 1   # int64 uniform in [-2^40, 2^40]
KIND_F32_NORMAL = 2  # float32, mean 0 variance 1, sum of twelve 32-bit uniforms (Irwin-Hall), full 24-bit mantissas
KIND_I32_FULL = 3   # int32 uniform over the full range
KIND_U64_FULL = 4   # uint64 uniform

KIND_DTYPE = {
    KIND_I32_PM20: np.int32, KIND_I64_PM40: np.int64, KIND_F32_NORMAL: np.float32,
    KIND_I32_FULL: np.int32, KIND_U64_FULL: np.uint64,
}


def splitmix64(z: np.ndarray) -> np.ndarray:
    """Output function of splitmix64 on an array of already advanced states."""
    z = z.astype(np.uint64, copy=True)
    z ^= z >> np.uint64(30)
    z *= M1
    z ^= z >> np.uint64(27)
    z *= M2
    z ^= z >> np.uint64(31)
    return z


def _hash(seed: int, counter: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        return splitmix64(np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + GAMMA * (counter + np.uint64(1)))


def gen_inputs(kind: int, seed: int, scenario_ids, P: int, k: int) -> np.ndarray:
    """Inputs ``[len(scenario_ids), P, k]`` of the given kind; element (s, p, e) depends only on
    (seed, s, p, e)."""
    sid = np.asarray(scenario_ids, dtype=np.uint64).reshape(-1, 1, 1)
    p = np.arange(P, dtype=np.uint64).reshape(1, -1, 1)
    e = np.arange(k, dtype=np.uint64).reshape(1, 1, -1)
    with np.errstate(over="ignore"):
        lin = (sid * np.uint64(P) + p) * np.uint64(k) + e          # element counter
    if kind == KIND_F32_NORMAL:
        total = np.zeros(lin.shape, dtype=np.int64)
        with np.errstate(over="ignore"):
            for t in range(6):
                h = _hash(seed, lin * np.uint64(6) + np.uint64(t))
                total += (h & np.uint64(0xFFFFFFFF)).astype(np.int64) + (h >> np.uint64(32)).astype(np.int64)
        # twelve uniforms on [0, 2^32): mean 6*(2^32-1), variance ~ 2^64. Twice the centred sum is an integer below 2^37;
        # its conversion to float32 rounds to nearest (the one rounding), the scale 2^-33 is exact. The values carry full
        # 24-bit mantissas, so float32 sums of them round at almost every addition (the fold order shows).
        centred = 2 * total - 12 * ((1 << 32) - 1)
        return centred.astype(np.float32) * np.float32(2.0 ** -33)
    h = _hash(seed, lin)
    if kind == KIND_I32_PM20:
        return ((h % np.uint64((1 << 21) + 1)).astype(np.int64) - (1 << 20)).astype(np.int32)
    if kind == KIND_I64_PM40:
        return (h % np.uint64((1 << 41) + 1)).astype(np.int64) - np.int64(1 << 40)
    if kind == KIND_I32_FULL:
        return (h & np.uint64(0xFFFFFFFF)).astype(np.uint32).view(np.int32)
    if kind == KIND_U64_FULL:
        return h
    raise ValueError(f"unknown value kind {kind}")


# ----------------------------------------------------------------------------------------------
# failure patterns
# ----------------------------------------------------------------------------------------------

def mask_words(P: int) -> int:
    return (P + 31) // 32


def sets_to_masks(sets, P: int) -> np.ndarray:
    """List of iterables of process ids -> uint32 bitmasks [S][ceil(P/32)] (bit p = process p)."""
    out = np.zeros((len(sets), mask_words(P)), dtype=np.uint32)
    for i, st in enumerate(sets):
        for p in st:
            out[i, p >> 5] |= np.uint32(1 << (p & 31))
    return out


def all_failure_sets(P: int, max_size: int):
    """Every subset of [0, P) with at most max_size members, by size then lexicographically."""
    out = []
    for n in range(max_size + 1):
        out.extend(itertools.combinations(range(P), n))
    return out


def random_subsets(rng: np.random.Generator, S: int, P: int, sizes: np.ndarray, lo: int = 0) -> np.ndarray:
    """For each scenario a uniformly random subset of [lo, P) of the given size, as an int64 array
    [S][max_size] padded with -1."""
    mx = int(sizes.max()) if S else 0
    picks = np.full((S, max(mx, 1)), -1, dtype=np.int64)
    for c in range(mx):
        need = sizes > c
        col = rng.integers(lo, P, size=S)
        while True:
            dup = np.zeros(S, dtype=bool)
            for prev in range(c):
                dup |= picks[:, prev] == col
            dup &= need
            if not dup.any():
                break
            col[dup] = rng.integers(lo, P, size=int(dup.sum()))
        picks[need, c] = col[need]
    return picks


def picks_to_masks(picks: np.ndarray, P: int) -> np.ndarray:
    S = picks.shape[0]
    out = np.zeros((S, mask_words(P)), dtype=np.uint32)
    rows = np.arange(S)
    for c in range(picks.shape[1]):
        ok = picks[:, c] >= 0
        p = picks[ok, c]
        np.bitwise_or.at(out, (rows[ok], p >> 5), (np.uint32(1) << (p & 31).astype(np.uint32)))
    return out


@dataclass
class Workload:
    """One batch of scenarios, host side. ``inputs`` is None when they are to be generated on the
    device from (kind, seed, first_scenario)."""
    name: str
    collective: str            # "reduce" or "allreduce"
    P: int
    f: int
    k: int
    kind: int
    op: str                    # "sum" | "max" | "xor"
    seed: int
    S: int
    prefail: np.ndarray        # [S][W] uint32
    inop: np.ndarray | None    # [S][max_inop][2] uint32 (victim, round) or None
    roots: np.ndarray | None   # [S] uint32 or None
    root: int = 0
    first_scenario: int = 0
    inputs: np.ndarray | None = None
    note: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def dtype(self):
        return KIND_DTYPE[self.kind]

    def host_inputs(self, idx=None) -> np.ndarray:
        ids = np.arange(self.S) if idx is None else np.asarray(idx)
        return gen_inputs(self.kind, self.seed, ids + self.first_scenario, self.P, self.k)


BASE_SEED = 0x26022445


def config1() -> Workload:
    """Reduce, P=8, f=1, root 0, k=1 int32 in [-2^20, 2^20], sum; all failure sets of size <= 1."""
    P, f = 8, 1
    sets = all_failure_sets(P, 1)
    return Workload("C1", "reduce", P, f, 1, KIND_I32_PM20, "sum", BASE_SEED + 1, len(sets),
                    sets_to_masks(sets, P), None, None, extra={"sets": sets})


def config2(draws: int = 16) -> Workload:
    """Reduce, P=64, f=2, root 0, k=8 int64 in [-2^40, 2^40], sum; all failure sets of size <= 2,
    each under `draws` input draws."""
    P, f = 64, 2
    sets = all_failure_sets(P, 2)
    masks = np.repeat(sets_to_masks(sets, P), draws, axis=0)
    return Workload("C2", "reduce", P, f, 8, KIND_I64_PM40, "sum", BASE_SEED + 2, masks.shape[0],
                    masks, None, None, extra={"sets": sets, "draws": draws})


def config3(S: int = 1 << 20, first: int = 0) -> Workload:
    """Allreduce, P=1024, f=3, k=16 float32 ~N(0,1), sum; failure-set size uniform in 0..3."""
    P, f = 1024, 3
    rng = np.random.Generator(np.random.PCG64([BASE_SEED + 3, first]))
    sizes = rng.integers(0, f + 1, size=S)
    masks = picks_to_masks(random_subsets(rng, S, P, sizes), P)
    return Workload("C3", "allreduce", P, f, 16, KIND_F32_NORMAL, "sum", BASE_SEED + 3, S, masks, None, None,
                    first_scenario=first)


def config4(rounds_per_attempt: int, S: int = 1 << 18, first: int = 0) -> Workload:
    """Allreduce, P=4096, f=4, k=32 int32 full range, max; up to 2 pre-operation failures and up to 2
    in-operation failures (victims outside the root candidates 0..f, distinct from the pre-failed),
    each at a uniformly random round in [1, rounds_per_attempt)."""
    P, f = 4096, 4
    rng = np.random.Generator(np.random.PCG64([BASE_SEED + 4, first]))
    n_pre = rng.integers(0, 3, size=S)
    n_in = rng.integers(0, 3, size=S)
    drawn = random_subsets(rng, S, P, n_pre)
    pre = np.full((S, 2), -1, dtype=np.int64)
    pre[:, :drawn.shape[1]] = drawn[:, :2]
    vic = np.full((S, 2), -1, dtype=np.int64)
    for c in range(2):
        need = n_in > c
        col = rng.integers(f + 1, P, size=S)
        while True:
            dup = np.zeros(S, dtype=bool)
            for prev in range(2):
                dup |= pre[:, prev] == col
            for prev in range(c):
                dup |= vic[:, prev] == col
            dup &= need
            if not dup.any():
                break
            col[dup] = rng.integers(f + 1, P, size=int(dup.sum()))
        vic[need, c] = col[need]
    rounds = rng.integers(1, rounds_per_attempt, size=(S, 2))
    inop = np.zeros((S, 2, 2), dtype=np.uint32)
    inop[:, :, 0] = np.where(vic >= 0, vic, UNUSED).astype(np.uint32)
    inop[:, :, 1] = np.where(vic >= 0, rounds, 0).astype(np.uint32)
    return Workload("C4", "allreduce", P, f, 32, KIND_I32_FULL, "max", BASE_SEED + 4, S,
                    picks_to_masks(pre, P), inop, None, first_scenario=first)


def config5(collective: str = "allreduce", op: str = "sum", S: int = 1 << 14, first: int = 0) -> Workload:
    """Reduce or allreduce, P=65536, f=8, k=4 uint64 uniform, sum or xor; failure-set size uniform in
    0..8, root (first root candidate) uniform per scenario."""
    P, f = 65536, 8
    rng = np.random.Generator(np.random.PCG64([BASE_SEED + 5, first]))
    sizes = rng.integers(0, f + 1, size=S)
    masks = picks_to_masks(random_subsets(rng, S, P, sizes), P)
    roots = rng.integers(0, P, size=S).astype(np.uint32)
    return Workload("C5", collective, P, f, 4, KIND_U64_FULL, op, BASE_SEED + 5, S, masks, None, roots,
                    root=-1, first_scenario=first)


def inop_sweep(P: int, f: int, k: int, kind: int, op: str, pre_sets, rounds, collective: str = "reduce",
               victims=None, seed: int = BASE_SEED + 6) -> Workload:
    """Exhaustive in-operation sweep: every pre-operation failure set of `pre_sets` x every victim x every failure
    round of `rounds` (victims that are in the pre-failed set are skipped). One in-operation slot per scenario."""
    victims = range(P) if victims is None else victims
    masks, inop = [], []
    for st in pre_sets:
        for v in victims:
            if v in st:
                continue
            for t in rounds:
                masks.append(st)
                inop.append((v, t))
    S = len(masks)
    io = np.asarray(inop, dtype=np.uint32).reshape(S, 1, 2)
    return Workload("inop-sweep", collective, P, f, k, kind, op, seed, S, sets_to_masks(masks, P), io, None,
                    extra={"sets": masks})
