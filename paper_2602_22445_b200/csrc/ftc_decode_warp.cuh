// Decode of one scenario by one warp, in registers: for process counts up to 1024 (one word of the failure mask per
// lane) and scenarios that stay within the tolerated number of failures. It yields the same facts as
// decode_scenario() and count_holders() (which play everything else, and share nothing but the definitions with
// this file): the root of the attempt that counts, the root child whose value the root takes, the arrival mask
// of the up-correction messages at the selected subtree's members, the fields of the status record.
// Ballots and shuffles take the place of shared memory, atomics and block-wide barriers.
#pragma once
#include "ftc_device.cuh"

namespace ftc {

struct WarpScen {
    // the same in every lane
    uint32_t code, sstar, attempts, root, base, npre, nexcl, inop_incl, holders, G;
    uint32_t any_victim;     // some in-operation slot counts (its victim is in range and had not failed before the operation)
    // per lane
    uint32_t incw;           // word `lane` of the arrival mask over renumbered ranks (0 beyond the mask)
    uint32_t iv;             // in-operation slot `lane`: its victim, or FTC_INOP_UNUSED when the slot does not count
};

constexpr uint32_t kFullWarp = 0xFFFFFFFFu;

// x / m and x % m for x below 2^26 without a division (p.m_magic = ceil(2^32 / m), m <= 32: the rounding error of the
// reciprocal times x stays below one unit of the quotient's last place)
__device__ __forceinline__ uint32_t div_m(const Params& p, uint32_t x) { return p.m == 1 ? x : __umulhi(x, p.m_magic); }

// The warp is cut into groups of L lanes (L = 32: the whole warp; 16 or 8: several scenarios at once), every group
// decodes its own scenario (W <= L mask words, max_inop <= L, f+1 <= L). All 32 lanes execute every ballot and
// shuffle, so nothing here returns early or loops a group-dependent number of times; ballots are cut to the group's
// lanes, shuffles and reductions stay inside the group. Facts that are "the same in every lane" of WarpScen are the
// same in every lane of a group.
// pfw: word `lane within the group` of the scenario's pre-operation mask, bits >= P cleared, 0 beyond the mask.
// ev / er: in-operation slot `lane within the group` as the caller passed it (beyond max_inop: anything).
// `slow` is set where the scenario is left to the general routines: a root out of range, or more failed processes
// (before and during the operation) than the f the schedule tolerates; the other outputs are then meaningless but
// harmless (G = 0 makes every fold read row 0 only).
// ALLRED_ / INOP_: 0 or 1 = compile-time copies of p.is_allreduce != 0 and p.max_inop != 0 (code that cannot run is
// left out); 2 = look at p when running.
template <int L> struct LaneGroup {
    static constexpr uint32_t kLanes = L == 32 ? 0xFFFFFFFFu : ((1u << L) - 1u);
    uint32_t lg, base, mask;                                       // lane within the group, the group's first lane and lanes
    __device__ __forceinline__ LaneGroup() { const uint32_t lane = threadIdx.x & 31; lg = lane & (L - 1); base = lane & ~(uint32_t)(L - 1); mask = kLanes << base; }
    __device__ __forceinline__ uint32_t ballot(bool pred) const { return (__ballot_sync(kFullWarp, pred) >> base) & kLanes; }
    __device__ __forceinline__ uint32_t shfl(uint32_t v, uint32_t src) const { return __shfl_sync(kFullWarp, v, src, L); }
    __device__ __forceinline__ uint32_t sum(uint32_t v) const { return __reduce_add_sync(mask, v); }
    __device__ __forceinline__ uint32_t any_or(uint32_t v) const { return __reduce_or_sync(mask, v); }
};

template <int L, int ALLRED_, int INOP_>
__device__ __forceinline__ void decode_group(const Params& p, uint32_t pfw, uint32_t ev, uint32_t er, uint32_t first_root, WarpScen& o, bool& slow) {
    const bool ALLRED = ALLRED_ == 2 ? p.is_allreduce != 0 : ALLRED_ != 0;
    const bool INOP = INOP_ == 2 ? p.max_inop != 0 : INOP_ != 0;
    const LaneGroup<L> g;
    const uint32_t lg = g.lg;
    slow = first_root >= p.P;
    if (slow) first_root = 0;                                          // keeps every index below in range
    const uint32_t npre = g.sum(__popc(pfw));

    uint32_t v = (INOP && lg < p.max_inop && ev < p.P) ? ev : FTC_INOP_UNUSED;
    uint32_t rmin = (INOP && lg < p.max_inop) ? er : 0u;
    uint32_t ifirst = 0;
    o.any_victim = 0;
    if (INOP) {                                                        // the same in every lane of the warp
        const uint32_t word = g.shfl(pfw, v == FTC_INOP_UNUSED ? 0u : v >> 5);
        const bool pre = v != FTC_INOP_UNUSED && ((word >> (v & 31)) & 1u);
        bool first = true;
        const uint32_t r0 = rmin;
        for (uint32_t j = 0; j < p.max_inop; ++j) {
            const uint32_t vj = g.shfl(v, j), rj = g.shfl(r0, j);
            if (vj == v) { rmin = min(rmin, rj); if (j < lg) first = false; }
        }
        if (pre) v = FTC_INOP_UNUSED;
        o.any_victim = g.ballot(v != FTC_INOP_UNUSED);
        ifirst = g.ballot(v != FTC_INOP_UNUSED && first);
    }
    if (npre + __popc(ifirst) > p.f) slow = true;
    const uint32_t iv = v, ir = rmin;

    auto fail_round_of = [&](uint32_t proc) {                          // proc may differ from lane to lane
        const uint32_t word = g.shfl(pfw, proc >> 5);
        uint32_t fr = ((word >> (proc & 31)) & 1u) ? 0u : kNever;
        if (INOP)
            for (uint32_t j = 0; j < p.max_inop; ++j) {
                const uint32_t vj = g.shfl(iv, j), rj = g.shfl(ir, j);
                if (fr == kNever && vj == proc) fr = rj;
            }
        return fr;
    };
    uint32_t code = FTC_ST_OK, root = first_root, base = 0, attempts = 1;
    if (!ALLRED) {
        if (fail_round_of(first_root) < p.Rred) code = FTC_ST_ROOT_FAILED;
    } else {
        uint32_t c = first_root + (lg < p.m ? lg : 0u);
        if (c >= p.P) c -= p.P;
        const uint32_t fr = fail_round_of(c);
        const uint32_t inopc = g.ballot(lg < p.m && fr != 0 && fr != kNever);
        const uint32_t alive = g.ballot(lg < p.m && fr != 0);
        if (inopc) { code = FTC_ST_PRECONDITION_INOP_ROOT; attempts = 0; }
        else if (!alive) { code = FTC_ST_NO_LIVE_ROOT_CANDIDATE; attempts = p.m; }
        else {
            const uint32_t a = __ffs(alive) - 1;
            root = first_root + a; if (root >= p.P) root -= p.P;
            base = a * p.Ratt; attempts = a + 1;
        }
    }
    o.code = code; o.root = root; o.base = base; o.attempts = attempts; o.npre = npre; o.iv = iv;

    uint32_t F = 0;
    for (uint32_t word = pfw; word; word &= word - 1) {                // lane-local: no shuffle inside
        const uint32_t vr = renumber((lg << 5) + (__ffs(word) - 1), root);
        if (vr) F |= 1u << ((vr - 1) - div_m(p, vr - 1) * p.m);
    }
    const uint32_t vren = (INOP && iv != FTC_INOP_UNUSED) ? renumber(iv, root) : 0u;
    const uint32_t t = INOP ? local_round(ir, base) : kNever;
    uint32_t j = 0, sv = 0;
    if (INOP && vren) {
        j = div_m(p, vren - 1); sv = (vren - 1) - j * p.m;
        const uint32_t d = 1 + heap_level(p.arity, j);
        if (!(p.f + p.H - d < t)) F |= 1u << sv;
    }
    F = g.any_or(F);
    const uint32_t all = p.m >= 32 ? 0xFFFFFFFFu : ((1u << p.m) - 1u);
    const uint32_t clean = ~F & all;
    if (!clean) slow = true;                                           // cannot happen with at most f failures
    const uint32_t sstar = clean ? __ffs(clean) - 1 : 0u;
    const bool ok = code == FTC_ST_OK && !slow;
    o.sstar = ok ? sstar : 0xFFu;
    o.G = ok ? p.q + (sstar < p.r ? 1u : 0u) : 0u;

    const uint32_t W = p.W;
    uint32_t incw = 0;
    if (lg < W) {
        incw = ~pfw;
        if (lg == W - 1 && (p.P & 31)) incw &= (1u << (p.P & 31)) - 1u;
    }
    {
        const uint32_t b0 = g.shfl(incw, 0) & 1u;
        if (root != 0) {
            if (lg == 0) incw |= 1u;
            if (lg == (root >> 5)) incw = b0 ? (incw | (1u << (root & 31))) : (incw & ~(1u << (root & 31)));
        }
    }
    o.nexcl = 0; o.inop_incl = 0;
    if (INOP) {
        bool included = true;
        if (vren) {
            const bool member_in_subtree = j < p.q || sstar < p.r;
            if (member_in_subtree) { if (sv != sstar) included = partner_slot(p, j, sv, sstar) < t; }
            else included = t > root_slot(p);
        }
        o.inop_incl = g.ballot(iv != FTC_INOP_UNUSED && included);
        const uint32_t excl = g.ballot(iv != FTC_INOP_UNUSED && !included);
        o.nexcl = __popc(excl & ifirst);
        for (uint32_t jj = 0; jj < p.max_inop; ++jj) {                 // every lane of the warp loops alike
            const uint32_t vj = g.shfl(vren, jj);
            if (((excl >> jj) & 1u) && lg == (vj >> 5)) incw &= ~(1u << (vj & 31));
        }
    }
    o.incw = incw;
    o.holders = 0;
    if (ALLRED) {
        const uint32_t dead_end = INOP ? (g.ballot(iv != FTC_INOP_UNUSED && t < p.Ratt) & ifirst) : 0u;
        o.holders = p.P - npre - __popc(dead_end);
    }
}

// Work items of the staged kernel that need the careful path or the masked folds, for a block of one warp whose
// tiles and groups of upper rows number at most 32: the same marks as mark_special_items(), as two words.
// pfw: this lane's word of the pre-operation mask; iv: this lane's in-operation slot (victim or FTC_INOP_UNUSED).
__device__ __forceinline__ void mark_special_warp(const Params& p, uint32_t pfw, uint32_t iv, uint32_t root, uint32_t G, uint32_t Lt,
                                                  uint32_t D, bool below, uint32_t grows, uint32_t ngroups, uint32_t& spec, uint32_t& mask) {
    const uint32_t lane = threadIdx.x & 31, ntiles = 1u << Lt, ntop = ntiles - 1;
    auto item_bit = [&](uint32_t j) -> uint32_t {
        const uint32_t lvl = ilog2u(j + 1);
        if (below && lvl >= Lt + D) return 0u;                      // rows under the tiles are folded one by one anyway
        return 1u << (lvl >= Lt ? ((j + 1) >> (lvl - Lt)) - ntiles : ntiles + j / grows);
    };
    uint32_t mk = 0, sp = 0;
    for (uint32_t word = pfw; word; word &= word - 1) {
        const uint32_t v = renumber((lane << 5) + (__ffs(word) - 1), root);
        if (v) { const uint32_t j = div_m(p, v - 1); if (j < G) mk |= item_bit(j); }
    }
    if (iv != FTC_INOP_UNUSED) {
        const uint32_t v = renumber(iv, root);
        if (v) { const uint32_t j = div_m(p, v - 1); if (j < G) mk |= item_bit(j); }
    }
    if (lane == 0) {
        if (root != 0 && div_m(p, root - 1) < G) sp |= item_bit(div_m(p, root - 1));   // the slot that holds process 0's input
        if (G > p.q) sp |= item_bit(p.q);                                              // the short last group
    }
    if (lane < ntiles && ((((ntop + lane + 2) << (D >= 2 ? D - 2 : 0)) - 2 >= G) || (!below && ((ntop + lane + 1) << D) - 1 < G)))
        sp |= 1u << lane;
    if (lane < ngroups && ((lane + 1) * grows > ntop || (lane + 1) * grows > G)) sp |= 1u << (ntiles + lane);
    mask = __reduce_or_sync(kFullWarp, mk);
    spec = __reduce_or_sync(kFullWarp, sp);
}

}  // namespace ftc
