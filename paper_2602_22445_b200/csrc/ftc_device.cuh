// Device-side pieces shared by the kernels: launch parameters, the reduction functions, and the
// per-scenario decode that turns failure masks into the facts the data pass needs.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>
#include "../../include/ftc.h"

namespace ftc {

constexpr uint32_t kNever = 0xFFFFFFFFu;   // failure round of a process that never fails

struct Params {
    uint32_t P, f, m, k, W;          // m = f+1 (group size = root children); W = mask words per scenario
    uint32_t q, r, H, Rred, Ratt;    // P-1 = q*m + r; deepest node; rounds of a reduce / of an allreduce attempt
    uint32_t Gmax;                   // nodes of the largest root subtree: q + (r > 0)
    uint32_t arity;                  // children per node below the root's children (2: binary heap; 1: binomial tree)
    uint32_t pdesc;                  // 1: group partners are visited in descending rank, the root last
    uint32_t max_inop, flags;
    int32_t  root;
    int32_t  is_allreduce;
    uint32_t kbytes;                 // bytes of one process' vector
    uint64_t S;
    const void* in;
    const uint32_t* prefail;
    const ftc_inop_t* inop;
    const uint32_t* roots;
    void* out;
    uint32_t* status;
    void* ws;
    uint64_t ws_bytes;               // bytes the caller's workspace offers at ws (0: none)
    // tiled kernel geometry
    uint32_t C;        // 16-byte chunks per process vector
    uint32_t cw_log2;  // log2 of lanes along the chunk dimension (= log2 C)
    uint32_t Lt;       // heap level at which the warp tiles are rooted; levels above go through shared memory
    uint32_t swz_mask; // swizzled tiles: XOR mask of the 16-byte chunk bits (0x70: 128-byte lines, 0x30: 64-byte lines)
    uint32_t row_shift; // swizzled tiles of 64-byte groups: tile rows after the first sit one row further (128-byte aligned levels)
    uint32_t below;    // 1: the heap's sparsely filled last level lies below the tiles (its rows are folded one by one)
    uint32_t m_magic;  // ceil(2^32 / m): floor(x / m) = (x * m_magic) >> 32 for every x below 2^26 (m <= 32)
    uint32_t* grid_query;  // host side only: when set, a launcher stores the number of blocks it would launch and launches nothing
};

// Per-scenario facts, in shared memory.
struct Ctx {
    uint32_t root;      // physical id of the root of the attempt that counts
    uint32_t base;      // first round of that attempt on the global clock
    uint32_t code, sstar, attempts;
    uint32_t Fmask;     // bit s: the subtree of root child s contains a process that does not send up the tree
    uint32_t npre;      // processes failed before the operation
    uint32_t nexcl;     // in-operation victims whose value does not reach the selected subtree
    uint32_t inop_incl; // in-operation slots whose victim is included
    uint32_t G;         // nodes of the selected subtree
    uint32_t holders;
    uint32_t ndead_end; // in-operation victims (not pre-failed) that are dead at the end of the attempt
    uint32_t unreached_lost;
    uint32_t reserved;
    uint32_t iv[FTC_MAX_INOP];   // victim (physical id) per slot, FTC_INOP_UNUSED if the slot does not count
    uint32_t ir[FTC_MAX_INOP];   // its failure round on the global clock (minimum over slots naming it)
    uint32_t ifirst;             // bit i: slot i is the first slot naming its victim
};

__device__ __forceinline__ uint32_t ilog2u(uint32_t v) { return 31u - __clz(v); }
__device__ __forceinline__ bool test_bit(const uint32_t* bm, uint32_t i) { return (bm[i >> 5] >> (i & 31)) & 1u; }

// ---- subtree shape: below each root child a heap on the local index j with p.arity children per node ----
// Level l holds the arity^l indices that follow those of the levels above; node j has children a*j+1 .. a*j+a.
// arity 1 stands for the binomial tree: the parent of j is j without its lowest set bit, so j's children are j + 2^i
// for every 2^i below that bit (all of them for j = 0), its level is its number of set bits, and everything below
// it is the index range (j, j + lowest set bit).
__device__ __forceinline__ uint32_t heap_level(uint32_t arity, uint32_t j) {
    if (arity == 2) return ilog2u(j + 1);
    if (arity == 1) return (uint32_t)__popc(j);
    uint32_t l = 0; uint64_t start = 0, width = 1;
    while (j >= start + width) { start += width; width *= arity; ++l; }
    return l;
}
// First index of level l (the levels above hold (a^l - 1)/(a - 1) indices); saturates far beyond any index.
__device__ __forceinline__ uint64_t heap_level_start(uint32_t arity, uint32_t l) {
    if (arity == 2) return ((uint64_t)1 << l) - 1;
    uint64_t start = 0, width = 1;
    for (uint32_t i = 0; i < l && start < ((uint64_t)1 << 40); ++i) { start += width; width *= arity; }
    return start;
}
// Sets in `bm` (bits = renumbered ranks) every process below local index j of root subtree sv, which has Gs nodes.
// All lanes of a warp call it with the same arguments.
__device__ __forceinline__ void mark_descendants(uint32_t arity, uint32_t m, uint32_t* bm, uint32_t j, uint32_t sv,
                                                 uint32_t Gs, uint32_t lane) {
    if (arity == 1) {
        const uint64_t end = j ? min((uint64_t)j + (j & (0u - j)), (uint64_t)Gs) : Gs;
        for (uint64_t i = (uint64_t)j + 1 + lane; i < end; i += 32) {
            const uint32_t u = (uint32_t)i * m + sv + 1;
            atomicOr(&bm[u >> 5], 1u << (u & 31));
        }
        return;
    }
    for (uint64_t lo = (uint64_t)arity * j + 1, n = arity; lo < Gs; lo = arity * lo + 1, n *= arity)
        for (uint64_t i = lane; i < n && lo + i < Gs; i += 32) {
            const uint32_t u = (uint32_t)(lo + i) * m + sv + 1;
            atomicOr(&bm[u >> 5], 1u << (u & 31));
        }
}

// n <= 32 bits of a bitmask starting at bit `pos`; the mask has one zero word of padding at its end.
__device__ __forceinline__ uint32_t extract_bits(const uint32_t* bm, uint32_t pos, uint32_t n) {
    uint32_t w = pos >> 5;
    uint32_t v = __funnelshift_r(bm[w], bm[w + 1], pos & 31);
    return n >= 32 ? v : (v & ((1u << n) - 1u));
}

// The root swaps numbers with process 0 (section "Reduce"); the map is its own inverse.
__device__ __forceinline__ uint32_t renumber(uint32_t x, uint32_t root) { return x == 0 ? root : (x == root ? 0u : x); }

// ---- reduction functions: accumulator is the left operand ----
enum { OP_SUM = 0, OP_MAX = 1, OP_XOR = 2 };
template <typename T, int OP> struct Comb;
template <typename T> struct Comb<T, OP_SUM> { static __device__ __forceinline__ T f(T a, T b) { return a + b; } };
template <> struct Comb<float, OP_SUM> { static __device__ __forceinline__ float f(float a, float b) { return __fadd_rn(a, b); } };
template <typename T> struct Comb<T, OP_MAX> { static __device__ __forceinline__ T f(T a, T b) { return a >= b ? a : b; } };
template <typename T> struct Comb<T, OP_XOR> { static __device__ __forceinline__ T f(T a, T b) { return a ^ b; } };

// Failure round of physical process p on the global clock: 0 = failed before the operation.
__device__ __forceinline__ uint32_t fail_round(const Params& p, const Ctx* cx, const uint32_t* pf, uint32_t proc) {
    if (test_bit(pf, proc)) return 0;
    for (uint32_t i = 0; i < p.max_inop; ++i)
        if (cx->iv[i] == proc) return cx->ir[i];
    return kNever;
}
// Same on the clock of the attempt that counts: rounds already over read as 0.
__device__ __forceinline__ uint32_t local_round(uint32_t fr, uint32_t base) {
    return fr == kNever ? kNever : (fr <= base ? 0u : fr - base);
}

// Index of partner (row, sp) in the partner list of member (row, sv), sv != sp: ascending rank with the root first
// in the short last group, or (p.pdesc) descending rank with the root last.
__device__ __forceinline__ uint32_t partner_slot(const Params& p, uint32_t row, uint32_t sv, uint32_t sp) {
    if (p.pdesc) return (row < p.q ? p.m : p.r) - 1 - sp - (sv > sp ? 1u : 0u);
    return (sp < sv ? sp : sp - 1) + (row == p.q ? 1u : 0u);
}
// Index of the root in the partner list of a member of the short last group.
__device__ __forceinline__ uint32_t root_slot(const Params& p) { return p.pdesc ? p.r - 1 : 0u; }

// Decode one scenario. All threads of the block call it. On return (after its last barrier) cx, pf (physical
// pre-failure bits) and inc (bit v: the input of renumbered process v reaches the selected subtree's member of
// its group) are valid. pf and inc have W+1 words, the last one zero.
static __device__ void decode_scenario(const Params& p, uint64_t s, Ctx* cx, uint32_t* pf, uint32_t* inc) {
    const uint32_t tid = threadIdx.x, nt = blockDim.x, lane = tid & 31;
    const uint32_t* gpf = p.prefail + s * p.W;
    if (tid == 0) {
        cx->Fmask = 0; cx->npre = 0; cx->nexcl = 0; cx->inop_incl = 0; cx->holders = 0; cx->ndead_end = 0;
        cx->unreached_lost = 0; cx->code = FTC_ST_OK; cx->sstar = 0xFF; cx->attempts = 0; cx->base = 0; cx->root = 0;
        cx->G = 0; cx->ifirst = 0;
        pf[p.W] = 0; inc[p.W] = 0;
    }
    if (tid < FTC_MAX_INOP) {
        uint32_t v = FTC_INOP_UNUSED, rd = 0;
        if (tid < p.max_inop) { ftc_inop_t e = p.inop[s * p.max_inop + tid]; v = e.victim < p.P ? e.victim : FTC_INOP_UNUSED; rd = e.round; }
        cx->iv[tid] = v; cx->ir[tid] = rd;
    }
    __syncthreads();
    uint32_t cnt = 0;
    for (uint32_t w = tid; w < p.W; w += nt) {
        uint32_t word = gpf[w];
        if (w == p.W - 1 && (p.P & 31)) word &= (1u << (p.P & 31)) - 1u;
        pf[w] = word; cnt += __popc(word);
    }
    cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
    if (lane == 0 && cnt) atomicAdd(&cx->npre, cnt);
    __syncthreads();

    // warp 0: drop victims that are pre-failed, merge slots naming the same victim, pick the root
    if (tid < 32) {
        uint32_t v = cx->iv[lane], rmin = cx->ir[lane];
        bool valid = v != FTC_INOP_UNUSED && !test_bit(pf, v);
        bool first = true;
        for (uint32_t j = 0; j < p.max_inop; ++j)
            if (cx->iv[j] == v) { rmin = min(rmin, cx->ir[j]); if (j < lane) first = false; }
        __syncwarp();
        cx->iv[lane] = valid ? v : FTC_INOP_UNUSED; cx->ir[lane] = rmin;
        uint32_t fm = __ballot_sync(0xFFFFFFFFu, valid && first);
        __syncwarp();
        uint32_t first_root = p.root >= 0 ? (uint32_t)p.root : p.roots[s];
        uint32_t code = FTC_ST_OK, root = first_root, base = 0, attempts = 1;
        if (first_root >= p.P) { code = FTC_ST_BAD_ROOT; attempts = 0; root = 0; }
        else if (!p.is_allreduce) {
            // the root must be alive when the last tree messages arrive (round f+H-1)
            if (fail_round(p, cx, pf, first_root) < p.Rred) code = FTC_ST_ROOT_FAILED;
        } else {
            uint32_t fr = kNever;
            if (lane < p.m) { uint32_t c = (first_root + lane) % p.P; fr = fail_round(p, cx, pf, c); }
            uint32_t inopc = __ballot_sync(0xFFFFFFFFu, fr != 0 && fr != kNever);
            uint32_t alive = __ballot_sync(0xFFFFFFFFu, lane < p.m && fr != 0);
            if (inopc) { code = FTC_ST_PRECONDITION_INOP_ROOT; attempts = 0; }
            else if (!alive) { code = FTC_ST_NO_LIVE_ROOT_CANDIDATE; attempts = p.m; }
            else { uint32_t a = __ffs(alive) - 1; root = (first_root + a) % p.P; base = a * p.Ratt; attempts = a + 1; }
        }
        if (lane == 0) { cx->ifirst = fm; cx->code = code; cx->root = root; cx->base = base; cx->attempts = attempts; }
    }
    __syncthreads();
    if (cx->code != FTC_ST_OK) return;          // uniform: every thread reads the same shared word

    // failed bits of the root's children: a subtree is unclean iff one of its processes does not send up the tree
    const uint32_t root = cx->root, base = cx->base;
    uint32_t F = 0;
    for (uint32_t w = tid; w < p.W; w += nt) {
        uint32_t word = pf[w];
        while (word) {
            uint32_t b = __ffs(word) - 1; word &= word - 1;
            uint32_t v = renumber((w << 5) + b, root);
            if (v) F |= 1u << ((v - 1) % p.m);
        }
    }
    if (tid < p.max_inop && cx->iv[tid] != FTC_INOP_UNUSED) {
        uint32_t v = renumber(cx->iv[tid], root);
        if (v) {
            uint32_t j = (v - 1) / p.m, d = 1 + heap_level(p.arity, j);
            uint32_t t = local_round(cx->ir[tid], base);
            if (!(p.f + p.H - d < t)) F |= 1u << ((v - 1) % p.m);     // tree send of depth d is round f+H-d
        }
    }
    F = __reduce_or_sync(0xFFFFFFFFu, F);
    if (lane == 0 && F) atomicOr(&cx->Fmask, F);
    for (uint32_t w = tid; w < p.W; w += nt) {
        uint32_t word = ~pf[w];
        if (w == p.W - 1 && (p.P & 31)) word &= (1u << (p.P & 31)) - 1u;
        inc[w] = word;
    }
    __syncthreads();

    if (tid < 32) {
        uint32_t Fm = cx->Fmask, all = p.m >= 32 ? 0xFFFFFFFFu : ((1u << p.m) - 1u);
        uint32_t clean = ~Fm & all;
        if (!clean) { if (lane == 0) cx->code = FTC_ST_NO_CLEAN_SUBTREE; }
        else {
            const uint32_t sstar = __ffs(clean) - 1;
            if (lane == 0) {
                cx->sstar = sstar; cx->G = p.q + (sstar < p.r ? 1u : 0u);
                if (root != 0) {                  // renumbered bit 0 is the root (alive), bit `root` is process 0
                    uint32_t b0 = inc[0] & 1u;
                    inc[0] |= 1u;
                    if (b0) inc[root >> 5] |= 1u << (root & 31); else inc[root >> 5] &= ~(1u << (root & 31));
                }
            }
            __syncwarp();
            if (lane < p.max_inop && cx->iv[lane] != FTC_INOP_UNUSED) {
                uint32_t v = renumber(cx->iv[lane], root);
                bool included = true;
                if (v) {
                    uint32_t j = (v - 1) / p.m, sv = (v - 1) % p.m;
                    uint32_t t = local_round(cx->ir[lane], base);
                    bool member_in_subtree = j < p.q || sstar < p.r;   // does group j have a member below child sstar?
                    if (member_in_subtree) { if (sv != sstar) included = partner_slot(p, j, sv, sstar) < t; }
                    else included = t > root_slot(p);                  // the group's values reach the root itself
                }
                if (included) atomicOr(&cx->inop_incl, 1u << lane);
                else {
                    atomicAnd(&inc[v >> 5], ~(1u << (v & 31)));
                    if ((cx->ifirst >> lane) & 1u) atomicAdd(&cx->nexcl, 1u);
                }
            }
        }
    }
    __syncthreads();
}

// Broadcast of the allreduce: how many processes are alive at the end of the attempt and hold the value.
// `unr` (W+1 words) receives bit v for every renumbered process the tree-down phase does not reach.
// `hold` (optional, W+1 words) receives the holders as a bitmask over the caller's process ids.
// All threads of the block call it after decode_scenario returned with code OK.
static __device__ void count_holders(const Params& p, Ctx* cx, const uint32_t* pf, uint32_t* unr, uint32_t* hold = nullptr) {
    const uint32_t tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, wid = tid >> 5, nw = nt >> 5;
    const uint32_t root = cx->root, base = cx->base;
    // With at most f failed processes one root subtree is free of failures: all its processes are reached by the
    // tree and alive throughout, every group has a member in it (the short last group has the root instead), so
    // the correction phase reaches every process that is alive at the end. No marking is needed then.
    if (cx->npre + __popc(cx->ifirst) <= p.f) {            // uniform: shared values, read after a barrier
        for (uint32_t w = tid; hold && w <= p.W; w += nt) {
            uint32_t word = w < p.W ? ~pf[w] : 0u;
            if (w == p.W - 1 && (p.P & 31)) word &= (1u << (p.P & 31)) - 1u;
            hold[w] = word;
        }
        __syncthreads();
        if (tid < p.max_inop && cx->iv[tid] != FTC_INOP_UNUSED && ((cx->ifirst >> tid) & 1u) &&
            local_round(cx->ir[tid], base) < p.Ratt) {
            atomicAdd(&cx->ndead_end, 1u);
            if (hold) atomicAnd(&hold[cx->iv[tid] >> 5], ~(1u << (cx->iv[tid] & 31)));
        }
        __syncthreads();
        if (tid == 0) cx->holders = p.P - cx->npre - cx->ndead_end;
        __syncthreads();
        return;
    }
    for (uint32_t w = tid; w <= p.W; w += nt) {
        unr[w] = 0;
        if (hold) {                                   // start from everybody who had not failed before the operation
            uint32_t word = w < p.W ? ~pf[w] : 0u;
            if (w == p.W - 1 && (p.P & 31)) word &= (1u << (p.P & 31)) - 1u;
            hold[w] = word;
        }
    }
    __syncthreads();
    // every process that does not forward the value down the tree cuts off all its descendants
    const uint32_t nwords_round = (p.W + 31) & ~31u;
    for (uint32_t w0 = wid * 32; w0 < nwords_round; w0 += nw * 32) {
        uint32_t w = w0 + lane;
        uint32_t word = w < p.W ? pf[w] : 0u;
        // in-operation victims that die before their tree-down send behave the same
        uint32_t pend = __ballot_sync(0xFFFFFFFFu, word != 0);
        while (pend) {
            uint32_t src = __ffs(pend) - 1; pend &= pend - 1;
            uint32_t ww = __shfl_sync(0xFFFFFFFFu, word, src), wbase = (w0 + src) << 5;
            while (ww) {
                uint32_t b = __ffs(ww) - 1; ww &= ww - 1;
                uint32_t v = renumber(wbase + b, root);
                if (!v) continue;
                uint32_t j = (v - 1) / p.m, sv = (v - 1) % p.m, Gs = p.q + (sv < p.r ? 1u : 0u);
                mark_descendants(p.arity, p.m, unr, j, sv, Gs, lane);
            }
        }
    }
    if (wid == 0) {
        for (uint32_t i = 0; i < p.max_inop; ++i) {
            if (cx->iv[i] == FTC_INOP_UNUSED || !((cx->ifirst >> i) & 1u)) continue;
            uint32_t v = renumber(cx->iv[i], root), t = local_round(cx->ir[i], base);
            if (lane == 0 && t < p.Ratt) {
                atomicAdd(&cx->ndead_end, 1u);
                if (hold) atomicAnd(&hold[cx->iv[i] >> 5], ~(1u << (cx->iv[i] & 31)));
            }
            if (!v) continue;
            uint32_t j = (v - 1) / p.m, sv = (v - 1) % p.m, Gs = p.q + (sv < p.r ? 1u : 0u), d = 1 + heap_level(p.arity, j);
            if (t > p.Rred + d) continue;                  // it does forward: tree-down send of depth d is round f+H+d
            mark_descendants(p.arity, p.m, unr, j, sv, Gs, lane);
        }
    }
    __syncthreads();
    // an unreached process still gets the value if a partner that the tree reached sends it in the correction phase
    uint32_t lost = 0;
    for (uint32_t w = tid; w < p.W; w += nt) {
        uint32_t word = unr[w];
        while (word) {
            uint32_t b = __ffs(word) - 1; word &= word - 1;
            uint32_t v = (w << 5) + b;                                     // renumbered, v >= 1
            uint32_t tv = local_round(fail_round(p, cx, pf, renumber(v, root)), base);
            if (tv < p.Ratt) continue;                                     // dead at the end: counted elsewhere
            uint32_t j = (v - 1) / p.m, sv = (v - 1) % p.m;
            uint32_t mj = j < p.q ? p.m : p.r;
            bool rescued = (j == p.q);                                     // the root is a member of the short group
            for (uint32_t su = 0; su < mj && !rescued; ++su) {
                if (su == sv) continue;
                uint32_t u = j * p.m + su + 1;
                if (test_bit(unr, u)) continue;
                uint32_t tu = local_round(fail_round(p, cx, pf, renumber(u, root)), base);
                if (tu > p.Rred + p.H + partner_slot(p, j, su, sv)) rescued = true;
            }
            if (!rescued) {
                ++lost;
                if (hold) { const uint32_t ph = renumber(v, root); atomicAnd(&hold[ph >> 5], ~(1u << (ph & 31))); }
            }
        }
    }
    lost = __reduce_add_sync(0xFFFFFFFFu, lost);
    if (lane == 0 && lost) atomicAdd(&cx->unreached_lost, lost);
    __syncthreads();
    if (tid == 0) cx->holders = p.P - cx->npre - cx->ndead_end - cx->unreached_lost;
    __syncthreads();
}

}  // namespace ftc
