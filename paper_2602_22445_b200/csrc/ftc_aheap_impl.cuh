// Level kernel: the shared-memory path for subtrees that are a-ary heaps (FTC_TREE_ARITY(a), a = 2..32; the paper's
// I(f)-tree fixes only the root's f+1 children and their subtree sizes, so any such shape is one). The heap of the
// selected subtree's rows is cut into tiles as in the staged kernel -- a tile is a forest of neighbouring sub-heaps of D
// levels, each level one contiguous run of rows, brought into shared memory by one bulk copy per level -- but a tile is
// evaluated level by level in shared memory instead of in registers and shuffles, which works for any number of children
// per node:
//   1. every (row, 16-byte chunk) of the tile folds its group (Algorithm "Up-correction": own input, then the partners
//      whose message arrived, in the schedule's order) and leaves the result in place of the row's first member;
//   2. the tile's levels are combined from the leaves up (Algorithm "reduce_non_root": data, then child 1, child 2, ...),
//      again in place, with a warp-level barrier between levels;
//   3. the tile's root goes to the block's heap array, which is combined level by level as in the staged kernel.
// Each row decides by itself whether the plain fold from its staged copy serves it (a full group under its arrival mask)
// or the general fold is needed (a renumbered slot, the short last group): no marking pass.
// Binomial subtrees (FTC_TREE_BINOMIAL, arity 1 internally) run here too: a tile is 2^D rows from a multiple of 2^D, which
// is the binomial subtree of its first row and one contiguous run; step 2 becomes D doubling steps, and step 3 the same
// doubling steps on the tile index.
#pragma once
#include "ftc_staged_impl.cuh"
#include "ftc_decode_warp.cuh"

namespace ftc {

constexpr uint32_t kAheapMaxLevels = 24;
#ifndef FTC_AHEAP_MINB
#define FTC_AHEAP_MINB 2
#endif
constexpr uint32_t kAheapWarpsPerSM = 8 * FTC_AHEAP_MINB;   // what the register bound of the kernel lets an SM hold

// A work item of the tile kind is a forest: n neighbouring nodes of heap level Lt with everything below them, d levels in
// all. Neighbouring nodes have neighbouring children, so every level of the forest is one contiguous run of rows. The
// heap's last level is filled from the left only: the first nA nodes of level Lt have rows on it (forests of D levels, n1
// nodes each), the others end one level higher (forests of D - 1 levels, n2 nodes each, n2 > n1), so that both kinds fill
// a warp's buffer about equally.
struct AheapGeom {
    uint32_t nwarps, tile_cap;             // warps per block, bytes of a warp's buffer
    uint32_t D, Lt;                        // levels of a deep forest; heap level of the forests' roots
    uint32_t n1, n2, nA, nroots;           // roots per deep / shallow forest; roots with rows on the last level; all roots
    uint32_t itemsA, itemsB, ngroups;      // deep forests, shallow forests, work items over the rows above level Lt
    uint32_t cap_rows;                     // rows a warp's buffer holds
    uint32_t ntop, nheap;                  // rows above level Lt; rows of the block's heap array (levels 0 .. Lt)
    uint32_t lstart[kAheapMaxLevels + 1];  // first row of heap level l: (a^l - 1) / (a - 1)
    uint32_t tstart[5], apow[5];           // a forest's level u per root: nodes above it, (a^u - 1) / (a - 1), and nodes on it, a^u
    uint32_t off_rootv, off_hv, off_bar, off_gaveup, off_tiles, smem_bytes;
    uint32_t c_magic;                      // 0: the vector is a power-of-two number of 16-byte chunks; else ceil(2^32 / chunks)
};

// NP2: the vector is not a power-of-two number of 16-byte chunks. M: the group size f + 1 when it is one of the usual ones (its
// fold is then straight-line code with all loads issued together: the fold is most of the instruction stream), 0: any.
template <typename T, int OP, bool NP2, int M>
__global__ void __launch_bounds__(kStagedMaxThreads, FTC_AHEAP_MINB) aheap_kernel(Params p, const __grid_constant__ AheapGeom g) {
    extern __shared__ __align__(128) uint32_t smem[];
    char* sbase = reinterpret_cast<char*>(smem);
    Ctx* cx = reinterpret_cast<Ctx*>(smem);
    uint32_t* pf = smem + sizeof(Ctx) / 4;
    uint32_t* inc = pf + p.W + 1;
    uint32_t* unr = inc + p.W + 1;
    uint4* rootv = reinterpret_cast<uint4*>(sbase + g.off_rootv);
    uint4* hv = reinterpret_cast<uint4*>(sbase + g.off_hv);
    volatile uint32_t* gaveup = reinterpret_cast<volatile uint32_t*>(sbase + g.off_gaveup);

    const uint32_t tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, wid = tid >> 5, nw = nt >> 5;
    const uint32_t a = p.arity, C = p.C;
    // unit u of a run of rows = (row u / C, chunk u % C); C is a power of two (shift and mask) or not (multiply by the
    // reciprocal g.c_magic = ceil(2^32 / C): exact for u below 2^26)
    const uint32_t cwl = p.cw_log2, cmagic = g.c_magic;
    auto urow = [&](uint32_t u) -> uint32_t { return NP2 ? __umulhi(u, cmagic) : u >> cwl; };
    auto uchunk = [&](uint32_t u, uint32_t t) -> uint32_t { return NP2 ? u - t * C : u & (C - 1); };
    const uint32_t D = g.D, Lt = g.Lt, ntop = g.ntop;
    const bool binom = a == 1;                                         // binomial subtrees: D = log2 of a tile's rows
    const uint32_t itemsAB = g.itemsA + g.itemsB, nitems = itemsAB + g.ngroups + 1;
    const uint32_t rowbytes = p.m * p.kbytes;
    const uint64_t scen_bytes = (uint64_t)p.P * p.kbytes;
    const uint32_t tries = (p.flags & FTC_DEBUG_ONE_POLL) ? 1u : kWaitTries;
    // forest `it`: first root (position on level Lt), roots, levels
    auto forest = [&](uint32_t it, uint32_t& x0, uint32_t& n, uint32_t& d) {
        if (it < g.itemsA) { x0 = it * g.n1; n = min(g.n1, g.nA - x0); d = D; }
        else { x0 = g.nA + (it - g.itemsA) * g.n2; n = min(g.n2, g.nroots - x0); d = D - 1; }
    };

    const uint32_t bar0 = smem_addr(sbase + g.off_bar) + wid * 8;
    char* tile = sbase + g.off_tiles + (size_t)wid * g.tile_cap;
    if (lane == 0) mbar_init(bar0, 1);
    if (tid == 0) *gaveup = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    uint32_t phase = 0;
    bool pending = false, stop = false;

    // ---- this warp's copy pipeline over the flat sequence (scenario, work item): one buffer, refilled as soon as it is free ----
    const uint32_t n_my = wid < nitems ? (nitems - wid + nw - 1) / nw : 0;
    uint64_t is_s = blockIdx.x;
    const char* is_src = reinterpret_cast<const char*>(p.in) + is_s * scen_bytes;
    uint32_t is_i = 0;
    uint32_t my_pw = 0, my_ts = 0, my_ls = 0;                         // lane u < D copies level u of a forest
    if (!binom && lane < D) { my_pw = g.apow[lane]; my_ts = g.tstart[lane]; my_ls = g.lstart[Lt + lane]; }
    auto issue_next = [&]() {
        if (n_my == 0 || is_s >= p.S || stop) return;
        const uint32_t it = wid + is_i * nw;
        uint64_t first_row = 0; uint32_t nrows = 0, dst_off = 0;
        if (binom) {
            if (it < itemsAB && lane == 0) { first_row = (uint64_t)it << D; nrows = 1u << D; }
        } else if (it < itemsAB) {
            uint32_t x0, n, d; forest(it, x0, n, d);
            if (lane < d) { first_row = (uint64_t)my_ls + (uint64_t)x0 * my_pw; nrows = n * my_pw; dst_off = n * my_ts * rowbytes; }
        } else if (it < itemsAB + g.ngroups) {
            if (lane == 0) { first_row = (uint64_t)(it - itemsAB) * g.cap_rows; nrows = min(g.cap_rows, ntop - (uint32_t)first_row); }
        }
        const uint64_t b0 = first_row * rowbytes + p.kbytes;
        uint32_t bytes = 0;
        if (nrows && b0 < scen_bytes) bytes = (uint32_t)min((uint64_t)nrows * rowbytes, scen_bytes - b0);
        const uint32_t total = __reduce_add_sync(0xFFFFFFFFu, bytes);
        if (total) {
            if (lane == 0) mbar_expect_tx(bar0, total);
            __syncwarp();
            if (bytes) bulk_g2s(smem_addr(tile + dst_off), is_src + b0, bytes, bar0);
            pending = true;
        }
        if (++is_i == n_my) { is_i = 0; is_s += gridDim.x; is_src += (uint64_t)gridDim.x * scen_bytes; }
    };
    auto acquire = [&]() {
        if (pending && !stop) {
            bool ok = mbar_wait_bounded(bar0, phase, tries);
            if (!__all_sync(0xFFFFFFFFu, ok)) {
                if (__any_sync(0xFFFFFFFFu, ok) && !ok) ok = mbar_wait_bounded(bar0, phase, kWaitTries);
                ok = __all_sync(0xFFFFFFFFu, ok);
            }
            if (ok) { phase ^= 1u; pending = false; }
            else { stop = true; if (lane == 0) atomicOr(const_cast<uint32_t*>(gaveup), 1u); }
        }
    };
    // values were written into the tile in place: order those writes before the next copy into the same bytes
    auto release = [&]() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); __syncwarp(); issue_next(); };
    issue_next();

    // A block of one warp whose masks are one word per lane decodes in registers (ftc_decode_warp.cuh) and fetches the
    // next scenario's mask word, in-operation entry and root while the current scenario is played.
    const bool warp_decode = nw == 1 && p.W <= 32 && p.max_inop <= 32;
    uint32_t nx_pf = 0, nx_vic = FTC_INOP_UNUSED, nx_rnd = 0, nx_root = 0;
    auto fetch_small = [&](uint64_t s) {
        nx_pf = 0; nx_vic = FTC_INOP_UNUSED; nx_rnd = 0; nx_root = 0;
        if (s >= p.S) return;
        if (lane < p.W) nx_pf = __ldg(p.prefail + s * p.W + lane);
        if (lane < p.max_inop) { const ftc_inop_t* e = p.inop + s * p.max_inop + lane; nx_vic = __ldg(&e->victim); nx_rnd = __ldg(&e->round); }
        if (p.root < 0) nx_root = __ldg(p.roots + s);
    };
    if (warp_decode) fetch_small(blockIdx.x);

    for (uint64_t s = blockIdx.x; s < p.S; s += gridDim.x) {
        const char* in_s = reinterpret_cast<const char*>(p.in) + s * scen_bytes;
        const bool dead = *gaveup != 0;
        if (dead) stop = true;
        bool decoded = false;
        if (warp_decode) {
            uint32_t pfw = nx_pf;
            if (lane == p.W - 1 && (p.P & 31)) pfw &= (1u << (p.P & 31)) - 1u;
            const uint32_t ev = nx_vic, er = nx_rnd, first_root = p.root >= 0 ? (uint32_t)p.root : nx_root;
            fetch_small(s + gridDim.x);
            WarpScen w; bool slow;
            decode_group<32, 2, 2>(p, pfw, ev, er, first_root, w, slow);
            if (!slow) {
                if (lane == 0) {
                    cx->code = w.code; cx->sstar = w.sstar; cx->attempts = w.attempts; cx->root = w.root; cx->base = w.base;
                    cx->npre = w.npre; cx->nexcl = w.nexcl; cx->inop_incl = w.inop_incl; cx->holders = w.holders; cx->G = w.G;
                    pf[p.W] = 0;
                }
                if (lane < p.W) pf[lane] = pfw;
                if (lane <= p.W) inc[lane] = w.incw;
                if (p.W == 32 && lane == 0) inc[32] = 0;
                decoded = true;
                __syncwarp();
            }
        }
        if (!decoded) decode_scenario(p, s, cx, pf, inc);
        char* out_s = reinterpret_cast<char*>(p.out) + s * p.kbytes;
        if (cx->code != FTC_ST_OK || dead) {
            if (tid < C) reinterpret_cast<uint4*>(out_s)[tid] = make_uint4(0, 0, 0, 0);
            for (uint32_t i = 0; i < n_my; ++i) { acquire(); release(); }
            __syncthreads();
            if (tid == 0) {
                if (*gaveup) cx->code = FTC_ST_INTERNAL_TIMEOUT;
                write_status_rec(p, s, cx);
            }
            __syncthreads();
            continue;
        }
        if (p.is_allreduce && !decoded) count_holders(p, cx, pf, unr);
        const uint32_t root = cx->root, sstar = cx->sstar, G = cx->G;
        // a row's value after up-correction (Algorithm "Up-correction") from its staged copy: folded as a plain group at once
        // (the loads do not wait for the row's mask), and once more by the general rules where the group is not plain
        auto fold_row = [&](const char* srow_lc, const char* in_lc, uint32_t row) -> uint4 {
            const uint4 v = fold16_full<T, OP, M>(srow_lc, p.kbytes, M ? (uint32_t)M : p.m, sstar, LdShared(), p.pdesc != 0);
            if (group_is_plain(p, root, inc, row)) return v;
            return fold_staged_call<T, OP, false>(fold_shape(p), root, sstar, inc, in_lc, srow_lc, row);
        };

        for (uint32_t i = 0; i < n_my; ++i) {
            const uint32_t it = wid + i * nw;
            acquire();
            if (binom && it < itemsAB) {
                // rows [it * 2^D, (it + 1) * 2^D) are the binomial subtree of the tile's first row: node x takes its children
                // x + 1, x + 2, x + 4, ... in that order, each complete before it is taken (it ends on fewer zero bits)
                const uint32_t r0 = it << D, nr = 1u << D;
                if (r0 < G) {
                    for (uint32_t u = lane; u < nr * C; u += 32) {
                        const uint32_t t = urow(u), c = uchunk(u, t);
                        if (r0 + t >= G) continue;
                        char* srow = tile + (size_t)t * rowbytes + c * 16;
                        *reinterpret_cast<uint4*>(srow) = fold_row(srow, in_s + c * 16, r0 + t);
                    }
                    __syncwarp();
                    for (uint32_t i = 0; i < D; ++i) {
                        for (uint32_t u = lane; u < (nr >> (i + 1)) * C; u += 32) {
                            const uint32_t ur = urow(u), x = ur << (i + 1), c = uchunk(u, ur);
                            if (r0 + x + (1u << i) >= G) continue;
                            char* mine = tile + (size_t)x * rowbytes + c * 16;
                            const uint4 child = *reinterpret_cast<const uint4*>(mine + ((size_t)rowbytes << i));
                            *reinterpret_cast<uint4*>(mine) = comb16<T, OP>(*reinterpret_cast<const uint4*>(mine), child);
                        }
                        __syncwarp();
                    }
                    if (lane < C) hv[(size_t)it * C + lane] = *reinterpret_cast<const uint4*>(tile + lane * 16);
                }
            } else if (it < itemsAB) {
                uint32_t x0, n, d; forest(it, x0, n, d);
                // local node t of forest level l is row rb_l + t; level l starts at local node th_l
                const uint32_t th1 = d > 1 ? n * g.tstart[1] : 0xFFFFFFFFu, th2 = d > 2 ? n * g.tstart[2] : 0xFFFFFFFFu,
                               th3 = d > 3 ? n * g.tstart[3] : 0xFFFFFFFFu;
                const uint32_t rb0 = g.lstart[Lt] + x0, rb1 = g.lstart[Lt + 1] + x0 * g.apow[1] - th1,
                               rb2 = g.lstart[Lt + 2] + x0 * g.apow[2] - th2, rb3 = g.lstart[Lt + 3] + x0 * g.apow[3] - th3;
                if (rb0 < G) {
                    // 1. every (row, chunk) folds its group; the result takes the place of the row's first member
                    const uint32_t units = n * g.tstart[d] * C;
                    for (uint32_t u = lane; u < units; u += 32) {
                        const uint32_t t = urow(u), c = uchunk(u, t);
                        const uint32_t row = t + (t >= th3 ? rb3 : t >= th2 ? rb2 : t >= th1 ? rb1 : rb0);
                        if (row >= G) continue;
                        char* srow = tile + (size_t)t * rowbytes + c * 16;
                        *reinterpret_cast<uint4*>(srow) = fold_row(srow, in_s + c * 16, row);
                    }
                    __syncwarp();
                    // 2. the levels of the forest, leaves first: data, then the children in ascending order
                    for (int lv = (int)d - 2; lv >= 0; --lv) {
                        const uint32_t t0 = n * g.tstart[lv], t1 = n * g.tstart[lv + 1], nn = n * g.apow[lv];
                        const uint32_t rbl = g.lstart[Lt + lv] + x0 * g.apow[lv];
                        for (uint32_t u = lane; u < nn * C; u += 32) {
                            const uint32_t pos = urow(u), c = uchunk(u, pos), row = rbl + pos, first = a * row + 1;
                            if (row >= G || first >= G) continue;
                            const uint32_t cnt = min(a, G - first);
                            char* mine = tile + (size_t)(t0 + pos) * rowbytes + c * 16;
                            const char* child = tile + (size_t)(t1 + a * pos) * rowbytes + c * 16;
                            uint4 v = *reinterpret_cast<const uint4*>(mine);
                            for (uint32_t ch = 0; ch < cnt; ++ch) v = comb16<T, OP>(v, *reinterpret_cast<const uint4*>(child + (size_t)ch * rowbytes));
                            *reinterpret_cast<uint4*>(mine) = v;
                        }
                        __syncwarp();
                    }
                    // 3. the forest's roots
                    for (uint32_t u = lane; u < n * C; u += 32) {
                        const uint32_t t = urow(u), c = uchunk(u, t);
                        hv[(size_t)(rb0 + t) * C + c] = *reinterpret_cast<const uint4*>(tile + (size_t)t * rowbytes + c * 16);
                    }
                }
            } else if (it < itemsAB + g.ngroups) {
                // rows above the forests: fold now, combine later
                const uint32_t r0 = (it - itemsAB) * g.cap_rows;
                for (uint32_t u = lane; u < g.cap_rows * C; u += 32) {
                    const uint32_t t = urow(u), c = uchunk(u, t), row = r0 + t;
                    if (row >= ntop || row >= G) break;
                    hv[(size_t)row * C + c] = fold_row(tile + (size_t)t * rowbytes + c * 16, in_s + c * 16, row);
                }
            } else if (sstar >= p.r) {
                if (lane < C) rootv[lane] = fold_root16<T, OP, LdGlobal>(p, root, inc, in_s + lane * 16);
            }
            release();
        }
        __syncthreads();
        // ---- binomial subtrees: the tiles' first rows form a binomial tree on the tile index ----
        if (binom) {
            const uint32_t used = (G + (1u << D) - 1) >> D;
            for (uint32_t i = 0; (1u << i) < used; ++i) {
                for (uint32_t u = tid; u < ((used >> (i + 1)) + 1) * C; u += nt) {
                    const uint32_t ur = urow(u), X = ur << (i + 1), Y = X + (1u << i), c = uchunk(u, ur);
                    if (Y < used) hv[(size_t)X * C + c] = comb16<T, OP>(hv[(size_t)X * C + c], hv[(size_t)Y * C + c]);
                }
                __syncthreads();
            }
        }
        // ---- levels above the forests, leaves first ----
        for (int lvl = (int)Lt - 1; lvl >= 0; --lvl) {
            const uint32_t lo = g.lstart[lvl], n = g.lstart[lvl + 1] - lo;
            for (uint32_t u = tid; u < n * C; u += nt) {
                const uint32_t ur = urow(u), row = lo + ur, c = uchunk(u, ur), first = a * row + 1;
                if (row >= G || first >= G) continue;
                const uint32_t cnt = min(a, G - first);
                uint4 v = hv[(size_t)row * C + c];
                for (uint32_t ch = 0; ch < cnt; ++ch) v = comb16<T, OP>(v, hv[(size_t)(first + ch) * C + c]);
                hv[(size_t)row * C + c] = v;
            }
            __syncthreads();
        }
        // ---- the root (Algorithm "reduce_root") ----
        const bool bad = *gaveup != 0;
        if (tid < C) {
            uint4 recv = hv[tid];
            recv = sstar < p.r ? recv : comb16<T, OP>(rootv[tid], recv);
            reinterpret_cast<uint4*>(out_s)[tid] = bad ? make_uint4(0, 0, 0, 0) : recv;
        }
        if (tid == 0) {
            if (bad) cx->code = FTC_ST_INTERNAL_TIMEOUT;
            write_status_rec(p, s, cx);
        }
        __syncthreads();
    }
    if (pending) mbar_wait_bounded(bar0, phase, kWaitTries);          // only after a wait gave up: a copy may still be in flight
}

// ---- host side ----
#ifndef FTC_AHEAP_TILE_KB
#define FTC_AHEAP_TILE_KB 14
#endif
constexpr uint64_t kAheapTileBytes = FTC_AHEAP_TILE_KB * 1024;   // a warp's buffer: forests are sized to fill it
constexpr size_t kAheapMaxHeapBytes = 96 * 1024;                 // the block's heap array (levels 0 .. Lt)
constexpr size_t kAheapSmallHeapBytes = 32 * 1024;               // a heap array that leaves the buffers room
#ifndef FTC_AHEAP_MAX_WARPS
#define FTC_AHEAP_MAX_WARPS 8
#endif
#ifndef FTC_AHEAP_ITEMS_PER_WARP
#define FTC_AHEAP_ITEMS_PER_WARP 4
#endif
constexpr uint32_t kAheapMaxWarps = FTC_AHEAP_MAX_WARPS;
constexpr uint32_t kAheapItemsPerWarp = FTC_AHEAP_ITEMS_PER_WARP; // a block gets a further warp only if each then has this many items a scenario

// The geometry for one buffer size; `inflight` = bytes of buffers the blocks of an SM hold together.
static bool aheap_geometry_at(Params& p, int smem_optin, AheapGeom& g, uint64_t tile_bytes, uint64_t& inflight) {
    if (p.kbytes % 16 || p.arity < 1) return false;
    const uint32_t C = p.kbytes / 16, a = p.arity;
    if (C == 0 || C > 32) return false;
    uint32_t cwl = 0; while ((1u << cwl) < C) ++cwl;
    p.C = C; p.cw_log2 = cwl; p.swz_mask = 0; p.row_shift = 0;       // plain tiles
    g.c_magic = (C & (C - 1)) ? (uint32_t)((((uint64_t)1 << 32) + C - 1) / C) : 0u;
    const uint64_t rowbytes = (uint64_t)p.m * p.kbytes;
    const uint64_t budget = tile_bytes > rowbytes ? tile_bytes : rowbytes;
    uint64_t cap_rows = 0;
    if (a == 1) {
        // binomial subtrees: a tile is 2^D rows starting at a multiple of 2^D (the binomial subtree of its first row), one
        // contiguous run; the tiles' first rows form a binomial tree again, on the tile index
        uint32_t t = 0;
        while (t < 12 && ((uint64_t)2 << t) * rowbytes <= budget && ((uint64_t)1 << t) < p.Gmax) ++t;
        const uint64_t ntiles = ((uint64_t)p.Gmax + ((uint64_t)1 << t) - 1) >> t;
        if (ntiles > (1u << 20)) return false;
        for (uint32_t l = 0; l <= kAheapMaxLevels; ++l) g.lstart[l] = 0;
        for (uint32_t u = 0; u < 5; ++u) { g.tstart[u] = 0; g.apow[u] = 0; }
        g.D = t; g.Lt = 0; g.n1 = 1u << t; g.n2 = 1; g.nA = g.nroots = (uint32_t)ntiles;
        g.itemsA = (uint32_t)ntiles; g.itemsB = 0; g.ngroups = 0; g.ntop = 0; g.nheap = (uint32_t)ntiles;
        cap_rows = (uint64_t)1 << t; g.cap_rows = (uint32_t)cap_rows;
    } else {
        // levels of the heap: first row of each level
        uint32_t Hmax = 0; uint64_t start = 0, width = 1;
        g.lstart[0] = 0;
        while (start < p.Gmax) {
            start += width; width *= a; ++Hmax;
            if (Hmax + 4 > kAheapMaxLevels) return false;
            g.lstart[Hmax] = (uint32_t)(start < 0xFFFFFFFFull ? start : 0xFFFFFFFFull);
        }
        for (uint32_t l = Hmax + 1; l <= kAheapMaxLevels; ++l) g.lstart[l] = 0xFFFFFFFFu;
        // the deepest forest of one root within the budget (at most four levels)
        uint32_t D = 1; uint64_t R = 1, w = a;
        while (D < 4 && D < Hmax && (R + w) * rowbytes <= budget) { R += w; w *= a; ++D; }
        { uint64_t s0 = 0, pw = 1; for (uint32_t u = 0; u < 5; ++u) { g.tstart[u] = (uint32_t)s0; g.apow[u] = (uint32_t)pw; s0 += pw; pw *= a; } }
        g.D = D; g.Lt = Hmax - D;
        const uint64_t Rshallow = g.tstart[D - 1];                                   // rows of a root with D - 1 levels (0: D = 1)
        uint64_t nroots = 1; for (uint32_t l = 0; l < g.Lt; ++l) nroots *= a;
        if (nroots > (1u << 20)) return false;
        const uint64_t nlast = p.Gmax - g.lstart[Hmax - 1];                          // rows on the heap's last level
        const uint64_t per_root_last = g.apow[D - 1];
        g.nA = (uint32_t)((nlast + per_root_last - 1) / per_root_last);
        g.nroots = D == 1 ? g.nA : (uint32_t)nroots;
        g.n1 = (uint32_t)(budget / (R * rowbytes)); if (g.n1 < 1) g.n1 = 1;
        g.n2 = Rshallow ? (uint32_t)(budget / (Rshallow * rowbytes)) : 1;
        // where the deep forests hold most of the rows the buffer is sized for them: no larger shallow forests
        if (Rshallow && (uint64_t)g.nA * R >= (g.nroots - g.nA) * Rshallow && g.n2 * Rshallow > g.n1 * R) g.n2 = (uint32_t)(g.n1 * R / Rshallow);
        if (g.n2 < 1) g.n2 = 1;
        g.itemsA = (g.nA + g.n1 - 1) / g.n1;
        g.itemsB = (g.nroots - g.nA + g.n2 - 1) / g.n2;
        cap_rows = g.n1 * R; if (g.n2 * Rshallow > cap_rows) cap_rows = g.n2 * Rshallow;
        g.cap_rows = (uint32_t)cap_rows;
        g.ntop = g.lstart[g.Lt]; g.nheap = g.ntop + (uint32_t)nroots;
        g.ngroups = (g.ntop + g.cap_rows - 1) / g.cap_rows;
    }
    const size_t hv_bytes = (size_t)g.nheap * C * 16;
    if (hv_bytes > kAheapMaxHeapBytes) return false;
    g.tile_cap = (uint32_t)((cap_rows * rowbytes + 127) & ~(uint64_t)127);
    const uint32_t nitems = g.itemsA + g.itemsB + g.ngroups + 1;
    size_t o = sizeof(Ctx) + 3 * (size_t)(p.W + 1) * 4;
    o = (o + 15) & ~(size_t)15; g.off_rootv = (uint32_t)o; o += (size_t)C * 16;
    g.off_hv = (uint32_t)o; o += hv_bytes;
    g.off_bar = (uint32_t)o; o += 8 * 8;
    g.off_gaveup = (uint32_t)o; o += 8;
    o = (o + 127) & ~(size_t)127; g.off_tiles = (uint32_t)o;
    // Warps per block: what counts is how many buffers the blocks of an SM keep in flight together (each warp waits for
    // its one buffer, folds it and asks for the next), so take the count that fits the most, among those that leave every
    // warp a few items per scenario; on a tie the smaller blocks, whose decodes overlap the others' streaming.
    const size_t per_sm = (size_t)smem_optin + 1024, limit = (size_t)smem_optin - 1024;
    uint32_t warps = 0, best = 0;
    for (uint32_t w = 1; w <= kAheapMaxWarps; ++w) {
        const size_t block = o + (size_t)w * g.tile_cap;
        if (block > limit) break;
        if (w > 1 && w * kAheapItemsPerWarp > nitems) break;
        size_t blocks = per_sm / (block + 1024);
        const size_t by_regs = kAheapWarpsPerSM / w, by_slots = 32;
        if (blocks > by_regs) blocks = by_regs;
        if (blocks > by_slots) blocks = by_slots;
        if (blocks * w > best) { best = (uint32_t)(blocks * w); warps = w; }
    }
    if (!warps) return false;
    o += (size_t)warps * g.tile_cap;
    g.nwarps = warps; g.smem_bytes = (uint32_t)o;
    inflight = (uint64_t)best * g.tile_cap;
    return true;
}

// Buffer size: a larger buffer can take forests one level deeper, which divides the forests' roots -- and with them the
// block's heap array -- by the arity. The smallest size whose heap array leaves most of the shared memory to the buffers
// is taken; where none does, the size that keeps the most bytes in flight.
static bool aheap_geometry(Params& p, int smem_optin, AheapGeom& g) {
    bool found = false; uint64_t best = 0;
    for (uint64_t tile = kAheapTileBytes; tile <= kAheapTileBytes + 12 * 1024; tile += 4 * 1024) {
        AheapGeom t; Params q = p; uint64_t inflight = 0;
        if (!aheap_geometry_at(q, smem_optin, t, tile, inflight)) continue;
        const size_t hv_bytes = (size_t)t.nheap * q.C * 16;
        if (hv_bytes <= kAheapSmallHeapBytes) { p = q; g = t; return true; }
        if (!found || inflight > best) { found = true; best = inflight; p = q; g = t; }
    }
    return found;
}

template <typename T, int OP, bool NP2, int M>
static cudaError_t launch_aheap_k(const Params& p, const AheapGeom& g, int sm_count, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(aheap_kernel<T, OP, NP2, M>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem_bytes);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, aheap_kernel<T, OP, NP2, M>, (int)g.nwarps * 32, g.smem_bytes);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    const uint64_t cap = (uint64_t)sm_count * per_sm;
    const uint32_t grid = (uint32_t)(p.S < cap ? p.S : cap);
    if (p.grid_query) { *p.grid_query = grid; return cudaSuccess; }
    aheap_kernel<T, OP, NP2, M><<<grid, g.nwarps * 32, g.smem_bytes, st>>>(p, g);
    return cudaGetLastError();
}

template <typename T, int OP>
static cudaError_t launch_aheap_t(Params p, int sm_count, int smem_optin, cudaStream_t st) {
    AheapGeom g;
    if (!aheap_geometry(p, smem_optin, g)) return cudaErrorInvalidConfiguration;
    if (g.c_magic) return launch_aheap_k<T, OP, true, 0>(p, g, sm_count, st);
    switch (p.m) {                                                  // the group sizes of f = 2, 3, 4 and 8
    case 3: return launch_aheap_k<T, OP, false, 3>(p, g, sm_count, st);
    case 4: return launch_aheap_k<T, OP, false, 4>(p, g, sm_count, st);
    case 5: return launch_aheap_k<T, OP, false, 5>(p, g, sm_count, st);
    case 9: return launch_aheap_k<T, OP, false, 9>(p, g, sm_count, st);
    default: return launch_aheap_k<T, OP, false, 0>(p, g, sm_count, st);
    }
}

cudaError_t launch_aheap_u64(const Params& p, int tsel, int sm_count, int smem_optin, cudaStream_t st);
cudaError_t launch_aheap_b32(const Params& p, int tsel, int sm_count, int smem_optin, cudaStream_t st);
cudaError_t launch_aheap_b64(const Params& p, int tsel, int sm_count, int smem_optin, cudaStream_t st);

}  // namespace ftc
