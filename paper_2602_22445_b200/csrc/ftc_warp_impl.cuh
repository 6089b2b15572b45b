// Warp kernel: scenarios of a few KB, one warp (= one block) per scenario at a time. For such scenarios the work
// per scenario that is not combining -- decoding the masks, barriers between the threads of a block, setting up
// copies -- outweighs the combining, so everything here is warp-local: the masks are decoded in registers
// (ftc_decode_warp.cuh), consecutive scenarios arrive several at a time by one bulk copy into the warp's own double
// buffer, their masks, in-operation entries and roots are fetched one group ahead into registers, and the whole
// subtree heap of a scenario is one warp tile (lanes = lane rows x 16-byte chunks, lane-local sub-heaps below,
// shuffles above), evaluated by the same routines as the tiles of the staged kernel. The tile has exactly as many
// levels as the heap (fewer lane rows are used when the heap is shallow), so it is complete down to its
// second-to-last level and the check-free folds serve every scenario; only the short last group, one row, is
// folded by the general routine.
// Before the evaluation the warp exchanges the vectors of process 0 and of the root in its copy of the scenario, so
// that the copy is in renumbered order (section "Reduce": the root swaps numbers with process 0) and no group needs
// special addressing. Scenarios the register decode leaves out (more failures than tolerated, a root out of range)
// go through decode_scenario()/count_holders(), which a one-warp block can call as they are.
#pragma once
#include "ftc_staged_impl.cuh"
#include "ftc_decode_warp.cuh"

namespace ftc {

struct WarpGeom {
    uint32_t lanes;        // lanes that play one scenario: 32, or 16 / 8 when the tile needs no more (several scenarios per warp)
    uint32_t lw;           // levels of the tile combined with shuffles: 2^lw lane rows are used
    uint32_t group;        // scenarios per buffer (consecutive scenarios, one bulk copy)
    uint32_t buf_bytes;    // bytes per buffer (multiple of 128)
    uint32_t off_bar, off_buf, smem_bytes;
};

// blocks (= warps) per SM the register budget allows: sub-heaps of three levels keep eight rows per lane in registers
// (several scenarios per warp need a few more registers: 24 warps then)
template <int XL, int L = 32> struct WarpMinBlocks { static constexpr int value = XL >= 3 ? 16 : (L < 32 ? 24 : 32); };

// MODE: bit 0 = allreduce, bit 1 = the call has in-operation slots.
// L: lanes per scenario. L < 32: the warp plays 32 / L scenarios at a time, one per group of L lanes, with one
// instruction stream: the decode is decode_group<L>, the tile's shuffles stay inside the group, and what used to be
// the same for the whole warp (root, selected child, masks) is the same within a group. A pair that holds a scenario
// for the general routines is played one scenario after the other, all groups on the same scenario.
template <typename T, int OP, int XL, int MODE, int L>
__global__ void __launch_bounds__(32, WarpMinBlocks<XL, L>::value) warp_kernel(Params p, WarpGeom g) {
    constexpr bool ALLRED = (MODE & 1) != 0, INOP = (MODE & 2) != 0;
    constexpr uint32_t NS = 32 / L;
    extern __shared__ __align__(128) uint32_t smem[];
    char* sbase = reinterpret_cast<char*>(smem);
    Ctx* cx = reinterpret_cast<Ctx*>(smem);
    uint32_t* pf = smem + sizeof(Ctx) / 4;
    uint32_t* inc = pf + p.W + 1;
    uint32_t* unr = inc + p.W + 1;
    uint32_t* ginc = unr + p.W + 1;                                     // L < 32: one arrival mask (W + 1 words) per group
    const uint32_t lane = threadIdx.x;
    const uint32_t lg = lane & (L - 1), gi = lane / L;                  // lane within its group, group within the warp
    const uint32_t cwl = p.cw_log2, lw = g.lw, RW = 1u << lw;
    const uint32_t lr_real = lg >> cwl, lc = lg & (p.C - 1);
    const uint32_t lr = lr_real < RW ? lr_real : 0u;                    // lane rows beyond the tile repeat lane row 0 (their results are unused)
    const uint32_t nq = p.C < 8 ? 8u / p.C : 1u, gq = min(nq, p.m & (0u - p.m));
    const uint32_t rot = (lr >> ilog2u(nq / gq)) & (gq - 1);          // starting member of this lane row's folds (bank spread)
    const uint32_t rowbytes = p.m * p.kbytes;
    const uint64_t scen_bytes = (uint64_t)p.P * p.kbytes;
    const uint32_t tries = (p.flags & FTC_DEBUG_ONE_POLL) ? 1u : kWaitTries;
    const uint32_t bar0 = smem_addr(sbase + g.off_bar);
    char* bufs = sbase + g.off_buf;
    if (lane < 2) mbar_init(bar0 + lane * 8, 1);
    if (lane == 0) { pf[p.W] = 0; inc[p.W] = 0; }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();

    const uint64_t ngroups = (p.S + g.group - 1) / g.group;
    uint32_t phase_bits = 0, pending = 0;
    bool dead = false;                  // a bounded wait gave up: no further copies or waits, every later scenario reports it
    auto group_size = [&](uint64_t grp) { return (uint32_t)min((uint64_t)g.group, p.S - grp * g.group); };
    auto issue = [&](uint64_t grp, uint32_t b) {
        if (dead) return;
        const uint32_t bytes = group_size(grp) * (uint32_t)scen_bytes;
        if (lane == 0) {
            mbar_expect_tx(bar0 + b * 8, bytes);
            bulk_g2s(smem_addr(bufs + (size_t)b * g.buf_bytes), reinterpret_cast<const char*>(p.in) + grp * g.group * scen_bytes,
                     bytes, bar0 + b * 8);
        }
        pending |= 1u << b;
    };
    // masks, in-operation entries and roots of a group, one register each (group * W, group * max_inop and group are at most 32)
    struct Small { uint32_t pfw, vic, rnd, root; };
    auto fetch = [&](uint64_t grp) {
        Small s{0, FTC_INOP_UNUSED, 0, 0};
        const uint32_t n = group_size(grp);
        const uint64_t s0 = grp * g.group;
        if (lane < n * p.W) s.pfw = __ldg(p.prefail + s0 * p.W + lane);
        if (lane < n * p.max_inop) { const ftc_inop_t* e = p.inop + s0 * p.max_inop + lane; s.vic = __ldg(&e->victim); s.rnd = __ldg(&e->round); }
        if (p.root < 0 && lane < n) s.root = __ldg(p.roots + s0 + lane);
        return s;
    };

    uint64_t grp = blockIdx.x;
    uint32_t b = 0;
    Small cur{0, FTC_INOP_UNUSED, 0, 0};
    if (grp < ngroups) { issue(grp, 0); cur = fetch(grp); }
    for (; grp < ngroups; grp += gridDim.x, b ^= 1u) {
        const uint64_t nxt = grp + gridDim.x;
        Small nx{0, FTC_INOP_UNUSED, 0, 0};
        if (nxt < ngroups) { issue(nxt, b ^ 1u); nx = fetch(nxt); }
        if (!dead && ((pending >> b) & 1u)) {
            bool ok = mbar_wait_bounded(bar0 + b * 8, (phase_bits >> b) & 1u, tries);
            if (!__all_sync(kFullWarp, ok)) {
                if (__any_sync(kFullWarp, ok) && !ok) ok = mbar_wait_bounded(bar0 + b * 8, (phase_bits >> b) & 1u, kWaitTries);
                ok = __all_sync(kFullWarp, ok);
            }
            if (ok) { phase_bits ^= 1u << b; pending &= ~(1u << b); }
            else dead = true;
        }
        const uint32_t n = group_size(grp);
        if constexpr (L == 32) {
        for (uint32_t i = 0; i < n; ++i) {
                const uint64_t s = grp * g.group + i;
                char* out_s = reinterpret_cast<char*>(p.out) + s * p.kbytes;
                uint32_t pfw = __shfl_sync(kFullWarp, cur.pfw, lane < p.W ? i * p.W + lane : 0u);
                if (lane >= p.W) pfw = 0;
                else if (lane == p.W - 1 && (p.P & 31)) pfw &= (1u << (p.P & 31)) - 1u;
                uint32_t ev = FTC_INOP_UNUSED, er = 0;
                if (INOP) {
                    const uint32_t src = lane < p.max_inop ? i * p.max_inop + lane : 0u;
                    ev = __shfl_sync(kFullWarp, cur.vic, src); er = __shfl_sync(kFullWarp, cur.rnd, src);
                }
                const uint32_t first_root = p.root >= 0 ? (uint32_t)p.root : __shfl_sync(kFullWarp, cur.root, i);
                WarpScen w; bool slow;
                decode_group<32, (ALLRED ? 1 : 0), (INOP ? 1 : 0)>(p, pfw, ev, er, first_root, w, slow);
                if (!slow) {
                    if (lane <= p.W) inc[lane] = w.incw;
                    if (p.W == 32 && lane == 0) inc[32] = 0;
                    __syncwarp();
                } else {
                    // the general routines (a block of one warp may call them): everything outside the register decode
                    decode_scenario(p, s, cx, pf, inc);
                    if (cx->code == FTC_ST_OK && ALLRED) count_holders(p, cx, pf, unr);
                    w.code = cx->code; w.sstar = cx->sstar; w.attempts = cx->attempts; w.root = cx->root; w.base = cx->base;
                    w.npre = cx->npre; w.nexcl = cx->nexcl; w.inop_incl = cx->inop_incl; w.holders = cx->holders; w.G = cx->G;
                    w.any_victim = 1;
                    __syncwarp();
                }
                const bool okc = w.code == FTC_ST_OK && !dead;
                if (!okc) {
                    if (lane < p.C) reinterpret_cast<uint4*>(out_s)[lane] = make_uint4(0, 0, 0, 0);
                } else {
                    char* sc = bufs + (size_t)b * g.buf_bytes + (size_t)i * scen_bytes;
                    // renumbered order: the vectors of process 0 and of the root change places (the copy is the warp's own)
                    if (w.root != 0) {
                        if (lane < p.C) {
                            uint4* a = reinterpret_cast<uint4*>(sc) + lane;
                            uint4* c = reinterpret_cast<uint4*>(sc + (size_t)w.root * p.kbytes) + lane;
                            const uint4 va = *a, vc = *c;
                            *a = vc; *c = va;
                        }
                        __syncwarp();
                    }
                    const uint32_t sstar = w.sstar, G = w.G;
                    const char* in_lc = sc + lc * 16;
                    // the one tile: heap rows 0 .. 2^D - 2; lane row lr owns row lr of the upper levels and the sub-heap under row RW-1+lr
                    const uint32_t tA = RW - 1 + lr, rowA = tA, tB = ilog2u(lr + 1), idxB = lr + 1 - (1u << tB), rowB = lr;
                    const bool masked = w.npre != 0 || w.any_victim != 0;
                    uint4 valA, valB;
                    const bool hasB = lr < RW - 1;
                    fold_tile_fast<T, OP, XL, true, false, true>(p, 0u, sstar, inc, in_lc, in_lc, rowbytes, 0u, lr, rot, rowB, hasB, tA, rowA, G, masked, valA, valB,
                                                                 G > p.q ? p.q : 0xFFFFFFFFu);
                    valB = tile_tree_phase<T, OP, (XL > 1), true>(valA, valB, lw, cwl, p.C, lane, lc, tB, idxB, rowB, hasB, G);
                    // the root (Algorithm "reduce_root"): its own data on the left unless the child's subtree holds it already
                    if (lr_real == 0) {
                        uint4 recv = lw ? valB : valA;
                        if (sstar >= p.r) recv = comb16<T, OP>(fold_root16<T, OP, LdShared>(p, 0u, inc, in_lc), recv);
                        reinterpret_cast<uint4*>(out_s)[lc] = recv;
                    }
                }
                if (lane == 0) {
                    uint4 rec;
                    const uint32_t code = dead ? (uint32_t)FTC_ST_INTERNAL_TIMEOUT : w.code;
                    rec.x = code | ((okc ? w.sstar : 0xFFu) << 8) | (w.attempts << 16);
                    rec.y = okc ? p.P - w.npre - w.nexcl : 0u;
                    rec.z = okc ? w.inop_incl : 0u;
                    rec.w = (okc && ALLRED) ? w.holders : 0u;
                    *reinterpret_cast<uint4*>(p.status + s * FTC_STATUS_WORDS) = rec;
                }
                __syncwarp();
            }
        } else {
            // ---- 32 / L scenarios at a time, one per group of L lanes ----
            auto evaluate = [&](const WarpScen& w, const uint32_t* incp, char* sc, bool writer, uint64_t s) {
                const bool okc = w.code == FTC_ST_OK && !dead;
                // renumbered order: the vectors of process 0 and of the root change places (the copy is the warp's own)
                if (okc && writer && w.root != 0 && lg < p.C) {
                    uint4* a = reinterpret_cast<uint4*>(sc) + lg;
                    uint4* c = reinterpret_cast<uint4*>(sc + (size_t)w.root * p.kbytes) + lg;
                    const uint4 va = *a, vc = *c;
                    *a = vc; *c = va;
                }
                __syncwarp();
                const uint32_t sstar = okc ? w.sstar : 0u, G = okc ? w.G : 0u;   // G = 0: every fold reads row 0, results unused
                const char* in_lc = sc + lc * 16;
                const uint32_t tA = RW - 1 + lr, rowA = tA, tB = ilog2u(lr + 1), idxB = lr + 1 - (1u << tB), rowB = lr;
                const bool masked = okc && (w.npre != 0 || w.any_victim != 0);
                uint4 valA, valB;
                const bool hasB = lr < RW - 1;
                fold_tile_fast<T, OP, XL, true, false, true>(p, 0u, sstar, incp, in_lc, in_lc, rowbytes, 0u, lr, rot, rowB, hasB, tA, rowA, G, masked, valA, valB,
                                                             (okc && G > p.q) ? p.q : 0xFFFFFFFFu);
                valB = tile_tree_phase<T, OP, (XL > 1), true, L>(valA, valB, lw, cwl, p.C, lg, lc, tB, idxB, rowB, hasB, G);
                if (writer) {
                    if (lr_real == 0) {
                        uint4 recv = make_uint4(0, 0, 0, 0);
                        if (okc) {
                            recv = lw ? valB : valA;
                            if (sstar >= p.r) recv = comb16<T, OP>(fold_root16<T, OP, LdShared>(p, 0u, incp, in_lc), recv);
                        }
                        reinterpret_cast<uint4*>(reinterpret_cast<char*>(p.out) + s * p.kbytes)[lc] = recv;
                    }
                    if (lg == 0) {
                        uint4 rec;
                        const uint32_t code = dead ? (uint32_t)FTC_ST_INTERNAL_TIMEOUT : w.code;
                        rec.x = code | ((okc ? w.sstar : 0xFFu) << 8) | (w.attempts << 16);
                        rec.y = okc ? p.P - w.npre - w.nexcl : 0u;
                        rec.z = okc ? w.inop_incl : 0u;
                        rec.w = (okc && ALLRED) ? w.holders : 0u;
                        *reinterpret_cast<uint4*>(p.status + s * FTC_STATUS_WORDS) = rec;
                    }
                }
                __syncwarp();
            };
            char* buf = bufs + (size_t)b * g.buf_bytes;
            for (uint32_t i = 0; i < n; i += NS) {
                const uint32_t si = i + gi;
                const bool active = si < n;
                const bool has_word = active && lg < p.W;
                uint32_t pfw = __shfl_sync(kFullWarp, cur.pfw, has_word ? si * p.W + lg : 0u);
                if (!has_word) pfw = 0;
                else if (lg == p.W - 1 && (p.P & 31)) pfw &= (1u << (p.P & 31)) - 1u;
                uint32_t ev = FTC_INOP_UNUSED, er = 0;
                if (INOP) {
                    const uint32_t src = (active && lg < p.max_inop) ? si * p.max_inop + lg : 0u;
                    ev = __shfl_sync(kFullWarp, cur.vic, src); er = __shfl_sync(kFullWarp, cur.rnd, src);
                    if (!active) ev = FTC_INOP_UNUSED;
                }
                const uint32_t rsrc = __shfl_sync(kFullWarp, cur.root, active ? si : 0u);
                const uint32_t first_root = p.root >= 0 ? (uint32_t)p.root : rsrc;
                WarpScen w; bool slow;
                decode_group<L, (ALLRED ? 1 : 0), (INOP ? 1 : 0)>(p, pfw, ev, er, first_root, w, slow);
                if (__any_sync(kFullWarp, active && slow)) {
                    // rare: a scenario for the general routines (a block of one warp may call them). The scenarios of this
                    // round are played one after the other, every group on the same scenario, the first group writing.
                    for (uint32_t gg = 0; gg < NS && i + gg < n; ++gg) {
                        const uint64_t s = grp * g.group + i + gg;
                        decode_scenario(p, s, cx, pf, inc);
                        if (cx->code == FTC_ST_OK && ALLRED) count_holders(p, cx, pf, unr);
                        WarpScen w1;
                        w1.code = cx->code; w1.sstar = cx->sstar; w1.attempts = cx->attempts; w1.root = cx->root; w1.base = cx->base;
                        w1.npre = cx->npre; w1.nexcl = cx->nexcl; w1.inop_incl = cx->inop_incl; w1.holders = cx->holders; w1.G = cx->G;
                        w1.any_victim = 1; w1.incw = 0; w1.iv = 0;
                        __syncwarp();
                        evaluate(w1, inc, buf + (size_t)(i + gg) * scen_bytes, gi == 0, s);
                    }
                } else {
                    uint32_t* incp = ginc + gi * (p.W + 1);
                    if (lg <= p.W) incp[lg] = w.incw;
                    if (p.W == L && lg == 0) incp[L] = 0;
                    if (!active) w.code = FTC_ST_BAD_ROOT;              // nothing to play: G = 0, nothing written
                    __syncwarp();
                    evaluate(w, incp, buf + (size_t)(active ? si : 0u) * scen_bytes, active, grp * g.group + si);
                }
            }
        }
        cur = nx;
    }
    // only after a wait gave up: a copy may still be in flight toward this block's shared memory
    for (uint32_t bb = 0; bb < 2; ++bb)
        if ((pending >> bb) & 1u) mbar_wait_bounded(bar0 + bb * 8, (phase_bits >> bb) & 1u, kWaitTries);
}

// ---- host side ----
// Shapes: 16-byte chunks, a power-of-two chunk count of at most 32, at most 1024 processes (one mask word per lane), a
// subtree heap that fits one warp tile with a lane-local sub-heap of at most three levels, scenarios of at most
// kWarpMaxBytes. XL: the shallowest sub-heap that holds the heap.
constexpr uint64_t kWarpMaxBytes = 8 * 1024;
constexpr uint32_t kWarpBufTarget = 2560;       // a buffer holds as many consecutive scenarios as fit in this (at least one)

static bool warp_geometry(Params& p, int smem_optin, uint32_t& XL, WarpGeom& g) {
    if (p.kbytes % 16 || p.W > 32) return false;
    const uint32_t C = p.kbytes / 16;
    if (C == 0 || C > 32 || (C & (C - 1))) return false;
    const uint64_t scen_bytes = (uint64_t)p.P * p.kbytes;
    if (scen_bytes > kWarpMaxBytes) return false;
    uint32_t cwl = 0; while ((1u << cwl) < C) ++cwl;
    const uint32_t lw = 5 - cwl;
    uint32_t Hmax = 1; while ((1u << Hmax) <= p.Gmax) ++Hmax;
    if (Hmax > lw + 3) return false;
    g.lw = Hmax - 1 < lw ? Hmax - 1 : lw;                      // a shallow heap uses fewer lane rows
    XL = Hmax - g.lw;
    // Half a warp per scenario where the tile fits 16 lanes: two scenarios then share one instruction stream, and for
    // scenarios of a KB or so that stream is what bounds them. (Fewer lane rows with deeper lane-local sub-heaps, to make
    // 2 KB scenarios fit as well, measured slower: 1.4 instead of 2.2 TB/s.)
    g.lanes = (p.W <= 16 && p.m <= 16 && p.max_inop <= 16 && (C << g.lw) <= 16 && XL <= 2) ? 16 : 32;
    p.C = C; p.cw_log2 = cwl; p.Lt = 0; p.below = 0; p.swz_mask = 0; p.row_shift = 0;
    uint32_t group = (uint32_t)(kWarpBufTarget / scen_bytes);
    if (group < 1) group = 1;
    while (group > 1 && (group * p.W > 32 || group * p.max_inop > 32 || group > 32)) --group;
    if (p.max_inop > 32) return false;
    g.group = group;
    // behind the last scenario: room for the bytes a full group would have beyond the short last group (read, not used)
    g.buf_bytes = (uint32_t)((group * scen_bytes + (uint64_t)p.m * p.kbytes + 127) & ~(uint64_t)127);
    size_t o = sizeof(Ctx) + (3 + 32 / g.lanes) * (size_t)(p.W + 1) * 4;      // the general routines' masks, then one arrival mask per group
    o = (o + 15) & ~(size_t)15; g.off_bar = (uint32_t)o; o += 16;
    o = (o + 127) & ~(size_t)127; g.off_buf = (uint32_t)o;
    o += 2 * (size_t)g.buf_bytes;
    g.smem_bytes = (uint32_t)o;
    return o <= (size_t)smem_optin - 1024;
}

template <typename T, int OP, int XL, int MODE, int L>
static cudaError_t launch_warp_l(const Params& p, const WarpGeom& g, int sm_count, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(warp_kernel<T, OP, XL, MODE, L>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem_bytes);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, warp_kernel<T, OP, XL, MODE, L>, 32, g.smem_bytes);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    const uint64_t ngroups = (p.S + g.group - 1) / g.group, cap = (uint64_t)sm_count * per_sm;
    const uint32_t grid = (uint32_t)(ngroups < cap ? ngroups : cap);
    if (p.grid_query) { *p.grid_query = grid; return cudaSuccess; }
    warp_kernel<T, OP, XL, MODE, L><<<grid, 32, g.smem_bytes, st>>>(p, g);
    return cudaGetLastError();
}

template <typename T, int OP, int XL, int MODE>
static cudaError_t launch_warp_m(const Params& p, const WarpGeom& g, int sm_count, cudaStream_t st) {
    if constexpr (XL <= 2) {
        if (g.lanes == 16) return launch_warp_l<T, OP, XL, MODE, 16>(p, g, sm_count, st);
    }
    return launch_warp_l<T, OP, XL, MODE, 32>(p, g, sm_count, st);
}

template <typename T, int OP, int XL>
static cudaError_t launch_warp_x(const Params& p, const WarpGeom& g, int sm_count, cudaStream_t st) {
    switch ((p.is_allreduce ? 1 : 0) | (p.max_inop ? 2 : 0)) {
    case 0: return launch_warp_m<T, OP, XL, 0>(p, g, sm_count, st);
    case 1: return launch_warp_m<T, OP, XL, 1>(p, g, sm_count, st);
    case 2: return launch_warp_m<T, OP, XL, 2>(p, g, sm_count, st);
    default: return launch_warp_m<T, OP, XL, 3>(p, g, sm_count, st);
    }
}

template <typename T, int OP>
static cudaError_t launch_warp_t(Params p, int sm_count, int smem_optin, cudaStream_t st) {
    WarpGeom g; uint32_t XL = 1;
    if (!warp_geometry(p, smem_optin, XL, g)) return cudaErrorInvalidConfiguration;
    switch (XL) {
    case 1: return launch_warp_x<T, OP, 1>(p, g, sm_count, st);
    case 2: return launch_warp_x<T, OP, 2>(p, g, sm_count, st);
    default: return launch_warp_x<T, OP, 3>(p, g, sm_count, st);
    }
}

}  // namespace ftc
