// Level kernel: the shared-memory path for subtrees that are a-ary heaps (FTC_TREE_ARITY(a), a = 2..32; the paper's
// I(f)-tree fixes only the root's f+1 children and their subtree sizes, so any such shape is one). The heap of the
// selected subtree's rows is cut into tiles as in the staged kernel -- a tile is a sub-heap of D levels, each level one
// contiguous run of rows, brought into shared memory by one bulk copy per level -- but a tile is evaluated level by
// level in shared memory instead of in registers and shuffles, which works for any number of children per node:
//   1. every (row, 16-byte chunk) of the tile folds its group (Algorithm "Up-correction": own input, then the partners
//      whose message arrived, in the schedule's order) and leaves the result in place of the row's first member;
//   2. the tile's levels are combined from the leaves up (Algorithm "reduce_non_root": data, then child 1, child 2, ...),
//      again in place, with a warp-level barrier between levels;
//   3. the tile's root goes to the block's heap array, which is combined level by level as in the staged kernel.
// Each row decides by itself whether the plain fold from its staged copy serves it (a full group under its arrival mask)
// or the general fold is needed (a renumbered slot, the short last group): no marking pass.
#pragma once
#include "ftc_staged_impl.cuh"

namespace ftc {

constexpr uint32_t kAheapMaxLevels = 24;

struct AheapGeom {
    uint32_t nwarps, tile_cap;             // warps per block, bytes of a warp's buffer
    uint32_t D, Lt;                        // levels of a tile; heap level at which the tiles are rooted
    uint32_t R;                            // rows of a tile: (a^D - 1) / (a - 1)
    uint32_t ntop, ntiles, nheap;          // rows above the tiles, tiles, rows of the heap array (ntop + ntiles)
    uint32_t ngroups;                      // work items over the rows above the tiles (R rows each)
    uint32_t lstart[kAheapMaxLevels + 1];  // first row of heap level l: (a^l - 1) / (a - 1)
    uint32_t tstart[4], apow[4];           // tile level u: its first node, and a^u (0xFFFFFFFF / 0 beyond the tile's levels)
    uint32_t off_rootv, off_hv, off_bar, off_gaveup, off_tiles, smem_bytes;
};

template <typename T, int OP>
__global__ void __launch_bounds__(kStagedMaxThreads, 2) aheap_kernel(Params p, const __grid_constant__ AheapGeom g) {
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
    const uint32_t a = p.arity, C = p.C, cwl = p.cw_log2, Cmask = C - 1;
    const uint32_t D = g.D, R = g.R, ntop = g.ntop, ntiles = g.ntiles;
    const uint32_t nitems = ntiles + g.ngroups + 1;
    const uint32_t rowbytes = p.m * p.kbytes;
    const uint64_t scen_bytes = (uint64_t)p.P * p.kbytes;
    const uint32_t tries = (p.flags & FTC_DEBUG_ONE_POLL) ? 1u : kWaitTries;
    // a^u for the tile level u that holds tile node t
    const uint32_t ts1 = g.tstart[1], ts2 = g.tstart[2], ts3 = g.tstart[3], a2 = a * a, a3 = a2 * a;
    auto level_width = [&](uint32_t t) { return t >= ts3 ? a3 : t >= ts2 ? a2 : t >= ts1 ? a : 1u; };

    const uint32_t bar0 = smem_addr(sbase + g.off_bar) + wid * 8;
    char* tile = sbase + g.off_tiles + (size_t)wid * g.tile_cap;
    if (lane == 0) mbar_init(bar0, 1);
    if (tid == 0) *gaveup = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    uint32_t phase = 0;
    bool pending = false, stop = false;

    // ---- this warp's copy pipeline over the flat sequence (scenario, work item), one buffer, one item ahead ----
    const uint32_t n_my = wid < nitems ? (nitems - wid + nw - 1) / nw : 0;
    uint64_t is_s = blockIdx.x;
    const char* is_src = reinterpret_cast<const char*>(p.in) + is_s * scen_bytes;
    uint32_t is_i = 0;
    uint32_t my_rows = 0, my_start = 0;                               // lane u < D copies level u of a tile
    if (lane < D) { my_rows = g.apow[lane]; my_start = g.tstart[lane]; }
    auto issue_next = [&]() {
        if (n_my == 0 || is_s >= p.S || stop) return;
        const uint32_t it = wid + is_i * nw;
        uint64_t first_row = 0; uint32_t nrows = 0, dst_off = 0;
        if (it < ntiles) {
            if (lane < D) { first_row = (uint64_t)my_rows * (ntop + it) + my_start; nrows = my_rows; dst_off = my_start * rowbytes; }
        } else if (it < ntiles + g.ngroups) {
            if (lane == 0) { first_row = (uint64_t)(it - ntiles) * R; nrows = min(R, ntop - (uint32_t)first_row); }
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

    for (uint64_t s = blockIdx.x; s < p.S; s += gridDim.x) {
        const char* in_s = reinterpret_cast<const char*>(p.in) + s * scen_bytes;
        const bool dead = *gaveup != 0;
        if (dead) stop = true;
        decode_scenario(p, s, cx, pf, inc);
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
        if (p.is_allreduce) count_holders(p, cx, pf, unr);
        const uint32_t root = cx->root, sstar = cx->sstar, G = cx->G;

        for (uint32_t i = 0; i < n_my; ++i) {
            const uint32_t it = wid + i * nw;
            acquire();
            if (it < ntiles) {
                const uint32_t j0 = ntop + it;
                if (j0 < G) {
                    // 1. every (row, chunk) folds its group; the result takes the place of the row's first member
                    for (uint32_t u = lane; u < R * C; u += 32) {
                        const uint32_t t = u >> cwl, c = u & Cmask, row = level_width(t) * j0 + t;
                        if (row >= G) continue;
                        char* srow = tile + (size_t)t * rowbytes + c * 16;
                        *reinterpret_cast<uint4*>(srow) = fold_staged<T, OP, false>(p, root, sstar, inc, in_s + c * 16, srow, row);
                    }
                    __syncwarp();
                    // 2. the levels of the tile, leaves first: data, then the children in ascending order
                    for (int lv = (int)D - 2; lv >= 0; --lv) {
                        const uint32_t t0 = g.tstart[lv], nn = g.apow[lv];
                        for (uint32_t u = lane; u < nn * C; u += 32) {
                            const uint32_t t = t0 + (u >> cwl), c = u & Cmask, row = nn * j0 + t;
                            if (row >= G) continue;
                            uint4 v = *reinterpret_cast<const uint4*>(tile + (size_t)t * rowbytes + c * 16);
                            for (uint32_t ch = 1; ch <= a; ++ch)
                                if ((uint64_t)a * row + ch < G) v = comb16<T, OP>(v, *reinterpret_cast<const uint4*>(tile + (size_t)(a * t + ch) * rowbytes + c * 16));
                            *reinterpret_cast<uint4*>(tile + (size_t)t * rowbytes + c * 16) = v;
                        }
                        __syncwarp();
                    }
                    // 3. the tile's root
                    if (lane < C) hv[(size_t)j0 * C + lane] = *reinterpret_cast<const uint4*>(tile + lane * 16);
                }
            } else if (it < ntiles + g.ngroups) {
                // rows above the tiles: fold now, combine later
                const uint32_t r0 = (it - ntiles) * R;
                for (uint32_t u = lane; u < R * C; u += 32) {
                    const uint32_t t = u >> cwl, c = u & Cmask, row = r0 + t;
                    if (row >= ntop || row >= G) continue;
                    hv[(size_t)row * C + c] = fold_staged<T, OP, false>(p, root, sstar, inc, in_s + c * 16, tile + (size_t)t * rowbytes + c * 16, row);
                }
            } else if (sstar >= p.r) {
                if (lane < C) rootv[lane] = fold_root16<T, OP, LdGlobal>(p, root, inc, in_s + lane * 16);
            }
            release();
        }
        __syncthreads();
        // ---- levels above the tiles, leaves first ----
        for (int lvl = (int)g.Lt - 1; lvl >= 0; --lvl) {
            const uint32_t lo = g.lstart[lvl], n = g.lstart[lvl + 1] - lo;
            for (uint32_t u = tid; u < n * C; u += nt) {
                const uint32_t row = lo + (u >> cwl), c = u & Cmask;
                if (row >= G) continue;
                uint4 v = hv[(size_t)row * C + c];
                for (uint32_t ch = 1; ch <= a; ++ch)
                    if ((uint64_t)a * row + ch < G) v = comb16<T, OP>(v, hv[(size_t)(a * row + ch) * C + c]);
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
#define FTC_AHEAP_TILE_KB 24
#endif
constexpr uint64_t kAheapTileBytes = FTC_AHEAP_TILE_KB * 1024;   // a tile takes as many whole levels as fit into this
constexpr size_t kAheapMaxHeapBytes = 96 * 1024;                 // the block's heap array (tile roots and the rows above them)

static bool aheap_geometry(Params& p, int smem_optin, AheapGeom& g) {
    if (p.kbytes % 16 || p.arity < 2) return false;
    const uint32_t C = p.kbytes / 16, a = p.arity;
    if (C == 0 || C > 32 || (C & (C - 1))) return false;
    uint32_t cwl = 0; while ((1u << cwl) < C) ++cwl;
    p.C = C; p.cw_log2 = cwl;
    const uint64_t rowbytes = (uint64_t)p.m * p.kbytes;
    // levels of the heap: first row of each level
    uint32_t Hmax = 0; uint64_t start = 0, width = 1;
    g.lstart[0] = 0;
    while (start < p.Gmax) {
        start += width; width *= a; ++Hmax;
        if (Hmax > kAheapMaxLevels) return false;
        g.lstart[Hmax] = (uint32_t)(start < 0xFFFFFFFFull ? start : 0xFFFFFFFFull);
    }
    for (uint32_t l = Hmax + 1; l <= kAheapMaxLevels; ++l) g.lstart[l] = 0xFFFFFFFFu;
    // the deepest tile within the byte budget (at most four levels)
    uint32_t D = 1; uint64_t R = 1, w = a;
    while (D < 4 && D < Hmax && (R + w) * rowbytes <= kAheapTileBytes) { R += w; w *= a; ++D; }
    if (R * rowbytes > 64 * 1024) return false;
    g.D = D; g.R = (uint32_t)R;
    { uint32_t s0 = 0, pw = 1; for (uint32_t u = 0; u < 4; ++u) { g.tstart[u] = u < D ? s0 : 0xFFFFFFFFu; g.apow[u] = u < D ? pw : 0; s0 += pw; pw *= a; } }
    g.Lt = Hmax > D ? Hmax - D : 0;
    g.ntop = g.lstart[g.Lt];
    uint64_t nt = 1; for (uint32_t l = 0; l < g.Lt; ++l) nt *= a;
    if (nt > (1u << 20)) return false;
    g.ntiles = (uint32_t)nt; g.nheap = g.ntop + g.ntiles;
    g.ngroups = (g.ntop + g.R - 1) / g.R;
    const size_t hv_bytes = (size_t)g.nheap * C * 16;
    if (hv_bytes > kAheapMaxHeapBytes) return false;
    g.tile_cap = (uint32_t)((R * rowbytes + 127) & ~(uint64_t)127);
    const uint32_t nitems = g.ntiles + g.ngroups + 1;
    uint32_t warps = 1;
    while (warps < 8 && warps * 2 * 8 <= nitems) warps *= 2;
    size_t o = sizeof(Ctx) + 3 * (size_t)(p.W + 1) * 4;
    o = (o + 15) & ~(size_t)15; g.off_rootv = (uint32_t)o; o += (size_t)C * 16;
    g.off_hv = (uint32_t)o; o += hv_bytes;
    g.off_bar = (uint32_t)o; o += 8 * 8;
    g.off_gaveup = (uint32_t)o; o += 8;
    o = (o + 127) & ~(size_t)127; g.off_tiles = (uint32_t)o;
    while (warps > 1 && o + (size_t)warps * g.tile_cap > (size_t)smem_optin - 1024) warps /= 2;
    o += (size_t)warps * g.tile_cap;
    if (o > (size_t)smem_optin - 1024) return false;
    g.nwarps = warps; g.smem_bytes = (uint32_t)o;
    return true;
}

template <typename T, int OP>
static cudaError_t launch_aheap_t(Params p, int sm_count, int smem_optin, cudaStream_t st) {
    AheapGeom g;
    if (!aheap_geometry(p, smem_optin, g)) return cudaErrorInvalidConfiguration;
    cudaError_t e = cudaFuncSetAttribute(aheap_kernel<T, OP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem_bytes);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, aheap_kernel<T, OP>, (int)g.nwarps * 32, g.smem_bytes);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    const uint64_t cap = (uint64_t)sm_count * per_sm;
    const uint32_t grid = (uint32_t)(p.S < cap ? p.S : cap);
    if (p.grid_query) { *p.grid_query = grid; return cudaSuccess; }
    aheap_kernel<T, OP><<<grid, g.nwarps * 32, g.smem_bytes, st>>>(p, g);
    return cudaGetLastError();
}

cudaError_t launch_aheap_u64(const Params& p, int tsel, int sm_count, int smem_optin, cudaStream_t st);

}  // namespace ftc
