// What every root child delivers (Algorithm "reduce_root": "receive from any child (data, failure information)";
// section "Failure information", second and third scheme), on the tiles of the staged kernel, for the exactly
// associative operations (integer sum, max, xor). The batch kernels evaluate only the child the root selects;
// here all f+1 subtrees are played, nodes that deliver nothing included, in one pass over the inputs.
//
// What makes one pass cheap: a group none of whose members failed, before or during the operation, has the same
// value at every member after up-correction when the operation is exactly associative and commutative (every
// member folds the same f+1 inputs). So a warp tile without a failed process, a renumbered slot or the short last
// group is evaluated once and its value serves all f+1 subtrees; only the few tiles that hold such a row are played
// child by child with the full rules: a node that does not send delivers nothing, its parent sets the failed bit
// and counts it, the list sizes add up.
//
// Per node and child the kernel carries a value and a word: exists | present | failed bit | size of the failed list.
// Above the tiles the same split holds: the heap array of tile roots and upper rows is combined once in shared memory
// for all children ("common" values, as in the staged kernel); only the nodes that have a specially played row
// somewhere below them ("dirty": the ancestors of the few special rows) carry one value and word per child, in a
// per-block slice of the workspace that is touched at those nodes only.
#pragma once
#include "ftc_staged_impl.cuh"

namespace ftc {

constexpr uint32_t kNoRow = 0xFFFFFFFFu, kManyRows = 0xFFFFFFFEu;
constexpr uint32_t kMetaExists = 1u << 31, kMetaPresent = 1u << 30, kMetaFailed = 1u << 29, kMetaCount = (1u << 29) - 1;

// A node takes one child's delivery: a child that sent is combined, its failed bit and list size taken over; a child
// that sent nothing sets the failed bit and is noted (Algorithm "reduce_non_root" with the second scheme's size).
template <typename T, int OP>
__device__ __forceinline__ void take_child(uint4& acc, uint32_t& meta, uint4 cv, uint32_t cm) {
    if (!(cm & kMetaExists)) return;
    if (cm & kMetaPresent) { acc = comb16<T, OP>(acc, cv); meta = (meta | (cm & kMetaFailed)) + (cm & kMetaCount); }
    else meta = (meta | kMetaFailed) + 1u;
}

// Facts of the scenario the child-by-child folds need (shared memory).
struct CandScen {
    const Ctx* cx;
    const uint32_t* alive;   // bit v (renumbered): v had not failed before the operation
    const uint32_t* snd;     // bit v (renumbered): v performs its tree send
    uint32_t root, base, troot;
};

// Node (row, sc) of root subtree sc after up-correction (Algorithm "Up-correction"): own input, the root's if it is a
// partner and its message was sent, then the partners whose message arrived. `in_lc`: the scenario in the caller's
// process order (global memory) at this lane's chunk; `srow_lc`: the row's staged copy in shared memory (its first
// member, this lane's chunk), which serves every member but the one whose input sits in the renumbered slot.
// The caller guarantees that the node exists (sc < members of the row).
template <typename T, int OP>
__device__ __noinline__ uint4 cand_fold(const Params& p, CandScen cs, const char* in_lc, const char* srow_lc, uint32_t row, uint32_t sc, uint32_t& meta) {
    auto member = [&](uint32_t sp, uint32_t vr) -> uint4 {
        return vr == cs.root ? ld_stream(in_lc) : *reinterpret_cast<const uint4*>(srow_lc + (size_t)sp * p.kbytes);
    };
    const uint32_t mj = row < p.q ? p.m : p.r, vbase = row * p.m + 1, v = vbase + sc;
    if (!test_bit(cs.snd, v)) { meta = kMetaExists; return make_uint4(0, 0, 0, 0); }
    uint32_t mask = extract_bits(cs.alive, vbase, mj);
    for (uint32_t i = 0; i < p.max_inop; ++i) {              // a dying partner's message arrives iff it was still sent
        const uint32_t vic = cs.cx->iv[i];
        if (vic == FTC_INOP_UNUSED) continue;
        const uint32_t vr = renumber(vic, cs.root);
        if (vr < vbase || vr >= vbase + mj || vr == v) continue;
        const uint32_t sv = vr - vbase, t = local_round(cs.cx->ir[i], cs.base);
        if (!(partner_slot(p, row, sv, sc) < t)) mask &= ~(1u << sv);
    }
    uint4 acc = member(sc, v);
    // the root's up-correction send to member sc of its group is its send number sc (descending order: r-1-sc); in the
    // fold the root comes first among the partners (descending order: last)
    const bool from_root = row == p.q && (p.pdesc ? p.r - 1 - sc : sc) < cs.troot;
    if (from_root && !p.pdesc) acc = comb16<T, OP>(acc, ld_stream(in_lc + (size_t)cs.root * p.kbytes));
    for (uint32_t i = 0; i < mj; ++i) {
        const uint32_t sp = p.pdesc ? mj - 1 - i : i, vr = vbase + sp;
        if (sp != sc && ((mask >> sp) & 1u)) acc = comb16<T, OP>(acc, member(sp, vr));
    }
    if (from_root && p.pdesc) acc = comb16<T, OP>(acc, ld_stream(in_lc + (size_t)cs.root * p.kbytes));
    meta = kMetaExists | kMetaPresent | (mj - __popc(mask) + ((row == p.q && !from_root) ? 1u : 0u));
    return acc;
}

// A lane's sub-heap of XL levels for child sc: node, then child 1, then child 2. Rows >= G do not exist.
template <typename T, int OP, int XL, int U>
struct SubHeapCand {
    static __device__ __forceinline__ uint4 eval(const Params& p, const CandScen& cs, const char* in_lc, const char* buf_lc, uint32_t rowbytes,
                                                 uint32_t trow, uint32_t grow, uint32_t G, uint32_t sc, uint32_t& meta) {
        if (grow >= G) { meta = 0; return make_uint4(0, 0, 0, 0); }
        uint4 v = cand_fold<T, OP>(p, cs, in_lc, buf_lc + (size_t)trow * rowbytes, grow, sc, meta);
        if (U + 1 < XL && (meta & kMetaPresent)) {           // what the children of a node that does not send deliver is lost
            constexpr int UN = (U + 1 < XL ? U + 1 : U);
            uint32_t cm;
            uint4 cv = SubHeapCand<T, OP, XL, UN>::eval(p, cs, in_lc, buf_lc, rowbytes, 2 * trow + 1, 2 * grow + 1, G, sc, cm);
            take_child<T, OP>(v, meta, cv, cm);
            cv = SubHeapCand<T, OP, XL, UN>::eval(p, cs, in_lc, buf_lc, rowbytes, 2 * trow + 2, 2 * grow + 2, G, sc, cm);
            take_child<T, OP>(v, meta, cv, cm);
        }
        return v;
    }
};

// Tree phase inside a warp tile with the words riding along (see tile_tree_phase for the lane roles).
template <typename T, int OP>
__device__ __forceinline__ uint4 tile_tree_phase_cand(uint4 valA, uint32_t mA, uint4 valB, uint32_t& mB, uint32_t lw, uint32_t cwl, uint32_t C,
                                                      uint32_t lane, uint32_t lc, uint32_t tB, uint32_t idxB, bool hasB) {
    if (lw) {
        const bool mine = hasB && tB == lw - 1;
        const uint32_t src1 = mine ? (((2 * idxB) << cwl) | lc) : lane, src2 = mine ? src1 + C : lane;
        const uint4 c1 = shfl16(valA, src1), c2 = shfl16(valA, src2);
        const uint32_t m1 = __shfl_sync(0xFFFFFFFFu, mA, src1), m2 = __shfl_sync(0xFFFFFFFFu, mA, src2);
        if (mine && (mB & kMetaPresent)) { take_child<T, OP>(valB, mB, c1, m1); take_child<T, OP>(valB, mB, c2, m2); }
    }
    for (int t = (int)lw - 2; t >= 0; --t) {
        const bool mine = hasB && tB == (uint32_t)t;
        const uint32_t src1 = mine ? ((((2u << t) - 1 + 2 * idxB) << cwl) | lc) : lane, src2 = mine ? src1 + C : lane;
        const uint4 c1 = shfl16(valB, src1), c2 = shfl16(valB, src2);
        const uint32_t m1 = __shfl_sync(0xFFFFFFFFu, mB, src1), m2 = __shfl_sync(0xFFFFFFFFu, mB, src2);
        if (mine && (mB & kMetaPresent)) { take_child<T, OP>(valB, mB, c1, m1); take_child<T, OP>(valB, mB, c2, m2); }
    }
    return valB;
}

// What the out-of-line tile routines need.
struct TileJob {
    CandScen cs;
    const char* in_s;        // the scenario in global memory (process order)
    char* tile;              // the warp's staged copy of the tile's rows (tile-heap order); the out-of-line routines overwrite it
    uint4* hv; uint32_t* hm; // per-child values and words of the heap array (workspace slice)
    uint4* hvc;              // common values of the heap array (shared memory)
    uint32_t nheap, j0, srow, Lt, D, Gc, rowbytes;
};

// Several special rows in one tile (rare): the whole tile child by child.
template <typename T, int OP, int XL>
__device__ __forceinline__ void cand_tile_many(const Params& p, const TileJob& jb) {
    const uint32_t lane = threadIdx.x & 31, cwl = p.cw_log2, lw = 5 - cwl, RW = 1u << lw;
    const uint32_t lr = lane >> cwl, lc = lane & (p.C - 1), j0 = jb.j0;
    const uint32_t tA = RW - 1 + lr, rowA = ((j0 + 1) << lw) - 1 + lr;
    const uint32_t tB = ilog2u(lr + 1), idxB = lr + 1 - (1u << tB), rowB = ((j0 + 1) << tB) - 1 + idxB;
    const char* in_lc = jb.in_s + lc * 16;
    const char* buf_lc = jb.tile + lc * 16;
    for (uint32_t sc = 0; sc < p.m; ++sc) {
        const uint32_t G = p.q + (sc < p.r ? 1u : 0u);
        uint32_t mA = 0, mB = 0;
        uint4 valA = SubHeapCand<T, OP, XL, 0>::eval(p, jb.cs, in_lc, buf_lc, jb.rowbytes, tA, rowA, G, sc, mA), valB = make_uint4(0, 0, 0, 0);
        const bool hasB = lr < RW - 1;
        if (hasB && rowB < G) valB = cand_fold<T, OP>(p, jb.cs, in_lc, buf_lc + (size_t)lr * jb.rowbytes, rowB, sc, mB);
        valB = tile_tree_phase_cand<T, OP>(valA, mA, valB, mB, lw, cwl, p.C, lane, lc, tB, idxB, hasB);
        if (lr == 0) {
            jb.hv[((size_t)sc * jb.nheap + j0) * p.C + lc] = lw ? valB : valA;
            if (lc == 0) jb.hm[(size_t)sc * jb.nheap + j0] = lw ? mB : mA;
        }
    }
}

// A ragged tile, or one special row in it. First the common value of every node's subtree, by the plain definition
// (valid wherever no special row lies below): own folds, then level by level. The value of a node takes the place of
// its row's first member in the staged copy (no further shared memory is needed); the special row and its ancestors
// keep their inputs, their values are not common anyway. Then, for one special row, its path to the tile's root, one
// lane per (child, chunk): what hangs off the path is common.
template <typename T, int OP>
__device__ __forceinline__ void cand_tile_one(const Params& p, const TileJob& jb) {
    const uint32_t lane = threadIdx.x & 31, cwl = p.cw_log2, Cmask = p.C - 1, j0 = jb.j0, Gc = jb.Gc, D = jb.D, rowbytes = jb.rowbytes;
    char* tile = jb.tile;
    const uint32_t nnodes = (1u << D) - 1;
    const uint32_t srow = jb.srow;
    // tile-heap index of the special row (none: beyond every node)
    const uint32_t su = srow == kNoRow ? 0u : ilog2u(srow + 1) - jb.Lt;
    const uint32_t st0 = srow == kNoRow ? 0xFFFFFFFFu : (1u << su) - 1 + (srow + 1 - ((j0 + 1) << su));
    auto row_of_node = [&](uint32_t t) { const uint32_t u = ilog2u(t + 1); return ((j0 + 1) << u) - 1 + (t + 1 - (1u << u)); };
    auto on_path = [&](uint32_t t) {                              // t is the special row's node or one of its ancestors
        const uint32_t u = ilog2u(t + 1);
        return srow != kNoRow && u <= su && ((st0 + 1) >> (su - u)) == t + 1;
    };
    auto tsub = [&](uint32_t t, uint32_t c) -> uint4& { return *reinterpret_cast<uint4*>(tile + (size_t)t * rowbytes + c * 16); };
    for (uint32_t u = lane; u < nnodes * p.C; u += 32) {
        const uint32_t t = u >> cwl, c = u & Cmask;
        if (row_of_node(t) < Gc && !on_path(t)) tsub(t, c) = fold_plain_staged<T, OP>(p, 0u, tile + (size_t)t * rowbytes + c * 16);
    }
    __syncwarp();
    for (int lv = (int)D - 2; lv >= 0; --lv) {
        const uint32_t t0 = (1u << lv) - 1;
        for (uint32_t u = lane; u < (t0 + 1) * p.C; u += 32) {
            const uint32_t t = t0 + (u >> cwl), c = u & Cmask, row = row_of_node(t);
            if (row >= Gc || on_path(t)) continue;
            uint4 v = tsub(t, c);
            if (2 * row + 1 < Gc) v = comb16<T, OP>(v, tsub(2 * t + 1, c));
            if (2 * row + 2 < Gc) v = comb16<T, OP>(v, tsub(2 * t + 2, c));
            tsub(t, c) = v;
        }
        __syncwarp();
    }
    if (srow == kNoRow) {                          // ragged only: the same for every child
        if (lane < p.C && j0 < Gc) jb.hvc[(size_t)j0 * p.C + lane] = tsub(0, lane);
        return;
    }
    for (uint32_t base_u = 0; base_u < p.m * p.C; base_u += 32) {
        const uint32_t unit = base_u + lane;
        if (unit >= p.m * p.C) continue;
        const uint32_t sc = unit >> cwl, c = unit & Cmask;
        const uint32_t G = p.q + (sc < p.r ? 1u : 0u);
        const char* in_c = jb.in_s + c * 16;
        uint32_t t = st0, row = srow, meta = 0;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (row < G) {
            v = cand_fold<T, OP>(p, jb.cs, in_c, tile + (size_t)t * rowbytes + c * 16, row, sc, meta);
            if ((meta & kMetaPresent) && su + 1 < D) {          // its own children are common
                if (2 * row + 1 < Gc) take_child<T, OP>(v, meta, tsub(2 * t + 1, c), kMetaExists | kMetaPresent);
                if (2 * row + 2 < Gc) take_child<T, OP>(v, meta, tsub(2 * t + 2, c), kMetaExists | kMetaPresent);
            }
        }
        while (t > 0) {
            const uint32_t tp = (t - 1) >> 1, rp = (row - 1) >> 1;
            uint32_t pm;
            uint4 pv = cand_fold<T, OP>(p, jb.cs, in_c, tile + (size_t)tp * rowbytes + c * 16, rp, sc, pm);
            if (pm & kMetaPresent) {
                const bool first = (t & 1u) != 0;                  // the path's node is child 1 of its parent
                const uint32_t ts = first ? t + 1 : t - 1, rs = first ? row + 1 : row - 1;
                const uint4 sv = tsub(ts, c);
                const uint32_t sm = rs < Gc ? (kMetaExists | kMetaPresent) : 0u;
                if (first) { take_child<T, OP>(pv, pm, v, meta); take_child<T, OP>(pv, pm, sv, sm); }
                else { take_child<T, OP>(pv, pm, sv, sm); take_child<T, OP>(pv, pm, v, meta); }
            }
            v = pv; meta = pm; t = tp; row = rp;
        }
        jb.hv[((size_t)sc * jb.nheap + j0) * p.C + c] = v;
        if (c == 0) jb.hm[(size_t)sc * jb.nheap + j0] = meta;
    }
}

struct CandGeom {
    StagedGeom st;
    uint64_t slice_bytes;       // workspace per block: f+1 heap arrays of values, then the words
    uint32_t nheap, ntop;       // rows of a heap array (tile roots and above): 2^(Lt+1) - 1; rows above the tiles: 2^Lt - 1
};

template <typename T, int OP, int XL>
__global__ void __launch_bounds__(kStagedMaxThreads, 2) cand_kernel(Params p, CandGeom cg, T* cand, uint32_t* info) {
    const StagedGeom& g = cg.st;
    extern __shared__ __align__(128) uint32_t smem[];
    char* sbase = reinterpret_cast<char*>(smem);
    Ctx* cx = reinterpret_cast<Ctx*>(smem);
    uint32_t* pf = smem + sizeof(Ctx) / 4;
    uint32_t* alive = pf + p.W + 1;
    uint32_t* snd = alive + p.W + 1;
    uint32_t* tspec = reinterpret_cast<uint32_t*>(sbase + g.off_special);
    uint32_t* dirty = reinterpret_cast<uint32_t*>(sbase + g.off_dirty);          // bit n: node n of the heap array is played per child
    uint32_t* rspec = dirty + ((cg.nheap + 31) / 32 + 1);                        // bit j: row j above the tiles is a special row
    uint32_t* trowv = rspec + ((cg.ntop + 31) / 32 + 1);                        // per tile: its one special row, kNoRow or kManyRows
    uint4* hvc = reinterpret_cast<uint4*>(sbase + g.off_hv);                     // common values, heap order
    volatile uint32_t* gaveup = reinterpret_cast<volatile uint32_t*>(sbase + g.off_gaveup);
    // ORD: the combine order is observable (float32): every member of a group folds in its own order, nothing is common
    // to the children; every node carries a value and a word per child, all in shared memory.
    constexpr bool ORD = Ordered<T>::value;
    // per block: values hv[sc][row][chunk], combined words hm[sc][row], own words of the rows above the tiles hmo[sc][row]
    // (a slice of the workspace, touched at the dirty nodes only; ORD: shared memory, every node)
    char* slice = ORD ? sbase + g.off_hv : static_cast<char*>(p.ws) + (size_t)blockIdx.x * cg.slice_bytes;
    uint4* hv = reinterpret_cast<uint4*>(slice);
    uint32_t* hm = ORD ? reinterpret_cast<uint32_t*>(sbase + g.off_words) : reinterpret_cast<uint32_t*>(slice + (size_t)p.m * cg.nheap * p.C * 16);
    uint32_t* hmo = hm + (size_t)p.m * cg.nheap;

    const uint32_t tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, wid = tid >> 5, nw = nt >> 5;
    const uint32_t cwl = p.cw_log2, lw = 5 - cwl, RW = 1u << lw, Cmask = p.C - 1;
    const uint32_t lr = lane >> cwl, lc = lane & Cmask;
    const uint32_t D = lw + XL;
    const uint32_t Lt = p.Lt, ntiles = 1u << Lt, ntop = ntiles - 1;
    const uint32_t GR = min((1u << XL) - 1, max(1u, (ntop + RW - 1) >> lw)), grows = RW * GR;
    const uint32_t ngroups = (ntop + grows - 1) / grows;
    const uint32_t nitems = ntiles + ngroups;
    const uint32_t rowbytes = p.m * p.kbytes;
    const uint64_t scen_bytes = (uint64_t)p.P * p.kbytes;
    const uint32_t tries = (p.flags & FTC_DEBUG_ONE_POLL) ? 1u : kWaitTries;
    const uint32_t Gc = p.q;                                       // rows every root subtree has; row q exists below children s < r only

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
    const uint32_t lvl_rows = lane < D ? 1u << lane : 0u, lvl_dst = (lvl_rows ? lvl_rows - 1 : 0u) * rowbytes;
    auto issue_next = [&]() {
        if (n_my == 0 || is_s >= p.S || stop) return;
        const uint32_t it = wid + is_i * nw;
        uint32_t first_row = 0, nrows = 0, dst_off = 0;
        if (it < ntiles) {
            const uint32_t j0 = ntop + it;
            if (j0 < p.Gmax) { first_row = ((j0 + 1) << lane) - 1; nrows = lvl_rows; dst_off = lvl_dst; }
        } else if (lane == 0) { first_row = (it - ntiles) * grows; nrows = min(grows, ntop - first_row); }
        const uint64_t b0 = (uint64_t)first_row * rowbytes + p.kbytes;
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
        decode_scenario(p, s, cx, pf, alive);                      // `alive` is scratch for its arrival mask here
        T* cand_s = cand + s * (uint64_t)p.m * p.k;
        uint32_t* info_s = info + s * (uint64_t)p.m * 2;
        const uint32_t code = cx->code;
        if (code == FTC_ST_BAD_ROOT || code == FTC_ST_PRECONDITION_INOP_ROOT || dead) {    // no attempt is played
            for (uint32_t u = tid; u < p.m * p.C; u += nt) reinterpret_cast<uint4*>(cand_s)[u] = make_uint4(0, 0, 0, 0);
            for (uint32_t u = tid; u < p.m; u += nt) { info_s[2 * u] = dead ? 3u : 2u; info_s[2 * u + 1] = 0; }
            for (uint32_t i = 0; i < n_my; ++i) { acquire(); release(); }
            __syncthreads();
            continue;
        }
        uint32_t root = cx->root, base = cx->base;
        if (code == FTC_ST_NO_LIVE_ROOT_CANDIDATE) {                // the last attempt, toward a dead root
            const uint32_t first = p.root >= 0 ? (uint32_t)p.root : p.roots[s];
            root = (first + p.f) % p.P; base = p.f * p.Ratt;
        }
        const uint32_t troot = local_round(fail_round(p, cx, pf, root), base);
        __syncthreads();                                           // decode's arrival mask is no longer read
        // who had not failed beforehand and who sends up the tree, over renumbered ranks
        for (uint32_t w = tid; w <= p.W; w += nt) {
            uint32_t word = w < p.W ? ~pf[w] : 0u;
            if (w == p.W - 1 && (p.P & 31)) word &= (1u << (p.P & 31)) - 1u;
            alive[w] = word; snd[w] = word;
        }
        __syncthreads();
        if (tid == 0 && root != 0) {                               // bit `root` is process 0, bit 0 the root
            const uint32_t b0 = alive[0] & 1u, bit = 1u << (root & 31);
            alive[0] |= 1u;
            if (b0) { alive[root >> 5] |= bit; snd[root >> 5] |= bit; } else { alive[root >> 5] &= ~bit; snd[root >> 5] &= ~bit; }
        }
        __syncthreads();
        if (tid < p.max_inop && cx->iv[tid] != FTC_INOP_UNUSED) {
            const uint32_t v = renumber(cx->iv[tid], root);
            if (v) {
                const uint32_t d = 1 + ilog2u((v - 1) / p.m + 1), t = local_round(cx->ir[tid], base);
                if (!(p.f + p.H - d < t)) atomicAnd(&snd[v >> 5], ~(1u << (v & 31)));      // tree send of depth d is round f+H-d
            }
        }
        // ---- work items that are played child by child: those with a failed process, a renumbered slot, the short last
        // group, or not complete above their last level. One bit per item (tile i, then groups of rows above the tiles);
        // and the nodes of the heap array whose value differs from child to child: the ancestors of every special row.
        for (uint32_t w = tid; w < (nitems + 31) / 32 + 1; w += nt) tspec[w] = 0;
        for (uint32_t w = tid; w < (cg.nheap + 31) / 32 + 1 + (cg.ntop + 31) / 32 + 1; w += nt) dirty[w] = 0;      // dirty and rspec
        for (uint32_t w = tid; w < ntiles; w += nt) trowv[w] = kNoRow;
        __syncthreads();
        {
            auto mark_dirty_from = [&](uint32_t n) {
                for (;;) { atomicOr(&dirty[n >> 5], 1u << (n & 31)); if (n == 0) break; n = (n - 1) >> 1; }
            };
            auto mark_row = [&](uint32_t j) {
                const uint32_t lvl = ilog2u(j + 1);
                const uint32_t it = lvl >= Lt ? ((j + 1) >> (lvl - Lt)) - ntiles : ntiles + j / grows;
                atomicOr(&tspec[it >> 5], 1u << (it & 31));
                if (lvl < Lt) atomicOr(&rspec[j >> 5], 1u << (j & 31));
                else {                                              // the tile remembers its special row while it is the only one
                    const uint32_t old = atomicCAS(&trowv[it], kNoRow, j);
                    if (old != kNoRow && old != j) trowv[it] = kManyRows;
                }
                mark_dirty_from(lvl >= Lt ? ((j + 1) >> (lvl - Lt)) - 1 : j);
            };
            for (uint32_t w = tid; w < p.W; w += nt) {
                uint32_t word = pf[w];
                while (word) {
                    const uint32_t b = __ffs(word) - 1; word &= word - 1;
                    const uint32_t v = renumber((w << 5) + b, root);
                    if (v) mark_row((v - 1) / p.m);
                }
            }
            if (tid < p.max_inop && cx->iv[tid] != FTC_INOP_UNUSED) {
                const uint32_t v = renumber(cx->iv[tid], root);
                if (v) mark_row((v - 1) / p.m);
            }
            if (tid == 0) {
                if (root != 0) mark_row((root - 1) / p.m);          // the slot that holds process 0's input
                if (p.r) mark_row(p.q);                             // the short last group
            }
            // tiles that exist but are not complete down to their second-to-last level: the check-free folds do not fit them
            for (uint32_t it = tid; it < ntiles; it += nt)
                if (ntop + it < Gc && ((ntop + it + 2) << (D >= 2 ? D - 2 : 0)) - 2 >= Gc) atomicOr(&tspec[it >> 5], 1u << (it & 31));
            for (uint32_t gi = tid; gi < ngroups; gi += nt)
                if ((gi + 1) * grows > ntop || (gi + 1) * grows > Gc) atomicOr(&tspec[(ntiles + gi) >> 5], 1u << ((ntiles + gi) & 31));
        }
        __syncthreads();
        const CandScen cs{cx, alive, snd, root, base, troot};
        const char* in_lc = in_s + lc * 16;

        for (uint32_t i = 0; i < n_my; ++i) {
            const uint32_t it = wid + i * nw;
            acquire();
            const char* buf_lc = tile + lc * 16;
            const bool special = test_bit(tspec, it);              // warp-uniform
            if (it < ntiles) {
                const uint32_t j0 = ntop + it;
                const uint32_t tA = RW - 1 + lr, rowA = ((j0 + 1) << lw) - 1 + lr;
                const uint32_t tB = ilog2u(lr + 1), idxB = lr + 1 - (1u << tB);
                const uint32_t rowB = ((j0 + 1) << tB) - 1 + idxB;
                if (ORD) {
                    if (!special) {
                        // every group whole: child sc's member folds its own input first, then the partners in the schedule's order
                        for (uint32_t sc = 0; sc < p.m; ++sc) {
                            uint4 valA = make_uint4(0, 0, 0, 0), valB = make_uint4(0, 0, 0, 0);
                            if (j0 < Gc) {
                                if (XL > 1 || rowA < Gc) valA = SubHeapPlain<T, OP, XL, 0, false, false>::eval(p, sc, alive, buf_lc, rowbytes, tA, rowA, Gc);
                                const bool hasB = lr < RW - 1;
                                if (hasB) valB = fold_plain_staged<T, OP>(p, sc, buf_lc + staged_row_offset<false>(p, rowbytes, lr, rowB));
                                valB = tile_tree_phase<T, OP, (XL > 1), true>(valA, valB, lw, cwl, p.C, lane, lc, tB, idxB, rowB, hasB, Gc);
                            }
                            if (lr == 0) {
                                hv[((size_t)sc * cg.nheap + j0) * p.C + lc] = lw ? valB : valA;
                                if (lc == 0) hm[(size_t)sc * cg.nheap + j0] = j0 < Gc ? (kMetaExists | kMetaPresent) : 0u;
                            }
                        }
                    } else {
                        const TileJob job{cs, in_s, tile, hv, hm, nullptr, cg.nheap, j0, kManyRows, Lt, D, Gc, rowbytes};
                        cand_tile_many<T, OP, XL>(p, job);
                    }
                    release();
                } else if (!special) {
                    // every group of the tile is whole: one value per row serves all children (exact operations)
                    if (j0 < Gc) {
                        uint4 valA = make_uint4(0, 0, 0, 0), valB = make_uint4(0, 0, 0, 0);
                        const bool hasB = lr < RW - 1;
                        // the group size as a constant where it is that of f = 4 or f = 8: one uniform branch per tile
                        auto folds = [&](auto mtag) {
                            constexpr int M = decltype(mtag)::value;
                            if (XL > 1 || rowA < Gc) valA = SubHeapPlain<T, OP, XL, 0, false, false, M>::eval(p, 0u, alive, buf_lc, rowbytes, tA, rowA, Gc);
                            if (hasB) valB = fold_plain_m<T, OP, M>(p, 0u, buf_lc + staged_row_offset<false>(p, rowbytes, lr, rowB));
                        };
                        if (p.m == 5) folds(std::integral_constant<int, 5>());
                        else if (p.m == 9) folds(std::integral_constant<int, 9>());
                        else folds(std::integral_constant<int, 0>());
                        valB = tile_tree_phase<T, OP, (XL > 1), true>(valA, valB, lw, cwl, p.C, lane, lc, tB, idxB, rowB, hasB, Gc);
                        if (lr == 0) hvc[(size_t)j0 * p.C + lc] = lw ? valB : valA;
                    }
                    release();
                } else {
                    // the few tiles with a special row or a ragged end: out of line, so that the common path stays compact
                    const TileJob job{cs, in_s, tile, hv, hm, hvc, cg.nheap, j0, trowv[it], Lt, D, Gc, rowbytes};
                    if (job.srow == kManyRows) cand_tile_many<T, OP, XL>(p, job);
                    else cand_tile_one<T, OP>(p, job);
                    release();
                }
            } else if (ORD) {
                // ---- rows above the tiles, every child's member in its own order ----
                for (uint32_t gs = 0; gs < GR; ++gs) {
                    const uint32_t rloc = gs * RW + lr, row = (it - ntiles) * grows + rloc;
                    if (row >= ntop) continue;
                    const bool plain = !special || (row < Gc && !test_bit(rspec, row));
                    for (uint32_t sc = 0; sc < p.m; ++sc) {
                        const uint32_t G = p.q + (sc < p.r ? 1u : 0u);
                        uint32_t mo = 0;
                        uint4 v = make_uint4(0, 0, 0, 0);
                        if (plain) { v = fold_plain_staged<T, OP>(p, sc, buf_lc + (size_t)rloc * rowbytes); mo = kMetaExists | kMetaPresent; }
                        else if (row < G) v = cand_fold<T, OP>(p, cs, in_lc, buf_lc + (size_t)rloc * rowbytes, row, sc, mo);
                        hv[((size_t)sc * cg.nheap + row) * p.C + lc] = v;
                        if (lc == 0) hmo[(size_t)sc * cg.ntop + row] = mo;
                    }
                }
                release();
            } else {
                // ---- rows above the tiles: fold now, combine later ----
                if (!special) {
                    for (uint32_t gs = 0; gs < GR; ++gs) {
                        const uint32_t rloc = gs * RW + lr;
                        hvc[(size_t)((it - ntiles) * grows + rloc) * p.C + lc] = fold_plain_staged<T, OP>(p, 0u, buf_lc + (size_t)rloc * rowbytes);
                    }
                } else {
                    for (uint32_t gs = 0; gs < GR; ++gs) {
                        const uint32_t rloc = gs * RW + lr, row = (it - ntiles) * grows + rloc;
                        if (row >= ntop) continue;
                        if (!test_bit(rspec, row)) {               // an ordinary row of a group that holds a special one, or a ragged end
                            if (row < Gc) hvc[(size_t)row * p.C + lc] = fold_plain_staged<T, OP>(p, 0u, buf_lc + (size_t)rloc * rowbytes);
                            continue;
                        }
                        for (uint32_t sc = 0; sc < p.m; ++sc) {
                            const uint32_t G = p.q + (sc < p.r ? 1u : 0u);
                            uint32_t mo = 0;
                            uint4 v = make_uint4(0, 0, 0, 0);
                            if (row < G) v = cand_fold<T, OP>(p, cs, in_lc, buf_lc + (size_t)rloc * rowbytes, row, sc, mo);
                            hv[((size_t)sc * cg.nheap + row) * p.C + lc] = v;
                            if (lc == 0) hmo[(size_t)sc * cg.ntop + row] = mo;
                        }
                    }
                }
                release();
            }
        }
        __syncthreads();
        // ---- levels above the tiles, leaves first (Algorithm "reduce_non_root") ----
        for (int lvl = ORD ? (int)Lt - 1 : -1; lvl >= 0; --lvl) {              // ORD: every node, per child
            const uint32_t lo = (1u << lvl) - 1u, n = lo + 1u;
            for (uint32_t u = tid; u < n * p.m * p.C; u += nt) {
                const uint32_t c = u & Cmask, x = u >> cwl, sc = x % p.m, row = lo + x / p.m;
                const size_t me = (size_t)sc * cg.nheap + row;
                uint32_t meta = hmo[(size_t)sc * cg.ntop + row];
                uint4 v = hv[me * p.C + c];
                if (meta & kMetaPresent) {
                    const size_t c1 = (size_t)sc * cg.nheap + 2 * row + 1;
                    take_child<T, OP>(v, meta, hv[c1 * p.C + c], hm[c1]);
                    take_child<T, OP>(v, meta, hv[(c1 + 1) * p.C + c], hm[c1 + 1]);
                    hv[me * p.C + c] = v;
                }
                if (c == 0) hm[me] = meta;
            }
            __syncthreads();
        }
        for (int lvl = ORD ? -1 : (int)Lt - 1; lvl >= 0; --lvl) {
            const uint32_t lo = (1u << lvl) - 1u, n = lo + 1u;
            // nodes played per child: own value (a special row's per-child fold, else the row's common fold), then each
            // child's delivery (per child if that node is played per child, else its common value)
            for (uint32_t u = tid; u < n * p.m * p.C; u += nt) {
                const uint32_t c = u & Cmask, x = u >> cwl, row = lo + x / p.m;
                if (!test_bit(dirty, row)) continue;
                const uint32_t sc = x % p.m;
                const size_t me = (size_t)sc * cg.nheap + row;
                uint32_t meta = kMetaExists | kMetaPresent;
                uint4 v;
                if (test_bit(rspec, row)) { meta = hmo[(size_t)sc * cg.ntop + row]; v = hv[me * p.C + c]; }
                else v = hvc[(size_t)row * p.C + c];
                if (meta & kMetaPresent) {
#pragma unroll
                    for (uint32_t k2 = 1; k2 <= 2; ++k2) {
                        const uint32_t ch = 2 * row + k2;
                        if (test_bit(dirty, ch)) take_child<T, OP>(v, meta, hv[((size_t)sc * cg.nheap + ch) * p.C + c], hm[(size_t)sc * cg.nheap + ch]);
                        else if (ch < Gc) take_child<T, OP>(v, meta, hvc[(size_t)ch * p.C + c], kMetaExists | kMetaPresent);
                    }
                }
                hv[me * p.C + c] = v;
                if (c == 0) hm[me] = meta;
            }
            __syncthreads();
            // common values
            for (uint32_t u = tid; u < n * p.C; u += nt) {
                const uint32_t row = lo + (u >> cwl), c = u & Cmask;
                if (row >= Gc) continue;
                uint4 v = hvc[(size_t)row * p.C + c];
                if (2 * row + 1 < Gc) v = comb16<T, OP>(v, hvc[(size_t)(2 * row + 1) * p.C + c]);
                if (2 * row + 2 < Gc) v = comb16<T, OP>(v, hvc[(size_t)(2 * row + 2) * p.C + c]);
                hvc[(size_t)row * p.C + c] = v;
            }
            __syncthreads();
        }
        // ---- what the root receives from each child ----
        const bool bad = *gaveup != 0;
        const bool per_child = ORD || test_bit(dirty, 0u);         // else: nothing failed anywhere, every child delivers the common value
        for (uint32_t u = tid; u < p.m * p.C; u += nt) {
            const uint32_t sc = u >> cwl, c = u & Cmask;
            const uint32_t meta = per_child ? hm[(size_t)sc * cg.nheap] : (kMetaExists | kMetaPresent);
            const bool got = (meta & kMetaPresent) && !bad;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (got) v = per_child ? hv[((size_t)sc * cg.nheap) * p.C + c] : hvc[c];
            reinterpret_cast<uint4*>(cand_s)[u] = v;
            if (c == 0) {
                info_s[2 * sc] = bad ? 3u : (meta & kMetaPresent) ? ((meta & kMetaFailed) ? 1u : 0u) : 2u;
                info_s[2 * sc + 1] = got ? (meta & kMetaCount) : 0u;
            }
        }
        __syncthreads();
    }
    if (pending) mbar_wait_bounded(bar0, phase, kWaitTries);      // only after a wait gave up: a copy may still be in flight
}

// ---- host side ----
static bool cand_geometry(Params& p, int smem_optin, int sm_count, uint32_t& XL, CandGeom& cg, bool ordered) {
    if (p.arity != 2) return false;
    XL = staged_xl(p);
    p.ws_bytes = 0; p.swz_mask = 0; p.row_shift = 0;               // its own slices; plain tiles
    if (!staged_geometry(p, smem_optin, sm_count, XL, cg.st, /*all_children=*/ordered ? 2 : 1)) return false;
    if (cg.st.whole || cg.st.nbuf != 1) return false;
    cg.nheap = (2u << p.Lt) - 1; cg.ntop = (1u << p.Lt) - 1;
    cg.slice_bytes = ordered ? 0 : (((uint64_t)p.m * cg.nheap * p.C * 16 + (uint64_t)p.m * (cg.nheap + cg.ntop) * 4) + 255) & ~(uint64_t)255;
    return true;
}

template <typename T, int OP, int XL>
static cudaError_t launch_cand_x(const Params& p, const CandGeom& cg, T* cand, uint32_t* info, int sm_count, cudaStream_t st, uint32_t* grid_out) {
    cudaError_t e = cudaFuncSetAttribute(cand_kernel<T, OP, XL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cg.st.smem_bytes);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, cand_kernel<T, OP, XL>, (int)cg.st.nwarps * 32, cg.st.smem_bytes);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    if (cg.slice_bytes && per_sm > 4) per_sm = 4;                 // workspace slices of all blocks stay in L2
    const uint64_t cap = (uint64_t)sm_count * per_sm;
    const uint32_t grid = (uint32_t)(p.S < cap ? p.S : cap);
    if (grid_out) { *grid_out = (uint32_t)cap; return cudaSuccess; }      // one workspace slice per block
    cand_kernel<T, OP, XL><<<grid, cg.st.nwarps * 32, cg.st.smem_bytes, st>>>(p, cg, cand, info);
    return cudaGetLastError();
}

template <typename T, int OP>
static cudaError_t launch_cand_t(Params p, void* cand, uint32_t* info, int sm_count, int smem_optin, cudaStream_t st, uint32_t* grid_out) {
    CandGeom cg; uint32_t XL;
    if (!cand_geometry(p, smem_optin, sm_count, XL, cg, Ordered<T>::value)) return cudaErrorInvalidConfiguration;
    switch (XL) {
    case 2: return launch_cand_x<T, OP, 2>(p, cg, static_cast<T*>(cand), info, sm_count, st, grid_out);
    case 3: return launch_cand_x<T, OP, 3>(p, cg, static_cast<T*>(cand), info, sm_count, st, grid_out);
    default: return launch_cand_x<T, OP, 1>(p, cg, static_cast<T*>(cand), info, sm_count, st, grid_out);
    }
}

}  // namespace ftc
