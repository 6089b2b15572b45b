// Staged kernel: the main fast path. One block plays one scenario at a time; the selected subtree's heap of
// up-correction groups ("rows") is cut into warp tiles, and the levels above the tiles are combined in a heap array
// (shared memory, or the caller's workspace when it is large). The input bytes of a tile travel global -> shared
// memory asynchronously, one copy per heap level of the tile (each level of a sub-heap is one contiguous run of
// rows), tracked by an mbarrier per buffer: untiled bulk copies, or tiled tensor copies with a swizzle where the
// plain layout would put the rows of different lanes into the same banks. Each warp runs its own copy pipeline over
// the flat sequence of its work items, across scenario boundaries, so the bytes in flight do not depend on
// registers and no lane spends instructions on global addresses.
//
// A tile has lw + XL levels (lw = log2 of the lane rows, 32 / chunks per vector): each lane row evaluates a
// sub-heap of XL levels by itself (values in registers), the lw levels above are combined with warp shuffles.
// Groups that are not "plain" (a missing member, a renumbered slot, the short last group) take slower folds; they
// are a handful per scenario.
//
// Variants, chosen on the host (template parameter MINB is a tag, see the constants before the kernel):
//   - large blocks (4-8 warps, 128 registers): rows folded one by one with fully inlined code -- C4, C5;
//   - lean blocks (1-2 warps, ~96 registers) and large blocks with groups of at most 128 bytes: all rows of a lane
//     folded together member by member, rare folds as function calls -- C3;
//   - the same two fed by swizzled tensor copies: float32 vectors of 16 and 32 bytes;
//   - scenarios staged whole by one copy (up to 12-16 KB): 64 registers.
#pragma once
#include <cuda.h>
#include <type_traits>
#include "ftc_tile_common.cuh"
#include "ftc_decode_warp.cuh"
#include "ftc_kernels.h"

namespace ftc {

// ---- mbarrier / bulk-copy primitives (shared::cta addresses as 32-bit) ----
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after `tries` polls and says so. A caller whose wait gave up never arms or waits on that
// barrier again except for one last bounded wait before the block ends (the copy may still be in flight), marks the
// block (sticky flag in shared memory) and lets every scenario the block still plays end as FTC_ST_INTERNAL_TIMEOUT.
// tries = 1 (FTC_DEBUG_ONE_POLL) polls once without suspending, so that the give-up path can be exercised.
constexpr uint32_t kWaitTries = 1u << 22;
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t tries) {
    if (tries == 1) return mbar_test_wait(bar, parity);
    for (uint32_t i = 0; i < tries; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// words of one per-item bitmap
__host__ __device__ inline uint32_t nitems_words(uint32_t Lt, uint32_t lw) {
    const uint32_t ntiles = 1u << Lt, nitems = ntiles + ((ntiles - 1 + (1u << lw) - 1) >> lw);
    return (nitems + 31) / 32 + 1;
}

struct StagedGeom {
    uint32_t nwarps, nbuf, tile_cap;       // warps per block, buffers per warp, bytes per buffer (multiple of 128)
    uint32_t whole;                        // 1: the whole scenario is staged in one block-wide buffer
    uint32_t off_special, off_rootv, off_hv, off_bar, off_gaveup, off_tiles, smem_bytes;
    uint32_t off_dirty;                    // all-children kernel: bitmaps over the rows of the heap array, then one word per tile
    uint32_t off_words;                    // all-children kernel, observable order: a word per node and child
    uint32_t hv_global;                    // 1: the heap array of tile roots and upper rows lives in the workspace
    uint64_t hv_bytes;                     // its size per block
};

// Where a row's bytes sit: at tile-heap position trow of the warp's buffer, or (WHOLE) at their place in the
// block-wide copy of the scenario (grow = global row).
// SW (swizzled tiles): with 64-byte groups every tile row but the first sits one row further, so that each level
// starts on a 128-byte boundary (tensor copies need that); p.row_shift is 0 otherwise.
template <bool WHOLE, bool SW = false>
__device__ __forceinline__ uint32_t staged_row_offset(const Params& p, uint32_t rowbytes, uint32_t trow, uint32_t grow) {
    if (WHOLE) return (grow * p.m + 1) * p.kbytes;
    return SW ? (trow + (trow ? p.row_shift : 0u)) * rowbytes : trow * rowbytes;
}

// 16 bytes of a staged row. SW: the tile came in by tiled tensor copies with the 128-byte swizzle, which exchanges
// the 16-byte chunks within each line by the line number (128-byte lines: bits 7-9 of the shared-memory address
// XORed into bits 4-6; 64-byte lines: bits 7-8 into bits 4-5); rows of different lane rows, 128 bytes or a multiple apart, then sit in different banks.
template <bool SW>
struct LdStaged {
    uint32_t mask;        // 0x70 for 128-byte lines, 0x30 for 64-byte lines
    __device__ __forceinline__ explicit LdStaged(uint32_t m) : mask(m) {}
    __device__ __forceinline__ uint4 operator()(const char* q) const {
        if (SW) {
            uint32_t a = smem_addr(q);
            a ^= (a >> 3) & mask;
            return *reinterpret_cast<const uint4*>(__cvta_shared_to_generic(a));
        }
        return *reinterpret_cast<const uint4*>(q);
    }
};

// Fold of a plain group from its staged copy.
template <typename T, int OP, bool SW = false>
__device__ __forceinline__ uint4 fold_plain_staged(const Params& p, uint32_t sstar, const char* srow_lc) {
    return fold16_full<T, OP, 0>(srow_lc, p.kbytes, p.m, sstar, LdStaged<SW>(p.swz_mask), p.pdesc != 0);
}

// Fold of one group on the careful path: a full group without a renumbered slot comes from its staged copy
// (`srow_lc`, NULL when the row is not in the buffer) under its arrival mask; the others by the general routine from the scenario in process order (`in_lc`: global
// memory, or the block-wide shared copy when WHOLE).
template <typename T, int OP, bool WHOLE>
__device__ __forceinline__ uint4 fold_staged(const Params& p, uint32_t root, uint32_t sstar, const uint32_t* inc,
                                             const char* in_lc, const char* srow_lc, uint32_t row) {
    const uint32_t vbase = row * p.m + 1;
    if (srow_lc && row < p.q && root - vbase >= p.m)      // full group, no renumbered slot in it: its staged copy serves
        return fold16_masked<T, OP>(srow_lc, p.kbytes, p.m, extract_bits(inc, vbase, p.m), sstar, LdShared(), p.pdesc != 0);
    if (WHOLE) return fold16_careful<T, OP, LdShared>(p, root, sstar, inc, in_lc, row);
    return fold16_careful<T, OP, LdGlobal>(p, root, sstar, inc, in_lc, row);
}

// A lane's sub-heap in a tile whose rows are all plain and that is complete down to its second-to-last level:
// only the children at the tile's last level (U + 1 == XL - 1) may be missing.
// MASKED: groups may miss members (fold under the arrival mask in `inc`), otherwise the same.
template <typename T, int OP, bool MASKED>
__device__ __forceinline__ uint4 fold_fast_staged(const Params& p, uint32_t sstar, const uint32_t* inc, const char* srow_lc, uint32_t grow) {
    if (MASKED) return fold16_masked<T, OP>(srow_lc, p.kbytes, p.m, extract_bits(inc, grow * p.m + 1, p.m), sstar, LdShared(), p.pdesc != 0);
    return fold_plain_staged<T, OP>(p, sstar, srow_lc);
}

// Fold of a plain group from its staged copy with the group size as a constant (M = f + 1: straight-line code, all loads
// issued together); M = 0: the size is read from p.
template <typename T, int OP, int M>
__device__ __forceinline__ uint4 fold_plain_m(const Params& p, uint32_t sstar, const char* srow_lc) {
    return fold16_full<T, OP, M>(srow_lc, p.kbytes, M ? (uint32_t)M : p.m, sstar, LdShared(), p.pdesc != 0);
}

// M: the group size as a constant for the plain folds (the large-block kernel picks it once per tile), 0: from p
template <typename T, int OP, int XL, int U, bool WHOLE, bool MASKED, int M = 0>
struct SubHeapPlain {
    static __device__ __forceinline__ uint4 eval(const Params& p, uint32_t sstar, const uint32_t* inc, const char* buf_lc, uint32_t rowbytes,
                                                 uint32_t trow, uint32_t grow, uint32_t G) {
        const char* srow = buf_lc + staged_row_offset<WHOLE>(p, rowbytes, trow, grow);
        uint4 v = (M && !MASKED) ? fold_plain_m<T, OP, M>(p, sstar, srow) : fold_fast_staged<T, OP, MASKED>(p, sstar, inc, srow, grow);
        if (U + 1 < XL) {
            constexpr int UN = (U + 1 < XL ? U + 1 : U);
            if (U + 2 < XL || 2 * grow + 1 < G)
                v = comb16<T, OP>(v, SubHeapPlain<T, OP, XL, UN, WHOLE, MASKED, M>::eval(p, sstar, inc, buf_lc, rowbytes, 2 * trow + 1, 2 * grow + 1, G));
            if (U + 2 < XL || 2 * grow + 2 < G)
                v = comb16<T, OP>(v, SubHeapPlain<T, OP, XL, UN, WHOLE, MASKED, M>::eval(p, sstar, inc, buf_lc, rowbytes, 2 * trow + 2, 2 * grow + 2, G));
        }
        return v;
    }
};

// ---- the lean variant (blocks of one or two warps) ----
// Small scenarios run as one- or two-warp blocks, many per SM, and each warp alternates between waiting for its
// copy and computing: what counts there is the length of the dependent instruction chain per tile and the
// registers per warp. So the lean variant folds all rows of a lane together (independent chains), and the folds
// that few rows need are real function calls, which keeps the code every row runs through small.

// Fold of one group by every rule: a full group without a renumbered slot comes from its staged copy (`srow_lc`,
// NULL when the row is not in the buffer) under its arrival mask; the others by the general routine from the
// scenario in process order (`in_lc`: global memory, or the block-wide shared copy when WHOLE).
template <typename T, int OP, bool WHOLE, bool SW = false>
__device__ __noinline__ uint4 fold_staged_call(FoldShape fs, uint32_t root, uint32_t sstar, const uint32_t* inc,
                                               const char* in_lc, const char* srow_lc, uint32_t row) {
    const uint32_t vbase = row * fs.m + 1;
    if (srow_lc && row < fs.q && root - vbase >= fs.m)      // full group, no renumbered slot in it: its staged copy serves
        return fold16_masked<T, OP>(srow_lc, fs.kbytes, fs.m, extract_bits(inc, vbase, fs.m), sstar, LdStaged<SW>(fs.swz_mask), fs.pdesc != 0);
    if (WHOLE) return fold16_general<T, OP, 0, LdShared, FoldShape>(fs, root, sstar, inc, in_lc, row);
    return fold16_general<T, OP, 0, LdGlobal, FoldShape>(fs, root, sstar, inc, in_lc, row);
}

// A full group some of whose members' messages are missing, from its staged copy.
template <typename T, int OP, bool SW = false>
__device__ __noinline__ uint4 fold_masked_call(const char* srow_lc, uint32_t kbytes, uint32_t m, uint32_t mask, uint32_t sstar, uint32_t swz_mask, bool desc) {
    return fold16_masked<T, OP>(srow_lc, kbytes, m, mask, sstar, LdStaged<SW>(swz_mask), desc);
}

// One row from its staged copy; `masked`: the work item holds a group with a missing member, so look at the mask.
template <typename T, int OP, bool SW = false>
__device__ __forceinline__ uint4 fold_row_lean(const Params& p, uint32_t sstar, const uint32_t* inc, const char* srow_lc,
                                               uint32_t grow, bool masked) {
    if (masked) {
        const uint32_t mask = extract_bits(inc, grow * p.m + 1, p.m), full = p.m >= 32 ? 0xFFFFFFFFu : (1u << p.m) - 1u;
        if (mask != full) return fold_masked_call<T, OP, SW>(srow_lc, p.kbytes, p.m, mask, sstar, p.swz_mask, p.pdesc != 0);
    }
    return fold_plain_staged<T, OP, SW>(p, sstar, srow_lc);
}

__host__ __device__ constexpr int clog2(int v) { return v <= 1 ? 0 : 1 + clog2(v >> 1); }

// Tree phase inside a lane's sub-heap from the folded rows, breadth-first index B (slot 1 + B of `acc`): the
// node's own fold, then child 1, then child 2. Children on the tile's last level may be missing; children on the
// heap's sparse last level, which is left out of the tiles, are leaves folded by the general routine.
template <typename T, int OP, int XL, int B, bool WHOLE>
struct SubComb {
    static __device__ __forceinline__ uint4 eval(const Params& p, uint32_t root, uint32_t sstar, const uint32_t* inc, const char* in_lc,
                                                 const uint4* acc, const uint32_t* grow, uint32_t G) {
        constexpr int U = clog2(B + 1);
        uint4 v = acc[1 + B];
        if (U + 1 < XL) {
            constexpr int C1 = (U + 1 < XL) ? 2 * B + 1 : B, C2 = (U + 1 < XL) ? 2 * B + 2 : B;
            if (U + 2 < XL || grow[1 + C1] < G) v = comb16<T, OP>(v, SubComb<T, OP, XL, C1, WHOLE>::eval(p, root, sstar, inc, in_lc, acc, grow, G));
            if (U + 2 < XL || grow[1 + C2] < G) v = comb16<T, OP>(v, SubComb<T, OP, XL, C2, WHOLE>::eval(p, root, sstar, inc, in_lc, acc, grow, G));
        } else if (p.below) {
            const uint32_t c1 = 2 * grow[1 + B] + 1;
            if (c1 < G) v = comb16<T, OP>(v, fold_staged_call<T, OP, WHOLE>(fold_shape(p), root, sstar, inc, in_lc, nullptr, c1));
            if (c1 + 1 < G) v = comb16<T, OP>(v, fold_staged_call<T, OP, WHOLE>(fold_shape(p), root, sstar, inc, in_lc, nullptr, c1 + 1));
        }
        return v;
    }
};

// Fast path of one tile for one lane: the rows it owns -- slot 0 its node of the tile's upper levels (tile heap
// index lr, global row rowB, present iff hasB), slots 1.. the XL-level sub-heap rooted at tile heap index tA
// (global row rowA), breadth first -- are folded together, one group member at a time across all rows (own input
// of the selected subtree's member first, then the partners ascending: Algorithm "Up-correction"), so that the
// loads and adds of different rows overlap; then the sub-heap is combined. The tile has no renumbered slot, no
// short group and is complete down to its second-to-last level. `masked`: some group of the tile misses a member.
// SHORT: the tile may hold the short last group (row `short_row`; its members end before a full group's would, the
// bytes behind them are readable): whatever the common fold made of that row is replaced by the general fold.
template <typename T, int OP, int XL, bool WHOLE, bool SW = false, bool SHORT = false>
__device__ __forceinline__ void fold_tile_fast(const Params& p, uint32_t root, uint32_t sstar, const uint32_t* inc, const char* in_lc,
                                               const char* buf_lc, uint32_t rowbytes, uint32_t j0, uint32_t lr, uint32_t rot, uint32_t rowB, bool hasB,
                                               uint32_t tA, uint32_t rowA, uint32_t G, bool masked, uint4& valA, uint4& valB,
                                               uint32_t short_row = 0xFFFFFFFFu) {
    constexpr int NS = 1 << XL;
    const LdStaged<SW> lds(p.swz_mask);
    uint32_t off[NS], grow[NS];
    const uint32_t off0 = staged_row_offset<WHOLE, SW>(p, rowbytes, 0, j0);        // the tile's root: always there
    grow[0] = hasB ? rowB : j0;
    off[0] = hasB ? staged_row_offset<WHOLE, SW>(p, rowbytes, lr, rowB) : off0;
#pragma unroll
    for (int b = 0; b < NS - 1; ++b) {
        const int u = clog2(b + 1), pos = b + 1 - (1 << u);
        const uint32_t t = ((tA + 1) << u) - 1 + pos, g = ((rowA + 1) << u) - 1 + pos;
        grow[1 + b] = g;
        off[1 + b] = g < G ? staged_row_offset<WHOLE, SW>(p, rowbytes, t, g) : off0;   // a missing row reads the root's bytes, unused
    }
    uint4 acc[NS];
    if (!Ordered<T>::value && !masked) {
        // Any member order gives the same bits: each lane row starts at member `rot`, chosen so that the lane rows
        // that load together (a quarter warp) read from different shared-memory banks.
        uint32_t mem = rot;
        const char* src = buf_lc + mem * p.kbytes;
#pragma unroll
        for (int s = 0; s < NS; ++s) acc[s] = lds(src + off[s]);
#pragma unroll 1
        for (uint32_t i = 1; i < p.m; ++i) {
            if (++mem == p.m) mem = 0;
            src = buf_lc + mem * p.kbytes;
#pragma unroll
            for (int s = 0; s < NS; ++s) acc[s] = comb16<T, OP>(acc[s], lds(src + off[s]));
        }
    } else {
        const char* own = buf_lc + sstar * p.kbytes;
#pragma unroll
        for (int s = 0; s < NS; ++s) acc[s] = lds(own + off[s]);
        // the partners in the schedule's order (ascending rank, or descending), own skipped: one pointer walks the group
        const bool desc = Ordered<T>::value && p.pdesc != 0;
        const int32_t step = desc ? -(int32_t)p.kbytes : (int32_t)p.kbytes;
        const char* mem = desc ? buf_lc + (p.m - 1) * p.kbytes : buf_lc;
        if (!masked) {
#pragma unroll 1
            for (uint32_t i = 1; i < p.m; ++i) {
                if (mem == own) mem += step;
#pragma unroll
                for (int s = 0; s < NS; ++s) acc[s] = comb16<T, OP>(acc[s], lds(mem + off[s]));
                mem += step;
            }
        } else {
            uint32_t mask[NS];
#pragma unroll
            for (int s = 0; s < NS; ++s) mask[s] = grow[s] < G ? extract_bits(inc, grow[s] * p.m + 1, p.m) : 0u;
            uint32_t sp = desc ? p.m - 1 : 0u;
#pragma unroll 1
            for (uint32_t i = 1; i < p.m; ++i) {
                if (mem == own) { mem += step; sp += desc ? 0xFFFFFFFFu : 1u; }
#pragma unroll
                for (int s = 0; s < NS; ++s)
                    if ((mask[s] >> sp) & 1u) acc[s] = comb16<T, OP>(acc[s], lds(mem + off[s]));
                mem += step; sp += desc ? 0xFFFFFFFFu : 1u;
            }
        }
    }
    if (SHORT) {
#pragma unroll
        for (int s = 0; s < NS; ++s)
            if (grow[s] == short_row) acc[s] = fold_staged_call<T, OP, WHOLE, SW>(fold_shape(p), root, sstar, inc, in_lc, nullptr, short_row);
    }
    valB = acc[0];
    valA = SubComb<T, OP, XL, 0, WHOLE>::eval(p, root, sstar, inc, in_lc, acc, grow, G);
}

// Value of the node at level u (of XL) of a lane's sub-heap: its group's fold, then child 1, then child 2.
// trow/grow: tile-heap index and global row of the node. Its bytes sit at tile-heap position trow of the warp's
// buffer, or (WHOLE) at their place in the block-wide copy of the scenario.
// CALL: the fold is a function call (lean variant) instead of inline code.
template <typename T, int OP, int XL, int U, bool WHOLE, bool CALL = false, bool SW = false>
struct SubHeap {
    static __device__ __forceinline__ uint4 eval(const Params& p, uint32_t root, uint32_t sstar, const uint32_t* inc,
                                                 const char* in_lc, const char* buf_lc, uint32_t rowbytes,
                                                 uint32_t trow, uint32_t grow, uint32_t G) {
        // the deepest level of this recursion lies below the tile: its rows are not in the warp's buffer
        const char* srow = (WHOLE || U + 1 < XL) ? buf_lc + staged_row_offset<WHOLE, SW>(p, rowbytes, trow, grow) : nullptr;
        uint4 v = CALL ? fold_staged_call<T, OP, WHOLE, SW>(fold_shape(p), root, sstar, inc, in_lc, srow, grow)
                       : fold_staged<T, OP, WHOLE>(p, root, sstar, inc, in_lc, srow, grow);
        if (U + 1 < XL) {
            if (2 * grow + 1 < G)
                v = comb16<T, OP>(v, SubHeap<T, OP, XL, (U + 1 < XL ? U + 1 : U), WHOLE, CALL, SW>::eval(p, root, sstar, inc, in_lc, buf_lc, rowbytes, 2 * trow + 1, 2 * grow + 1, G));
            if (2 * grow + 2 < G)
                v = comb16<T, OP>(v, SubHeap<T, OP, XL, (U + 1 < XL ? U + 1 : U), WHOLE, CALL, SW>::eval(p, root, sstar, inc, in_lc, buf_lc, rowbytes, 2 * trow + 2, 2 * grow + 2, G));
        }
        return v;
    }
};

constexpr int kStagedMaxThreads = 256;
constexpr int kStagedLeanThreads = 64;      // lean variant: at most two warps, about 96 registers a thread
constexpr int kStagedLeanMinBlocks = 10;
constexpr int kStagedBatchedTag = 3;         // large blocks running the lean variant's code (small groups, exact operations)
constexpr int kStagedLeanSwzTag = 21;        // lean variant fed by swizzled tensor copies (float32, small vectors)
constexpr int kStagedBatchedSwzTag = 5;      // the same in large blocks

// Tensor maps of the swizzled variant: one per tile level (its box is that level's rows); unused otherwise.
struct alignas(64) TmaMaps { CUtensorMap lvl[8]; };

// GM: the group size f + 1 as a constant for the plain folds of the large-block kernel (5, 9: the configurations with many
// processes), 0: read from p
template <typename T, int OP, int XL, bool WHOLE, int MINB, int GM = 0>
__global__ void __launch_bounds__((MINB == kStagedLeanMinBlocks || MINB == kStagedLeanSwzTag) ? kStagedLeanThreads : kStagedMaxThreads,
                                  (MINB == kStagedBatchedTag || MINB == kStagedBatchedSwzTag) ? 2 : (MINB == kStagedLeanSwzTag ? kStagedLeanMinBlocks : MINB))
staged_kernel(Params p, StagedGeom g, const __grid_constant__ TmaMaps maps) {
    constexpr bool SWZ = MINB == kStagedLeanSwzTag || MINB == kStagedBatchedSwzTag;
    constexpr bool LEAN = MINB == kStagedLeanMinBlocks || MINB == kStagedBatchedTag || SWZ;
    extern __shared__ __align__(128) uint32_t smem[];
    char* sbase = reinterpret_cast<char*>(smem);
    Ctx* cx = reinterpret_cast<Ctx*>(smem);
    uint32_t* pf = smem + sizeof(Ctx) / 4;
    uint32_t* inc = pf + p.W + 1;
    uint32_t* unr = inc + p.W + 1;
    uint32_t* tspec = reinterpret_cast<uint32_t*>(sbase + g.off_special);            // items that need every check
    uint32_t* tmask = tspec + (nitems_words(p.Lt, 5 - p.cw_log2));                     // items with missing group members only
    uint4* rootv = reinterpret_cast<uint4*>(sbase + g.off_rootv);
    // node values of the tile roots and of the rows above them, heap order: in shared memory, or, when that would
    // crowd out resident blocks, in this block's slice of the workspace (it stays in L2: written and read once)
    uint4* hv = g.hv_global ? reinterpret_cast<uint4*>(static_cast<char*>(p.ws) + (size_t)blockIdx.x * g.hv_bytes)
                            : reinterpret_cast<uint4*>(sbase + g.off_hv);

    const uint32_t tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, wid = tid >> 5, nw = nt >> 5;
    const uint32_t cwl = p.cw_log2, lw = 5 - cwl, RW = 1u << lw, Cmask = p.C - 1;
    const uint32_t lr = lane >> cwl, lc = lane & Cmask;
    const uint32_t D = lw + XL;                                   // levels of a tile
    // Starting member of this lane row's folds for the exactly associative operations. A quarter warp holds
    // nq = 8/C lane rows whose rows start m*C chunks apart; with g = gcd(m, nq), rows nq/g apart share their banks,
    // and g different starting members (all < m) separate them.
    const uint32_t nq = p.C < 8 ? 8u / p.C : 1u, gq = min(nq, p.m & (0u - p.m));
    const uint32_t rot = (lr >> ilog2u(nq / gq)) & (gq - 1);
    // rows above the tiles come as work items of `grows` rows: as many per lane row as a tile's sub-heap has (one when
    // the tiles are swizzled: the tensor map of that box is the one of a tile level)
    const uint32_t Lt = p.Lt, ntiles = 1u << Lt, ntop = ntiles - 1;
    const uint32_t GR = SWZ ? 1u : min((1u << XL) - 1, max(1u, (ntop + RW - 1) >> lw)), grows = RW * GR;
    const uint32_t ngroups = (ntop + grows - 1) / grows;
    const uint32_t nitems = ntiles + ngroups + 1;
    const uint32_t rowbytes = p.m * p.kbytes;
    const uint64_t scen_bytes = (uint64_t)p.P * p.kbytes;

    const uint32_t bar0 = smem_addr(sbase + g.off_bar) + wid * g.nbuf * 8;
    char* tiles = sbase + g.off_tiles + (size_t)wid * g.nbuf * g.tile_cap;
    const uint32_t cbar = smem_addr(sbase + g.off_bar) + g.nwarps * g.nbuf * 8;   // block-wide barrier (WHOLE)
    char* wbuf = sbase + g.off_tiles;                                            // block-wide scenario copy (WHOLE)
    // set, and never cleared, once a bounded wait of this block gave up (decode_scenario does not touch it)
    volatile uint32_t* gaveup = reinterpret_cast<volatile uint32_t*>(sbase + g.off_gaveup);
    const uint32_t tries = (p.flags & FTC_DEBUG_ONE_POLL) ? 1u : kWaitTries;
    if (lane < g.nbuf) mbar_init(bar0 + lane * 8, 1);
    if (WHOLE && tid == 0) mbar_init(cbar, 1);
    if (tid == 0) *gaveup = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    uint32_t phase_bits = 0;                                      // bit b: parity to wait for on buffer b
    uint32_t cphase = 0;
    bool cfail = false;                                           // WHOLE: this thread's wait for the block-wide copy gave up
    bool stop = false;                                            // this warp issues no further copies (a wait of the block gave up)

    // ---- the copy pipeline of this warp: it runs over the flat sequence (scenario, work item) of everything the
    // warp will process, g.nbuf items ahead of the item being computed, across scenario boundaries. What is copied
    // depends on the geometry only (rows that exist for the largest subtree), never on a scenario's decode.
    const uint32_t n_my = wid < nitems ? (nitems - wid + nw - 1) / nw : 0;     // work items of this warp per scenario
    uint64_t is_s = blockIdx.x;                                   // scenario and local item of the next copy to issue
    const char* is_src = reinterpret_cast<const char*>(p.in) + is_s * scen_bytes;
    uint32_t is_i = 0, ibuf = 0, cbuf = 0;                        // buffer of the next copy to issue / item to consume
    uint32_t pending = 0;                                         // bit b: buffer b has a copy in flight
    // lane t copies level t of a tile: 2^t rows, placed after the 2^t - 1 rows of the levels above
    const uint32_t lvl_rows = lane < D ? 1u << lane : 0u, lvl_dst = (lvl_rows ? lvl_rows - 1 : 0u) * rowbytes;
    auto issue_next = [&]() {
        if (WHOLE || n_my == 0 || is_s >= p.S || stop) return;
        const uint32_t it = wid + is_i * nw, b = ibuf;
        uint32_t first_row = 0, nrows = 0, dst_off = 0;
        if (it < ntiles) {
            const uint32_t j0 = ntop + it;
            if (j0 < p.Gmax) { first_row = ((j0 + 1) << lane) - 1; nrows = lvl_rows; dst_off = lvl_dst; }
        } else if (it < ntiles + ngroups) {
            if (lane == 0) { first_row = (it - ntiles) * grows; nrows = SWZ ? RW : min(grows, ntop - first_row); }
        }
        if (SWZ) {
            // Tiled tensor copies over the view [scenario][128-byte line][32 words] of the full groups: lane t brings
            // level t with the map whose box is 2^t rows (rows above the tiles: the map of 2^lw rows). A box always
            // delivers its full byte count; lines past the last full group arrive as zeros and are never read.
            const uint32_t bytes = (nrows && first_row < p.q) ? nrows * rowbytes : 0u;
            const uint32_t total = __reduce_add_sync(0xFFFFFFFFu, bytes);
            if (total) {
                if (lane == 0) mbar_expect_tx(bar0 + b * 8, total);
                __syncwarp();
                if (bytes) {
                    const CUtensorMap* map = &maps.lvl[it < ntiles ? lane : lw];
                    // 64-byte groups: level t >= 1 of a tile starts at row slot 2^t (a 128-byte boundary), one further than usual
                    if (p.row_shift && it < ntiles && lane) dst_off = rowbytes << lane;
                    const uint32_t lines_per_row = p.swz_mask == 0x70u ? rowbytes >> 7 : 1u;
                    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                                 ::"r"(smem_addr(tiles + (size_t)b * g.tile_cap + dst_off)), "l"(map), "r"(0),
                                   "r"((int)(first_row * lines_per_row)), "r"((int)is_s), "r"(bar0 + b * 8) : "memory");
                }
                pending |= 1u << b;
            }
            if (++ibuf == g.nbuf) ibuf = 0;
            if (++is_i == n_my) { is_i = 0; is_s += gridDim.x; is_src += (uint64_t)gridDim.x * scen_bytes; }
            return;
        }
        // rows first_row .. first_row+nrows-1 are bytes [first_row*rowbytes + kbytes, ...) of the scenario, cut at its end
        const uint64_t b0 = (uint64_t)first_row * rowbytes + p.kbytes;
        uint32_t bytes = 0;
        if (nrows && b0 < scen_bytes) bytes = (uint32_t)min((uint64_t)nrows * rowbytes, scen_bytes - b0);
        const uint32_t total = __reduce_add_sync(0xFFFFFFFFu, bytes);
        if (total) {
            if (lane == 0) mbar_expect_tx(bar0 + b * 8, total);
            __syncwarp();
            if (bytes) bulk_g2s(smem_addr(tiles + (size_t)b * g.tile_cap + dst_off), is_src + b0, bytes, bar0 + b * 8);
            pending |= 1u << b;
        }
        if (++ibuf == g.nbuf) ibuf = 0;
        if (++is_i == n_my) { is_i = 0; is_s += gridDim.x; is_src += (uint64_t)gridDim.x * scen_bytes; }
    };
    // the buffer of the item about to be computed: wait for its copy if one was issued. A warp whose wait gave up
    // keeps the buffer marked as in flight (its barrier's phase never completed: it is not armed or waited on again
    // before the last wait at the end of the kernel), stops issuing and waiting, and marks the block.
    auto acquire = [&]() {
        const uint32_t b = WHOLE ? 0u : cbuf;
        if (!WHOLE && ((pending >> b) & 1u) && !stop) {
            bool ok = mbar_wait_bounded(bar0 + b * 8, (phase_bits >> b) & 1u, tries);
            if (!__all_sync(0xFFFFFFFFu, ok)) {
                // a lane that saw the phase complete proves the copy landed: the others look once more (returns at once)
                if (__any_sync(0xFFFFFFFFu, ok) && !ok) ok = mbar_wait_bounded(bar0 + b * 8, (phase_bits >> b) & 1u, kWaitTries);
                ok = __all_sync(0xFFFFFFFFu, ok);
            }
            if (ok) { phase_bits ^= 1u << b; pending &= ~(1u << b); }
            else { stop = true; if (lane == 0) atomicOr(const_cast<uint32_t*>(gaveup), 1u); }
        }
        return b;
    };
    // every lane is done with the buffer: hand it to the next copy
    auto release = [&]() { __syncwarp(); if (!WHOLE && ++cbuf == g.nbuf) cbuf = 0; issue_next(); };
    if (!WHOLE) for (uint32_t i = 0; i < g.nbuf; ++i) issue_next();

    // Blocks of one warp whose masks are one word per lane decode in registers (ftc_decode_warp.cuh) and fetch the next
    // scenario's mask word, in-operation entry and root while the current scenario is played.
    const bool warp_decode = LEAN && !WHOLE && nw == 1 && p.W <= 32 && ntiles + ngroups <= 32;
    uint32_t nx_pf = 0, nx_vic = FTC_INOP_UNUSED, nx_rnd = 0, nx_root = 0;
    auto fetch_small = [&](uint64_t s) {
        nx_pf = 0; nx_vic = FTC_INOP_UNUSED; nx_rnd = 0; nx_root = 0;
        if (s >= p.S) return;
        if (lane < p.W) nx_pf = __ldg(p.prefail + s * p.W + lane);
        if (lane < p.max_inop) { const ftc_inop_t* e = p.inop + s * p.max_inop + lane; nx_vic = __ldg(&e->victim); nx_rnd = __ldg(&e->round); }
        if (p.root < 0) nx_root = __ldg(p.roots + s);
    };
    if (LEAN && warp_decode) fetch_small(blockIdx.x);

    for (uint64_t s = blockIdx.x; s < p.S; s += gridDim.x) {
        const char* in_s = reinterpret_cast<const char*>(p.in) + s * scen_bytes;
        // uniform: the flag is only written between the barriers of a scenario, and a barrier ended the previous one
        const bool dead = *gaveup != 0;
        if (dead) stop = true;
        if (WHOLE && wid == 0 && !dead) {
            // the whole scenario, in pieces of at most 32 KB, lands while the masks are decoded
            if (lane == 0) mbar_expect_tx(cbar, (uint32_t)scen_bytes);
            __syncwarp();
            for (uint64_t o = (uint64_t)lane * 32768; o < scen_bytes; o += 32u * 32768)
                bulk_g2s(smem_addr(wbuf + o), in_s + o, (uint32_t)min((uint64_t)32768, scen_bytes - o), cbar);
        }
        bool marked = false;
        if (LEAN && warp_decode) {
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
                if (w.code == FTC_ST_OK) {
                    uint32_t spec, mask;
                    mark_special_warp(p, pfw, w.iv, w.root, w.G, Lt, D, p.below != 0, grows, ngroups, spec, mask);
                    if (lane == 0) { tspec[0] = spec; tspec[1] = 0; tmask[0] = mask; tmask[1] = 0; }
                }
                marked = true;
                __syncwarp();
            } else decode_scenario(p, s, cx, pf, inc);
        } else decode_scenario(p, s, cx, pf, inc);
        char* out_s = reinterpret_cast<char*>(p.out) + s * p.kbytes;
        if (WHOLE && !dead) {
            // every thread sees the copy complete before it reads it or leaves the iteration
            if (mbar_wait_bounded(cbar, cphase, tries)) cphase ^= 1u;
            else { cfail = true; atomicOr(const_cast<uint32_t*>(gaveup), 1u); }
        }
        if (cx->code != FTC_ST_OK || dead) {
            if (tid < p.C) reinterpret_cast<uint4*>(out_s)[tid] = make_uint4(0, 0, 0, 0);
            for (uint32_t i = 0; i < n_my; ++i) { acquire(); release(); }        // its copies were issued: consume them unused
            __syncthreads();                                                     // a wait that gave up just now is seen by thread 0
            if (tid == 0) {
                if (*gaveup) cx->code = FTC_ST_INTERNAL_TIMEOUT;
                write_status_rec(p, s, cx);
            }
            __syncthreads();
            continue;
        }
        if (!marked) {                 // warp-uniform, and the block is one warp when it is set
            if (p.is_allreduce) count_holders(p, cx, pf, unr);
            mark_special_items(p, cx, pf, tspec, tmask, Lt, lw, D, LEAN && p.below != 0, grows, ngroups);
        }
        const uint32_t root = cx->root, sstar = cx->sstar, G = cx->G;
        const char* in_lc = (WHOLE ? wbuf : in_s) + lc * 16;      // the scenario in process order, for the general fold

        for (uint32_t i = 0; i < n_my; ++i) {
            const uint32_t it = wid + i * nw, b = acquire();
            const char* buf_lc = (WHOLE ? wbuf : tiles + (size_t)b * g.tile_cap) + lc * 16;
            const bool careful = it < ntiles + ngroups && test_bit(tspec, it);      // warp-uniform
            const bool masked = it < ntiles + ngroups && test_bit(tmask, it);
            if (it < ntiles) {
                const uint32_t j0 = ntop + it;
                const uint32_t tA = RW - 1 + lr, rowA = ((j0 + 1) << lw) - 1 + lr;     // root of this lane row's sub-heap
                const uint32_t tB = ilog2u(lr + 1), idxB = lr + 1 - (1u << tB);
                const uint32_t rowB = ((j0 + 1) << tB) - 1 + idxB;                     // this lane row's node above
                if (LEAN) {
                    if (!careful) {
                        uint4 valA, valB;
                        const bool hasB = lr < RW - 1;
                        fold_tile_fast<T, OP, XL, WHOLE, SWZ>(p, root, sstar, inc, in_lc, buf_lc, rowbytes, j0, lr, rot, rowB, hasB, tA, rowA, G, masked, valA, valB);
                        valB = tile_tree_phase<T, OP, (XL > 1), true>(valA, valB, lw, cwl, p.C, lane, lc, tB, idxB, rowB, hasB, G);
                        if (lr == 0) hv[(size_t)j0 * p.C + lc] = lw ? valB : valA;
                    } else if (j0 < G) {
                        uint4 valA = make_uint4(0, 0, 0, 0), valB = make_uint4(0, 0, 0, 0);
                        if (rowA < G) valA = SubHeap<T, OP, XL + 1, 0, WHOLE, true, SWZ>::eval(p, root, sstar, inc, in_lc, buf_lc, rowbytes, tA, rowA, G);
                        const bool hasB = lr < RW - 1 && rowB < G;
                        if (hasB) valB = fold_staged_call<T, OP, WHOLE, SWZ>(fold_shape(p), root, sstar, inc, in_lc, buf_lc + staged_row_offset<WHOLE, SWZ>(p, rowbytes, lr, rowB), rowB);
                        valB = tile_tree_phase<T, OP>(valA, valB, lw, cwl, p.C, lane, lc, tB, idxB, rowB, hasB, G);
                        if (lr == 0) hv[(size_t)j0 * p.C + lc] = lw ? valB : valA;
                    }
                } else if (!careful && !masked) {
                    // XL == 1: the bottom rows are the tile's last level and may be missing; XL > 1: they exist
                    uint4 valA = make_uint4(0, 0, 0, 0), valB = make_uint4(0, 0, 0, 0);
                    const bool hasB = lr < RW - 1;
                    // the tile's folds, with the group size as a constant in the instantiations that have one
                    auto folds = [&](auto mtag) {
                        constexpr int M = decltype(mtag)::value;
                        if (XL > 1 || rowA < G) valA = SubHeapPlain<T, OP, XL, 0, WHOLE, false, M>::eval(p, sstar, inc, buf_lc, rowbytes, tA, rowA, G);
                        if (hasB) valB = fold_plain_m<T, OP, M>(p, sstar, buf_lc + staged_row_offset<WHOLE>(p, rowbytes, lr, rowB));
                    };
                    folds(std::integral_constant<int, GM>());
                    valB = tile_tree_phase<T, OP, (XL > 1), true>(valA, valB, lw, cwl, p.C, lane, lc, tB, idxB, rowB, hasB, G);
                    if (lr == 0) hv[(size_t)j0 * p.C + lc] = lw ? valB : valA;
                } else if (!careful) {
                    // the same with some group members missing
                    uint4 valA = make_uint4(0, 0, 0, 0), valB = make_uint4(0, 0, 0, 0);
                    if (XL > 1 || rowA < G) valA = SubHeapPlain<T, OP, XL, 0, WHOLE, true>::eval(p, sstar, inc, buf_lc, rowbytes, tA, rowA, G);
                    const bool hasB = lr < RW - 1;
                    if (hasB) valB = fold_fast_staged<T, OP, true>(p, sstar, inc, buf_lc + staged_row_offset<WHOLE>(p, rowbytes, lr, rowB), rowB);
                    valB = tile_tree_phase<T, OP, (XL > 1), true>(valA, valB, lw, cwl, p.C, lane, lc, tB, idxB, rowB, hasB, G);
                    if (lr == 0) hv[(size_t)j0 * p.C + lc] = lw ? valB : valA;
                } else if (j0 < G) {
                    uint4 valA = make_uint4(0, 0, 0, 0), valB = make_uint4(0, 0, 0, 0);
                    if (rowA < G) valA = SubHeap<T, OP, XL + 1, 0, WHOLE>::eval(p, root, sstar, inc, in_lc, buf_lc, rowbytes, tA, rowA, G);   // one level deeper: rows below the tile
                    const bool hasB = lr < RW - 1 && rowB < G;
                    if (hasB) valB = fold_staged<T, OP, WHOLE>(p, root, sstar, inc, in_lc, buf_lc + staged_row_offset<WHOLE>(p, rowbytes, lr, rowB), rowB);
                    valB = tile_tree_phase<T, OP>(valA, valB, lw, cwl, p.C, lane, lc, tB, idxB, rowB, hasB, G);
                    if (lr == 0) hv[(size_t)j0 * p.C + lc] = lw ? valB : valA;
                }
            } else if (it < ntiles + ngroups) {
                for (uint32_t gs = 0; gs < GR; ++gs) {
                    const uint32_t rloc = gs * RW + lr, row = (it - ntiles) * grows + rloc;     // row rloc of the item's buffer
                    const char* srow = buf_lc + staged_row_offset<WHOLE>(p, rowbytes, rloc, row);
                    if (LEAN) {
                        if (!careful) hv[(size_t)row * p.C + lc] = fold_row_lean<T, OP, SWZ>(p, sstar, inc, srow, row, masked);
                        else if (row < ntop && row < G) hv[(size_t)row * p.C + lc] = fold_staged_call<T, OP, WHOLE, SWZ>(fold_shape(p), root, sstar, inc, in_lc, srow, row);
                    } else if (!careful && !masked) hv[(size_t)row * p.C + lc] = fold_plain_staged<T, OP>(p, sstar, srow);
                    else if (!careful) hv[(size_t)row * p.C + lc] = fold_fast_staged<T, OP, true>(p, sstar, inc, srow, row);
                    else if (row < ntop && row < G) hv[(size_t)row * p.C + lc] = fold_staged<T, OP, WHOLE>(p, root, sstar, inc, in_lc, srow, row);
                }
            } else if (sstar >= p.r) {
                if (lr == 0) rootv[lc] = WHOLE ? fold_root16<T, OP, LdShared>(p, root, inc, in_lc) : fold_root16<T, OP, LdGlobal>(p, root, inc, in_lc);
            }
            release();
        }
        __syncthreads();
        // ---- levels above the tiles, leaves first (Algorithm "reduce_non_root") ----
        for (int lvl = (int)Lt - 1; lvl >= 0; --lvl) {
            const uint32_t lo = (1u << lvl) - 1u, n = min(lo + 1u, G > lo ? G - lo : 0u);
            for (uint32_t u = tid; u < n * p.C; u += nt) {
                const uint32_t row = lo + (u >> cwl), c = u & Cmask;
                uint4 v = hv[(size_t)row * p.C + c];
                if (2 * row + 1 < G) v = comb16<T, OP>(v, hv[(size_t)(2 * row + 1) * p.C + c]);
                if (2 * row + 2 < G) v = comb16<T, OP>(v, hv[(size_t)(2 * row + 2) * p.C + c]);
                hv[(size_t)row * p.C + c] = v;
            }
            __syncthreads();
        }
        // ---- the root (Algorithm "reduce_root") ----
        // a wait that gave up during this scenario was flagged before the barrier that followed the work items:
        // every thread reads the same value here; the result is then not valid and zero bytes are written instead
        const bool bad = *gaveup != 0;
        if (tid < p.C) {
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
    // Only after a wait gave up: a copy may still be in flight toward this block's shared memory. One more bounded
    // wait per such buffer before the block ends and the SM hands the memory to another block.
    if (!WHOLE) {
        for (uint32_t b = 0; b < g.nbuf; ++b)
            if ((pending >> b) & 1u) mbar_wait_bounded(bar0 + b * 8, (phase_bits >> b) & 1u, kWaitTries);
    } else if (cfail) mbar_wait_bounded(cbar, cphase, kWaitTries);
}

// ---- host side ----
// The heap array moves to the workspace when it is at least this large and the workspace has a slice for every block
// (at most kHvGlobalBlocksPerSm blocks per SM are launched then).
// Scenarios up to this size are staged whole with one copy.
constexpr uint64_t kWholeMaxBytes = 12 * 1024;
constexpr size_t kHvGlobalMinBytes = 24 * 1024;
constexpr size_t kHvGlobalMaxBytes = 512 * 1024;   // beyond this the slices of all blocks no longer stay in L2
constexpr int kHvGlobalBlocksPerSm = 4;

// all_children: geometry for the kernel that plays every root child (ftc_cand_impl.cuh): every heap level is tiled and
// the heap arrays live in the workspace, never in shared memory.
// all_children == 2: its variant for an observable combine order (float32): one heap array per root child, all in
// shared memory, with their words.
static bool staged_geometry(Params& p, int smem_optin, int sm_count, uint32_t XL, StagedGeom& g, int all_children = 0) {
    if (p.kbytes % 16) return false;
    const uint32_t C = p.kbytes / 16;
    if (C == 0 || C > 32 || (C & (C - 1))) return false;
    uint32_t cwl = 0; while ((1u << cwl) < C) ++cwl;
    const uint32_t lw = 5 - cwl, D = lw + XL;
    uint32_t Hmax = 1; while ((1u << Hmax) <= p.Gmax) ++Hmax;      // levels of the largest subtree heap
    // a last level filled to less than an eighth stays out of the tiles (its few rows go the careful way), so that
    // the tiles, and with them the copy buffers, are full
    const uint32_t last_rows = p.Gmax - ((1u << (Hmax - 1)) - 1);
    const uint32_t Heff = (!all_children && Hmax >= 2 && last_rows * 8 < (1u << (Hmax - 1))) ? Hmax - 1 : Hmax;
    p.C = C; p.cw_log2 = cwl; p.Lt = Heff > D ? Heff - D : 0;
    p.below = (Heff < Hmax && Heff >= D) ? 1u : 0u;
    if (p.Lt > 16) return false;
    const uint64_t rowbytes = (uint64_t)p.m * p.kbytes;
    const uint64_t cap = ((((uint64_t)1 << D) - 1 + p.row_shift) * rowbytes + 127) & ~(uint64_t)127;
    if (cap > 64 * 1024) return false;

    const uint32_t RW = 1u << lw, ntiles = 1u << p.Lt;
    const uint32_t gr_max = (1u << XL) - 1, gr_need = (ntiles - 1 + RW - 1) >> lw;
    const uint32_t grows = RW * (p.swz_mask ? 1u : (gr_need < 1 ? 1u : (gr_need < gr_max ? gr_need : gr_max)));
    const uint32_t nitems = ntiles + (ntiles - 1 + grows - 1) / grows + 1;
    // Launch shape, from sweeps on B200: what limits the kernel is the number of resident warps doing the combine
    // work, and shared memory per warp decides that number. So: one buffer per warp, and blocks just large enough
    // to give every warp at least 16 work items per scenario (at most 8 warps).
    // Vectors of 256 and 512 bytes leave one or two lane rows, so their tiles are small sub-heaps and their work items
    // many and short: there 8 items per warp and at most 4 warps did better in the sweeps.
    const uint32_t per_warp = C >= 16 ? 8u : 16u, max_warps = C >= 16 ? 4u : 8u;
    uint32_t warps = 1;
    while (warps < max_warps && warps * 2 * per_warp <= nitems) warps *= 2;
    uint32_t nbuf = 1;
    // tiny scenarios are staged whole with one copy, larger ones tile by tile (at 16 KB the tiles already win)
    const uint64_t scen_bytes = (uint64_t)p.P * p.kbytes;
    g.whole = scen_bytes <= (C >= 16 ? 16 * 1024 : kWholeMaxBytes) ? 1u : 0u;      // a few wide vectors: one copy up to 16 KB
    if (g.whole) nbuf = 0;
    size_t o = sizeof(Ctx) + 3 * (size_t)(p.W + 1) * 4;
    o = (o + 15) & ~(size_t)15; g.off_special = (uint32_t)o;
    o += (2 * (size_t)nitems_words(p.Lt, lw) * 4 + 15) & ~(size_t)15;
    g.off_rootv = (uint32_t)o; o += (size_t)C * 16;
    g.hv_bytes = (((uint64_t)2 << p.Lt) - 1) * C * 16;
    g.hv_global = (!g.whole && g.hv_bytes >= kHvGlobalMinBytes && g.hv_bytes <= kHvGlobalMaxBytes &&
                   p.ws_bytes / ((uint64_t)sm_count * kHvGlobalBlocksPerSm) >= g.hv_bytes) ? 1u : 0u;
    if (all_children == 2 && (g.hv_global || g.hv_bytes * p.m > 64 * 1024)) return false;
    g.off_hv = (uint32_t)o; if (!g.hv_global) o += (size_t)g.hv_bytes * (all_children == 2 ? p.m : 1u);
    g.off_dirty = (uint32_t)o;
    if (all_children) o += ((((((size_t)3 << p.Lt) + 31) / 32 + 4) + ((size_t)1 << p.Lt)) * 4 + 15) & ~(size_t)15;   // keeps the barriers behind it 8-byte aligned
    g.off_words = (uint32_t)o;
    if (all_children == 2) o += ((size_t)p.m * (((size_t)3 << p.Lt)) * 4 + 15) & ~(size_t)15;       // words of every node and child
    g.off_bar = (uint32_t)o; o += (size_t)(kStagedMaxThreads / 32) * 4 * 8 + 8;      // room for any warps x nbuf, plus one
    g.off_gaveup = (uint32_t)o; o += 8;
    o = (o + 127) & ~(size_t)127; g.off_tiles = (uint32_t)o;
    if (g.whole) {
        o += (size_t)((scen_bytes + 127) & ~(uint64_t)127);
    } else {
        while (nbuf > 1 && o + (size_t)warps * nbuf * cap > (size_t)smem_optin - 1024) --nbuf;
        while (warps > 1 && o + (size_t)warps * nbuf * cap > (size_t)smem_optin - 1024) --warps;
        o += (size_t)warps * nbuf * cap;
    }
    if (o > (size_t)smem_optin - 1024) return false;
    g.nwarps = warps; g.nbuf = nbuf; g.tile_cap = (uint32_t)cap; g.smem_bytes = (uint32_t)o;
    return true;
}

static uint32_t staged_xl(const Params& p) {
    uint32_t xl;
    // deepest lane-local sub-heap that keeps a tile (all its levels, every member) within 12 KB; 20 KB for vectors of
    // 256 and 512 bytes, whose tiles would otherwise be three rows
    if (p.kbytes % 16 || p.kbytes > 512) return 1;
    uint32_t C = p.kbytes / 16, cwl = 0; while ((1u << cwl) < C) ++cwl;
    const uint32_t lw = 5 - cwl, budget = (C >= 16 ? 20u : 12u) * 1024u;
    for (xl = 3; xl > 1; --xl)
        if ((((uint64_t)1 << (lw + xl)) - 1) * p.m * p.kbytes <= budget) break;
    return xl;
}

static const TmaMaps kNoMaps = {};

// Tensor maps for the swizzled variant (host side, below).
static bool staged_tensor_maps(const Params& p, uint32_t D, TmaMaps& maps);

template <typename T, int OP, int XL, bool WHOLE, int MINB, int GM = 0>
static cudaError_t launch_staged_w(const Params& p, const StagedGeom& g, int sm_count, cudaStream_t st, const TmaMaps& maps = kNoMaps) {
    cudaError_t e = cudaFuncSetAttribute(staged_kernel<T, OP, XL, WHOLE, MINB, GM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem_bytes);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, staged_kernel<T, OP, XL, WHOLE, MINB, GM>, (int)g.nwarps * 32, g.smem_bytes);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    if (g.hv_global && per_sm > kHvGlobalBlocksPerSm) per_sm = kHvGlobalBlocksPerSm;      // one workspace slice per block
    const uint64_t cap = (uint64_t)sm_count * per_sm;
    const uint32_t grid = (uint32_t)(p.S < cap ? p.S : cap);
    if (p.grid_query) { *p.grid_query = grid; return cudaSuccess; }
    staged_kernel<T, OP, XL, WHOLE, MINB, GM><<<grid, g.nwarps * 32, g.smem_bytes, st>>>(p, g, maps);
    return cudaGetLastError();
}

// Which instantiation plays a shape. The names are what ftc_kernel_variant() reports.
enum StagedVariant { SV_NONE = 0, SV_WHOLE, SV_WHOLE_LARGE, SV_LEAN, SV_LEAN_SWZ, SV_BATCHED_LEAN, SV_BATCHED_SWZ, SV_LARGE };
static inline const char* staged_variant_name(StagedVariant v) {
    switch (v) {
    case SV_WHOLE: return "staged/whole";
    case SV_WHOLE_LARGE: return "staged/whole-large";
    case SV_LEAN: return "staged/lean";
    case SV_LEAN_SWZ: return "staged/lean-swz";
    case SV_BATCHED_LEAN: return "staged/batched-lean";
    case SV_BATCHED_SWZ: return "staged/batched-swz";
    case SV_LARGE: return "staged/large";
    default: return "none";
    }
}

// Can the batch be described by the tensor maps of the swizzled variant (everything but the driver's own checks)?
static inline bool staged_tensor_maps_possible(const Params& p, uint32_t D) {
    const uint64_t rowbytes = (uint64_t)p.m * p.kbytes, line = p.swz_mask == 0x70u ? 128 : 64;
    const uint64_t scen_bytes = (uint64_t)p.P * p.kbytes;
    if (D > 8 || p.q == 0 || scen_bytes % 16 || rowbytes % line) return false;
    return ((rowbytes / line) << (D - 1)) <= 256;
}

// Geometry and instantiation for a shape; `ordered`: the combine order is observable (float32); `allow_swz`: the
// swizzled variants may be chosen (the launch retries without them when the driver refuses a tensor map).
static StagedVariant staged_plan(Params& p, bool ordered, bool allow_swz, uint32_t XL, int smem_optin, int sm_count, StagedGeom& g) {
    // float32 with vectors of 16 or 32 bytes: the fold order is fixed, so the rows of different lane rows would meet in
    // the same banks when groups are a multiple of 128 bytes or 64 bytes (4- and 8-way conflicts); their tiles come in
    // by tensor copies with the matching swizzle instead
    const uint64_t gbytes = (uint64_t)p.m * p.kbytes;
    bool swizzled = allow_swz && ordered && p.kbytes <= 32 && (gbytes % 128 == 0 || gbytes == 64) && p.S < (1ull << 31) &&
                    (uint64_t)p.P * p.kbytes > kWholeMaxBytes;
    p.swz_mask = 0; p.row_shift = 0;
    if (swizzled) { p.swz_mask = gbytes == 64 ? 0x30u : 0x70u; p.row_shift = gbytes == 64 ? 1u : 0u; }
    if (swizzled && !(staged_geometry(p, smem_optin, sm_count, XL, g) && !g.whole && staged_tensor_maps_possible(p, (5 - p.cw_log2) + XL))) {
        swizzled = false; p.swz_mask = 0; p.row_shift = 0;
    }
    if (!swizzled && !staged_geometry(p, smem_optin, sm_count, XL, g)) return SV_NONE;
    // one- and two-warp blocks get the lean variant; its register cap (about 96) matches the blocks that fit by shared
    // memory. Scenarios staged whole are so small that many more blocks fit: for them 64 registers, so that the
    // SM's block limit and not the register file decides
    const bool lean = g.nwarps <= 2;
    if (g.whole) return lean ? SV_WHOLE : SV_WHOLE_LARGE;
    if (swizzled) return lean ? SV_LEAN_SWZ : SV_BATCHED_SWZ;
    if (lean) return SV_LEAN;
    // Groups of at most 128 bytes: a row is so little data that the instructions around it count, so large blocks
    // run the lean variant's code too (rows of a lane folded together, starting members rotated). Not for float32:
    // its bank conflicts weigh more there than the saved instructions.
    if (!ordered && gbytes <= 128) return SV_BATCHED_LEAN;
    return SV_LARGE;
}

template <typename T, int OP, int XL>
static cudaError_t launch_staged_t(Params p, int sm_count, int smem_optin, cudaStream_t st) {
    StagedGeom g;
    StagedVariant v = staged_plan(p, Ordered<T>::value, true, XL, smem_optin, sm_count, g);
    if constexpr (Ordered<T>::value) {
        if (v == SV_LEAN_SWZ || v == SV_BATCHED_SWZ) {
            TmaMaps maps = kNoMaps;
            if (p.grid_query || staged_tensor_maps(p, (5 - p.cw_log2) + XL, maps))
                return v == SV_LEAN_SWZ ? launch_staged_w<T, OP, XL, false, kStagedLeanSwzTag>(p, g, sm_count, st, maps)
                                        : launch_staged_w<T, OP, XL, false, kStagedBatchedSwzTag>(p, g, sm_count, st, maps);
            v = staged_plan(p, true, false, XL, smem_optin, sm_count, g);      // no tensor maps: the plain layout after all
        }
    }
    switch (v) {
    case SV_WHOLE: return launch_staged_w<T, OP, XL, true, 4>(p, g, sm_count, st);
    case SV_WHOLE_LARGE: return launch_staged_w<T, OP, XL, true, 2>(p, g, sm_count, st);
    case SV_LEAN: return launch_staged_w<T, OP, XL, false, kStagedLeanMinBlocks>(p, g, sm_count, st);
    case SV_BATCHED_LEAN:
        if constexpr (!Ordered<T>::value) return launch_staged_w<T, OP, XL, false, kStagedBatchedTag>(p, g, sm_count, st);
        return cudaErrorInvalidConfiguration;
    case SV_LARGE:
        if (p.m == 5) return launch_staged_w<T, OP, XL, false, 2, 5>(p, g, sm_count, st);
        if (p.m == 9) return launch_staged_w<T, OP, XL, false, 2, 9>(p, g, sm_count, st);
        return launch_staged_w<T, OP, XL, false, 2>(p, g, sm_count, st);
    default: return cudaErrorInvalidConfiguration;
    }
}

typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                      const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The scenario batch as a tensor [S][lines][line words]: line = 128 bytes (64 for 64-byte groups), counted from the first group of each scenario
// (process 1), full groups only; consecutive scenarios lie P*k*e bytes apart. Map t has a box of 2^t rows. Returns
// false when the driver entry point is missing or a map cannot be encoded (the caller then takes the untiled copies).
static bool staged_tensor_maps(const Params& p, uint32_t D, TmaMaps& maps) {
    static TensorMapEncodeFn encode = [] {
        void* fn = nullptr; cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) fn = nullptr;
        return reinterpret_cast<TensorMapEncodeFn>(fn);
    }();
    const uint64_t rowbytes = (uint64_t)p.m * p.kbytes, line = p.swz_mask == 0x70u ? 128 : 64;
    const uint64_t lines_per_row = rowbytes / line, scen_bytes = (uint64_t)p.P * p.kbytes;
    if (!encode || !staged_tensor_maps_possible(p, D)) return false;
    void* base = const_cast<char*>(static_cast<const char*>(p.in)) + p.kbytes;
    const cuuint64_t dims[3] = {line / 4, (cuuint64_t)p.q * lines_per_row, (cuuint64_t)p.S};
    const cuuint64_t strides[2] = {line, scen_bytes};
    const cuuint32_t elem_strides[3] = {1, 1, 1};
    for (uint32_t t = 0; t < D; ++t) {
        const uint64_t box_lines = lines_per_row << t;
        if (box_lines > 256) return false;
        const cuuint32_t box[3] = {(cuuint32_t)(line / 4), (cuuint32_t)box_lines, 1};
        if (encode(&maps.lvl[t], CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, base, dims, strides, box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   line == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return false;
    }
    for (uint32_t t = D; t < 8; ++t) maps.lvl[t] = maps.lvl[0];
    return true;
}

template <typename T, int OP>
static cudaError_t launch_staged_x(const Params& p, int sm_count, int smem_optin, cudaStream_t st) {
    switch (staged_xl(p)) {
    case 2: return launch_staged_t<T, OP, 2>(p, sm_count, smem_optin, st);
    case 3: return launch_staged_t<T, OP, 3>(p, sm_count, smem_optin, st);
    default: return launch_staged_t<T, OP, 1>(p, sm_count, smem_optin, st);
    }
}

}  // namespace ftc
