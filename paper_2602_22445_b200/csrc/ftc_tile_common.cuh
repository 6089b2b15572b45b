// Pieces shared by the register-tiled and the shared-memory-staged kernels: 16-byte vector combine, the group
// fold from global memory, the warp-shuffle tree phase of a tile, the status record.
#pragma once
#include "ftc_device.cuh"

namespace ftc {

template <typename T> struct Vec16 { static constexpr int N = 16 / sizeof(T); };

template <typename T, int OP>
__device__ __forceinline__ uint4 comb16(uint4 a, uint4 b) {
    union U { uint4 v; T t[Vec16<T>::N]; } A, B;
    A.v = a; B.v = b;
#pragma unroll
    for (int i = 0; i < Vec16<T>::N; ++i) A.t[i] = Comb<T, OP>::f(A.t[i], B.t[i]);
    return A.v;
}

__device__ __forceinline__ uint4 ld_stream(const char* ptr) {
    return __ldg(reinterpret_cast<const uint4*>(ptr));
}

// WIDTH < 32: the warp is cut into groups of WIDTH lanes and `src` counts within the caller's group.
template <int WIDTH = 32>
__device__ __forceinline__ uint4 shfl16(uint4 v, uint32_t src) {
    uint4 r;
    r.x = __shfl_sync(0xFFFFFFFFu, v.x, src, WIDTH); r.y = __shfl_sync(0xFFFFFFFFu, v.y, src, WIDTH);
    r.z = __shfl_sync(0xFFFFFFFFu, v.z, src, WIDTH); r.w = __shfl_sync(0xFFFFFFFFu, v.w, src, WIDTH);
    return r;
}

// Is the combine order observable? Integer sum, max and xor are exactly associative and commutative, so any order
// gives the same bits; float32 addition is not, so there the schedule's order is kept.
template <typename T> struct Ordered { static constexpr bool value = false; };
template <> struct Ordered<float> { static constexpr bool value = true; };

struct LdGlobal { __device__ __forceinline__ uint4 operator()(const char* q) const { return ld_stream(q); } };
struct LdShared { __device__ __forceinline__ uint4 operator()(const char* q) const { return *reinterpret_cast<const uint4*>(q); } };

// Chunk lc of group `row` as the selected subtree's member holds it after up-correction, read from a copy of the
// scenario in the caller's process order (global memory, or shared memory when LD = LdShared):
// own input, then (short last group only) the root's, then the partners whose message arrived, ascending.
// Handles every case (missing members, the renumbered slots, the short group). MCAP > 0: loads of up to MCAP
// members are issued together; MCAP = 0: batches of four.
template <typename T, int OP, int MCAP, typename LD = LdGlobal, typename SHAPE = Params>
__device__ __forceinline__ uint4 fold16_general(const SHAPE& p, uint32_t root, uint32_t sstar, const uint32_t* inc,
                                                const char* in_lc, uint32_t row) {
    const LD ld{};
    const uint32_t mj = row < p.q ? p.m : p.r, vbase = row * p.m + 1;
    const uint32_t mask = extract_bits(inc, vbase, mj);
    uint4 acc = make_uint4(0, 0, 0, 0);
    if (Ordered<T>::value && p.pdesc) {
        // the other partner order: own input, then the partners whose message arrived in descending rank, the root last
        const uint32_t vo = vbase + sstar;
        acc = ld(in_lc + (size_t)(vo == root ? 0u : vo) * p.kbytes);
        for (uint32_t sp = mj; sp-- > 0;) {
            const uint32_t vr = vbase + sp;
            if (sp != sstar && ((mask >> sp) & 1u)) acc = comb16<T, OP>(acc, ld(in_lc + (size_t)(vr == root ? 0u : vr) * p.kbytes));
        }
        if (row == p.q) acc = comb16<T, OP>(acc, ld(in_lc + (size_t)root * p.kbytes));
        return acc;
    }
    if (MCAP > 0) {
        uint4 v[MCAP > 0 ? MCAP : 1];
#pragma unroll
        for (int sp = 0; sp < MCAP; ++sp) {
            v[sp] = make_uint4(0, 0, 0, 0);
            if ((uint32_t)sp < mj && ((mask >> sp) & 1u)) {
                const uint32_t vr = vbase + sp;
                v[sp] = ld(in_lc + (size_t)(vr == root ? 0u : vr) * p.kbytes);
            }
        }
        uint4 vroot = make_uint4(0, 0, 0, 0);
        if (row == p.q) vroot = ld(in_lc + (size_t)root * p.kbytes);
#pragma unroll
        for (int sp = 0; sp < MCAP; ++sp) if ((uint32_t)sp == sstar) acc = v[sp];
        if (row == p.q) acc = comb16<T, OP>(acc, vroot);
#pragma unroll
        for (int sp = 0; sp < MCAP; ++sp)
            if ((uint32_t)sp < mj && (uint32_t)sp != sstar && ((mask >> sp) & 1u)) acc = comb16<T, OP>(acc, v[sp]);
    } else {
        const uint32_t vo = vbase + sstar;
        acc = ld(in_lc + (size_t)(vo == root ? 0u : vo) * p.kbytes);
        if (row == p.q) acc = comb16<T, OP>(acc, ld(in_lc + (size_t)root * p.kbytes));
        for (uint32_t s0 = 0; s0 < mj; s0 += 4) {
            uint4 v[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t sp = s0 + i, vr = vbase + sp;
                v[i] = make_uint4(0, 0, 0, 0);
                if (sp < mj && sp != sstar && ((mask >> sp) & 1u)) v[i] = ld(in_lc + (size_t)(vr == root ? 0u : vr) * p.kbytes);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t sp = s0 + i;
                if (sp < mj && sp != sstar && ((mask >> sp) & 1u)) acc = comb16<T, OP>(acc, v[i]);
            }
        }
    }
    return acc;
}

// Position in memory of the i-th operand of a full group's fold: for float the member of the selected subtree
// comes first, then the others ascending (desc: descending); for the exactly associative operations simply ascending.
template <typename T>
__device__ __forceinline__ uint32_t fold_member(uint32_t i, uint32_t sstar, uint32_t m = 0, bool desc = false) {
    if (!Ordered<T>::value) return i;
    if (i == 0) return sstar;
    if (desc) { const uint32_t c = m - i; return c - (c <= sstar ? 1u : 0u); }
    return i - (i <= sstar ? 1u : 0u);
}

// Fold of a full group all of whose members' messages are present, from m vectors `stride` bytes apart starting
// at `ptr` (global or shared memory, LD loads 16 bytes). MCAP > 0: all loads issued together.
template <typename T, int OP, int MCAP, typename LD>
__device__ __forceinline__ uint4 fold16_full(const char* ptr, uint32_t stride, uint32_t m, uint32_t sstar, LD ld, bool desc = false) {
    uint4 acc;
    if (MCAP > 0) {
        uint4 v[MCAP > 0 ? MCAP : 1];
#pragma unroll
        for (int i = 0; i < MCAP; ++i)
            if ((uint32_t)i < m) v[i] = ld(ptr + fold_member<T>(i, sstar, m, desc) * stride);
        acc = v[0];
#pragma unroll
        for (int i = 1; i < MCAP; ++i)
            if ((uint32_t)i < m) acc = comb16<T, OP>(acc, v[i]);
    } else {
        acc = ld(ptr + fold_member<T>(0, sstar) * stride);
#pragma unroll 4
        for (uint32_t i = 1; i < m; ++i) acc = comb16<T, OP>(acc, ld(ptr + fold_member<T>(i, sstar, m, desc) * stride));
    }
    return acc;
}

// Fold of a full-size group some of whose members' messages may be missing (`mask`), from a copy in which the
// members sit `stride` bytes apart in rank order: own input first, then the arrived ones ascending.
template <typename T, int OP, typename LD>
__device__ __forceinline__ uint4 fold16_masked(const char* ptr, uint32_t stride, uint32_t m, uint32_t mask, uint32_t sstar, LD ld, bool desc = false) {
    uint4 acc = ld(ptr + sstar * stride);
#pragma unroll 2
    for (uint32_t i = 0; i < m; ++i) {
        const uint32_t sp = (Ordered<T>::value && desc) ? m - 1 - i : i;
        if (sp != sstar && ((mask >> sp) & 1u)) acc = comb16<T, OP>(acc, ld(ptr + sp * stride));
    }
    return acc;
}

// A group is "plain" when it is full, every member's message reached the selected subtree's member, and neither
// renumbered slot lies in it; then its fold needs one base address and constant strides.
__device__ __forceinline__ bool group_is_plain(const Params& p, uint32_t root, const uint32_t* inc, uint32_t row) {
    const uint32_t vbase = row * p.m + 1;
    const uint32_t full = p.m >= 32 ? 0xFFFFFFFFu : ((1u << p.m) - 1u);
    return row < p.q && root - vbase >= p.m && extract_bits(inc, vbase, p.m) == full;   // unsigned wrap: root outside the row
}

// The four numbers the general fold needs, for passing by value.
struct FoldShape { uint32_t m, q, r, kbytes, swz_mask, pdesc; };
__device__ __forceinline__ FoldShape fold_shape(const Params& p) { return FoldShape{p.m, p.q, p.r, p.kbytes, p.swz_mask, p.pdesc}; }

// Any group, by the general routine (the careful path of the tiled kernels; rare). LD says where `in_lc`, the
// scenario in process order, lives.
template <typename T, int OP, typename LD>
__device__ __forceinline__ uint4 fold16_careful(const Params& p, uint32_t root, uint32_t sstar, const uint32_t* inc,
                                             const char* in_lc, uint32_t row) {
    return fold16_general<T, OP, 0, LD>(p, root, sstar, inc, in_lc, row);
}

// Tree phase inside a warp tile (Algorithm "reduce_non_root": data <- (data (op) child 1) (op) child 2).
// valA: this lane's row of the tile's bottom level (lane row lr); valB: its row of the levels above (tile heap
// index lr, level tB, position idxB; rowB its global row, hasB whether it exists). Returns the updated valB.
// FULL: every row of the tile's upper levels and of its bottom level exists (no existence checks at all);
// FULL_ABOVE: only the bottom level may be ragged (checked), everything above exists.
// WIDTH < 32: one tile per group of WIDTH lanes; `lane` is then the lane within the group.
template <typename T, int OP, bool FULL = false, bool FULL_ABOVE = false, int WIDTH = 32>
__device__ __forceinline__ uint4 tile_tree_phase(uint4 valA, uint4 valB, uint32_t lw, uint32_t cwl, uint32_t C,
                                                 uint32_t lane, uint32_t lc, uint32_t tB, uint32_t idxB, uint32_t rowB,
                                                 bool hasB, uint32_t G) {
    if (lw) {
        const bool mine = hasB && tB == lw - 1;
        const uint32_t src1 = mine ? (((2 * idxB) << cwl) | lc) : lane;
        const uint4 c1 = shfl16<WIDTH>(valA, src1), c2 = shfl16<WIDTH>(valA, mine ? src1 + C : lane);
        if (mine) {
            if (FULL || 2 * rowB + 1 < G) valB = comb16<T, OP>(valB, c1);
            if (FULL || 2 * rowB + 2 < G) valB = comb16<T, OP>(valB, c2);
        }
    }
    for (int t = (int)lw - 2; t >= 0; --t) {
        const bool mine = hasB && tB == (uint32_t)t;
        const uint32_t src1 = mine ? ((((2u << t) - 1 + 2 * idxB) << cwl) | lc) : lane;
        const uint4 c1 = shfl16<WIDTH>(valB, src1), c2 = shfl16<WIDTH>(valB, mine ? src1 + C : lane);
        if (mine) {
            if (FULL || FULL_ABOVE || 2 * rowB + 1 < G) valB = comb16<T, OP>(valB, c1);
            if (FULL || FULL_ABOVE || 2 * rowB + 2 < G) valB = comb16<T, OP>(valB, c2);
        }
    }
    return valB;
}

// Work items (warp tiles, then groups of rows above the tiles) that need the careful path: those containing a
// group that is not plain (a member failed or is an in-operation victim, a renumbered slot, the short last group)
// and those that are incomplete above their last level. One bit per item in `tspec`; all threads call.
// Item numbering: tile i (rooted at heap row 2^Lt - 1 + i, D levels) is item i; rows [g*grows, (g+1)*grows) above the
// tiles are item 2^Lt + g (grows = rows per such item, 0 = one per lane row).
// `tmask` gets the items whose only peculiarity is a group with missing members (fold under the arrival mask, no
// other checks needed); pass tmask = tspec to send those the careful way too.
// `below`: rows under the tiles' last level (a sparsely filled last heap level) are folded one by one by the general
// routine wherever a tile meets them, so they mark nothing.
static __device__ void mark_special_items(const Params& p, const Ctx* cx, const uint32_t* pf, uint32_t* tspec,
                                          uint32_t* tmask, uint32_t Lt, uint32_t lw, uint32_t D, bool below = false, uint32_t grows = 0,
                                          uint32_t ngroups = 0) {
    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    const uint32_t ntiles = 1u << Lt, ntop = ntiles - 1;
    if (grows == 0) { grows = 1u << lw; ngroups = (ntop + grows - 1) >> lw; }      // callers with other sizes pass both
    const uint32_t nitems = ntiles + ngroups, root = cx->root, G = cx->G;
    for (uint32_t w = tid; w < (nitems + 31) / 32 + 1; w += nt) { tspec[w] = 0; tmask[w] = 0; }
    __syncthreads();
    auto mark_row = [&](uint32_t j, uint32_t* bm) {
        const uint32_t lvl = ilog2u(j + 1);
        if (below && lvl >= Lt + D) return;
        const uint32_t it = lvl >= Lt ? ((j + 1) >> (lvl - Lt)) - ntiles : ntiles + j / grows;
        atomicOr(&bm[it >> 5], 1u << (it & 31));
    };
    for (uint32_t w = tid; w < p.W; w += nt) {
        uint32_t word = pf[w];
        while (word) {
            const uint32_t b = __ffs(word) - 1; word &= word - 1;
            const uint32_t v = renumber((w << 5) + b, root);
            if (v && (v - 1) / p.m < G) mark_row((v - 1) / p.m, tmask);
        }
    }
    if (tid < p.max_inop && cx->iv[tid] != FTC_INOP_UNUSED) {
        const uint32_t v = renumber(cx->iv[tid], root);
        if (v && (v - 1) / p.m < G) mark_row((v - 1) / p.m, tmask);
    }
    if (tid == 0) {
        if (root != 0 && (root - 1) / p.m < G) mark_row((root - 1) / p.m, tspec);   // the slot that holds process 0's input
        if (G > p.q) mark_row(p.q, tspec);                                          // the short last group
    }
    // tiles not complete down to their second-to-last level (the last row of level t of the tile rooted at j0 is
    // ((j0+2) << t) - 2); their last level may be ragged, the common path checks it. And the ragged last group.
    // Also tiles with rows of the subtree below their last level (a sparsely filled last heap level is left out
    // of the tiles: the first row below tile j0 is ((j0+1) << D) - 1).
    for (uint32_t it = tid; it < ntiles; it += nt)
        if (((ntop + it + 2) << (D >= 2 ? D - 2 : 0)) - 2 >= G || (!below && ((ntop + it + 1) << D) - 1 < G))
            atomicOr(&tspec[it >> 5], 1u << (it & 31));
    for (uint32_t g = tid; g < ngroups; g += nt)
        if ((g + 1) * grows > ntop || (g + 1) * grows > G) atomicOr(&tspec[(ntiles + g) >> 5], 1u << ((ntiles + g) & 31));
    __syncthreads();
}

// The root's data after up-correction, for the case that no member of its (short, last) group lies in the
// selected subtree: own input, then the members of that group whose message arrived.
template <typename T, int OP, typename LD = LdGlobal>
__device__ __forceinline__ uint4 fold_root16(const Params& p, uint32_t root, const uint32_t* inc, const char* in_lc) {
    const LD ld{};
    uint4 acc = ld(in_lc + (size_t)root * p.kbytes);
    if (p.r) {
        const uint32_t vbase = p.q * p.m + 1, mask = extract_bits(inc, vbase, p.r);
        for (uint32_t i = 0; i < p.r; ++i) {
            const uint32_t sp = (Ordered<T>::value && p.pdesc) ? p.r - 1 - i : i, vr = vbase + sp;
            if ((mask >> sp) & 1u) acc = comb16<T, OP>(acc, ld(in_lc + (size_t)(vr == root ? 0u : vr) * p.kbytes));
        }
    }
    return acc;
}

__device__ __forceinline__ void write_status_rec(const Params& p, uint64_t s, const Ctx* cx) {
    uint32_t* st = p.status + s * FTC_STATUS_WORDS;
    const bool ok = cx->code == FTC_ST_OK;
    uint4 rec;
    rec.x = cx->code | ((ok ? cx->sstar : 0xFFu) << 8) | (cx->attempts << 16);
    rec.y = ok ? p.P - cx->npre - cx->nexcl : 0u;
    rec.z = ok ? cx->inop_incl : 0u;
    rec.w = (ok && p.is_allreduce) ? cx->holders : 0u;
    *reinterpret_cast<uint4*>(st) = rec;
}

}  // namespace ftc
