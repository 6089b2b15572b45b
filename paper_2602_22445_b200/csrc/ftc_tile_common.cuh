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

__device__ __forceinline__ uint4 shfl16(uint4 v, uint32_t src) {
    uint4 r;
    r.x = __shfl_sync(0xFFFFFFFFu, v.x, src); r.y = __shfl_sync(0xFFFFFFFFu, v.y, src);
    r.z = __shfl_sync(0xFFFFFFFFu, v.z, src); r.w = __shfl_sync(0xFFFFFFFFu, v.w, src);
    return r;
}

// Is the combine order observable? Integer sum, max and xor are exactly associative and commutative, so any order
// gives the same bits; float32 addition is not, so there the schedule's order is kept.
template <typename T> struct Ordered { static constexpr bool value = false; };
template <> struct Ordered<float> { static constexpr bool value = true; };

// Chunk lc of group `row` as the selected subtree's member holds it after up-correction, read from global memory:
// own input, then (short last group only) the root's, then the partners whose message arrived, ascending.
// Handles every case (missing members, the renumbered slots, the short group). MCAP > 0: loads of up to MCAP
// members are issued together; MCAP = 0: batches of eight.
template <typename T, int OP, int MCAP>
__device__ __forceinline__ uint4 fold16_general(const Params& p, uint32_t root, uint32_t sstar, const uint32_t* inc,
                                                const char* in_lc, uint32_t row) {
    const uint32_t mj = row < p.q ? p.m : p.r, vbase = row * p.m + 1;
    const uint32_t mask = extract_bits(inc, vbase, mj);
    uint4 acc = make_uint4(0, 0, 0, 0);
    if (MCAP > 0) {
        uint4 v[MCAP > 0 ? MCAP : 1];
#pragma unroll
        for (int sp = 0; sp < MCAP; ++sp) {
            v[sp] = make_uint4(0, 0, 0, 0);
            if ((uint32_t)sp < mj && ((mask >> sp) & 1u)) {
                const uint32_t vr = vbase + sp;
                v[sp] = ld_stream(in_lc + (size_t)(vr == root ? 0u : vr) * p.kbytes);
            }
        }
        uint4 vroot = make_uint4(0, 0, 0, 0);
        if (row == p.q) vroot = ld_stream(in_lc + (size_t)root * p.kbytes);
#pragma unroll
        for (int sp = 0; sp < MCAP; ++sp) if ((uint32_t)sp == sstar) acc = v[sp];
        if (row == p.q) acc = comb16<T, OP>(acc, vroot);
#pragma unroll
        for (int sp = 0; sp < MCAP; ++sp)
            if ((uint32_t)sp < mj && (uint32_t)sp != sstar && ((mask >> sp) & 1u)) acc = comb16<T, OP>(acc, v[sp]);
    } else {
        const uint32_t vo = vbase + sstar;
        acc = ld_stream(in_lc + (size_t)(vo == root ? 0u : vo) * p.kbytes);
        if (row == p.q) acc = comb16<T, OP>(acc, ld_stream(in_lc + (size_t)root * p.kbytes));
        for (uint32_t s0 = 0; s0 < mj; s0 += 8) {
            uint4 v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t sp = s0 + i, vr = vbase + sp;
                v[i] = make_uint4(0, 0, 0, 0);
                if (sp < mj && sp != sstar && ((mask >> sp) & 1u)) v[i] = ld_stream(in_lc + (size_t)(vr == root ? 0u : vr) * p.kbytes);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t sp = s0 + i;
                if (sp < mj && sp != sstar && ((mask >> sp) & 1u)) acc = comb16<T, OP>(acc, v[i]);
            }
        }
    }
    return acc;
}

// Fold of a full group all of whose members' messages are present, from m vectors `stride` bytes apart starting
// at `ptr` (global or shared memory, LD loads 16 bytes). Own input first when the order is observable.
template <typename T, int OP, int MCAP, typename LD>
__device__ __forceinline__ uint4 fold16_full(const char* ptr, uint32_t stride, uint32_t m, uint32_t sstar, LD ld) {
    uint4 acc;
    if (MCAP > 0) {
        uint4 v[MCAP > 0 ? MCAP : 1];
#pragma unroll
        for (int sp = 0; sp < MCAP; ++sp)
            if ((uint32_t)sp < m) v[sp] = ld(ptr + (uint32_t)sp * stride);
        acc = v[0];
        if (Ordered<T>::value) {
#pragma unroll
            for (int sp = 1; sp < MCAP; ++sp) if ((uint32_t)sp == sstar) acc = v[sp];
#pragma unroll
            for (int sp = 0; sp < MCAP; ++sp)
                if ((uint32_t)sp < m && (uint32_t)sp != sstar) acc = comb16<T, OP>(acc, v[sp]);
        } else {
#pragma unroll
            for (int sp = 1; sp < MCAP; ++sp)
                if ((uint32_t)sp < m) acc = comb16<T, OP>(acc, v[sp]);
        }
    } else {
        acc = ld(ptr + (Ordered<T>::value ? sstar : 0u) * stride);
        for (uint32_t sp = 0; sp < m; ++sp)
            if (sp != (Ordered<T>::value ? sstar : 0u)) acc = comb16<T, OP>(acc, ld(ptr + sp * stride));
    }
    return acc;
}

struct LdGlobal { __device__ __forceinline__ uint4 operator()(const char* q) const { return ld_stream(q); } };

// A group is "plain" when it is full, every member's message reached the selected subtree's member, and neither
// renumbered slot lies in it; then its fold needs one base address and constant strides.
__device__ __forceinline__ bool group_is_plain(const Params& p, uint32_t root, const uint32_t* inc, uint32_t row) {
    const uint32_t vbase = row * p.m + 1;
    const uint32_t full = p.m >= 32 ? 0xFFFFFFFFu : ((1u << p.m) - 1u);
    return row < p.q && root - vbase >= p.m && extract_bits(inc, vbase, p.m) == full;   // unsigned wrap: root outside the row
}

template <typename T, int OP, int MCAP>
__device__ __forceinline__ uint4 fold16(const Params& p, uint32_t root, uint32_t sstar, const uint32_t* inc,
                                        const char* in_lc, uint32_t row) {
    if (group_is_plain(p, root, inc, row))
        return fold16_full<T, OP, MCAP>(in_lc + (size_t)(row * p.m + 1) * p.kbytes, p.kbytes, p.m, sstar, LdGlobal());
    return fold16_general<T, OP, MCAP>(p, root, sstar, inc, in_lc, row);
}

// Tree phase inside a warp tile (Algorithm "reduce_non_root": data <- (data (op) child 1) (op) child 2).
// valA: this lane's row of the tile's bottom level (lane row lr); valB: its row of the levels above (tile heap
// index lr, level tB, position idxB; rowB its global row, hasB whether it exists). Returns the updated valB.
template <typename T, int OP>
__device__ __forceinline__ uint4 tile_tree_phase(uint4 valA, uint4 valB, uint32_t lw, uint32_t cwl, uint32_t C,
                                                 uint32_t lane, uint32_t lc, uint32_t tB, uint32_t idxB, uint32_t rowB,
                                                 bool hasB, uint32_t G) {
    if (lw) {
        const bool mine = hasB && tB == lw - 1;
        const uint32_t src1 = mine ? (((2 * idxB) << cwl) | lc) : lane;
        const uint4 c1 = shfl16(valA, src1), c2 = shfl16(valA, mine ? src1 + C : lane);
        if (mine) {
            if (2 * rowB + 1 < G) valB = comb16<T, OP>(valB, c1);
            if (2 * rowB + 2 < G) valB = comb16<T, OP>(valB, c2);
        }
    }
    for (int t = (int)lw - 2; t >= 0; --t) {
        const bool mine = hasB && tB == (uint32_t)t;
        const uint32_t src1 = mine ? ((((2u << t) - 1 + 2 * idxB) << cwl) | lc) : lane;
        const uint4 c1 = shfl16(valB, src1), c2 = shfl16(valB, mine ? src1 + C : lane);
        if (mine) {
            if (2 * rowB + 1 < G) valB = comb16<T, OP>(valB, c1);
            if (2 * rowB + 2 < G) valB = comb16<T, OP>(valB, c2);
        }
    }
    return valB;
}

// The root's data after up-correction, for the case that no member of its (short, last) group lies in the
// selected subtree: own input, then the members of that group whose message arrived.
template <typename T, int OP>
__device__ __forceinline__ uint4 fold_root16(const Params& p, uint32_t root, const uint32_t* inc, const char* in_lc) {
    uint4 acc = ld_stream(in_lc + (size_t)root * p.kbytes);
    if (p.r) {
        const uint32_t vbase = p.q * p.m + 1, mask = extract_bits(inc, vbase, p.r);
        for (uint32_t sp = 0; sp < p.r; ++sp) {
            const uint32_t vr = vbase + sp;
            if ((mask >> sp) & 1u) acc = comb16<T, OP>(acc, ld_stream(in_lc + (size_t)(vr == root ? 0u : vr) * p.kbytes));
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
