// Tiled kernel: the fast path for process vectors made of a power-of-two number (<= 32) of 16-byte chunks.
//
// One block plays one scenario at a time (grid-stride over the batch). After the decode, the selected root
// subtree -- a binary heap over the up-correction groups ("rows"; row j holds the f+1 processes j(f+1)+1 ..
// (j+1)(f+1), contiguous in memory) -- is cut at heap level Lt:
//   * every sub-heap rooted at level Lt is a TILE evaluated by one warp in registers: lane (lr, lc) handles
//     16-byte chunk lc of row lr of the tile's bottom level plus one row of the levels above, folds the row's
//     members with 128-bit loads (up-correction), and the tile's levels are combined with warp shuffles (tree
//     phase);
//   * rows above level Lt are folded by the same lanes into shared memory and combined there level by level.
// Every input byte is read from global memory exactly once; the combine order is the schedule's order, so
// float32 sums come out bit-identical to a message-by-message execution.
#include "ftc_tile_common.cuh"
#include "ftc_kernels.h"

namespace ftc {

constexpr int kTiledMaxThreads = 256;

template <typename T, int OP, int MCAP, int MINB>
__global__ void __launch_bounds__(kTiledMaxThreads, MINB) tiled_kernel(Params p) {
    extern __shared__ __align__(16) uint32_t smem[];
    Ctx* cx = reinterpret_cast<Ctx*>(smem);
    uint32_t* pf = smem + sizeof(Ctx) / 4;
    uint32_t* inc = pf + p.W + 1;
    uint32_t* unr = inc + p.W + 1;
    const uint32_t mask_words = ((sizeof(Ctx) / 4 + 3 * (p.W + 1)) + 3u) & ~3u;
    uint4* rootv = reinterpret_cast<uint4*>(smem + mask_words);      // [C] the root's own data after up-correction
    uint4* hv = rootv + p.C;                                          // [2^(Lt+1)-1][C] node values, heap order
    uint32_t* tspec = reinterpret_cast<uint32_t*>(hv + (((size_t)2 << p.Lt) - 1) * p.C);   // careful-path bit per work item

    const uint32_t tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, wid = tid >> 5, nw = nt >> 5;
    const uint32_t cwl = p.cw_log2, lw = 5 - cwl, RW = 1u << lw, Cmask = p.C - 1;
    const uint32_t lr = lane >> cwl, lc = lane & Cmask;
    const uint32_t Lt = p.Lt, ntiles = 1u << Lt, ntop = ntiles - 1, ngroups = (ntop + RW - 1) >> lw;
    const uint32_t nitems = ntiles + ngroups + 1;

    for (uint64_t s = blockIdx.x; s < p.S; s += gridDim.x) {
        decode_scenario(p, s, cx, pf, inc);
        char* out_s = reinterpret_cast<char*>(p.out) + s * p.kbytes;
        if (cx->code != FTC_ST_OK) {
            if (tid < p.C) reinterpret_cast<uint4*>(out_s)[tid] = make_uint4(0, 0, 0, 0);
            if (tid == 0) write_status_rec(p, s, cx);
            __syncthreads();
            continue;
        }
        if (p.is_allreduce) count_holders(p, cx, pf, unr);
        mark_special_items(p, cx, pf, tspec, tspec, Lt, lw, lw + 1);
        const uint32_t root = cx->root, sstar = cx->sstar, G = cx->G;
        const char* in_lc = reinterpret_cast<const char*>(p.in) + s * (size_t)p.P * p.kbytes + lc * 16;

        for (uint32_t it = wid; it < nitems; it += nw) {
            const bool careful = it < ntiles + ngroups && test_bit(tspec, it);      // warp-uniform
            if (it < ntiles) {
                // ---- one tile: the sub-heap below heap row j0, lw+1 levels ----
                const uint32_t j0 = ntop + it;
                const uint32_t rowA = ((j0 + 1) << lw) - 1 + lr;              // bottom level of the tile
                uint4 valA = make_uint4(0, 0, 0, 0), valB = make_uint4(0, 0, 0, 0);
                const uint32_t tB = ilog2u(lr + 1), idxB = lr + 1 - (1u << tB);
                const uint32_t rowB = ((j0 + 1) << tB) - 1 + idxB;            // this lane's row of the upper levels
                if (!careful) {
                    // all rows plain, the levels above the bottom complete: constant strides; only the bottom may be ragged
                    if (rowA < G) valA = fold16_full<T, OP, MCAP>(in_lc + (size_t)(rowA * p.m + 1) * p.kbytes, p.kbytes, p.m, sstar, LdGlobal(), p.pdesc != 0);
                    const bool hasBp = lr < RW - 1;
                    if (hasBp) valB = fold16_full<T, OP, MCAP>(in_lc + (size_t)(rowB * p.m + 1) * p.kbytes, p.kbytes, p.m, sstar, LdGlobal(), p.pdesc != 0);
                    valB = tile_tree_phase<T, OP, false, true>(valA, valB, lw, cwl, p.C, lane, lc, tB, idxB, rowB, hasBp, G);
                    if (lr == 0) hv[(size_t)j0 * p.C + lc] = lw ? valB : valA;
                    continue;
                }
                if (j0 >= G) continue;
                const bool hasB = lr < RW - 1 && rowB < G;
                if (rowA < G) valA = fold16_careful<T, OP, LdGlobal>(p, root, sstar, inc, in_lc, rowA);
                if (hasB) valB = fold16_careful<T, OP, LdGlobal>(p, root, sstar, inc, in_lc, rowB);
                valB = tile_tree_phase<T, OP>(valA, valB, lw, cwl, p.C, lane, lc, tB, idxB, rowB, hasB, G);
                if (lr == 0) hv[(size_t)j0 * p.C + lc] = lw ? valB : valA;
            } else if (it < ntiles + ngroups) {
                // ---- rows above the tiles: fold now, combine later ----
                const uint32_t row = ((it - ntiles) << lw) + lr;
                if (!careful) hv[(size_t)row * p.C + lc] = fold16_full<T, OP, MCAP>(in_lc + (size_t)(row * p.m + 1) * p.kbytes, p.kbytes, p.m, sstar, LdGlobal(), p.pdesc != 0);
                else if (row < ntop && row < G) hv[(size_t)row * p.C + lc] = fold16_careful<T, OP, LdGlobal>(p, root, sstar, inc, in_lc, row);
            } else if (sstar >= p.r) {
                if (lr == 0) rootv[lc] = fold_root16<T, OP>(p, root, inc, in_lc);
            }
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
        if (tid < p.C) {
            uint4 recv = hv[tid];
            reinterpret_cast<uint4*>(out_s)[tid] = sstar < p.r ? recv : comb16<T, OP>(rootv[tid], recv);
        }
        if (tid == 0) write_status_rec(p, s, cx);
        __syncthreads();
    }
}

static size_t tiled_smem_bytes(const Params& p) {
    size_t mask_words = ((sizeof(Ctx) / 4 + 3 * (size_t)(p.W + 1)) + 3u) & ~(size_t)3u;
    const uint32_t lw = 5 - p.cw_log2, ntiles = 1u << p.Lt;
    const size_t nitems = ntiles + ((ntiles - 1 + (1u << lw) - 1) >> lw);
    return mask_words * 4 + (size_t)p.C * 16 + (((size_t)2 << p.Lt) - 1) * p.C * 16 + ((nitems + 31) / 32 + 1) * 4;
}

bool tiled_supported(Params& p, int smem_optin_bytes) {
    if (p.kbytes % 16) return false;
    uint32_t C = p.kbytes / 16;
    if (C == 0 || C > 32 || (C & (C - 1))) return false;
    uint32_t cwl = 0; while ((1u << cwl) < C) ++cwl;
    uint32_t lw = 5 - cwl, D = lw + 1;
    uint32_t Hmax = 1; while ((1u << Hmax) <= p.Gmax) ++Hmax;      // levels of the largest subtree heap
    p.C = C; p.cw_log2 = cwl; p.Lt = Hmax > D ? Hmax - D : 0;
    if (p.Lt > 20) return false;
    return tiled_smem_bytes(p) <= (size_t)smem_optin_bytes - 1024;
}

static uint32_t tiled_threads(const Params& p) {
    const uint32_t lw = 5 - p.cw_log2, ntiles = 1u << p.Lt;
    const uint32_t nitems = ntiles + ((ntiles - 1 + (1u << lw) - 1) >> lw) + 1;
    uint32_t warps = nitems / 32;                 // about 32 work items per warp and scenario
    if (warps < 1) warps = 1;
    if (warps > 8) warps = 8;
    return warps * 32;
}

template <typename T, int OP, int MCAP, int MINB>
static cudaError_t launch_tiled_t(const Params& p, int sm_count, cudaStream_t st) {
    const size_t smem = tiled_smem_bytes(p);
    const uint32_t threads = tiled_threads(p);
    cudaError_t e = cudaFuncSetAttribute(tiled_kernel<T, OP, MCAP, MINB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, tiled_kernel<T, OP, MCAP, MINB>, (int)threads, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    uint64_t g = (uint64_t)sm_count * per_sm;
    const uint32_t grid = (uint32_t)(p.S < g ? p.S : g);
    if (p.grid_query) { *p.grid_query = grid; return cudaSuccess; }
    tiled_kernel<T, OP, MCAP, MINB><<<grid, threads, smem, st>>>(p);
    return cudaGetLastError();
}

// Register budget per MCAP (blocks of up to 256 threads): 3 blocks per SM (80 registers) for groups of up to four
// members, 2 (128 registers) for wider groups whose loads are all issued together.
template <typename T, int OP, int MCAP>
static cudaError_t launch_tiled_b(const Params& p, int sm_count, cudaStream_t st) {
    return launch_tiled_t<T, OP, MCAP, (MCAP == 4 ? 3 : 2)>(p, sm_count, st);
}

template <typename T, int OP>
static cudaError_t launch_tiled_m(const Params& p, int sm_count, cudaStream_t st) {
    if (p.m <= 4) return launch_tiled_b<T, OP, 4>(p, sm_count, st);
    if (p.m <= 6) return launch_tiled_b<T, OP, 6>(p, sm_count, st);
    if (p.m <= 9) return launch_tiled_b<T, OP, 9>(p, sm_count, st);
    return launch_tiled_b<T, OP, 0>(p, sm_count, st);
}

cudaError_t launch_tiled(const Params& p, int tsel, int sm_count, cudaStream_t st) {
    switch (tsel) {
    case TS_U32_SUM: return launch_tiled_m<uint32_t, OP_SUM>(p, sm_count, st);
    case TS_I32_MAX: return launch_tiled_m<int32_t, OP_MAX>(p, sm_count, st);
    case TS_U32_XOR: return launch_tiled_m<uint32_t, OP_XOR>(p, sm_count, st);
    case TS_U64_SUM: return launch_tiled_m<unsigned long long, OP_SUM>(p, sm_count, st);
    case TS_I64_MAX: return launch_tiled_m<long long, OP_MAX>(p, sm_count, st);
    case TS_U64_MAX: return launch_tiled_m<unsigned long long, OP_MAX>(p, sm_count, st);
    case TS_U64_XOR: return launch_tiled_m<unsigned long long, OP_XOR>(p, sm_count, st);
    case TS_F32_SUM: return launch_tiled_m<float, OP_SUM>(p, sm_count, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace ftc
