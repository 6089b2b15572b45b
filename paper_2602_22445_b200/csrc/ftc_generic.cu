// General kernel: any P, f, k. One block per scenario (grid-stride), the selected subtree is evaluated level by
// level from the leaves, node values pass through a per-block slice of the global workspace.
#include <mutex>
#include "ftc_tile_common.cuh"
#include "ftc_kernels.h"

namespace ftc {

// The unit a thread works on: one element, or (VEC) one 16-byte chunk of a process vector when vectors are a
// whole number of chunks.
template <typename T, int OP, bool VEC> struct Unit;
template <typename T, int OP> struct Unit<T, OP, false> {
    using V = T;
    static __device__ __forceinline__ V comb(V a, V b) { return Comb<T, OP>::f(a, b); }
    static __device__ __forceinline__ V zero() { return T(0); }
    static __device__ __forceinline__ V ld(const V* q) { return __ldg(q); }
};
template <typename T, int OP> struct Unit<T, OP, true> {
    using V = uint4;
    static __device__ __forceinline__ V comb(V a, V b) { return comb16<T, OP>(a, b); }
    static __device__ __forceinline__ V zero() { return make_uint4(0, 0, 0, 0); }
    static __device__ __forceinline__ V ld(const V* q) { return __ldg(q); }
};

// Value of group `row` as the selected subtree's member sees it after up-correction (Algorithm "Up-correction"):
// own input first, then the partners whose message arrived, in ascending rank (the root first in the short group).
// `in_s`: the scenario as units, `nu` units per process, `u` the unit.
template <typename U>
__device__ __forceinline__ typename U::V fold_group_unit(const Params& p, uint32_t root, uint32_t sstar, const uint32_t* inc,
                                                          const typename U::V* in_s, uint32_t nu, uint32_t row, uint32_t u) {
    const uint32_t mj = row < p.q ? p.m : p.r, vbase = row * p.m + 1;
    const uint32_t mask = extract_bits(inc, vbase, mj);
    typename U::V acc = U::ld(in_s + (size_t)renumber(vbase + sstar, root) * nu + u);
    if (p.pdesc) {                       // the other partner order: descending rank, the root last
        for (uint32_t sp = mj; sp-- > 0;)
            if (sp != sstar && ((mask >> sp) & 1u)) acc = U::comb(acc, U::ld(in_s + (size_t)renumber(vbase + sp, root) * nu + u));
        if (row == p.q) acc = U::comb(acc, U::ld(in_s + (size_t)root * nu + u));
        return acc;
    }
    if (row == p.q) acc = U::comb(acc, U::ld(in_s + (size_t)root * nu + u));
    for (uint32_t sp = 0; sp < mj; ++sp)
        if (sp != sstar && ((mask >> sp) & 1u)) acc = U::comb(acc, U::ld(in_s + (size_t)renumber(vbase + sp, root) * nu + u));
    return acc;
}

// The root's own data after up-correction when it is a member of the short last group whose other members all
// lie outside the selected subtree.
template <typename U>
__device__ __forceinline__ typename U::V fold_root_unit(const Params& p, uint32_t root, const uint32_t* inc,
                                                         const typename U::V* in_s, uint32_t nu, uint32_t u) {
    typename U::V acc = U::ld(in_s + (size_t)root * nu + u);
    if (p.r) {
        const uint32_t vbase = p.q * p.m + 1, mask = extract_bits(inc, vbase, p.r);
        for (uint32_t i = 0; i < p.r; ++i) {
            const uint32_t sp = p.pdesc ? p.r - 1 - i : i;
            if ((mask >> sp) & 1u) acc = U::comb(acc, U::ld(in_s + (size_t)renumber(vbase + sp, root) * nu + u));
        }
    }
    return acc;
}

static __device__ void write_status(const Params& p, uint64_t s, const Ctx* cx) {
    uint32_t* st = p.status + s * FTC_STATUS_WORDS;
    const bool ok = cx->code == FTC_ST_OK;
    st[0] = cx->code | ((ok ? cx->sstar : 0xFFu) << 8) | (cx->attempts << 16);
    st[1] = ok ? p.P - cx->npre - cx->nexcl : 0u;
    st[2] = ok ? cx->inop_incl : 0u;
    st[3] = (ok && p.is_allreduce) ? cx->holders : 0u;
}

template <typename T, int OP, bool VEC>
__global__ void __launch_bounds__(256, VEC ? 0 : 8) generic_kernel(Params p) {
    using U = Unit<T, OP, VEC>;
    using V = typename U::V;
    extern __shared__ uint32_t smem[];
    Ctx* cx = reinterpret_cast<Ctx*>(smem);
    uint32_t* pf = smem + sizeof(Ctx) / 4;
    uint32_t* inc = pf + p.W + 1;
    uint32_t* unr = inc + p.W + 1;
    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    const uint32_t nu = VEC ? p.kbytes / 16 : p.k;                 // units per process vector
    // a power-of-two group of `upw` lanes walks the units of one row; 32/upw rows per warp, no divisions
    uint32_t upw_log2 = 0; while ((1u << upw_log2) < nu && upw_log2 < 5) ++upw_log2;
    const uint32_t upw = 1u << upw_log2, rows_per_pass = nt >> upw_log2, r0 = tid >> upw_log2, u0 = tid & (upw - 1);
    V* ws = reinterpret_cast<V*>(p.ws) + (size_t)blockIdx.x * p.Gmax * nu;

    for (uint64_t s = blockIdx.x; s < p.S; s += gridDim.x) {
        decode_scenario(p, s, cx, pf, inc);
        V* out_s = reinterpret_cast<V*>(p.out) + s * nu;
        if (cx->code != FTC_ST_OK) {
            for (uint32_t u = tid; u < nu; u += nt) out_s[u] = U::zero();
            if (tid == 0) write_status(p, s, cx);
            __syncthreads();
            continue;
        }
        if (p.is_allreduce) count_holders(p, cx, pf, unr);
        const V* in_s = reinterpret_cast<const V*>(p.in) + s * (size_t)p.P * nu;
        const uint32_t G = cx->G, root = cx->root, sstar = cx->sstar;
        // tree phase (Algorithm "reduce_non_root"): data <- data (op) child 1 (op) child 2 ..., leaves first.
        // The rows of the last level are leaves: their value is their group's fold, which the thread that handles
        // the parent computes on the spot (most rows of a heap are leaves, so most values never touch the workspace).
        if (p.arity == 1) {
            // binomial subtrees: the nodes of one depth are scattered over the index range, so every level looks at
            // all rows and takes those with that many set bits; children of j are j + 2^i below j's lowest set bit
            for (int lvl = (int)p.H - 1; lvl >= 0; --lvl) {
                auto node = [&](uint32_t j, uint32_t u) {
                    V v = fold_group_unit<U>(p, root, sstar, inc, in_s, nu, j, u);
                    for (uint64_t bit = 1; (j == 0 || bit < (j & (0u - j))) && j + bit < G; bit <<= 1)
                        v = U::comb(v, ws[(size_t)(j + bit) * nu + u]);
                    ws[(size_t)j * nu + u] = v;
                };
                if (VEC) {
                    for (uint32_t j = r0; j < G; j += rows_per_pass)
                        if (__popc(j) == lvl) for (uint32_t u = u0; u < nu; u += upw) node(j, u);
                } else {
                    for (uint32_t x = tid; x < G * nu; x += nt)
                        if (__popc(x / nu) == lvl) node(x / nu, x % nu);
                }
                __syncthreads();
            }
        } else {
            const int last = (int)heap_level(p.arity, G - 1);
            const uint32_t leaf_lo = (uint32_t)heap_level_start(p.arity, last);
            for (int lvl = last > 0 ? last - 1 : 0; lvl >= 0; --lvl) {
                const uint32_t lo = (uint32_t)heap_level_start(p.arity, lvl);
                const uint32_t hi = (uint32_t)min(heap_level_start(p.arity, lvl + 1), (uint64_t)G);
                auto node = [&](uint32_t j, uint32_t u) {
                    const uint64_t c0 = (uint64_t)p.arity * j + 1, c1 = min(c0 + p.arity, (uint64_t)G);
                    V v = fold_group_unit<U>(p, root, sstar, inc, in_s, nu, j, u);
                    for (uint64_t c = c0; c < c1; ++c)
                        v = U::comb(v, (last > 0 && c >= leaf_lo) ? fold_group_unit<U>(p, root, sstar, inc, in_s, nu, (uint32_t)c, u)
                                                                  : ws[(size_t)c * nu + u]);
                    ws[(size_t)j * nu + u] = v;
                };
                if (VEC) {
                    for (uint32_t j = lo + r0; j < hi; j += rows_per_pass)
                        for (uint32_t u = u0; u < nu; u += upw) node(j, u);
                } else {
                    // single elements: every thread takes the next (row, element) pair of the level, whatever k is
                    for (uint32_t x = tid; x < (hi - lo) * nu; x += nt) node(lo + x / nu, x % nu);
                }
                __syncthreads();
            }
        }
        // root (Algorithm "reduce_root"): the selected child's value, combined with the root's own data unless the
        // child's subtree already holds it (it does iff it contains a member of the root's group)
        for (uint32_t u = tid; u < nu; u += nt) {
            V recv = ws[u];
            out_s[u] = sstar < p.r ? recv : U::comb(fold_root_unit<U>(p, root, inc, in_s, nu, u), recv);
        }
        if (tid == 0) write_status(p, s, cx);
        __syncthreads();
    }
}

size_t generic_smem_bytes(const Params& p) { return sizeof(Ctx) + 3 * (size_t)(p.W + 1) * 4; }

uint32_t generic_grid(const Params& p, int sm_count) {
    uint64_t g = (uint64_t)sm_count * 8;
    return (uint32_t)(p.S < g ? p.S : g);
}

// Threads of a block of the general reduce kernel: a level of the widest subtree keeps at most Gmax rows x the lanes
// that walk a row busy, so scenarios of a few dozen processes get one warp (cheap barriers, 32 blocks per SM) and
// large ones the full 256 threads.
uint32_t generic_reduce_threads(const Params& p) {
    const uint32_t nu = p.kbytes % 16 == 0 ? p.kbytes / 16 : p.k;
    uint32_t upw = 1; while (upw < nu && upw < 32) upw <<= 1;
    const uint64_t busy = (uint64_t)p.Gmax * upw;
    uint32_t t = 32; while (t < 256 && t < busy) t <<= 1;
    return t;
}

uint32_t generic_reduce_grid(const Params& p, int sm_count) {
    const uint32_t per_sm = 2048 / generic_reduce_threads(p) > 32 ? 32 : 2048 / generic_reduce_threads(p);
    uint64_t g = (uint64_t)sm_count * per_sm;
    return (uint32_t)(p.S < g ? p.S : g);
}

template <typename T, int OP, bool VEC>
static cudaError_t launch_generic_v(const Params& p, uint32_t grid, cudaStream_t st) {
    size_t smem = generic_smem_bytes(p);
    if (p.grid_query) { *p.grid_query = grid; return cudaSuccess; }
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(generic_kernel<T, OP, VEC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    generic_kernel<T, OP, VEC><<<grid, generic_reduce_threads(p), smem, st>>>(p);
    return cudaGetLastError();
}

// 16-byte units when the process vectors are a whole number of them (inputs, results and workspace are 16-byte aligned)
template <typename T, int OP>
static cudaError_t launch_generic_t(const Params& p, int sm_count, cudaStream_t st) {
    return p.kbytes % 16 == 0 ? launch_generic_v<T, OP, true>(p, generic_reduce_grid(p, sm_count), st)
                              : launch_generic_v<T, OP, false>(p, generic_reduce_grid(p, sm_count), st);
}

cudaError_t launch_generic(const Params& p, int tsel, int sm_count, cudaStream_t st) {
    switch (tsel) {
    case TS_U32_SUM: return launch_generic_t<uint32_t, OP_SUM>(p, sm_count, st);
    case TS_I32_MAX: return launch_generic_t<int32_t, OP_MAX>(p, sm_count, st);
    case TS_U32_XOR: return launch_generic_t<uint32_t, OP_XOR>(p, sm_count, st);
    case TS_U64_SUM: return launch_generic_t<unsigned long long, OP_SUM>(p, sm_count, st);
    case TS_I64_MAX: return launch_generic_t<long long, OP_MAX>(p, sm_count, st);
    case TS_U64_MAX: return launch_generic_t<unsigned long long, OP_MAX>(p, sm_count, st);
    case TS_U64_XOR: return launch_generic_t<unsigned long long, OP_XOR>(p, sm_count, st);
    case TS_F32_SUM: return launch_generic_t<float, OP_SUM>(p, sm_count, st);
    }
    return cudaErrorInvalidValue;
}

// ---------------------------------------------------------------------------------------------------------
// Built-in scratch for callers that cannot hand the library a workspace.
// The array lives in device memory of every GPU that loads the library, from load to process exit. Its name is
// only meaningful to device code; host code must ask the runtime for its device address (below) and may never
// pass the symbol itself to a kernel.
// ---------------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[FTC_NOALLOC_SCRATCH_BYTES];

static std::mutex g_static_mutex;
static void* g_static_ptr[64];          // device address of g_static_scratch, per device ordinal
static bool g_static_ready[64];

// First call on a device: looks the array's device address up (with that device current). Later calls reuse it.
static cudaError_t static_scratch_address(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ready[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        if (!ptr) return cudaErrorInvalidSymbol;
        g_static_ptr[dev] = ptr; g_static_ready[dev] = true;
    }
    *out = g_static_ptr[dev];
    return cudaSuccess;
}

template <typename T, int OP>
static cudaError_t launch_static_t(const Params& p, uint32_t grid, cudaStream_t st) {
    return p.kbytes % 16 == 0 ? launch_generic_v<T, OP, true>(p, grid, st) : launch_generic_v<T, OP, false>(p, grid, st);
}

// The general kernel with its node values in the built-in scratch: as many blocks as slices fit (at most the
// usual grid). *too_large is set when not even one block's slice fits.
cudaError_t launch_generic_static(Params p, int tsel, int sm_count, cudaStream_t st, bool* too_large) {
    const size_t slice = (size_t)p.Gmax * p.kbytes;
    *too_large = slice > (size_t)FTC_NOALLOC_SCRATCH_BYTES;
    if (*too_large) return cudaSuccess;
    void* ptr = nullptr;
    cudaError_t e = static_scratch_address(&ptr);
    if (e != cudaSuccess) return e;
    uint32_t grid = generic_reduce_grid(p, sm_count);
    const size_t fit = (size_t)FTC_NOALLOC_SCRATCH_BYTES / slice;
    if (grid > fit) grid = (uint32_t)fit;
    p.ws = ptr;
    switch (tsel) {
    case TS_U32_SUM: return launch_static_t<uint32_t, OP_SUM>(p, grid, st);
    case TS_I32_MAX: return launch_static_t<int32_t, OP_MAX>(p, grid, st);
    case TS_U32_XOR: return launch_static_t<uint32_t, OP_XOR>(p, grid, st);
    case TS_U64_SUM: return launch_static_t<unsigned long long, OP_SUM>(p, grid, st);
    case TS_I64_MAX: return launch_static_t<long long, OP_MAX>(p, grid, st);
    case TS_U64_MAX: return launch_static_t<unsigned long long, OP_MAX>(p, grid, st);
    case TS_U64_XOR: return launch_static_t<unsigned long long, OP_XOR>(p, grid, st);
    case TS_F32_SUM: return launch_static_t<float, OP_SUM>(p, grid, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace ftc
