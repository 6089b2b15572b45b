// General kernel: any P, f, k. One block per scenario (grid-stride), the selected subtree is evaluated level by
// level from the leaves, node values pass through a per-block slice of the global workspace.
#include <mutex>
#include "ftc_device.cuh"
#include "ftc_kernels.h"

namespace ftc {

// Value of group `row` as the selected subtree's member sees it after up-correction (Algorithm "Up-correction"):
// own input first, then the partners whose message arrived, in ascending rank (the root first in the short group).
template <typename T, int OP>
__device__ __forceinline__ T fold_group_scalar(const Params& p, const Ctx* cx, const uint32_t* inc, const T* in_s,
                                               uint32_t row, uint32_t e) {
    const uint32_t root = cx->root, sstar = cx->sstar;
    const uint32_t mj = row < p.q ? p.m : p.r, vbase = row * p.m + 1;
    const uint32_t mask = extract_bits(inc, vbase, mj);
    T acc = in_s[(size_t)renumber(vbase + sstar, root) * p.k + e];
    if (row == p.q) acc = Comb<T, OP>::f(acc, in_s[(size_t)root * p.k + e]);
    for (uint32_t sp = 0; sp < mj; ++sp)
        if (sp != sstar && ((mask >> sp) & 1u)) acc = Comb<T, OP>::f(acc, in_s[(size_t)renumber(vbase + sp, root) * p.k + e]);
    return acc;
}

// The root's own data after up-correction when it is a member of the short last group whose other members all
// lie outside the selected subtree.
template <typename T, int OP>
__device__ __forceinline__ T fold_root_scalar(const Params& p, const Ctx* cx, const uint32_t* inc, const T* in_s, uint32_t e) {
    const uint32_t root = cx->root;
    T acc = in_s[(size_t)root * p.k + e];
    if (p.r) {
        const uint32_t vbase = p.q * p.m + 1, mask = extract_bits(inc, vbase, p.r);
        for (uint32_t sp = 0; sp < p.r; ++sp)
            if ((mask >> sp) & 1u) acc = Comb<T, OP>::f(acc, in_s[(size_t)renumber(vbase + sp, root) * p.k + e]);
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

template <typename T, int OP>
__global__ void __launch_bounds__(256) generic_kernel(Params p) {
    extern __shared__ uint32_t smem[];
    Ctx* cx = reinterpret_cast<Ctx*>(smem);
    uint32_t* pf = smem + sizeof(Ctx) / 4;
    uint32_t* inc = pf + p.W + 1;
    uint32_t* unr = inc + p.W + 1;
    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    T* ws = reinterpret_cast<T*>(p.ws) + (size_t)blockIdx.x * p.Gmax * p.k;

    for (uint64_t s = blockIdx.x; s < p.S; s += gridDim.x) {
        decode_scenario(p, s, cx, pf, inc);
        T* out_s = reinterpret_cast<T*>(p.out) + s * p.k;
        if (cx->code != FTC_ST_OK) {
            for (uint32_t e = tid; e < p.k; e += nt) out_s[e] = T(0);
            if (tid == 0) write_status(p, s, cx);
            __syncthreads();
            continue;
        }
        if (p.is_allreduce) count_holders(p, cx, pf, unr);
        const T* in_s = reinterpret_cast<const T*>(p.in) + s * (size_t)p.P * p.k;
        const uint32_t G = cx->G;
        // tree phase (Algorithm "reduce_non_root"): data <- data (op) child 1 (op) child 2 ..., leaves first
        for (int lvl = (int)heap_level(p.arity, G - 1); lvl >= 0; --lvl) {
            const uint32_t lo = (uint32_t)heap_level_start(p.arity, lvl);
            const uint32_t hi = (uint32_t)min(heap_level_start(p.arity, lvl + 1), (uint64_t)G);
            for (uint32_t u = tid; u < (hi - lo) * p.k; u += nt) {
                const uint32_t j = lo + u / p.k, e = u % p.k;
                T v = fold_group_scalar<T, OP>(p, cx, inc, in_s, j, e);
                for (uint64_t c = (uint64_t)p.arity * j + 1; c <= (uint64_t)p.arity * j + p.arity && c < G; ++c)
                    v = Comb<T, OP>::f(v, ws[(size_t)c * p.k + e]);
                ws[(size_t)j * p.k + e] = v;
            }
            __syncthreads();
        }
        // root (Algorithm "reduce_root"): the selected child's value, combined with the root's own data unless the
        // child's subtree already holds it (it does iff it contains a member of the root's group)
        for (uint32_t e = tid; e < p.k; e += nt) {
            T recv = ws[e];
            out_s[e] = cx->sstar < p.r ? recv : Comb<T, OP>::f(fold_root_scalar<T, OP>(p, cx, inc, in_s, e), recv);
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

template <typename T, int OP>
static cudaError_t launch_generic_t(const Params& p, int sm_count, cudaStream_t st) {
    size_t smem = generic_smem_bytes(p);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(generic_kernel<T, OP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    generic_kernel<T, OP><<<generic_grid(p, sm_count), 256, smem, st>>>(p);
    return cudaGetLastError();
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
    size_t smem = generic_smem_bytes(p);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(generic_kernel<T, OP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    generic_kernel<T, OP><<<grid, 256, smem, st>>>(p);
    return cudaGetLastError();
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
    uint32_t grid = generic_grid(p, sm_count);
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
