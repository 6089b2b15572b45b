// Expanded allreduce output: the value every holder has, written into the slot of each process that is alive at
// the end of the operation and holds it (allreduce semantics: the value is the same at all of them), zeros into
// the slots of all others. Runs after the main kernel, which leaves the compact results in the workspace.
#include "ftc_device.cuh"
#include "ftc_kernels.h"

namespace ftc {

template <typename V>
__global__ void __launch_bounds__(256) expand_kernel(Params p, const V* compact, V* out, uint32_t vecs) {
    extern __shared__ uint32_t smem[];
    Ctx* cx = reinterpret_cast<Ctx*>(smem);
    uint32_t* pf = smem + sizeof(Ctx) / 4;
    uint32_t* inc = pf + p.W + 1;
    uint32_t* unr = inc + p.W + 1;
    uint32_t* hold = unr + p.W + 1;
    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    V zero; memset(&zero, 0, sizeof zero);
    for (uint64_t s = blockIdx.x; s < p.S; s += gridDim.x) {
        decode_scenario(p, s, cx, pf, inc);
        const bool ok = cx->code == FTC_ST_OK;
        if (ok) count_holders(p, cx, pf, unr, hold);
        V* out_s = out + s * (uint64_t)p.P * vecs;
        const V* val = compact + s * (uint64_t)vecs;
        const uint64_t n = (uint64_t)p.P * vecs;
        for (uint64_t u = tid; u < n; u += nt) {
            const uint32_t proc = (uint32_t)(u / vecs), c = (uint32_t)(u % vecs);
            out_s[u] = (ok && test_bit(hold, proc)) ? val[c] : zero;
        }
        __syncthreads();
    }
}

size_t expand_smem_bytes(const Params& p) { return sizeof(Ctx) + 4 * (size_t)(p.W + 1) * 4; }

cudaError_t launch_expand(const Params& p, const void* compact, void* out, int sm_count, cudaStream_t st) {
    const size_t smem = expand_smem_bytes(p);
    const uint64_t cap = (uint64_t)sm_count * 8;
    const uint32_t grid = (uint32_t)(p.S < cap ? p.S : cap);
    cudaError_t e;
    if (p.kbytes % 16 == 0) {
        if (smem > 48 * 1024 && (e = cudaFuncSetAttribute(expand_kernel<uint4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        expand_kernel<uint4><<<grid, 256, smem, st>>>(p, static_cast<const uint4*>(compact), static_cast<uint4*>(out), p.kbytes / 16);
    } else {
        if (smem > 48 * 1024 && (e = cudaFuncSetAttribute(expand_kernel<uint32_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        expand_kernel<uint32_t><<<grid, 256, smem, st>>>(p, static_cast<const uint32_t*>(compact), static_cast<uint32_t*>(out), p.kbytes / 4);
    }
    return cudaGetLastError();
}

}  // namespace ftc
