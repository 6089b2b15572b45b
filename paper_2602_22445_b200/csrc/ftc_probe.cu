// Read-bandwidth probe (a measurement aid, not part of the method): streams a device buffer once and does nothing
// else, in the two ways the batch kernels read their inputs -- 128-bit loads into registers, and asynchronous bulk
// copies into shared memory. The time of one launch over the same buffer a batch call reads is the ceiling a
// read-only kernel can reach on this GPU, which a copy benchmark (reads and writes) does not show.
#include "ftc_device.cuh"
#include "ftc_kernels.h"

namespace ftc {

// mode 0: every thread folds 16-byte words with xor, eight independent loads in flight per thread.
__global__ void __launch_bounds__(512, 2) probe_loads_kernel(const uint4* __restrict__ buf, uint64_t n16, unsigned long long* sink) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint4 a = make_uint4(0, 0, 0, 0);
    for (; i + 7 * stride < n16; i += 8 * stride) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = __ldg(buf + i + u * stride);
#pragma unroll
        for (int u = 0; u < 8; ++u) { a.x ^= v[u].x; a.y ^= v[u].y; a.z ^= v[u].z; a.w ^= v[u].w; }
    }
    for (; i < n16; i += stride) { const uint4 v = __ldg(buf + i); a.x ^= v.x; a.y ^= v.y; a.z ^= v.z; a.w ^= v.w; }
    uint32_t x = a.x ^ a.y ^ a.z ^ a.w;
    x = __reduce_xor_sync(0xFFFFFFFFu, x);
    if ((threadIdx.x & 31) == 0 && x == 0x9E3779B9u) atomicAdd(sink, 1ull);      // keeps the loads alive; almost never taken
}

// mode 1: every warp keeps kProbeBufs bulk copies of kProbeChunk bytes in flight into its own shared-memory buffers
// (global -> shared, completion on an mbarrier) and never looks at the bytes.
constexpr uint32_t kProbeChunk = 16 * 1024, kProbeBufs = 3, kProbeWarps = 4, kProbeTries = 1u << 22;

__global__ void __launch_bounds__(kProbeWarps * 32, 1) probe_bulk_kernel(const char* __restrict__ buf, uint64_t nchunks, unsigned long long* sink) {
    extern __shared__ __align__(128) unsigned char psm[];
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    unsigned char* mine = psm + 128 + (size_t)wid * kProbeBufs * kProbeChunk;
    const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(psm) + wid * kProbeBufs * 8;
    if (lane < kProbeBufs) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar0 + lane * 8), "r"(1) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    const uint64_t nw = (uint64_t)gridDim.x * kProbeWarps, w0 = (uint64_t)blockIdx.x * kProbeWarps + wid;
    uint64_t next = w0;                      // chunk of the next copy to issue
    uint32_t issued = 0, done = 0, gaveup = 0;
    auto issue = [&]() {
        if (next >= nchunks) return;
        const uint32_t b = issued % kProbeBufs, bar = bar0 + b * 8;
        if (lane == 0) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kProbeChunk) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"((uint32_t)__cvta_generic_to_shared(mine + (size_t)b * kProbeChunk)), "l"(buf + next * kProbeChunk),
                           "r"(kProbeChunk), "r"(bar) : "memory");
        }
        ++issued; next += nw;
    };
    for (uint32_t i = 0; i < kProbeBufs; ++i) issue();
    while (done < issued) {
        const uint32_t b = done % kProbeBufs, bar = bar0 + b * 8, parity = (done / kProbeBufs) & 1u;
        uint32_t ok = 0;
        for (uint32_t t = 0; t < kProbeTries && !ok; ++t)
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) { gaveup = 1; break; }      // bounded: report and stop issuing; the copies in flight get one more wait below
        ++done;
        __syncwarp();
        issue();
    }
    if (gaveup) {
        for (uint32_t d = done; d < issued; ++d) {
            const uint32_t bar = bar0 + (d % kProbeBufs) * 8, parity = (d / kProbeBufs) & 1u;
            uint32_t ok = 0;
            for (uint32_t t = 0; t < kProbeTries && !ok; ++t)
                asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                             : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        }
        if (lane == 0) atomicAdd(sink + 1, 1ull);
    }
}

cudaError_t launch_probe(uint32_t mode, const void* buf, uint64_t bytes, unsigned long long* sink, int sm_count, cudaStream_t st) {
    if (mode == 0) {
        probe_loads_kernel<<<sm_count * 2, 512, 0, st>>>(static_cast<const uint4*>(buf), bytes / 16, sink);
        return cudaGetLastError();
    }
    const size_t smem = 128 + (size_t)kProbeWarps * kProbeBufs * kProbeChunk;
    cudaError_t e = cudaFuncSetAttribute(probe_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    probe_bulk_kernel<<<sm_count, kProbeWarps * 32, smem, st>>>(static_cast<const char*>(buf), bytes / kProbeChunk, sink);
    return cudaGetLastError();
}

}  // namespace ftc
