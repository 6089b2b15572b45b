// Synthetic scenario inputs on the device: a stateless counter-based generator (splitmix64's output function on
// seed + GAMMA * (counter + 1)), one counter per element, so that the host can regenerate any scenario.
#include "ftc_kernels.h"

namespace ftc {

__device__ __forceinline__ uint64_t splitmix_out(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
__device__ __forceinline__ uint64_t hash_ctr(uint64_t seed, uint64_t ctr) {
    return splitmix_out(seed + 0x9E3779B97F4A7C15ull * (ctr + 1ull));
}

template <int KIND, typename T>
__global__ void fill_kernel(uint64_t seed, uint64_t first_elem, uint64_t n, T* out) {
    for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t lin = first_elem + i;
        if (KIND == 2) {
            // twelve uniforms on [0, 2^32) from six hashes; twice the centred sum (below 2^37) is rounded to float32 once
            // (to nearest), the scale to unit variance, 2^-33, is exact
            long long total = 0;
            for (int t = 0; t < 6; ++t) {
                uint64_t h = hash_ctr(seed, lin * 6ull + t);
                total += (long long)(h & 0xFFFFFFFFull) + (long long)(h >> 32);
            }
            long long centred = 2 * total - 12ll * ((1ll << 32) - 1);
            out[i] = (T)(__ll2float_rn(centred) * 1.1641532182693481e-10f);
        } else {
            uint64_t h = hash_ctr(seed, lin);
            if (KIND == 0) out[i] = (T)((long long)(h % ((1ull << 21) + 1ull)) - (1ll << 20));
            else if (KIND == 1) out[i] = (T)((long long)(h % ((1ull << 41) + 1ull)) - (1ll << 40));
            else if (KIND == 3) out[i] = (T)(int32_t)(uint32_t)(h & 0xFFFFFFFFull);
            else out[i] = (T)h;
        }
    }
}

cudaError_t launch_fill(uint32_t kind, uint64_t seed, uint64_t first, uint64_t S, uint32_t P, uint32_t k, void* out,
                        int sm_count, cudaStream_t st) {
    const uint64_t n = S * P * k, first_elem = first * P * k;
    if (n == 0) return cudaSuccess;
    uint64_t blocks = (n + 255) / 256, cap = (uint64_t)sm_count * 16;
    uint32_t grid = (uint32_t)(blocks < cap ? blocks : cap);
    switch (kind) {
    case 0: fill_kernel<0, int32_t><<<grid, 256, 0, st>>>(seed, first_elem, n, (int32_t*)out); break;
    case 1: fill_kernel<1, long long><<<grid, 256, 0, st>>>(seed, first_elem, n, (long long*)out); break;
    case 2: fill_kernel<2, float><<<grid, 256, 0, st>>>(seed, first_elem, n, (float*)out); break;
    case 3: fill_kernel<3, int32_t><<<grid, 256, 0, st>>>(seed, first_elem, n, (int32_t*)out); break;
    case 4: fill_kernel<4, unsigned long long><<<grid, 256, 0, st>>>(seed, first_elem, n, (unsigned long long*)out); break;
    default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace ftc
