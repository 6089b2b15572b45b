// Instantiations of the staged kernel for two (element type, reduction) pairs; split over several files so that
// they compile in parallel.
#include "ftc_staged_impl.cuh"

namespace ftc {

cudaError_t launch_staged_u32_xor(const Params& p, int sm_count, int smem_optin, cudaStream_t st) {
    return launch_staged_x<uint32_t, OP_XOR>(p, sm_count, smem_optin, st);
}

cudaError_t launch_staged_u64_sum(const Params& p, int sm_count, int smem_optin, cudaStream_t st) {
    return launch_staged_x<unsigned long long, OP_SUM>(p, sm_count, smem_optin, st);
}

}  // namespace ftc
