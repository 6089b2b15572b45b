// Instantiations of the staged kernel for two (element type, reduction) pairs; split over several files so that
// they compile in parallel.
#include "ftc_staged_impl.cuh"

namespace ftc {

cudaError_t launch_staged_i64_max(const Params& p, int sm_count, int smem_optin, cudaStream_t st) {
    return launch_staged_x<long long, OP_MAX>(p, sm_count, smem_optin, st);
}

cudaError_t launch_staged_u64_max(const Params& p, int sm_count, int smem_optin, cudaStream_t st) {
    return launch_staged_x<unsigned long long, OP_MAX>(p, sm_count, smem_optin, st);
}

}  // namespace ftc
