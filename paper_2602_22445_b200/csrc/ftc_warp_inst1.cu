// Warp kernel: the instantiations for the 8-byte element types (see ftc_warp_inst0.cu).
#include "ftc_warp_impl.cuh"

namespace ftc {

cudaError_t launch_warp_u64(const Params& p, int tsel, int sm_count, int smem_optin, cudaStream_t st) {
    switch (tsel) {
    case TS_U64_SUM: return launch_warp_t<unsigned long long, OP_SUM>(p, sm_count, smem_optin, st);
    case TS_I64_MAX: return launch_warp_t<long long, OP_MAX>(p, sm_count, smem_optin, st);
    case TS_U64_MAX: return launch_warp_t<unsigned long long, OP_MAX>(p, sm_count, smem_optin, st);
    case TS_U64_XOR: return launch_warp_t<unsigned long long, OP_XOR>(p, sm_count, smem_optin, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace ftc
