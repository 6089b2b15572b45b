// Level kernel (ftc_aheap_impl.cuh): the instantiations for uint64 sum and int64 max.
#include "ftc_aheap_impl.cuh"

namespace ftc {

cudaError_t launch_aheap_u64(const Params& p, int tsel, int sm_count, int smem_optin, cudaStream_t st) {
    switch (tsel) {
    case TS_U64_SUM: return launch_aheap_t<unsigned long long, OP_SUM>(p, sm_count, smem_optin, st);
    case TS_I64_MAX: return launch_aheap_t<long long, OP_MAX>(p, sm_count, smem_optin, st);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace ftc
