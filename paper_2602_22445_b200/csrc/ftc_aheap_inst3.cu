// Level kernel (ftc_aheap_impl.cuh): the instantiations for uint64 max and uint64 xor.
#include "ftc_aheap_impl.cuh"

namespace ftc {

cudaError_t launch_aheap_b64(const Params& p, int tsel, int sm_count, int smem_optin, cudaStream_t st) {
    switch (tsel) {
    case TS_U64_MAX: return launch_aheap_t<unsigned long long, OP_MAX>(p, sm_count, smem_optin, st);
    case TS_U64_XOR: return launch_aheap_t<unsigned long long, OP_XOR>(p, sm_count, smem_optin, st);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace ftc
