// Level kernel (ftc_aheap_impl.cuh): the instantiations for uint32 xor and float32 sum.
#include "ftc_aheap_impl.cuh"

namespace ftc {

cudaError_t launch_aheap_b32(const Params& p, int tsel, int sm_count, int smem_optin, cudaStream_t st) {
    switch (tsel) {
    case TS_U32_XOR: return launch_aheap_t<uint32_t, OP_XOR>(p, sm_count, smem_optin, st);
    case TS_F32_SUM: return launch_aheap_t<float, OP_SUM>(p, sm_count, smem_optin, st);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace ftc
