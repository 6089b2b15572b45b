// Every root child's delivery on the staged tiles: the instantiations for the 8-byte types (see ftc_cand_inst0.cu).
#include "ftc_cand_impl.cuh"

namespace ftc {

cudaError_t launch_cand_u64(const Params& p, int tsel, void* cand, uint32_t* info, int sm_count, int smem_optin, cudaStream_t st, uint32_t* grid_out) {
    switch (tsel) {
    case TS_U64_SUM: return launch_cand_t<unsigned long long, OP_SUM>(p, cand, info, sm_count, smem_optin, st, grid_out);
    case TS_I64_MAX: return launch_cand_t<long long, OP_MAX>(p, cand, info, sm_count, smem_optin, st, grid_out);
    case TS_U64_MAX: return launch_cand_t<unsigned long long, OP_MAX>(p, cand, info, sm_count, smem_optin, st, grid_out);
    case TS_U64_XOR: return launch_cand_t<unsigned long long, OP_XOR>(p, cand, info, sm_count, smem_optin, st, grid_out);
    }
    return cudaErrorInvalidValue;
}

}  // namespace ftc
