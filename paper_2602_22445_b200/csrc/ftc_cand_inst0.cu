// Every root child's delivery on the staged tiles (ftc_cand_impl.cuh): host side and the instantiations for the
// 4-byte integer types; those for the 8-byte types are in ftc_cand_inst1.cu.
#include "ftc_cand_impl.cuh"

namespace ftc {

cudaError_t launch_cand_u64(const Params& p, int tsel, void* cand, uint32_t* info, int sm_count, int smem_optin, cudaStream_t st, uint32_t* grid_out);

// Shapes the staged tiles cover (float32: with one heap array per root child in shared memory); everything else takes
// the general kernel.
bool cand_fast_supported(Params p, int tsel, int smem_optin_bytes, int sm_count) {
    if (p.flags & FTC_KERNEL_GENERIC) return false;
    CandGeom cg; uint32_t XL;
    return cand_geometry(p, smem_optin_bytes, sm_count, XL, cg, tsel == TS_F32_SUM);
}

size_t cand_fast_workspace_bytes(Params p, int tsel, int smem_optin_bytes, int sm_count) {
    CandGeom cg; uint32_t XL, blocks = 0;
    if (!cand_geometry(p, smem_optin_bytes, sm_count, XL, cg, tsel == TS_F32_SUM)) return 0;
    if (launch_cand_fast(p, tsel, nullptr, nullptr, sm_count, smem_optin_bytes, nullptr, &blocks) != cudaSuccess) blocks = (uint32_t)sm_count * 2;
    return (size_t)blocks * cg.slice_bytes;
}

cudaError_t launch_cand_fast(const Params& p, int tsel, void* cand, uint32_t* info, int sm_count, int smem_optin, cudaStream_t st, uint32_t* grid_out) {
    switch (tsel) {
    case TS_U32_SUM: return launch_cand_t<uint32_t, OP_SUM>(p, cand, info, sm_count, smem_optin, st, grid_out);
    case TS_I32_MAX: return launch_cand_t<int32_t, OP_MAX>(p, cand, info, sm_count, smem_optin, st, grid_out);
    case TS_U32_XOR: return launch_cand_t<uint32_t, OP_XOR>(p, cand, info, sm_count, smem_optin, st, grid_out);
    case TS_F32_SUM: return launch_cand_t<float, OP_SUM>(p, cand, info, sm_count, smem_optin, st, grid_out);
    default: return launch_cand_u64(p, tsel, cand, info, sm_count, smem_optin, st, grid_out);
    }
}

}  // namespace ftc
