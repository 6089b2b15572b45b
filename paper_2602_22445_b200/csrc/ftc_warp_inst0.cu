// Warp kernel, host side and the instantiations for the 4-byte element types; those for the 8-byte types are in
// ftc_warp_inst1.cu (two files so that they compile in parallel). The kernel itself is in ftc_warp_impl.cuh.
#include "ftc_warp_impl.cuh"

namespace ftc {

cudaError_t launch_warp_u64(const Params& p, int tsel, int sm_count, int smem_optin, cudaStream_t st);

bool warp_supported(Params p, int smem_optin_bytes) {
    WarpGeom g; uint32_t XL;
    return warp_geometry(p, smem_optin_bytes, XL, g);
}

uint32_t warp_lanes_per_scenario(Params p, int smem_optin_bytes) {
    WarpGeom g; uint32_t XL;
    return warp_geometry(p, smem_optin_bytes, XL, g) ? g.lanes : 0u;
}

cudaError_t launch_warp(const Params& p, int tsel, int sm_count, int smem_optin, cudaStream_t st) {
    switch (tsel) {
    case TS_U32_SUM: return launch_warp_t<uint32_t, OP_SUM>(p, sm_count, smem_optin, st);
    case TS_I32_MAX: return launch_warp_t<int32_t, OP_MAX>(p, sm_count, smem_optin, st);
    case TS_U32_XOR: return launch_warp_t<uint32_t, OP_XOR>(p, sm_count, smem_optin, st);
    case TS_F32_SUM: return launch_warp_t<float, OP_SUM>(p, sm_count, smem_optin, st);
    default: return launch_warp_u64(p, tsel, sm_count, smem_optin, st);
    }
}

}  // namespace ftc
