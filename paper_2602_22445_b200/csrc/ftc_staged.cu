// Staged kernel, host side: shape check and dispatch to the per-type instantiations (ftc_staged_inst*.cu); the
// kernel itself is in ftc_staged_impl.cuh.
#include "ftc_staged_impl.cuh"

namespace ftc {

cudaError_t launch_staged_u32_sum(const Params& p, int sm_count, int smem_optin, cudaStream_t st);
cudaError_t launch_staged_i32_max(const Params& p, int sm_count, int smem_optin, cudaStream_t st);
cudaError_t launch_staged_u32_xor(const Params& p, int sm_count, int smem_optin, cudaStream_t st);
cudaError_t launch_staged_u64_sum(const Params& p, int sm_count, int smem_optin, cudaStream_t st);
cudaError_t launch_staged_i64_max(const Params& p, int sm_count, int smem_optin, cudaStream_t st);
cudaError_t launch_staged_u64_max(const Params& p, int sm_count, int smem_optin, cudaStream_t st);
cudaError_t launch_staged_u64_xor(const Params& p, int sm_count, int smem_optin, cudaStream_t st);
cudaError_t launch_staged_f32_sum(const Params& p, int sm_count, int smem_optin, cudaStream_t st);

bool staged_supported(Params& p, int smem_optin_bytes, int sm_count) {
    StagedGeom g;
    return staged_geometry(p, smem_optin_bytes, sm_count, staged_xl(p), g);
}

size_t staged_workspace_bytes(Params p, int smem_optin_bytes, int sm_count) {
    StagedGeom g;
    p.ws_bytes = ~0ull;                       // what would be used if the workspace were there
    if (!staged_geometry(p, smem_optin_bytes, sm_count, staged_xl(p), g) || !g.hv_global) return 0;
    return (size_t)sm_count * kHvGlobalBlocksPerSm * (size_t)g.hv_bytes;
}

const char* staged_variant(Params p, int tsel, int smem_optin_bytes, int sm_count, uint32_t* grid_cap_blocks_per_sm) {
    if (grid_cap_blocks_per_sm) *grid_cap_blocks_per_sm = 0;
    if (warp_supported(p, smem_optin_bytes)) return warp_lanes_per_scenario(p, smem_optin_bytes) == 16 ? "staged/warp-pair" : "staged/warp";
    StagedGeom g;
    const StagedVariant v = staged_plan(p, tsel == TS_F32_SUM, true, staged_xl(p), smem_optin_bytes, sm_count, g);
    if (grid_cap_blocks_per_sm) *grid_cap_blocks_per_sm = g.hv_global ? (uint32_t)kHvGlobalBlocksPerSm : 0u;
    return staged_variant_name(v);
}

cudaError_t launch_staged(const Params& p, int tsel, int sm_count, int smem_optin, cudaStream_t st) {
    if (warp_supported(p, smem_optin)) return launch_warp(p, tsel, sm_count, smem_optin, st);
    switch (tsel) {
    case TS_U32_SUM: return launch_staged_u32_sum(p, sm_count, smem_optin, st);
    case TS_I32_MAX: return launch_staged_i32_max(p, sm_count, smem_optin, st);
    case TS_U32_XOR: return launch_staged_u32_xor(p, sm_count, smem_optin, st);
    case TS_U64_SUM: return launch_staged_u64_sum(p, sm_count, smem_optin, st);
    case TS_I64_MAX: return launch_staged_i64_max(p, sm_count, smem_optin, st);
    case TS_U64_MAX: return launch_staged_u64_max(p, sm_count, smem_optin, st);
    case TS_U64_XOR: return launch_staged_u64_xor(p, sm_count, smem_optin, st);
    case TS_F32_SUM: return launch_staged_f32_sum(p, sm_count, smem_optin, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace ftc
