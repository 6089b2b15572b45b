// Level kernel for a-ary heaps and binomial trees (ftc_aheap_impl.cuh): host side and the instantiations for uint32 sum and
// int32 max; the other types are in ftc_aheap_inst1.cu .. ftc_aheap_inst3.cu (split for parallel compilation).
#include "ftc_aheap_impl.cuh"

namespace ftc {

bool aheap_supported(Params p, int smem_optin_bytes) {
    if (p.flags & (FTC_KERNEL_GENERIC | FTC_KERNEL_DIRECT)) return false;
    AheapGeom g;
    return aheap_geometry(p, smem_optin_bytes, g);
}

cudaError_t launch_aheap(const Params& p, int tsel, int sm_count, int smem_optin, cudaStream_t st) {
    switch (tsel) {
    case TS_U32_SUM: return launch_aheap_t<uint32_t, OP_SUM>(p, sm_count, smem_optin, st);
    case TS_I32_MAX: return launch_aheap_t<int32_t, OP_MAX>(p, sm_count, smem_optin, st);
    case TS_U32_XOR: case TS_F32_SUM: return launch_aheap_b32(p, tsel, sm_count, smem_optin, st);
    case TS_U64_SUM: case TS_I64_MAX: return launch_aheap_u64(p, tsel, sm_count, smem_optin, st);
    default: return launch_aheap_b64(p, tsel, sm_count, smem_optin, st);
    }
}

}  // namespace ftc
