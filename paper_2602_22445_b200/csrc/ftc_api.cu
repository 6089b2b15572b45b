// extern "C" boundary: argument checks, schedule constants, kernel choice, host-buffer variants.
#include <cstring>
#include "ftc_device.cuh"
#include "ftc_kernels.h"

namespace ftc {


// level of index j in an a-ary heap (level l holds a^l indices)
static uint32_t heap_level_h(uint32_t arity, uint32_t j) {
    uint32_t l = 0; uint64_t start = 0, width = 1;
    while (j >= start + width) { start += width; width *= arity; ++l; }
    return l;
}
// children per node from the descriptor's flags: 0 = not given = binary; 1 and values above FTC_MAX_ARITY are invalid
// (internally 1 stands for the binomial tree, which FTC_TREE_BINOMIAL asks for)
static bool tree_arity(uint32_t flags, uint32_t& arity) {
    const uint32_t a = (flags >> 16) & 0xFFu;
    if (flags & FTC_TREE_BINOMIAL) { arity = 1u; return a == 0; }
    arity = a ? a : 2u;
    return a != 1 && a <= FTC_MAX_ARITY;
}
// deepest level among the local indices 0..G-1 of a subtree
static uint32_t deepest_level_h(uint32_t arity, uint32_t G) {
    if (arity != 1) return heap_level_h(arity, G - 1);
    const uint32_t M = G - 1;                 // most set bits of any index <= M
    uint32_t b = 0; while (b < 32 && (M >> b)) ++b;
    return (b && M == (uint32_t)((1ull << b) - 1)) ? b : (b ? b - 1 : 0);
}

static uint32_t elem_size(uint32_t dtype) { return (dtype == FTC_I32 || dtype == FTC_F32) ? 4u : 8u; }

static int type_select(uint32_t dtype, uint32_t op) {
    switch (dtype) {
    case FTC_I32: return op == FTC_SUM ? TS_U32_SUM : op == FTC_MAX ? TS_I32_MAX : op == FTC_XOR ? TS_U32_XOR : -1;
    case FTC_I64: return op == FTC_SUM ? TS_U64_SUM : op == FTC_MAX ? TS_I64_MAX : op == FTC_XOR ? TS_U64_XOR : -1;
    case FTC_U64: return op == FTC_SUM ? TS_U64_SUM : op == FTC_MAX ? TS_U64_MAX : op == FTC_XOR ? TS_U64_XOR : -1;
    case FTC_F32: return op == FTC_SUM ? TS_F32_SUM : -1;
    }
    return -1;
}

// Descriptor checks and schedule constants. Returns FTC_OK or the error.
static int fill_params(const ftc_desc_t* d, uint64_t S, int is_allreduce, Params& p) {
    if (!d) return FTC_EINVAL;
    if (d->dtype > FTC_F32 || d->op > FTC_XOR) return FTC_EUNSUPPORTED;
    if (type_select(d->dtype, d->op) < 0) return FTC_EUNSUPPORTED;
    if (d->k == 0 || d->f > FTC_MAX_F || d->P < d->f + 2 || d->max_inop > FTC_MAX_INOP) return FTC_EINVAL;
    if (d->root >= 0 && (uint32_t)d->root >= d->P) return FTC_EINVAL;
    if ((uint64_t)d->k * elem_size(d->dtype) > 0x7FFFFFFFull || (uint64_t)d->P * d->k > (1ull << 40)) return FTC_EINVAL;
    uint32_t arity;
    if (!tree_arity(d->flags, arity)) return FTC_EINVAL;
    std::memset(&p, 0, sizeof p);
    p.arity = arity;
    p.pdesc = (d->flags & FTC_PARTNERS_DESCENDING) ? 1u : 0u;
    p.P = d->P; p.f = d->f; p.m = d->f + 1; p.k = d->k; p.W = (d->P + 31) / 32;
    p.q = (d->P - 1) / p.m; p.r = (d->P - 1) % p.m;
    p.m_magic = (uint32_t)((0x100000000ull + p.m - 1) / p.m);
    p.Gmax = p.q + (p.r ? 1u : 0u);
    p.H = 1 + deepest_level_h(p.arity, p.Gmax);
    p.Rred = p.f + p.H; p.Ratt = 2 * p.Rred;
    p.max_inop = d->max_inop; p.flags = d->flags; p.root = d->root; p.is_allreduce = is_allreduce;
    p.kbytes = d->k * elem_size(d->dtype);
    p.S = S;
    return FTC_OK;
}

struct DeviceInfo { int sm_count; int smem_optin; };
static int device_info(DeviceInfo& di) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FTC_ECUDA;
    if (cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return FTC_ECUDA;
    if (cudaDeviceGetAttribute(&di.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return FTC_ECUDA;
    return FTC_OK;
}

// B200 figures, used where no device can be asked (sizing queries on a machine without a GPU).
static const DeviceInfo kB200 = {148, 232448};

enum KernelKind { K_GENERIC = 0, K_TILED = 1, K_STAGED = 2, K_LEVELS = 3 };
static KernelKind pick_kernel(Params& p, const DeviceInfo& di) {
    if (p.flags & FTC_KERNEL_GENERIC) return K_GENERIC;
    if (p.arity != 2 || (p.flags & FTC_KERNEL_LEVELS))                       // heaps of any arity, binomial trees: tiles evaluated level by level
        if (aheap_supported(p, di.smem_optin)) return K_LEVELS;
    if (p.arity != 2) return K_GENERIC;                                      // the register-tiled kernels are built on the binary heap
    if (!(p.flags & FTC_KERNEL_DIRECT) && staged_supported(p, di.smem_optin, di.sm_count)) return K_STAGED;
    if (tiled_supported(p, di.smem_optin)) return K_TILED;
    // vectors that are not a power-of-two number of 16-byte chunks: the register tiles cannot hold them, the level kernel can
    const uint32_t chunks = p.kbytes / 16;
    if (p.kbytes % 16 == 0 && (chunks & (chunks - 1)) && !(p.flags & FTC_KERNEL_DIRECT) && aheap_supported(p, di.smem_optin)) return K_LEVELS;
    return K_GENERIC;
}

static size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

// Bytes at the front of the workspace that hold the compact results while the expanded output is produced.
static size_t compact_area(const Params& p) {
    return (p.flags & FTC_OUT_EXPANDED) ? up256((size_t)p.S * p.kbytes) : 0;
}

// Workspace that lets the batch calls run at their best: the general kernel needs its slices; the staged kernel
// uses one for large heap arrays (without it the shape runs more slowly, or on another kernel).
static size_t workspace_for(Params& p, const DeviceInfo& di) {
    size_t need = compact_area(p);
    p.ws_bytes = ~0ull;
    const KernelKind kind = pick_kernel(p, di);
    if (kind == K_GENERIC) need += (size_t)generic_reduce_grid(p, di.sm_count) * p.Gmax * p.kbytes;
    else if (kind == K_STAGED) need += staged_workspace_bytes(p, di.smem_optin, di.sm_count);
    return need;
}

static bool aligned16(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }

static int run_batch(const ftc_desc_t* desc, uint64_t S, int is_allreduce, const void* d_in, const uint32_t* d_prefail,
                     const ftc_inop_t* d_inop, const uint32_t* d_roots, void* d_out, uint32_t* d_status,
                     void* d_ws, size_t ws_bytes, void* stream) {
    Params p;
    int rc = fill_params(desc, S, is_allreduce, p);
    if (rc != FTC_OK) return rc;
    const bool expanded = (desc->flags & FTC_OUT_EXPANDED) != 0;
    if (expanded && !is_allreduce) return FTC_EUNSUPPORTED;     // a reduce delivers at the root only
    if (S == 0) return FTC_OK;
    if (!d_in || !d_prefail || !d_out || !d_status) return FTC_EINVAL;
    if (p.max_inop && !d_inop) return FTC_EINVAL;
    if (p.root < 0 && !d_roots) return FTC_EINVAL;
    if (!aligned16(d_in) || !aligned16(d_out) || !aligned16(d_status)) return FTC_EINVAL;
    DeviceInfo di;
    if ((rc = device_info(di)) != FTC_OK) return rc;
    const size_t front = compact_area(p);
    if (expanded && (!d_ws || ws_bytes < front || (reinterpret_cast<uintptr_t>(d_ws) & 255u))) return FTC_EWORKSPACE;
    if (expanded && expand_smem_bytes(p) > (size_t)di.smem_optin) return FTC_EUNSUPPORTED;   // before anything is enqueued
    p.in = d_in; p.prefail = d_prefail; p.inop = d_inop; p.roots = d_roots; p.status = d_status;
    p.out = expanded ? d_ws : d_out;                            // compact results first, expanded afterwards
    if (expanded) { d_ws = static_cast<char*>(d_ws) + front; ws_bytes -= front; }
    const int tsel = type_select(desc->dtype, desc->op);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    p.ws = d_ws; p.ws_bytes = (d_ws && aligned16(d_ws)) ? ws_bytes : 0;
    const KernelKind kind = pick_kernel(p, di);
    if (kind == K_STAGED) {
        e = launch_staged(p, tsel, di.sm_count, di.smem_optin, st);
    } else if (kind == K_TILED) {
        e = launch_tiled(p, tsel, di.sm_count, st);
    } else if (kind == K_LEVELS) {
        e = launch_aheap(p, tsel, di.sm_count, di.smem_optin, st);
    } else {
        const size_t need = (size_t)generic_reduce_grid(p, di.sm_count) * p.Gmax * p.kbytes;
        if (!d_ws || ws_bytes < need || !aligned16(d_ws)) return FTC_EWORKSPACE;
        if (generic_smem_bytes(p) > (size_t)di.smem_optin) return FTC_EUNSUPPORTED;
        p.ws = d_ws;
        e = launch_generic(p, tsel, di.sm_count, st);
    }
    if (e == cudaSuccess && expanded) e = launch_expand(p, p.out, d_out, di.sm_count, st);
    return e == cudaSuccess ? FTC_OK : FTC_ECUDA;
}

struct StagingLayout { size_t in, prefail, inop, roots, out, status, ws, total; };
static StagingLayout staging_layout(Params& p, uint64_t chunk, const DeviceInfo& di) {
    StagingLayout L; size_t o = 0;
    L.in = o; o += up256(chunk * (size_t)p.P * p.kbytes);
    L.prefail = o; o += up256(chunk * (size_t)p.W * 4);
    L.inop = o; o += up256(chunk * (size_t)p.max_inop * sizeof(ftc_inop_t));
    L.roots = o; o += up256(chunk * 4);
    L.out = o; o += up256(chunk * (size_t)p.kbytes);
    L.status = o; o += up256(chunk * FTC_STATUS_WORDS * 4);
    p.S = chunk;
    L.ws = o; o += up256(workspace_for(p, di));
    L.total = o;
    return L;
}

static int run_batch_host(const ftc_desc_t* desc, uint64_t S, int is_allreduce, const void* h_in, const uint32_t* h_prefail,
                          const ftc_inop_t* h_inop, const uint32_t* h_roots, void* h_out, uint32_t* h_status,
                          void* d_staging, size_t staging_bytes, void* stream) {
    Params p;
    int rc = fill_params(desc, S, is_allreduce, p);
    if (rc != FTC_OK) return rc;
    if (desc->flags & FTC_OUT_EXPANDED) return FTC_EUNSUPPORTED;
    if (S == 0) return FTC_OK;
    if (!h_in || !h_prefail || !h_out || !h_status || !d_staging) return FTC_EINVAL;
    if (p.max_inop && !h_inop) return FTC_EINVAL;
    if (p.root < 0 && !h_roots) return FTC_EINVAL;
    if (reinterpret_cast<uintptr_t>(d_staging) & 255u) return FTC_EINVAL;
    DeviceInfo di;
    if ((rc = device_info(di)) != FTC_OK) return rc;
    // largest chunk the staging holds
    uint64_t chunk = S;
    while (chunk > 1 && staging_layout(p, chunk, di).total > staging_bytes) chunk = (chunk + 1) / 2;
    StagingLayout L = staging_layout(p, chunk, di);
    if (L.total > staging_bytes) return FTC_EWORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* base = static_cast<char*>(d_staging);
    const size_t scen_bytes = (size_t)p.P * p.kbytes;
    for (uint64_t s0 = 0; s0 < S; s0 += chunk) {
        const uint64_t n = (S - s0 < chunk) ? S - s0 : chunk;
        if (cudaMemcpyAsync(base + L.in, static_cast<const char*>(h_in) + s0 * scen_bytes, n * scen_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return FTC_ECUDA;
        if (cudaMemcpyAsync(base + L.prefail, h_prefail + s0 * p.W, n * p.W * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return FTC_ECUDA;
        if (p.max_inop && cudaMemcpyAsync(base + L.inop, h_inop + s0 * p.max_inop, n * p.max_inop * sizeof(ftc_inop_t), cudaMemcpyHostToDevice, st) != cudaSuccess) return FTC_ECUDA;
        if (p.root < 0 && cudaMemcpyAsync(base + L.roots, h_roots + s0, n * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return FTC_ECUDA;
        rc = run_batch(desc, n, is_allreduce, base + L.in, reinterpret_cast<const uint32_t*>(base + L.prefail),
                       p.max_inop ? reinterpret_cast<const ftc_inop_t*>(base + L.inop) : nullptr,
                       p.root < 0 ? reinterpret_cast<const uint32_t*>(base + L.roots) : nullptr,
                       base + L.out, reinterpret_cast<uint32_t*>(base + L.status), base + L.ws, L.total - L.ws, st);
        if (rc != FTC_OK) return rc;
        if (cudaMemcpyAsync(static_cast<char*>(h_out) + s0 * p.kbytes, base + L.out, n * p.kbytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return FTC_ECUDA;
        if (cudaMemcpyAsync(h_status + s0 * FTC_STATUS_WORDS, base + L.status, n * FTC_STATUS_WORDS * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return FTC_ECUDA;
    }
    return cudaStreamSynchronize(st) == cudaSuccess ? FTC_OK : FTC_ECUDA;
}

}  // namespace ftc

using namespace ftc;

extern "C" {

int ftc_reduce_batch(const ftc_desc_t* desc, uint64_t S, const void* d_in, const uint32_t* d_prefail,
                     const ftc_inop_t* d_inop, const uint32_t* d_roots, void* d_out, uint32_t* d_status,
                     void* d_workspace, size_t workspace_bytes, void* cuda_stream) {
    return run_batch(desc, S, 0, d_in, d_prefail, d_inop, d_roots, d_out, d_status, d_workspace, workspace_bytes, cuda_stream);
}

int ftc_allreduce_batch(const ftc_desc_t* desc, uint64_t S, const void* d_in, const uint32_t* d_prefail,
                        const ftc_inop_t* d_inop, const uint32_t* d_roots, void* d_out, uint32_t* d_status,
                        void* d_workspace, size_t workspace_bytes, void* cuda_stream) {
    return run_batch(desc, S, 1, d_in, d_prefail, d_inop, d_roots, d_out, d_status, d_workspace, workspace_bytes, cuda_stream);
}

int ftc_reduce_batch_noalloc(const ftc_desc_t* desc, uint64_t S, const void* d_in, const uint32_t* d_prefail,
                             const ftc_inop_t* d_inop, const uint32_t* d_roots, void* d_out, uint32_t* d_status,
                             void* cuda_stream) {
    Params p;
    int rc = fill_params(desc, S, 0, p);
    if (rc != FTC_OK) return rc;
    if (desc->flags & FTC_OUT_EXPANDED) return FTC_EUNSUPPORTED;
    if (S == 0) return FTC_OK;
    if (!d_in || !d_prefail || !d_out || !d_status) return FTC_EINVAL;
    if (p.max_inop && !d_inop) return FTC_EINVAL;
    if (p.root < 0 && !d_roots) return FTC_EINVAL;
    if (!aligned16(d_in) || !aligned16(d_out) || !aligned16(d_status)) return FTC_EINVAL;
    DeviceInfo di;
    if ((rc = device_info(di)) != FTC_OK) return rc;
    if (generic_smem_bytes(p) > (size_t)di.smem_optin) return FTC_EUNSUPPORTED;
    p.in = d_in; p.prefail = d_prefail; p.inop = d_inop; p.roots = d_roots; p.out = d_out; p.status = d_status;
    bool too_large = false;
    cudaError_t e = launch_generic_static(p, type_select(desc->dtype, desc->op), di.sm_count,
                                          static_cast<cudaStream_t>(cuda_stream), &too_large);
    if (too_large) return FTC_ETOOLARGE;
    return e == cudaSuccess ? FTC_OK : FTC_ECUDA;
}

int ftc_candidates_batch(const ftc_desc_t* desc, uint64_t S, int is_allreduce, const void* d_in, const uint32_t* d_prefail,
                         const ftc_inop_t* d_inop, const uint32_t* d_roots, void* d_cand, uint32_t* d_cand_info,
                         void* d_workspace, size_t workspace_bytes, void* cuda_stream) {
    Params p;
    int rc = fill_params(desc, S, is_allreduce ? 1 : 0, p);
    if (rc != FTC_OK) return rc;
    if (S == 0) return FTC_OK;
    if (!d_in || !d_prefail || !d_cand || !d_cand_info) return FTC_EINVAL;
    if (p.max_inop && !d_inop) return FTC_EINVAL;
    if (p.root < 0 && !d_roots) return FTC_EINVAL;
    if (!aligned16(d_in) || !aligned16(d_cand) || !aligned16(d_cand_info)) return FTC_EINVAL;
    DeviceInfo di;
    if ((rc = device_info(di)) != FTC_OK) return rc;
    const int tsel = type_select(desc->dtype, desc->op);
    p.in = d_in; p.prefail = d_prefail; p.inop = d_inop; p.roots = d_roots; p.ws = d_workspace;
    if (cand_fast_supported(p, tsel, di.smem_optin, di.sm_count)) {
        const size_t need = cand_fast_workspace_bytes(p, tsel, di.smem_optin, di.sm_count);
        if (need && (!d_workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(d_workspace) & 255u))) return FTC_EWORKSPACE;
        return launch_cand_fast(p, tsel, d_cand, d_cand_info, di.sm_count, di.smem_optin, static_cast<cudaStream_t>(cuda_stream), nullptr)
                   == cudaSuccess ? FTC_OK : FTC_ECUDA;
    }
    const size_t need = (size_t)generic_grid(p, di.sm_count) * candidates_slice_bytes(p);
    if (!d_workspace || workspace_bytes < need || !aligned16(d_workspace)) return FTC_EWORKSPACE;
    if (generic_smem_bytes(p) > (size_t)di.smem_optin) return FTC_EUNSUPPORTED;
    cudaError_t e = launch_candidates(p, tsel, d_cand, d_cand_info, di.sm_count, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? FTC_OK : FTC_ECUDA;
}

int ftc_message_counts_batch(const ftc_desc_t* desc, uint64_t S, int is_allreduce, const uint32_t* d_prefail,
                             const ftc_inop_t* d_inop, const uint32_t* d_roots, uint64_t* d_msgs, void* cuda_stream) {
    Params p;
    int rc = fill_params(desc, S, is_allreduce ? 1 : 0, p);
    if (rc != FTC_OK) return rc;
    if (S == 0) return FTC_OK;
    if (!d_prefail || !d_msgs) return FTC_EINVAL;
    if (p.max_inop && !d_inop) return FTC_EINVAL;
    if (p.root < 0 && !d_roots) return FTC_EINVAL;
    if (reinterpret_cast<uintptr_t>(d_msgs) & 7u) return FTC_EINVAL;
    DeviceInfo di;
    if ((rc = device_info(di)) != FTC_OK) return rc;
    if (messages_smem_bytes(p) > (size_t)di.smem_optin) return FTC_EUNSUPPORTED;
    p.prefail = d_prefail; p.inop = d_inop; p.roots = d_roots;
    cudaError_t e = launch_messages(p, reinterpret_cast<unsigned long long*>(d_msgs), di.sm_count,
                                    static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? FTC_OK : FTC_ECUDA;
}

int ftc_failed_list_batch(const ftc_desc_t* desc, uint64_t S, int is_allreduce, const uint32_t* d_prefail,
                          const ftc_inop_t* d_inop, const uint32_t* d_roots, uint32_t* d_failed, uint32_t* d_nfail,
                          void* cuda_stream) {
    Params p;
    int rc = fill_params(desc, S, is_allreduce ? 1 : 0, p);
    if (rc != FTC_OK) return rc;
    if (S == 0) return FTC_OK;
    if (!d_prefail || !d_failed || !d_nfail) return FTC_EINVAL;
    if (p.max_inop && !d_inop) return FTC_EINVAL;
    if (p.root < 0 && !d_roots) return FTC_EINVAL;
    DeviceInfo di;
    if ((rc = device_info(di)) != FTC_OK) return rc;
    if (messages_smem_bytes(p) > (size_t)di.smem_optin) return FTC_EUNSUPPORTED;
    p.prefail = d_prefail; p.inop = d_inop; p.roots = d_roots;
    cudaError_t e = launch_failed_list(p, d_failed, d_nfail, di.sm_count, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? FTC_OK : FTC_ECUDA;
}

const char* ftc_candidates_kernel_name(const ftc_desc_t* desc) {
    Params p;
    if (fill_params(desc, 1, 0, p) != FTC_OK) return "invalid";
    DeviceInfo di;
    if (device_info(di) != FTC_OK) di = kB200;
    return cand_fast_supported(p, type_select(desc->dtype, desc->op), di.smem_optin, di.sm_count) ? "staged" : "generic";
}

size_t ftc_candidates_workspace_bytes(const ftc_desc_t* desc, uint64_t S) {
    Params p;
    if (fill_params(desc, S, 0, p) != FTC_OK || S == 0) return 0;
    DeviceInfo di;
    const bool have_device = device_info(di) == FTC_OK;
    if (!have_device) di = kB200;
    const int tsel = type_select(desc->dtype, desc->op);
    if (have_device && cand_fast_supported(p, tsel, di.smem_optin, di.sm_count))
        return cand_fast_workspace_bytes(p, tsel, di.smem_optin, di.sm_count);
    return (size_t)generic_grid(p, di.sm_count) * candidates_slice_bytes(p);
}

size_t ftc_workspace_bytes(const ftc_desc_t* desc, uint64_t S, int is_allreduce) {
    Params p;
    if (fill_params(desc, S, is_allreduce, p) != FTC_OK || S == 0) return 0;
    DeviceInfo di;
    if (device_info(di) != FTC_OK) di = kB200;
    return workspace_for(p, di);
}

int ftc_reduce_batch_host(const ftc_desc_t* desc, uint64_t S, const void* h_in, const uint32_t* h_prefail,
                          const ftc_inop_t* h_inop, const uint32_t* h_roots, void* h_out, uint32_t* h_status,
                          void* d_staging, size_t staging_bytes, void* cuda_stream) {
    return run_batch_host(desc, S, 0, h_in, h_prefail, h_inop, h_roots, h_out, h_status, d_staging, staging_bytes, cuda_stream);
}

int ftc_allreduce_batch_host(const ftc_desc_t* desc, uint64_t S, const void* h_in, const uint32_t* h_prefail,
                             const ftc_inop_t* h_inop, const uint32_t* h_roots, void* h_out, uint32_t* h_status,
                             void* d_staging, size_t staging_bytes, void* cuda_stream) {
    return run_batch_host(desc, S, 1, h_in, h_prefail, h_inop, h_roots, h_out, h_status, d_staging, staging_bytes, cuda_stream);
}

size_t ftc_host_staging_bytes(const ftc_desc_t* desc, uint64_t chunk_scenarios) {
    Params p;
    if (fill_params(desc, chunk_scenarios, 0, p) != FTC_OK || chunk_scenarios == 0) return 0;
    DeviceInfo di;
    if (device_info(di) != FTC_OK) di = kB200;
    return staging_layout(p, chunk_scenarios, di).total;
}

int ftc_schedule_info(const ftc_desc_t* desc, ftc_sched_t* out) {
    uint32_t arity;
    if (!desc || !out || desc->f > FTC_MAX_F || desc->P < desc->f + 2 || !tree_arity(desc->flags, arity)) return FTC_EINVAL;
    const uint32_t m = desc->f + 1, q = (desc->P - 1) / m, r = (desc->P - 1) % m;
    out->q = q; out->r = r;
    out->H = 1 + deepest_level_h(arity, q + (r ? 1u : 0u));
    out->rounds_reduce = desc->f + out->H;
    out->rounds_attempt = 2 * out->rounds_reduce;
    out->msgs_upcorrection = (uint64_t)desc->f * m * q + (uint64_t)(r + 1) * r;
    out->msgs_tree = desc->P - 1;
    return FTC_OK;
}

int ftc_fill_inputs(uint32_t kind, uint64_t seed, uint64_t first_scenario, uint64_t S, uint32_t P, uint32_t k,
                    void* d_out, void* cuda_stream) {
    if (kind > 4 || (!d_out && S) || P == 0 || k == 0) return FTC_EINVAL;
    DeviceInfo di;
    int rc = device_info(di);
    if (rc != FTC_OK) return rc;
    return launch_fill(kind, seed, first_scenario, S, P, k, d_out, di.sm_count, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
               ? FTC_OK : FTC_ECUDA;
}

int ftc_read_bandwidth_probe(uint32_t mode, const void* d_buf, uint64_t bytes, uint64_t* d_sink, void* cuda_stream) {
    if (mode > 1 || !d_buf || !d_sink || !aligned16(d_buf) || (reinterpret_cast<uintptr_t>(d_sink) & 7u) || bytes % (16 * 1024)) return FTC_EINVAL;
    DeviceInfo di;
    int rc = device_info(di);
    if (rc != FTC_OK) return rc;
    return launch_probe(mode, d_buf, bytes, reinterpret_cast<unsigned long long*>(d_sink), di.sm_count,
                        static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? FTC_OK : FTC_ECUDA;
}

const char* ftc_kernel_name(const ftc_desc_t* desc, int is_allreduce) {
    Params p;
    if (fill_params(desc, 1, is_allreduce, p) != FTC_OK) return "invalid";
    DeviceInfo di;
    if (device_info(di) != FTC_OK) di = kB200;
    p.ws_bytes = ~0ull;                                   // given the workspace ftc_workspace_bytes() asks for
    const KernelKind kind = pick_kernel(p, di);
    return kind == K_STAGED ? "staged" : kind == K_TILED ? "tiled" : kind == K_LEVELS ? "levels" : "generic";
}

const char* ftc_kernel_variant(const ftc_desc_t* desc, int is_allreduce) {
    Params p;
    if (fill_params(desc, 1, is_allreduce, p) != FTC_OK) return "invalid";
    DeviceInfo di;
    if (device_info(di) != FTC_OK) di = kB200;
    p.ws_bytes = ~0ull;
    const KernelKind kind = pick_kernel(p, di);
    if (kind == K_STAGED) return staged_variant(p, type_select(desc->dtype, desc->op), di.smem_optin, di.sm_count, nullptr);
    return kind == K_TILED ? "tiled" : kind == K_LEVELS ? "levels" : "generic";
}

int ftc_launch_blocks(const ftc_desc_t* desc, uint64_t S, int is_allreduce, uint32_t* blocks) {
    Params p;
    int rc = fill_params(desc, S, is_allreduce, p);
    if (rc != FTC_OK) return rc;
    if (!blocks) return FTC_EINVAL;
    *blocks = 0;
    if (S == 0) return FTC_OK;
    DeviceInfo di;
    if ((rc = device_info(di)) != FTC_OK) return rc;
    p.ws_bytes = ~0ull;
    p.grid_query = blocks;
    const int tsel = type_select(desc->dtype, desc->op);
    const KernelKind kind = pick_kernel(p, di);
    cudaError_t e = kind == K_STAGED ? launch_staged(p, tsel, di.sm_count, di.smem_optin, nullptr)
                  : kind == K_TILED ? launch_tiled(p, tsel, di.sm_count, nullptr)
                  : kind == K_LEVELS ? launch_aheap(p, tsel, di.sm_count, di.smem_optin, nullptr) : launch_generic(p, tsel, di.sm_count, nullptr);
    return e == cudaSuccess ? FTC_OK : FTC_ECUDA;
}

const char* ftc_strerror(int code) {
    switch (code) {
    case FTC_OK: return "ok";
    case FTC_EINVAL: return "invalid argument (P < f+2, k = 0, root >= P, f > 31, max_inop > 32, NULL or misaligned pointer)";
    case FTC_EUNSUPPORTED: return "unsupported dtype/op combination or flag";
    case FTC_EWORKSPACE: return "workspace missing, misaligned or smaller than ftc_workspace_bytes()";
    case FTC_ECUDA: return "a CUDA call or kernel launch failed";
    case FTC_ETOOLARGE: return "shape too large for the built-in scratch: ceil((P-1)/(f+1)) * k * element size exceeds FTC_NOALLOC_SCRATCH_BYTES";
    }
    return "unknown error code";
}

uint32_t ftc_version(void) { return FTC_VERSION; }

}  // extern "C"
