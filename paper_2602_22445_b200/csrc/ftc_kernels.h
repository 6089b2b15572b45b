// Host-side declarations of the kernel launchers (internal to the library).
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

namespace ftc {

struct Params;

// (element type, reduction) pairs the kernels are instantiated for. Signed and unsigned sums and xors of the
// same width are the same bit operation, so int64 sum runs as uint64 sum, and so on.
enum TypeSel { TS_U32_SUM = 0, TS_I32_MAX, TS_U32_XOR, TS_U64_SUM, TS_I64_MAX, TS_U64_MAX, TS_U64_XOR, TS_F32_SUM, TS_COUNT };

size_t generic_smem_bytes(const Params& p);
uint32_t generic_grid(const Params& p, int sm_count);
uint32_t generic_reduce_threads(const Params& p);            // block size of the general reduce kernel for this shape
uint32_t generic_reduce_grid(const Params& p, int sm_count);  // its blocks (each needs a workspace slice of Gmax * kbytes)
cudaError_t launch_generic(const Params& p, int tsel, int sm_count, cudaStream_t st);

// General kernel on the library's built-in scratch array (no workspace from the caller).
cudaError_t launch_generic_static(Params p, int tsel, int sm_count, cudaStream_t st, bool* too_large);

// Tiled kernel: does the shape fit (16-byte chunks, power-of-two chunk count <= 32, shared memory)? Fills the
// tile geometry into p when it does.
bool tiled_supported(Params& p, int smem_optin_bytes);
cudaError_t launch_tiled(const Params& p, int tsel, int sm_count, cudaStream_t st);

// Staged kernel (bulk copies into shared memory): same shape limits plus room for the tile buffers.
// With a workspace (p.ws_bytes) large heap arrays move there, which frees shared memory: more shapes fit and more
// blocks are resident. staged_workspace_bytes: what that takes for this shape (0: nothing to gain).
bool staged_supported(Params& p, int smem_optin_bytes, int sm_count);
size_t staged_workspace_bytes(Params p, int smem_optin_bytes, int sm_count);
cudaError_t launch_staged(const Params& p, int tsel, int sm_count, int smem_optin_bytes, cudaStream_t st);
// Name of the instantiation launch_staged would run ("staged/lean", ...); p.S and p.ws_bytes matter.
const char* staged_variant(Params p, int tsel, int smem_optin_bytes, int sm_count, uint32_t* grid_cap_blocks_per_sm);

// Warp kernel (scenarios of a few KB, one warp per scenario): shape check and launch. The staged launcher and the
// variant query route to it when the shape fits.
bool warp_supported(Params p, int smem_optin_bytes);
uint32_t warp_lanes_per_scenario(Params p, int smem_optin_bytes);      // 32, or 16 when two scenarios share a warp; 0: not this kernel
cudaError_t launch_warp(const Params& p, int tsel, int sm_count, int smem_optin_bytes, cudaStream_t st);

// Level kernel: staged tiles evaluated level by level in shared memory, for subtrees that are a-ary heaps of any
// arity >= 2 (the binary heap takes it only on request).
bool aheap_supported(Params p, int smem_optin_bytes);
cudaError_t launch_aheap(const Params& p, int tsel, int sm_count, int smem_optin_bytes, cudaStream_t st);

// Every root child's delivery (value, flag, failed-list size): general kernel, workspace slices of candidates_slice_bytes().
size_t candidates_slice_bytes(const Params& p);
cudaError_t launch_candidates(const Params& p, int tsel, void* cand, uint32_t* info, int sm_count, cudaStream_t st);

// The same on the staged tiles, all root children in one pass over the inputs (exactly associative operations).
// grid_out != NULL: store the blocks a launch may use (the workspace holds one slice per block) and launch nothing.
bool cand_fast_supported(Params p, int tsel, int smem_optin_bytes, int sm_count);
size_t cand_fast_workspace_bytes(Params p, int tsel, int smem_optin_bytes, int sm_count);
cudaError_t launch_cand_fast(const Params& p, int tsel, void* cand, uint32_t* info, int sm_count, int smem_optin_bytes, cudaStream_t st, uint32_t* grid_out);

// Message counts per scenario (FTC_MSG_WORDS 64-bit words each); reads the failure pattern only.
size_t messages_smem_bytes(const Params& p);
cudaError_t launch_messages(const Params& p, unsigned long long* out, int sm_count, cudaStream_t st);

// The failed-process list the root ends up with (bitmask over process ids, and its size); reads the failure pattern only.
cudaError_t launch_failed_list(const Params& p, uint32_t* failed, uint32_t* nfail, int sm_count, cudaStream_t st);

// Expanded allreduce output from the compact results (one value per scenario) left by the main kernel.
size_t expand_smem_bytes(const Params& p);
cudaError_t launch_expand(const Params& p, const void* compact, void* out, int sm_count, cudaStream_t st);

// Read-bandwidth probe: mode 0 = 128-bit loads, mode 1 = bulk copies into shared memory; sink = two 64-bit words.
cudaError_t launch_probe(uint32_t mode, const void* buf, uint64_t bytes, unsigned long long* sink, int sm_count, cudaStream_t st);

cudaError_t launch_fill(uint32_t kind, uint64_t seed, uint64_t first, uint64_t S, uint32_t P, uint32_t k, void* out,
                        int sm_count, cudaStream_t st);

}  // namespace ftc
