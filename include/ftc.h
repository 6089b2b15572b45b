/*
 * ftc.h -- C ABI of the batched executor for the correction-based fault-tolerant
 * reduce and allreduce (Kuettler & Haertig, "Fault-tolerant Reduce and Allreduce
 * operations based on correction").
 *
 * The library plays the paper's message schedule for S independent scenarios at once
 * on one NVIDIA B200 (sm_100a). A scenario is one input vector of k elements for each
 * of P logical processes plus a failure pattern; the result is the value the root
 * (reduce) or every surviving process (allreduce) ends up with, and a status record.
 *
 * Conventions for every entry point
 *   - plain C linkage, no exceptions, no global state (except where an entry point
 *     says otherwise); pointers named d_* are DEVICE pointers, h_* HOST pointers;
 *   - the caller owns every buffer and the stream; inputs are read-only; the library
 *     allocates nothing and never synchronises the host unless stated;
 *   - work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL = the
 *     default stream) and is complete when that stream has drained;
 *   - the return value reports call-level errors only (0 = FTC_OK, negative = error,
 *     see ftc_strerror). What happens inside a scenario (failed root, no failure-free
 *     subtree, ...) is not an error: it is written to that scenario's status record.
 *
 * Readings of the paper that fix the schedule (the paper leaves them open):
 *   - the root swaps numbers with process 0 (section "Reduce"); all rules below apply
 *     to the renumbered ranks v;
 *   - up-correction group of v >= 1 is floor((v-1)/(f+1)); the root joins the last
 *     group iff that group is short (section "Up-Correction"); partners are visited in
 *     ascending rank, the root first;
 *   - v >= 1 lies below root child s = (v-1) mod (f+1) (proof of the first theorem of
 *     section "Properties"); within a subtree the nodes j = floor((v-1)/(f+1)) form a
 *     heap, binary unless FTC_TREE_ARITY(a) in the flags asks for a children per node: children a*j+1 .. a*j+a,
 *     received in that order, accumulator on the left (the paper's I(f)-tree fixes only the root's f+1 children
 *     and their subtree sizes; heaps of other arities and binomial trees run on the level kernel in shared memory
 *     where their shape fits it, else on the general kernel, which needs its workspace);
 *   - failure information is the single failed bit (third scheme of section "Failure
 *     information"); the root takes the lowest-numbered child that delivered with the
 *     bit clear (Algorithm "reduce_root");
 *   - rounds: up-correction iteration i is round i (0..f-1); a node at depth d sends up
 *     the tree in round f+H-d, H = 1+floor(log2(ceil((P-1)/(f+1)))); one reduce has
 *     f+H rounds. The broadcast of the allreduce sends down the same tree (depth d in
 *     round f+H+d) and then lets every process the tree reached send the value to its
 *     up-correction partners (iteration i in round f+2H+i); one allreduce attempt has
 *     2(f+H) rounds and attempt a starts at round a*2(f+H). A process with failure
 *     round t performs exactly the sends scheduled in rounds < t;
 *   - allreduce root candidates are first, first+1, ... (mod P), f+1 of them
 *     (Algorithm "Allreduce"; "at least f+1 processes must eventually be tried").
 */
#ifndef FTC_H
#define FTC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define FTC_API __attribute__((visibility("default")))
#else
#define FTC_API
#endif

#define FTC_VERSION 0x00010000u

/* element types and reduction functions (section "Reduce": associative and commutative) */
enum { FTC_I32 = 0, FTC_I64 = 1, FTC_U64 = 2, FTC_F32 = 3 };
enum { FTC_SUM = 0, FTC_MAX = 1, FTC_XOR = 2 };   /* integer sums wrap; FTC_F32 supports FTC_SUM only */

/* call-level return codes */
enum {
    FTC_OK = 0,
    FTC_EINVAL = -1,        /* P < f+2, k = 0, root >= P, NULL or misaligned required pointer, f > 31, max_inop > 32, tree arity 1 or > 32 */
    FTC_EUNSUPPORTED = -2,  /* unknown dtype/op, xor or max on f32, expanded output for so many processes that its bitmasks
                               exceed shared memory */
    FTC_EWORKSPACE = -3,    /* workspace missing or smaller than ftc_workspace_bytes() */
    FTC_ECUDA = -4,         /* a CUDA call or launch failed */
    FTC_ETOOLARGE = -5      /* ftc_reduce_batch_noalloc: the shape does not fit the built-in scratch */
};

/* per-scenario outcome, low byte of status word 0 */
enum {
    FTC_ST_OK = 0,
    FTC_ST_ROOT_FAILED = 1,             /* reduce to a failed root is a no-op (section "Semantics") */
    FTC_ST_NO_CLEAN_SUBTREE = 2,        /* Algorithm "reduce_root": "No failure-free subtree" (needs > f failures) */
    FTC_ST_NO_LIVE_ROOT_CANDIDATE = 3,  /* allreduce: all f+1 candidates had failed before the operation */
    FTC_ST_PRECONDITION_INOP_ROOT = 4,  /* allreduce: a root candidate is listed as failing in-operation */
    FTC_ST_BAD_ROOT = 5,                /* d_roots[s] >= P */
    FTC_ST_INTERNAL_TIMEOUT = 6         /* a bounded wait for a copy inside the kernel ran out: this scenario and every later one
                                           that the same thread block plays report this outcome; results are zero bytes */
};

/*
 * Status record, FTC_STATUS_WORDS uint32 per scenario:
 *   word 0: outcome | selected root child (0..f, 0xFF none) << 8 | attempts used << 16
 *   word 1: number of processes whose input is included in the result
 *   word 2: bit i set = the victim of in-operation slot i is included in the result
 *   word 3: allreduce: processes that are alive at the end and hold the result; reduce: 0
 * When the outcome is not FTC_ST_OK words 1..3 are 0 and the result is all zero bytes.
 */
#define FTC_STATUS_WORDS 4

/* An in-operation failure: `victim` performs exactly the sends scheduled in rounds < `round`.
 * victim = FTC_INOP_UNUSED marks an empty slot; a victim that is also pre-failed counts as pre-failed;
 * round 0 is the same as a pre-operation failure. (Sections "Introduction", "Failures".) */
typedef struct { uint32_t victim; uint32_t round; } ftc_inop_t;
#define FTC_INOP_UNUSED 0xFFFFFFFFu
#define FTC_MAX_INOP 32u
#define FTC_MAX_F 31u

/* flags */
#define FTC_OUT_EXPANDED   0x1u   /* allreduce: d_out is [S][P][k], zeros for processes that do not hold the result */
#define FTC_TREE_ARITY(a)  (((uint32_t)(a) & 0xFFu) << 16)  /* subtrees below the root's children are a-ary heaps, 2 <= a <= FTC_MAX_ARITY (not given: binary) */
#define FTC_MAX_ARITY 32u
#define FTC_TREE_BINOMIAL   0x1000000u /* subtrees below the root's children are binomial trees on the local index j: parent of j =
                                         j without its lowest set bit, children in ascending order, depth = 1 + set bits of j
                                         (not together with FTC_TREE_ARITY) */
#define FTC_PARTNERS_DESCENDING 0x2000000u /* up-correction (and the broadcast's correction) visits the group partners in descending
                                            rank, the root last, instead of ascending with the root first: the algorithm leaves the
                                            order open (every kernel plays it) */
#define FTC_KERNEL_GENERIC 0x100u /* force the general level-by-level kernel (needs the workspace) */
#define FTC_KERNEL_LEVELS  0x400u /* binary heaps: take the level kernel (shared-memory tiles evaluated level by level), which heaps of
                                     arity 3 and more and binomial trees use by default, where the shape allows it */
#define FTC_KERNEL_DIRECT  0x200u /* force the register-tiled kernel (direct global loads) where the shape allows it */
#define FTC_DEBUG_ONE_POLL 0x4000000u /* testing aid: the kernel's bounded waits for its asynchronous copies look once instead of
                                         polling, so most of them give up and the give-up path runs: affected scenarios report
                                         FTC_ST_INTERNAL_TIMEOUT with zero bytes, nothing waits without a limit and nothing is read
                                         or written out of bounds. Never set it in production calls */

typedef struct {
    uint32_t P;         /* processes, P >= f+2 (the root needs f+1 children: definition of the I(f)-tree) */
    uint32_t f;         /* failures to tolerate, 0..31; up-correction groups have f+1 members */
    uint32_t k;         /* elements per process */
    uint32_t dtype;     /* FTC_I32 ... */
    uint32_t op;        /* FTC_SUM ... */
    int32_t  root;      /* >= 0: root (reduce) / first root candidate (allreduce) of every scenario; -1: d_roots[s] */
    uint32_t max_inop;  /* in-operation slots per scenario in d_inop, 0..32 */
    uint32_t flags;
} ftc_desc_t;

/* Schedule constants under the readings above and the failure-free message counts of the theorem on the
 * number of messages (section "Properties"). */
typedef struct {
    uint32_t q, r;              /* full groups, size of the short last group without the root: P-1 = q(f+1)+r */
    uint32_t H;                 /* depth of the deepest node */
    uint32_t rounds_reduce;     /* f+H */
    uint32_t rounds_attempt;    /* 2(f+H): reduce plus broadcast */
    uint64_t msgs_upcorrection; /* f(f+1)q + a(a-1), a = r+1 */
    uint64_t msgs_tree;         /* P-1 */
} ftc_sched_t;

/*
 * Corrected reduce (Algorithms "Up-correction", "reduce_root", "reduce_non_root", "reduce") for S scenarios.
 *   d_in      [S][P][k] elements of desc->dtype, process order as the caller numbers them; 16-byte aligned
 *   d_prefail [S][ceil(P/32)] uint32, bit p of a scenario's words set = process p failed before the operation
 *   d_inop    [S][max_inop] or NULL when max_inop = 0
 *   d_roots   [S] or NULL; read only when desc->root < 0
 *   d_out     [S][k]: the value delivered at the root (zeros unless the outcome is FTC_ST_OK); 16-byte aligned
 *   d_status  [S][FTC_STATUS_WORDS] uint32; 16-byte aligned (one record is stored as one 16-byte word)
 *   d_workspace, workspace_bytes: scratch of at least ftc_workspace_bytes(desc, S, 0) bytes (may be NULL if that is 0),
 *             16-byte aligned; contents are undefined afterwards; calls that share a workspace must not overlap on
 *             the device. Shapes that run on the shared-memory kernels also run with less or none (large process
 *             counts with wide vectors then more slowly); shapes that need the general kernel get FTC_EWORKSPACE
 * S = 0 is valid and does nothing. Returns FTC_OK or an error before anything is enqueued.
 */
FTC_API int ftc_reduce_batch(const ftc_desc_t* desc, uint64_t S, const void* d_in, const uint32_t* d_prefail,
                     const ftc_inop_t* d_inop, const uint32_t* d_roots, void* d_out, uint32_t* d_status,
                     void* d_workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Corrected allreduce (Algorithm "Allreduce": reduce to a root candidate, broadcast from it, next candidate if
 * it had failed before the operation). Arguments as for ftc_reduce_batch; desc->root / d_roots give the first
 * candidate. d_out is [S][k] (the value every holder has) or, with FTC_OUT_EXPANDED, [S][P][k]: the value in the
 * slot of every process that is alive at the end and holds it, zero bytes in all other slots. The expanded form
 * needs ftc_workspace_bytes() of 256-byte aligned workspace (the compact results pass through it); the host-buffer
 * variants and ftc_reduce_batch do not offer it (FTC_EUNSUPPORTED).
 */
FTC_API int ftc_allreduce_batch(const ftc_desc_t* desc, uint64_t S, const void* d_in, const uint32_t* d_prefail,
                        const ftc_inop_t* d_inop, const uint32_t* d_roots, void* d_out, uint32_t* d_status,
                        void* d_workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Corrected reduce for callers that cannot give the library any scratch memory and cannot allocate it either.
 * (The paper has no counterpart to this entry point: it exists for the sake of the host program, not the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a latency-critical loop, where an
 * allocation's implicit device-wide synchronisation would stall unrelated streams; inside a plug-in or callback
 * of another framework that owns the memory budget and hands out no allocator; or after start-up in a service
 * whose device memory is fully accounted for. ftc_reduce_batch wants a caller-provided workspace for shapes that
 * run on the general kernel; this variant needs none.
 *
 * How: the general kernel's per-block node values go to an array of FTC_NOALLOC_SCRATCH_BYTES bytes that is part
 * of the library image. Every GPU that loads the library holds that array until the process exits. The call
 * allocates nothing (no cudaMalloc, cudaFree or allocating library routine), results and status records are
 * identical to ftc_reduce_batch's, and it is slower when fewer blocks than usual fit into the array.
 *   - Limit: one block's slice, ceil((P-1)/(f+1)) * k * element size bytes, must fit the array; otherwise
 *     FTC_ETOOLARGE is returned and nothing is enqueued.
 *   - The first call on each device looks the array's device address up (one runtime query, with that device
 *     current) and keeps it for the life of the process. Make that first call before starting any stream capture
 *     on that device. The address belongs to the device's primary context: a host program that destroys that
 *     context (cudaDeviceReset) must not call this entry point on that device afterwards.
 *   - All calls on a device share the one array, which keeps whatever the previous call left in it. Nothing in it
 *     needs clearing: within a scenario every slot is written before it is read. But two calls whose kernels can
 *     overlap on the same GPU (different streams, or different host threads) race on it: serialise them.
 * Arguments and all other rules as for ftc_reduce_batch, without the workspace pair. The always-general kernel
 * is used whatever the shape.
 */
#define FTC_NOALLOC_SCRATCH_BYTES (8u << 20)
FTC_API int ftc_reduce_batch_noalloc(const ftc_desc_t* desc, uint64_t S, const void* d_in, const uint32_t* d_prefail,
                                     const ftc_inop_t* d_inop, const uint32_t* d_roots, void* d_out,
                                     uint32_t* d_status, void* cuda_stream);

/*
 * What the root receives from each of its f+1 children (Algorithm "reduce_root": "receive from any child (data,
 * failure information)"; section "Failure information", second and third scheme), for S scenarios. The batch calls
 * above evaluate only the child the root selects; this call plays all f+1 subtrees, nodes that deliver nothing
 * included. is_allreduce != 0: the reduce of the allreduce attempt that counts (the last one if no candidate is alive).
 *   d_cand      [S][f+1][k]: the value child s delivers (zeros if it delivers nothing); 16-byte aligned
 *   d_cand_info [S][f+1][2] uint32: [0] 0 = delivered with the failed bit clear, 1 = delivered with the failed bit set,
 *               2 = nothing delivered, 3 = a bounded wait inside the kernel ran out (no value; as FTC_ST_INTERNAL_TIMEOUT);
 *               [1] size of the list of failed processes that came with the value
 *   workspace of at least ftc_candidates_workspace_bytes(desc, S) bytes, 256-byte aligned
 * Other arguments as for ftc_reduce_batch. Scenarios whose root is invalid or violates the allreduce precondition
 * play no attempt: zeros and "nothing delivered".
 * Two kernels (ftc_candidates_kernel_name): "staged" on binary heaps with vectors of 16..512 bytes (a power-of-two number of
 * 16-byte chunks) and scenarios above 12 KB -- one pass over the inputs on the tiles of the shared-memory kernel; for the
 * exactly associative operations (integer sum, max, xor) a group without a failed member is folded once for all children,
 * for float32 every child's member folds in its own order from the staged copy; "generic" (any k, other subtree shapes,
 * FTC_KERNEL_GENERIC) plays child after child.
 */
FTC_API int ftc_candidates_batch(const ftc_desc_t* desc, uint64_t S, int is_allreduce, const void* d_in,
                                 const uint32_t* d_prefail, const ftc_inop_t* d_inop, const uint32_t* d_roots,
                                 void* d_cand, uint32_t* d_cand_info, void* d_workspace, size_t workspace_bytes,
                                 void* cuda_stream);
FTC_API size_t ftc_candidates_workspace_bytes(const ftc_desc_t* desc, uint64_t S);
FTC_API const char* ftc_candidates_kernel_name(const ftc_desc_t* desc);

/*
 * The list of failed processes that the root holds when it delivers (section "Failure information", first scheme:
 * in the up-correction phase and in the tree phase every process appends the ids of the processes it could not
 * receive a value from; the lists travel up the tree with the values; "the root receives a complete list of failed
 * processes from each child ... that does not contain a failed process in the subtree spanned by it"). It is the list
 * that came with the value of the child the root selected, plus, when that child's subtree holds no member of the
 * root's own up-correction group, what the root noted itself. Under in-operation failures it lists exactly the
 * processes whose input is not part of the delivered result. is_allreduce != 0: the reduce of the attempt that counts.
 *   d_failed [S][ceil(P/32)] uint32: bit p of a scenario's words set = process p (the caller's numbering) is on the list
 *   d_nfail  [S] uint32: the size of the list (the second scheme sends only this); equals the number of set bits,
 *            since concatenated lists come from disjoint sets
 * Scenarios whose outcome is not FTC_ST_OK deliver nothing: all zero. Only the failure pattern is read; desc->k, dtype
 * and op must be valid but do not matter. Other arguments as for ftc_reduce_batch. No workspace.
 */
FTC_API int ftc_failed_list_batch(const ftc_desc_t* desc, uint64_t S, int is_allreduce, const uint32_t* d_prefail,
                                  const ftc_inop_t* d_inop, const uint32_t* d_roots, uint32_t* d_failed, uint32_t* d_nfail,
                                  void* cuda_stream);

/*
 * Messages sent in each scenario (theorem on the number of messages of the reduce and theorem on the messages of
 * the allreduce, section "Properties": failure-free f(f+1)q + a(a-1) up-correction and P-1 tree messages; no
 * process sends more when processes fail; an allreduce whose first candidates had failed repeats the reduce).
 * A message counts when its sender performs the send, whether or not the receiver is alive (section "Failures":
 * a send to a failed process completes). Only the failure pattern is read; desc->k, dtype and op must be valid
 * but do not matter.
 *   d_msgs [S][FTC_MSG_WORDS] uint64, 8-byte aligned:
 *     [0..3] over all attempts that are played: up-correction, tree, tree-down (broadcast), correction (broadcast)
 *     [4..7] the same four for the last attempt alone
 *   A reduce plays one attempt and has no broadcast ([2], [3], [6], [7] are 0), also when its root has failed
 *   (the others still send). An allreduce plays one attempt per root candidate up to the first one that had not
 *   failed before the operation; only that candidate broadcasts, and only if it found a failure-free subtree.
 *   Scenarios with outcome FTC_ST_BAD_ROOT or FTC_ST_PRECONDITION_INOP_ROOT play nothing: all zero.
 *   The broadcast numbers rest on this library's reading of the broadcast (see the top of this file), which the
 *   paper does not define.
 * Other arguments as for ftc_reduce_batch. No workspace.
 */
#define FTC_MSG_WORDS 8
FTC_API int ftc_message_counts_batch(const ftc_desc_t* desc, uint64_t S, int is_allreduce, const uint32_t* d_prefail,
                                     const ftc_inop_t* d_inop, const uint32_t* d_roots, uint64_t* d_msgs,
                                     void* cuda_stream);

/* Scratch bytes ftc_reduce_batch / ftc_allreduce_batch want for this descriptor and batch size: the general kernel's
 * node values, the compact results of the expanded output, and for many processes with wide vectors the shared-memory
 * kernel's array of tile results (0 otherwise). Returns 0 for an invalid descriptor as well; the batch calls report that. */
FTC_API size_t ftc_workspace_bytes(const ftc_desc_t* desc, uint64_t S, int is_allreduce);

/*
 * Same operations with HOST buffers (h_* as the d_* above): copies the inputs to the device in chunks, runs the
 * kernels, copies results and status back, all on `cuda_stream`, then synchronises that stream before returning.
 * d_staging is device scratch of at least ftc_host_staging_bytes(desc, 1) bytes; larger staging means larger
 * chunks. Pinned host memory makes the copies asynchronous but is not required.
 */
FTC_API int ftc_reduce_batch_host(const ftc_desc_t* desc, uint64_t S, const void* h_in, const uint32_t* h_prefail,
                          const ftc_inop_t* h_inop, const uint32_t* h_roots, void* h_out, uint32_t* h_status,
                          void* d_staging, size_t staging_bytes, void* cuda_stream);
FTC_API int ftc_allreduce_batch_host(const ftc_desc_t* desc, uint64_t S, const void* h_in, const uint32_t* h_prefail,
                             const ftc_inop_t* h_inop, const uint32_t* h_roots, void* h_out, uint32_t* h_status,
                             void* d_staging, size_t staging_bytes, void* cuda_stream);
/* Device staging bytes for chunks of `chunk_scenarios` scenarios (inputs, masks, outputs and workspace). */
FTC_API size_t ftc_host_staging_bytes(const ftc_desc_t* desc, uint64_t chunk_scenarios);

/* Schedule constants and failure-free message counts for (P, f) of the descriptor. FTC_EINVAL if P < f+2. */
FTC_API int ftc_schedule_info(const ftc_desc_t* desc, ftc_sched_t* out);

/*
 * Synthetic scenario inputs on the device (not part of the paper's method): element (s, p, e) of scenario
 * first_scenario+s is a function of (seed, scenario, p, e) only -- the splitmix64 output function applied to
 * seed + 0x9E3779B97F4A7C15 * (counter+1) -- mapped to one of the value kinds
 *   0 int32 in [-2^20, 2^20]   1 int64 in [-2^40, 2^40]   2 float32, sum of twelve 32-bit uniforms (six counters per
 *   element) centred, rounded to float32 once and scaled to unit variance: close to N(0,1), full mantissas
 *   3 int32 full range         4 uint64 full range
 * d_out is [S][P][k] of the kind's type. Returns FTC_OK, FTC_EINVAL (unknown kind, NULL) or FTC_ECUDA.
 */
FTC_API int ftc_fill_inputs(uint32_t kind, uint64_t seed, uint64_t first_scenario, uint64_t S, uint32_t P, uint32_t k,
                    void* d_out, void* cuda_stream);

/*
 * Measurement aid (not part of the paper's method): reads `bytes` bytes (a multiple of 16 KiB) at d_buf (16-byte
 * aligned) once and does nothing else. mode 0: 128-bit loads folded with xor in registers; mode 1: asynchronous bulk
 * copies into shared memory, the way the batch kernels stage their inputs. Timed over the buffer a batch call reads,
 * it gives the bandwidth a read-only kernel can reach on this GPU (a copy benchmark reads and writes).
 * d_sink: two uint64 words, zeroed by the caller; word 1 counts warps whose bounded wait for a copy gave up (0 in a valid run).
 */
FTC_API int ftc_read_bandwidth_probe(uint32_t mode, const void* d_buf, uint64_t bytes, uint64_t* d_sink, void* cuda_stream);

/* Name of the kernel family the batch calls would use for this descriptor: "staged", "tiled" or "generic". */
FTC_API const char* ftc_kernel_name(const ftc_desc_t* desc, int is_allreduce);

/* The same, down to the instantiation of the shared-memory kernel: "staged/warp" (scenarios of a few KB: one warp per
 * scenario), "staged/warp-pair" (two scenarios per warp, half a warp each), "staged/whole" (scenario staged by one copy),
 * "staged/lean" (blocks of one or two warps), "staged/large" (4-8 warps), "staged/batched-lean" (4-8 warps, groups of at
 * most 128 bytes, exact operations), "staged/lean-swz" and "staged/batched-swz" (float32 vectors of 16 or 32 bytes, tiles
 * by swizzled tensor copies), "staged/whole-large", "tiled", "generic"; assuming the workspace ftc_workspace_bytes() asks for. */
FTC_API const char* ftc_kernel_variant(const ftc_desc_t* desc, int is_allreduce);

/* Thread blocks the batch calls would launch for S scenarios on the current device (given the workspace
 * ftc_workspace_bytes() asks for). Block b plays scenarios b, b + blocks, b + 2*blocks, ... one after the other (the warp
 * kernel for scenarios of a few KB hands out short runs of consecutive scenarios the same way); a batch keeps the whole
 * GPU busy when S is a few times this number. Needs a device. Launches nothing. */
FTC_API int ftc_launch_blocks(const ftc_desc_t* desc, uint64_t S, int is_allreduce, uint32_t* blocks);

FTC_API const char* ftc_strerror(int code);
FTC_API uint32_t ftc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FTC_H */
